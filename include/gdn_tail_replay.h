/*
 * gdn_tail_replay.h — C ABI of the B200 (sm_100a) Gated DeltaNet tail-replay library.
 *
 * What it computes.  For every request n and v-head h, starting from a zero state (or from
 * desc->init_state), the Gated DeltaNet recurrence of the paper's Eq. 1 is applied to the
 * request's rows of the packed inputs:
 *
 *     S_t = S_{t-1} * alpha_t * (I - beta_t k_t k_t^T) + beta_t v_t k_t^T       S in R^{dv x dk}
 *     o_t = S_t q_t                                                            (state after token t)
 *
 * with alpha_t = exp(g_t), g_t = log alpha_t <= 0.  gdn_tail_replay is Eq. 2 (the recurrence
 * restricted to the last k tokens of a matched prefix, zero start): the caller passes only the
 * tail rows.  gdn_full_prefill is the same function over whole prefixes (the paper's
 * full-prefill baseline).  tail_select is the replay-window arithmetic k = ceil(r m) of the
 * paper's Method section.
 *
 * Layouts (row-major, packed varlen, no batch dimension; T = cu_tail_lens[N]):
 *     q, k          [T, Hq, dk]   io_dtype (bf16 or fp32)
 *     v             [T, Hv, dv]   io_dtype
 *     g, beta       [T, Hv]       fp32
 *     cu_tail_lens  [N + 1]       int32, cu[0] = 0, non-decreasing; request n owns rows
 *                                 [cu[n], cu[n+1])
 *     out_o         [T, Hv, dv]   io_dtype
 *     out_state     [N, Hv, dk, dv] fp32, out_state[n,h,a,b] = S[b][a] (the transpose of S)
 * v-head h reads q/k head h / (Hv / Hq): consecutive v-heads share one q/k head.  No scaling
 * or normalisation is applied to q or k.  All pointers must be 16-byte aligned.
 *
 * Memory.  With desc->memory == GDN_MEM_DEVICE every data pointer is a device pointer.  With
 * GDN_MEM_HOST every data pointer (q, k, v, g, beta, cu_tail_lens, out_o, out_state,
 * init_state) is a host pointer (pinned memory makes the copies asynchronous); the library
 * stages through the caller's workspace, pipelined by groups of requests: inputs travel host to
 * device on one internal copy stream and results device to host on another while the kernels
 * run on desc->stream, which is also where the call ends (work enqueued on desc->stream after
 * the call sees the results).  The two copy streams and a few events are created once per
 * device on the first host-memory call; they are host-side objects, not device memory.
 * Ownership: every buffer is the caller's.  The library allocates no device memory, keeps no
 * state between calls and frees nothing (the one exception, gdn_tail_replay_static_scratch, says so below).  Calls are asynchronous on desc->stream; buffers
 * must stay alive until the stream has passed the call.  Valid output rows are fully
 * overwritten; no other byte of the outputs is touched.  A request of length 0 gets a zero
 * state (or its init_state) and no output rows.
 *
 * Errors.  Every function returns a gdn_status (tail_select: a length, or -1); nothing
 * aborts or throws.  Problems visible on the host (null pointers, bad head counts,
 * unsupported dims or chunk, workspace too small, misaligned pointers) are reported before
 * any GPU work is enqueued.  Device data (g > 0, NaN, non-monotone cu_tail_lens on the
 * device) is not validated.  The tensor-core path reads whole 64-row tiles, so the last tile of
 * a request covers rows of the request that follows it in the packed arrays: those rows never
 * influence the result as long as they hold finite values (any magnitude), but an infinity or
 * a NaN in the first rows of a request can reach the last tile of its predecessor.
 * A bounded device-side wait that expires writes
 * GDN_ERR_TIMEOUT to *desc->status_word (if given) and the kernel returns early.
 */
#ifndef GDN_TAIL_REPLAY_H_
#define GDN_TAIL_REPLAY_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define GDN_API __attribute__((visibility("default")))
#else
#define GDN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GDN_OK = 0,
    GDN_ERR_INVALID_ARG = -1,   /* null / misaligned pointer, inconsistent sizes */
    GDN_ERR_UNSUPPORTED = -2,   /* head dims, chunk, dtype or kernel choice not built */
    GDN_ERR_WORKSPACE = -3,     /* workspace missing or smaller than gdn_workspace_size() */
    GDN_ERR_CUDA = -4,          /* a CUDA runtime / driver call failed */
    GDN_ERR_TIMEOUT = -5,       /* device-side bounded wait expired (status_word only) */
    GDN_ERR_TOO_LARGE = -6      /* more requests than the built-in scratch of the no-allocation entry holds */
} gdn_status;

typedef enum { GDN_F32 = 0, GDN_BF16 = 1 } gdn_dtype;
typedef enum { GDN_MEM_DEVICE = 0, GDN_MEM_HOST = 1 } gdn_memory;

/* Which kernel family runs the recurrence. */
typedef enum {
    GDN_KERNEL_AUTO = 0,        /* tensor-core path when the shape allows it, else the fp32 path */
    GDN_KERNEL_FP32_SIMT = 1,   /* token-recurrent, all-fp32 FFMA; any supported shape and dtype */
    GDN_KERNEL_TCGEN05 = 2      /* chunkwise WY form on tcgen05/TMEM; bf16, dk = dv = 128, chunk 64 */
} gdn_kernel;

/* What the q, k, g and beta arguments of the forward calls hold. */
typedef enum {
    GDN_INPUT_READY = 0,        /* q, k as they enter Eq. 1 (normalised by the caller), g = log alpha, beta */
    GDN_INPUT_RAW = 1           /* raw projection outputs; the kernels apply the input stage themselves, see below */
} gdn_input_stage;

typedef struct gdn_desc {
    int32_t  num_qk_heads;      /* Hq */
    int32_t  num_v_heads;       /* Hv, a multiple of Hq */
    int32_t  head_k_dim;        /* dk: 64 or 128 */
    int32_t  head_v_dim;        /* dv: 64 or 128 */
    int32_t  io_dtype;          /* gdn_dtype of q, k, v, out_o */
    int32_t  num_seqs;          /* N */
    int64_t  total_tokens;      /* T = cu_tail_lens[N]; known to the caller, so no device sync */
    int32_t  memory;            /* gdn_memory */
    int32_t  kernel;            /* gdn_kernel */
    int32_t  input_stage;       /* gdn_input_stage */
    int32_t  reserved;          /* 0 */
    const float* init_state;    /* optional [N, Hv, dk, dv] fp32 start state; NULL = zero (Eq. 2) */
    void*    workspace;         /* caller-owned device scratch, 256-byte aligned */
    size_t   workspace_bytes;   /* >= gdn_workspace_size(desc) */
    int32_t* status_word;       /* optional device int32; written only on a device-side error */
    void*    stream;            /* cudaStream_t (NULL = the legacy default stream) */
} gdn_desc;

/*
 * Device scratch the two forward calls need for this descriptor (scheduler work list and
 * counter; plus staging for every input and output when desc->memory == GDN_MEM_HOST).
 * Returns 0 for an invalid descriptor.  Host-only; no CUDA call.
 */
GDN_API size_t gdn_workspace_size(const gdn_desc* desc);

/*
 * Tail replay (paper Eq. 2): rebuild each request's per-head state by running Eq. 1 over its
 * tail rows from a zero state, returning o_t for every tail token and the final state.
 * `chunk` is the chunk length of the chunkwise evaluation; the result does not depend on it
 * mathematically; 64 is the supported value.  out_o may be NULL to skip the outputs (state
 * rebuild only); out_state may be NULL to skip the states.
 */
GDN_API int32_t gdn_tail_replay(const gdn_desc* desc, const void* q, const void* k, const void* v,
                        const float* g, const float* beta, const int32_t* cu_tail_lens,
                        int32_t chunk, void* out_o, float* out_state);

/*
 * Fused input stage (desc->input_stage == GDN_INPUT_RAW).  The paper's replay feeds the cached hiddens through the
 * linear-attention layers, "which produce k, v, T and beta at each replay step" (Method section); it fixes neither
 * a normalisation nor a gate parametrisation.  With GDN_INPUT_RAW the forward calls take what the projections put
 * out and apply, in their load path (no extra pass over memory):
 *     q, k   each row (token, head) L2-normalised:  x / sqrt(sum(x^2) + 1e-6)
 *     g      holds the gate pre-activation a:       alpha = sigmoid(a),  i.e. log alpha = -log(1 + exp(-a))
 *     beta   holds the pre-activation b:            beta = sigmoid(b)
 * v is used as it is.  Available in gdn_tail_replay, gdn_full_prefill and gdn_tail_replay_static_scratch on both
 * kernel families; gdn_decode_step takes ready-made inputs only.
 */

/*
 * Full prefill (paper Eq. 1 over the whole matched prefix; the paper's "full" baseline):
 * same arguments and semantics, cu_tail_lens holding whole prefix lengths.
 */
GDN_API int32_t gdn_full_prefill(const gdn_desc* desc, const void* q, const void* k, const void* v,
                         const float* g, const float* beta, const int32_t* cu_tail_lens,
                         int32_t chunk, void* out_o, float* out_state);

/*
 * One decoding step from a given state (paper, Method section: after the replay "the model continues serving the
 * current request ... with the retrieved FA KV and reconstructed linear-attention states", i.e. Eq. 1 continued
 * one token at a time from the rebuilt state).  Every request contributes exactly one token:
 *     q, k [N, Hq, dk], v [N, Hv, dv] in io_dtype; g, beta [N, Hv] fp32;
 *     state_in, state_out [N, Hv, dk, dv] fp32 in the layout of out_state (they may be the same buffer);
 *     out_o [N, Hv, dv] in io_dtype, or NULL.
 * desc supplies the head counts and dims (dk, dv in {64, 128}), io_dtype, num_seqs = N and the stream;
 * total_tokens, workspace, init_state and kernel are ignored.  Device pointers only (GDN_MEM_HOST: UNSUPPORTED).
 * It is gdn_tail_replay with init_state = state_in and one-row requests, as a kernel of its own because it is bound
 * by reading and writing the states once, not by the chunk machinery.
 */
GDN_API int32_t gdn_decode_step(const gdn_desc* desc, const void* q, const void* k, const void* v,
                                const float* g, const float* beta, const float* state_in,
                                void* out_o, float* state_out);

/*
 * Tail replay for callers that have no device memory to hand over as workspace.  (The paper has no
 * counterpart: this entry point exists for integration reasons only.)
 *
 * Who needs it: a serving process that reserved the whole HBM for its own cache pool at start-up and can
 * neither spare a slice for a library nor risk a cudaMalloc in the middle of serving (it may fail outright,
 * and it stalls every stream of the device while it runs); and callers that only hold raw pointers handed
 * down from another runtime's allocator and have no allocator of their own to ask.
 *
 * It is gdn_tail_replay with the scheduler scratch (work counter + longest-first request order) taken from
 * an array that is compiled into the library's device image instead of from desc->workspace, which is
 * ignored together with desc->workspace_bytes.  The array is GDN_STATIC_SCRATCH_BYTES large and is held by
 * every GPU that loads the library until the process exits.  Limits and rules:
 *   - desc->num_seqs <= GDN_STATIC_SCRATCH_MAX_SEQS, otherwise GDN_ERR_TOO_LARGE (nothing is enqueued);
 *   - device pointers only (desc->memory == GDN_MEM_DEVICE), otherwise GDN_ERR_UNSUPPORTED: staging host
 *     buffers would need far more scratch than is built in;
 *   - the first call on each device looks up the array's device address (with that device current) and
 *     caches it; make that first call before starting any stream capture;
 *   - the call itself allocates and frees nothing, on the host side of CUDA or on the device;
 *   - every call on a device shares the one array and the array keeps the previous call's contents; the
 *     scheduler kernel rewrites the counter and the part of the order list it uses before the forward
 *     kernel reads them, so back-to-back calls on one stream are fine, but two calls that overlap on the
 *     GPU (different streams, or different host threads without ordering) race on it and are not allowed.
 * All other arguments, layouts, results and error codes are those of gdn_tail_replay.
 */
#define GDN_STATIC_SCRATCH_MAX_SEQS 4096
#define GDN_STATIC_SCRATCH_BYTES (256 + 4 * GDN_STATIC_SCRATCH_MAX_SEQS)
GDN_API int32_t gdn_tail_replay_static_scratch(const gdn_desc* desc, const void* q, const void* k, const void* v,
                                               const float* g, const float* beta, const int32_t* cu_tail_lens,
                                               int32_t chunk, void* out_o, float* out_state);

/*
 * Replay-window length k = ceil(budget_frac * prefix_len) (paper, Method section); the
 * window is rows [prefix_len - k, prefix_len).  Clamped to [0, prefix_len]; budget_frac >= 1
 * selects the whole prefix.  budget_frac is read as the decimal it was written as (the shortest
 * decimal that converts to the same double) and the ceiling is taken in integer arithmetic, for
 * any prefix_len up to 2^63 - 1: 0.07 * 100 gives 7, not the 8 of a binary64 product.  Returns -1
 * if prefix_len < 0, budget_frac < 0 or budget_frac is NaN.  Host-only.
 */
GDN_API int64_t tail_select(int64_t prefix_len, double budget_frac);

/* Static, human-readable text for a gdn_status value. */
GDN_API const char* gdn_status_string(int32_t status);

/*
 * Testing aid for the bounded device-side waits (no counterpart in the paper).  Every wait inside the
 * tensor-core kernel gives up after `wait_timeout_ns` (default 2 s; 0 restores the default), after which the
 * kernel stops blocking, finishes with unspecified results and writes GDN_ERR_TIMEOUT to desc->status_word.
 * `skip_kq_load_of_chunk` >= 0 makes each CTA leave out the K/Q tile copy of that chunk of its work list, so
 * that the wait for it provably runs out (-1, the default, skips nothing).  Nothing faults or hangs: the
 * point is to exercise the error path with the GPU context staying usable.  Process-wide; not thread-safe
 * against concurrent forward calls.
 */
GDN_API void gdn_test_hooks(uint64_t wait_timeout_ns, int32_t skip_kq_load_of_chunk);

/* Number of kernels the last forward call on this thread enqueued (for launch accounting). */
GDN_API int32_t gdn_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* GDN_TAIL_REPLAY_H_ */

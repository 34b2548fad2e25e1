// Shared declarations of the GDN tail-replay CUDA library (host + device).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "gdn_tail_replay.h"

namespace gdn {

// Device-side view of one forward call; all pointers are device pointers.
struct Problem {
    const void* q;            // [T, Hq, dk] io dtype
    const void* k;            // [T, Hq, dk]
    const void* v;            // [T, Hv, dv]
    const float* g;           // [T, Hv]  log-decay
    const float* beta;        // [T, Hv]
    const int32_t* cu;        // [N + 1]
    const float* init_state;  // [N, Hv, dk, dv] or nullptr
    void* out_o;              // [T, Hv, dv] io dtype or nullptr
    float* out_state;         // [N, Hv, dk, dv] or nullptr
    int32_t* status_word;     // optional device int32
    int32_t num_seqs, Hq, Hv, dk, dv;
    int32_t input_raw;        // 1: q, k un-normalised, g = gate pre-activation, beta = pre-activation (fused input stage)
    int64_t total_tokens;
};

constexpr float kNormEps = 1.0e-6f;   // added to the squared norm of q and k rows in the fused input stage

// Scheduler scratch at the head of the workspace.
struct SchedHeader {
    uint32_t next_item;       // dynamic work counter, reset by the scheduler kernel
    uint32_t pad[63];
};
static_assert(sizeof(SchedHeader) == 256, "header is one 256-byte line");

// Work list: requests ordered longest-first (paper is silent on scheduling; ragged tails from
// concurrent cache hits differ up to 8x in length, so long chains must start first).
struct Sched {
    SchedHeader* header;
    int32_t* order;           // [N] request indices, longest first; null: the requests in the order given (the
                              // tensor-core path with a single request, which then needs no scheduler kernel)
};

cudaError_t launch_scheduler(const int32_t* cu, int32_t num_seqs, const Sched& s, cudaStream_t stream);
cudaError_t launch_simt(const Problem& p, const Sched& s, int io_dtype, cudaStream_t stream, int* launches);
// Whether the tensor-core path can run this problem; launch_tcgen05 returns cudaErrorNotSupported when it cannot.
bool tcgen05_supported(const Problem& p);
cudaError_t launch_tcgen05(const Problem& p, const Sched& s, cudaStream_t stream, int* launches);
// One token per request from a given state (state_in and state_out may alias).
cudaError_t launch_decode(const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const float* state_in, float* state_out, void* out_o, int32_t num_seqs, int32_t Hq,
                          int32_t Hv, int32_t dk, int32_t dv, int io_dtype, cudaStream_t stream);

}  // namespace gdn

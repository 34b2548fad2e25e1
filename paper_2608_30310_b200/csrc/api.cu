// C-ABI entry points: argument validation, workspace carving, host staging and dispatch.
// Every step of the path itself runs in the kernels of sched.cu, gdn_simt.cu and gdn_tc.cu.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <mutex>
#include "common.cuh"

namespace {

// Built-in scheduler scratch of gdn_tail_replay_static_scratch: lives in the library's device image, one
// copy per GPU that loads it.  In host code this name is only a handle for cudaGetSymbolAddress, never a
// device address.
static __device__ __align__(256) unsigned char g_static_scratch[GDN_STATIC_SCRATCH_BYTES];
static_assert(GDN_STATIC_SCRATCH_BYTES == sizeof(gdn::SchedHeader) + sizeof(int32_t) * GDN_STATIC_SCRATCH_MAX_SEQS,
              "built-in scratch = scheduler header + one order entry per request");
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};
std::mutex g_static_scratch_mutex;

thread_local int g_last_launches = 0;

inline size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t io_size(int32_t dt) { return dt == GDN_BF16 ? 2 : 4; }

struct Sizes {
    size_t qk, v, gb, cu, o, state;       // bytes of each array
};

bool desc_shape_ok(const gdn_desc* d)
{
    if (!d) return false;
    if (d->num_qk_heads <= 0 || d->num_v_heads <= 0) return false;
    if (d->num_v_heads % d->num_qk_heads != 0) return false;
    if (d->num_seqs < 0 || d->total_tokens < 0 || d->total_tokens > 0x7fffffffLL) return false;
    if (d->io_dtype != GDN_F32 && d->io_dtype != GDN_BF16) return false;
    if (d->memory != GDN_MEM_DEVICE && d->memory != GDN_MEM_HOST) return false;
    if (d->input_stage != GDN_INPUT_READY && d->input_stage != GDN_INPUT_RAW) return false;
    if (d->head_k_dim <= 0 || d->head_v_dim <= 0) return false;
    return true;
}

Sizes sizes_of(const gdn_desc* d)
{
    Sizes s;
    const size_t T = (size_t)d->total_tokens, N = (size_t)d->num_seqs;
    s.qk = T * d->num_qk_heads * d->head_k_dim * io_size(d->io_dtype);
    s.v = T * d->num_v_heads * d->head_v_dim * io_size(d->io_dtype);
    s.gb = T * d->num_v_heads * sizeof(float);
    s.cu = (N + 1) * sizeof(int32_t);
    s.o = s.v;
    s.state = N * d->num_v_heads * d->head_k_dim * d->head_v_dim * sizeof(float);
    return s;
}

size_t sched_bytes(const gdn_desc* d)
{
    return sizeof(gdn::SchedHeader) + round256((size_t)(d->num_seqs > 0 ? d->num_seqs : 1) * sizeof(int32_t));
}

// Scheduler + forward kernel of one (sub-)batch on `stream`; sets the launch count of this thread.
int32_t run_kernels(gdn::Problem& p, gdn::Sched sched, bool use_tc, int32_t kernel, int32_t io_dtype, cudaStream_t stream)
{
    g_last_launches = 0;
    // A single request needs no ordering: the tensor-core path then runs without the scheduler kernel, which
    // matters for the batch-1 state rebuild (one call per layer, a few microseconds each).
    if (use_tc && p.num_seqs == 1 && p.total_tokens > 0 && gdn::tcgen05_supported(p)) {
        sched.order = nullptr;
    } else {
        if (gdn::launch_scheduler(p.cu, p.num_seqs, sched, stream) != cudaSuccess) return GDN_ERR_CUDA;
        g_last_launches += 1;
    }
    cudaError_t e = cudaErrorNotSupported;
    if (use_tc && p.total_tokens > 0) {                       // (a batch of empty requests only gets its states filled in)
        e = gdn::launch_tcgen05(p, sched, stream, &g_last_launches);
        if (e == cudaErrorNotSupported && kernel == GDN_KERNEL_TCGEN05) return GDN_ERR_UNSUPPORTED;
    }
    if (e == cudaErrorNotSupported) e = gdn::launch_simt(p, sched, io_dtype, stream, &g_last_launches);
    if (e == cudaErrorNotSupported) return GDN_ERR_UNSUPPORTED;
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

// Copy streams and events of the host-memory mode, made once per device on its first host-memory call (host-side
// objects only: no device memory is allocated).
constexpr int kMaxGroups = 16;
struct HostPipe {
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_start, ev_done, ev_in[kMaxGroups], ev_k[kMaxGroups];
};
HostPipe* host_pipe()
{
    static HostPipe pipes[kMaxDevices];
    static bool ready[kMaxDevices] = {};
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!ready[dev]) {
        HostPipe& hp = pipes[dev];
        bool ok = cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.ev_done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kMaxGroups; ++i)
            ok = cudaEventCreateWithFlags(&hp.ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.ev_k[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        ready[dev] = true;
    }
    return &pipes[dev];
}

int32_t forward(const gdn_desc* d, const void* q, const void* k, const void* v, const float* g,
                const float* beta, const int32_t* cu, int32_t chunk, void* out_o, float* out_state)
{
    g_last_launches = 0;
    if (!desc_shape_ok(d)) return GDN_ERR_INVALID_ARG;
    if (!q || !k || !v || !g || !beta || !cu) return GDN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(out_o) || !aligned16(out_state) || !aligned16(d->init_state))
        return GDN_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(cu) & 3u) != 0) return GDN_ERR_INVALID_ARG;
    const bool dims_ok = (d->head_k_dim == 64 || d->head_k_dim == 128) &&
                         (d->head_v_dim == 64 || d->head_v_dim == 128);
    if (!dims_ok) return GDN_ERR_UNSUPPORTED;
    if (chunk != 64) return GDN_ERR_UNSUPPORTED;
    if (d->kernel != GDN_KERNEL_AUTO && d->kernel != GDN_KERNEL_FP32_SIMT && d->kernel != GDN_KERNEL_TCGEN05)
        return GDN_ERR_INVALID_ARG;
    const bool tc_shape = d->io_dtype == GDN_BF16 && d->head_k_dim == 128 && d->head_v_dim == 128;
    if (d->kernel == GDN_KERNEL_TCGEN05 && !tc_shape) return GDN_ERR_UNSUPPORTED;
    if (d->num_seqs == 0) return GDN_OK;
    const size_t need = gdn_workspace_size(d);
    if (!d->workspace || d->workspace_bytes < need) return GDN_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(d->workspace) & 255u) != 0) return GDN_ERR_INVALID_ARG;
    if (d->memory == GDN_MEM_HOST) {
        // host arrays can be checked for consistency before anything is enqueued
        if (cu[0] != 0 || (int64_t)cu[d->num_seqs] != d->total_tokens) return GDN_ERR_INVALID_ARG;
        for (int32_t n = 0; n < d->num_seqs; ++n)
            if (cu[n + 1] < cu[n]) return GDN_ERR_INVALID_ARG;
    }

    cudaStream_t stream = (cudaStream_t)d->stream;
    char* ws = (char*)d->workspace;
    gdn::Sched sched;
    sched.header = (gdn::SchedHeader*)ws;
    sched.order = (int32_t*)(ws + sizeof(gdn::SchedHeader));
    ws += sched_bytes(d);

    gdn::Problem p;
    memset(&p, 0, sizeof p);
    p.num_seqs = d->num_seqs; p.Hq = d->num_qk_heads; p.Hv = d->num_v_heads;
    p.dk = d->head_k_dim; p.dv = d->head_v_dim; p.total_tokens = d->total_tokens;
    p.status_word = d->status_word;
    p.input_raw = d->input_stage == GDN_INPUT_RAW ? 1 : 0;
    const bool use_tc = tc_shape && d->kernel != GDN_KERNEL_FP32_SIMT;

    if (d->memory == GDN_MEM_DEVICE) {
        p.q = q; p.k = k; p.v = v; p.g = g; p.beta = beta; p.cu = cu;
        p.init_state = d->init_state; p.out_o = out_o; p.out_state = out_state;
        return run_kernels(p, sched, use_tc, d->kernel, d->io_dtype, stream);
    }

    // ---- host memory: staged through the workspace and pipelined by groups of requests over three streams: the
    // inputs of group i + 1 go host -> device on a copy stream while group i computes on the caller's stream and the
    // results of group i - 1 go device -> host on a second copy stream (the two directions of the link are independent).
    HostPipe* hp = host_pipe();
    if (!hp) return GDN_ERR_CUDA;
    const Sizes sz = sizes_of(d);
    auto carve = [&](size_t bytes) -> char* { char* r = ws; ws += round256(bytes); return r; };
    char* cu_d = carve(sz.cu);
    char* q_d = carve(sz.qk); char* k_d = carve(sz.qk); char* v_d = carve(sz.v);
    char* g_d = carve(sz.gb); char* b_d = carve(sz.gb);
    char* init_d = d->init_state ? carve(sz.state) : nullptr;
    char* o_d = out_o ? carve(sz.o) : nullptr;
    char* st_d = out_state ? carve(sz.state) : nullptr;
    p.cu = (const int32_t*)cu_d; p.q = q_d; p.k = k_d; p.v = v_d; p.g = (const float*)g_d; p.beta = (const float*)b_d;

    // Request groups by token count.  The link into the device is the busy resource from the first copy to the last, so
    // what a schedule can save is its tail: the compute and the copy back of the last group.  Six equal groups take
    // 86 % of the tokens, the last three 8 %, 4 % and 2 %; fewer, larger copies also mean fewer copy launches.
    const int32_t N = d->num_seqs;
    int32_t bounds[kMaxGroups + 1];
    int ngroups = 0;
    {
        static const double cum[] = {0.1433, 0.2867, 0.43, 0.5733, 0.7167, 0.86, 0.94, 0.98};
        const int64_t T = d->total_tokens;
        bounds[0] = 0;
        for (double f : cum) {
            const int64_t target = (int64_t)(f * (double)T);
            int32_t n = bounds[ngroups];
            while (n < N && cu[n] < target) ++n;
            if (n > bounds[ngroups] && n < N) bounds[++ngroups] = n;
        }
        bounds[++ngroups] = N;
    }
    const size_t row_qk = (size_t)d->num_qk_heads * d->head_k_dim * io_size(d->io_dtype);
    const size_t row_v = (size_t)d->num_v_heads * d->head_v_dim * io_size(d->io_dtype);
    const size_t state1 = (size_t)d->num_v_heads * d->head_k_dim * d->head_v_dim * sizeof(float);

    cudaError_t err = cudaEventRecord(hp->ev_start, stream);     // earlier work on the caller's stream (and the last
    if (err == cudaSuccess) err = cudaStreamWaitEvent(hp->s_in, hp->ev_start, 0);   // call's use of the workspace) first
    if (err == cudaSuccess) err = cudaStreamWaitEvent(hp->s_out, hp->ev_start, 0);
    if (err == cudaSuccess) err = cudaMemcpyAsync(cu_d, cu, sz.cu, cudaMemcpyHostToDevice, hp->s_in);
    auto copy = [&](void* dst, const void* src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st) {
        if (err == cudaSuccess && bytes) err = cudaMemcpyAsync(dst, src, bytes, kind, st);
    };
    // the small per-token arrays go in whole (1 / 64 of the input bytes at d = 128), the large ones group by group
    copy(g_d, g, sz.gb, cudaMemcpyHostToDevice, hp->s_in);
    copy(b_d, beta, sz.gb, cudaMemcpyHostToDevice, hp->s_in);
    int32_t status = GDN_OK;
    for (int gi = 0; gi < ngroups && err == cudaSuccess && status == GDN_OK; ++gi) {
        const int32_t n0 = bounds[gi], n1 = bounds[gi + 1];
        const size_t r0 = (size_t)cu[n0], rows = (size_t)cu[n1] - r0;
        copy(q_d + r0 * row_qk, (const char*)q + r0 * row_qk, rows * row_qk, cudaMemcpyHostToDevice, hp->s_in);
        copy(k_d + r0 * row_qk, (const char*)k + r0 * row_qk, rows * row_qk, cudaMemcpyHostToDevice, hp->s_in);
        copy(v_d + r0 * row_v, (const char*)v + r0 * row_v, rows * row_v, cudaMemcpyHostToDevice, hp->s_in);
        if (init_d)
            copy(init_d + n0 * state1, (const char*)d->init_state + n0 * state1, (n1 - n0) * state1, cudaMemcpyHostToDevice, hp->s_in);
        if (err == cudaSuccess) err = cudaEventRecord(hp->ev_in[gi], hp->s_in);
        if (err == cudaSuccess) err = cudaStreamWaitEvent(stream, hp->ev_in[gi], 0);
        if (err != cudaSuccess) break;
        gdn::Problem pg = p;
        pg.cu = p.cu + n0; pg.num_seqs = n1 - n0;
        // The rows of later groups are still on their way: the group sees the arrays only up to its own last row, so
        // that the tile that hangs over the end reads zeros instead of whatever the workspace held before.
        pg.total_tokens = (int64_t)cu[n1];
        pg.init_state = init_d ? (const float*)(init_d + n0 * state1) : nullptr;
        pg.out_o = o_d; pg.out_state = st_d ? (float*)(st_d + n0 * state1) : nullptr;
        gdn::Sched sg = sched;
        sg.order = sched.order + n0;
        const int before = g_last_launches;
        status = run_kernels(pg, sg, use_tc, d->kernel, d->io_dtype, stream);
        g_last_launches += before;
        if (status != GDN_OK) break;
        err = cudaEventRecord(hp->ev_k[gi], stream);
        if (err == cudaSuccess) err = cudaStreamWaitEvent(hp->s_out, hp->ev_k[gi], 0);
        if (out_o) copy((char*)out_o + r0 * row_v, o_d + r0 * row_v, rows * row_v, cudaMemcpyDeviceToHost, hp->s_out);
        if (out_state)
            copy((char*)out_state + n0 * state1, st_d + n0 * state1, (n1 - n0) * state1, cudaMemcpyDeviceToHost, hp->s_out);
    }
    // the caller's stream ends the call: it has the results once the last copy back is done
    cudaError_t e2 = cudaEventRecord(hp->ev_done, hp->s_out);
    if (e2 == cudaSuccess) e2 = cudaStreamWaitEvent(stream, hp->ev_done, 0);
    if (status != GDN_OK) return status;
    if (err != cudaSuccess || e2 != cudaSuccess) return GDN_ERR_CUDA;
    return GDN_OK;
}

}  // namespace

extern "C" {

size_t gdn_workspace_size(const gdn_desc* d)
{
    if (!desc_shape_ok(d)) return 0;
    size_t total = sched_bytes(d);
    if (d->memory == GDN_MEM_HOST) {
        const Sizes s = sizes_of(d);
        total += round256(s.cu) + 2 * round256(s.qk) + round256(s.v) + 2 * round256(s.gb) +
                 round256(s.o) + 2 * round256(s.state);
    }
    return total;
}

int32_t gdn_tail_replay(const gdn_desc* desc, const void* q, const void* k, const void* v,
                        const float* g, const float* beta, const int32_t* cu_tail_lens,
                        int32_t chunk, void* out_o, float* out_state)
{
    return forward(desc, q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state);
}

int32_t gdn_full_prefill(const gdn_desc* desc, const void* q, const void* k, const void* v,
                         const float* g, const float* beta, const int32_t* cu_tail_lens,
                         int32_t chunk, void* out_o, float* out_state)
{
    // Same function on longer rows; the persistent kernels size their grid from the chain count,
    // so a few very long chains simply occupy fewer SMs.
    return forward(desc, q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state);
}

int32_t gdn_tail_replay_static_scratch(const gdn_desc* desc, const void* q, const void* k, const void* v,
                                       const float* g, const float* beta, const int32_t* cu_tail_lens,
                                       int32_t chunk, void* out_o, float* out_state)
{
    if (!desc) return GDN_ERR_INVALID_ARG;
    if (desc->memory != GDN_MEM_DEVICE) return GDN_ERR_UNSUPPORTED;
    if (desc->num_seqs > GDN_STATIC_SCRATCH_MAX_SEQS) return GDN_ERR_TOO_LARGE;
    if (desc->num_seqs <= 0) return forward(desc, q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GDN_ERR_CUDA;
    void* scratch = nullptr;
    {
        // one-time set-up per device: resolve the array's address on the current device
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        if (!g_static_scratch_addr[dev]) {
            void* addr = nullptr;
            if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return GDN_ERR_CUDA;
            g_static_scratch_addr[dev] = addr;
        }
        scratch = g_static_scratch_addr[dev];
    }
    gdn_desc d = *desc;
    d.workspace = scratch;
    d.workspace_bytes = GDN_STATIC_SCRATCH_BYTES;
    return forward(&d, q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state);
}

int32_t gdn_decode_step(const gdn_desc* d, const void* q, const void* k, const void* v, const float* g,
                        const float* beta, const float* state_in, void* out_o, float* state_out)
{
    g_last_launches = 0;
    if (!desc_shape_ok(d)) return GDN_ERR_INVALID_ARG;
    if (!q || !k || !v || !g || !beta || !state_in || !state_out) return GDN_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) || !aligned16(beta) ||
        !aligned16(state_in) || !aligned16(state_out) || !aligned16(out_o))
        return GDN_ERR_INVALID_ARG;
    const bool dims_ok = (d->head_k_dim == 64 || d->head_k_dim == 128) && (d->head_v_dim == 64 || d->head_v_dim == 128);
    if (!dims_ok) return GDN_ERR_UNSUPPORTED;
    if (d->memory != GDN_MEM_DEVICE) return GDN_ERR_UNSUPPORTED;
    if (d->num_seqs == 0) return GDN_OK;
    const cudaError_t e = gdn::launch_decode(q, k, v, g, beta, state_in, state_out, out_o, d->num_seqs, d->num_qk_heads,
                                             d->num_v_heads, d->head_k_dim, d->head_v_dim, d->io_dtype,
                                             (cudaStream_t)d->stream);
    if (e == cudaErrorNotSupported) return GDN_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return GDN_ERR_CUDA;
    g_last_launches = 1;
    return GDN_OK;
}

int64_t tail_select(int64_t prefix_len, double budget_frac)
{
    if (prefix_len < 0 || budget_frac != budget_frac || budget_frac < 0.0) return -1;
    if (budget_frac >= 1.0) return prefix_len;
    if (budget_frac == 0.0 || prefix_len == 0) return 0;
    // The ratio is read as the decimal it was written as: its shortest decimal representation that converts back to
    // the same binary64, digits x 10^-scale.  The ceiling of prefix_len x digits / 10^scale is then taken in integers,
    // so that 0.07 x 100 is 7 and no genuine fraction is lost at any size.
    char buf[40];
    int prec = 1;
    for (; prec <= 17; ++prec) {
        snprintf(buf, sizeof buf, "%.*e", prec - 1, budget_frac);
        if (strtod(buf, nullptr) == budget_frac) break;
    }
    unsigned long long digits = 0;
    const char* c = buf;
    for (; *c && *c != 'e'; ++c)
        if (*c >= '0' && *c <= '9') digits = digits * 10ull + (unsigned long long)(*c - '0');
    const int exp10 = *c == 'e' ? atoi(c + 1) : 0;           // value = d.ddd x 10^exp10 = digits x 10^(exp10 - (prec - 1))
    const int scale = (prec - 1) - exp10;                      // > 0 for a ratio below 1
    const unsigned __int128 num = (unsigned __int128)(unsigned long long)prefix_len * digits;   // < 2^63 x 10^17
    if (scale > 36) return num > 0 ? 1 : 0;                    // 10^scale exceeds any possible numerator
    unsigned __int128 den = 1;
    for (int i = 0; i < scale; ++i) den *= 10u;
    const unsigned __int128 k = (num + den - 1) / den;
    return k > (unsigned __int128)(unsigned long long)prefix_len ? prefix_len : (int64_t)k;
}

const char* gdn_status_string(int32_t status)
{
    switch (status) {
        case GDN_OK: return "ok";
        case GDN_ERR_INVALID_ARG: return "invalid argument";
        case GDN_ERR_UNSUPPORTED: return "unsupported shape, dtype, chunk or kernel";
        case GDN_ERR_WORKSPACE: return "workspace missing or too small";
        case GDN_ERR_CUDA: return "CUDA call failed";
        case GDN_ERR_TIMEOUT: return "device-side wait timed out";
        case GDN_ERR_TOO_LARGE: return "more requests than the built-in scratch holds";
        default: return "unknown status";
    }
}

int32_t gdn_last_launch_count(void) { return g_last_launches; }

}  // extern "C"

// C-ABI entry points: argument validation, workspace carving, host staging and dispatch.
// Every step of the path itself runs in the kernels of sched.cu, gdn_simt.cu and gdn_tc.cu.
#include <math.h>
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

    const Sizes sz = sizes_of(d);
    void* o_stage = nullptr; float* st_stage = nullptr;
    if (d->memory == GDN_MEM_HOST) {
        auto stage_in = [&](const void* src, size_t bytes, cudaError_t& err) -> void* {
            void* dst = ws;
            ws += round256(bytes);
            if (err == cudaSuccess && bytes) err = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, stream);
            return dst;
        };
        cudaError_t err = cudaSuccess;
        p.cu = (const int32_t*)stage_in(cu, sz.cu, err);
        p.q = stage_in(q, sz.qk, err);
        p.k = stage_in(k, sz.qk, err);
        p.v = stage_in(v, sz.v, err);
        p.g = (const float*)stage_in(g, sz.gb, err);
        p.beta = (const float*)stage_in(beta, sz.gb, err);
        if (d->init_state) p.init_state = (const float*)stage_in(d->init_state, sz.state, err);
        if (out_o) { o_stage = ws; ws += round256(sz.o); }
        if (out_state) { st_stage = (float*)ws; ws += round256(sz.state); }
        p.out_o = o_stage; p.out_state = st_stage;
        if (err != cudaSuccess) return GDN_ERR_CUDA;
    } else {
        p.q = q; p.k = k; p.v = v; p.g = g; p.beta = beta; p.cu = cu;
        p.init_state = d->init_state; p.out_o = out_o; p.out_state = out_state;
    }

    const bool use_tc = tc_shape && d->kernel != GDN_KERNEL_FP32_SIMT;
    // A single request needs no ordering: the tensor-core path then runs without the scheduler kernel, which
    // matters for the batch-1 state rebuild (one call per layer, a few microseconds each).
    if (use_tc && p.num_seqs == 1 && gdn::tcgen05_supported(p)) {
        sched.order = nullptr;
    } else {
        if (gdn::launch_scheduler(p.cu, p.num_seqs, sched, stream) != cudaSuccess) return GDN_ERR_CUDA;
        g_last_launches += 1;
    }

    cudaError_t e = cudaErrorNotSupported;
    if (use_tc) {
        e = gdn::launch_tcgen05(p, sched, stream, &g_last_launches);
        if (e == cudaErrorNotSupported && d->kernel == GDN_KERNEL_TCGEN05) return GDN_ERR_UNSUPPORTED;
    }
    if (e == cudaErrorNotSupported) e = gdn::launch_simt(p, sched, d->io_dtype, stream, &g_last_launches);
    if (e == cudaErrorNotSupported) return GDN_ERR_UNSUPPORTED;
    if (e != cudaSuccess) return GDN_ERR_CUDA;

    if (d->memory == GDN_MEM_HOST) {
        cudaError_t err = cudaSuccess;
        if (out_o && sz.o) err = cudaMemcpyAsync(out_o, o_stage, sz.o, cudaMemcpyDeviceToHost, stream);
        if (err == cudaSuccess && out_state && sz.state)
            err = cudaMemcpyAsync(out_state, st_stage, sz.state, cudaMemcpyDeviceToHost, stream);
        if (err != cudaSuccess) return GDN_ERR_CUDA;
    }
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
    const double x = budget_frac * (double)prefix_len;
    const double eps = 1e-9 * fmax(1.0, x);
    int64_t k = (int64_t)ceil(x - eps);
    if (k < 0) k = 0;
    if (k > prefix_len) k = prefix_len;
    return k;
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

// Single-token step of Eq. 1 from a given state: what serving does after the replay, one token per request at a time.
//
// Per chain (request n, v-head h), with H = S^T (dk x dv, fp32, the layout of out_state), a = exp(g), b = beta:
//     r     = H^T k                      (dv)
//     delta = b (v - a r)
//     H'    = a H + k delta^T            (== S a (I - b k k^T) + b v k^T, transposed)
//     o     = H'^T q
// The step reads and writes the whole state once (2 x dk x dv x 4 bytes per chain) and does 6 dk dv flops on it: it
// is bound by HBM bandwidth.  One CTA of 256 threads per chain keeps the state in registers: a thread owns 4
// consecutive value columns of DK / RG rows (16-byte loads and stores, a warp covers whole 512-byte rows), the two
// reductions over rows go through shared memory.
#include "common.cuh"

namespace gdn {

template <typename T> __device__ __forceinline__ float dec_to_f32(T x);
template <> __device__ __forceinline__ float dec_to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float dec_to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T dec_from_f32(float x);
template <> __device__ __forceinline__ float dec_from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 dec_from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

struct DecodeArgs {
    const void* q; const void* k; const void* v;      // [N, Hq, dk], [N, Hq, dk], [N, Hv, dv]
    const float* g; const float* beta;                // [N, Hv]
    const float* state_in; float* state_out;          // [N, Hv, dk, dv]; may alias
    void* out_o;                                      // [N, Hv, dv] or nullptr
    int32_t num_seqs, Hq, Hv;
};

template <int DK, int DV, typename T>
__global__ void __launch_bounds__(256)
gdn_decode_kernel(const DecodeArgs a)
{
    constexpr int CG = DV / 4;             // threads across one state row (4 columns each)
    constexpr int RG = 256 / CG;           // row groups
    constexpr int RPT = DK / RG;           // rows per thread
    __shared__ __align__(16) float part[RG][DV];
    __shared__ float ks[DK], qs[DK];
    __shared__ __align__(16) float dl[DV];

    const int tid = threadIdx.x, cg = tid % CG, rg = tid / CG;
    const int chain = blockIdx.x, n = chain / a.Hv, h = chain % a.Hv, hq = h / (a.Hv / a.Hq);
    const T* __restrict__ qg = reinterpret_cast<const T*>(a.q) + ((size_t)n * a.Hq + hq) * DK;
    const T* __restrict__ kg = reinterpret_cast<const T*>(a.k) + ((size_t)n * a.Hq + hq) * DK;
    const T* __restrict__ vg = reinterpret_cast<const T*>(a.v) + ((size_t)n * a.Hv + h) * DV;
    const float* Hin = a.state_in + (size_t)chain * DK * DV;      // may be the same memory as Hout: every thread
    float* Hout = a.state_out + (size_t)chain * DK * DV;          // writes only the entries it has read itself

    // the state first: these loads are the kernel
    float4 Hr[RPT];
#pragma unroll
    for (int i = 0; i < RPT; ++i)
        Hr[i] = *reinterpret_cast<const float4*>(Hin + (size_t)(rg * RPT + i) * DV + 4 * cg);
    if (tid < DK) { ks[tid] = dec_to_f32<T>(kg[tid]); qs[tid] = dec_to_f32<T>(qg[tid]); }
    const float alpha = __expf(a.g[(size_t)n * a.Hv + h]);
    const float b = a.beta[(size_t)n * a.Hv + h];
    __syncthreads();

    // r = H^T k: partial sums over this thread's rows, then over the row groups
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const float kk = ks[rg * RPT + i];
        acc.x = fmaf(Hr[i].x, kk, acc.x); acc.y = fmaf(Hr[i].y, kk, acc.y);
        acc.z = fmaf(Hr[i].z, kk, acc.z); acc.w = fmaf(Hr[i].w, kk, acc.w);
    }
    *reinterpret_cast<float4*>(&part[rg][4 * cg]) = acc;
    __syncthreads();
    if (tid < DV) {
        float r = 0.f;
#pragma unroll
        for (int j = 0; j < RG; ++j) r += part[j][tid];
        dl[tid] = b * (dec_to_f32<T>(vg[tid]) - alpha * r);
    }
    __syncthreads();

    // H' = a H + k delta^T, stored; o = H'^T q accumulated on the way
    const float4 d4 = *reinterpret_cast<const float4*>(&dl[4 * cg]);
    acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const float kk = ks[rg * RPT + i], qq = qs[rg * RPT + i];
        float4 x = Hr[i];
        x.x = fmaf(alpha, x.x, kk * d4.x); x.y = fmaf(alpha, x.y, kk * d4.y);
        x.z = fmaf(alpha, x.z, kk * d4.z); x.w = fmaf(alpha, x.w, kk * d4.w);
        *reinterpret_cast<float4*>(Hout + (size_t)(rg * RPT + i) * DV + 4 * cg) = x;
        acc.x = fmaf(x.x, qq, acc.x); acc.y = fmaf(x.y, qq, acc.y);
        acc.z = fmaf(x.z, qq, acc.z); acc.w = fmaf(x.w, qq, acc.w);
    }
    if (a.out_o) {
        *reinterpret_cast<float4*>(&part[rg][4 * cg]) = acc;      // (every thread has read its part of r by now)
        __syncthreads();
        if (tid < DV) {
            float o = 0.f;
#pragma unroll
            for (int j = 0; j < RG; ++j) o += part[j][tid];
            reinterpret_cast<T*>(a.out_o)[((size_t)n * a.Hv + h) * DV + tid] = dec_from_f32<T>(o);
        }
    }
}

template <int DK, int DV>
static cudaError_t launch_dtype(const DecodeArgs& a, int io_dtype, cudaStream_t stream)
{
    const unsigned grid = (unsigned)a.num_seqs * (unsigned)a.Hv;
    if (io_dtype == GDN_BF16) gdn_decode_kernel<DK, DV, __nv_bfloat16><<<grid, 256, 0, stream>>>(a);
    else gdn_decode_kernel<DK, DV, float><<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_decode(const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const float* state_in, float* state_out, void* out_o, int32_t num_seqs, int32_t Hq,
                          int32_t Hv, int32_t dk, int32_t dv, int io_dtype, cudaStream_t stream)
{
    DecodeArgs a;
    a.q = q; a.k = k; a.v = v; a.g = g; a.beta = beta; a.state_in = state_in; a.state_out = state_out; a.out_o = out_o;
    a.num_seqs = num_seqs; a.Hq = Hq; a.Hv = Hv;
    if (dk == 128 && dv == 128) return launch_dtype<128, 128>(a, io_dtype, stream);
    if (dk == 64 && dv == 128) return launch_dtype<64, 128>(a, io_dtype, stream);
    if (dk == 128 && dv == 64) return launch_dtype<128, 64>(a, io_dtype, stream);
    if (dk == 64 && dv == 64) return launch_dtype<64, 64>(a, io_dtype, stream);
    return cudaErrorNotSupported;
}

}  // namespace gdn

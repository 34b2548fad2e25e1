// fp32 path of the GDN forward: token-recurrent evaluation of Eq. 1 with plain FFMA.
//
// One CTA walks one chain (request n, v-head h) at a time.  The dv x dk state S lives in
// registers: thread (j, part) owns 32 entries of row j of S.  Per token, with the state before
// the token S' and a = alpha_t, b = beta_t:
//     r = S' k,  p = S' q                      (row dot products, reduced over the row's threads)
//     delta = b (v - a r)
//     S = a S' + delta k^T                      (== S' a (I - b k k^T) + b v k^T, Eq. 1)
//     o = S q = a p + delta (k . q)
// This path serves fp32 io (tolerance 1e-4 rules out tf32/bf16 tensor cores) and every shape
// the tensor-core path does not cover.
#include "common.cuh"

namespace gdn {

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

constexpr int kTokBlock = 16;   // tokens staged in shared memory per step

template <int DK, int DV, typename T>
__global__ void __launch_bounds__(DV * (DK / 32))
gdn_simt_kernel(const Problem p, const Sched s)
{
    constexpr int TPR = DK / 32;           // threads per state row
    constexpr int NT = DV * TPR;
    constexpr int R = 32;                   // state entries per thread
    __shared__ __align__(16) float ks[kTokBlock][DK];
    __shared__ __align__(16) float qs[kTokBlock][DK];
    __shared__ float vs[kTokBlock][DV];
    __shared__ float os[kTokBlock][DV];
    __shared__ float as[kTokBlock], bs[kTokBlock], kqs[kTokBlock];
    __shared__ uint32_t item_s;

    const int tid = threadIdx.x;
    const int j = tid / TPR;               // state row (dv index)
    const int part = tid % TPR;            // which interleaved slice of dk
    const int lane = tid & 31, warp = tid >> 5;
    const int G = p.Hv / p.Hq;
    const uint32_t num_items = (uint32_t)p.num_seqs * (uint32_t)p.Hv;
    const T* __restrict__ qg = (const T*)p.q;
    const T* __restrict__ kg = (const T*)p.k;
    const T* __restrict__ vg = (const T*)p.v;
    T* __restrict__ og = (T*)p.out_o;

    for (;;) {
        if (tid == 0) item_s = atomicAdd(&s.header->next_item, 1u);
        __syncthreads();
        const uint32_t item = item_s;
        __syncthreads();
        if (item >= num_items) break;
        const int n = s.order[item / p.Hv];
        const int h = item % p.Hv;
        const int hq = h / G;
        const int64_t row_begin = p.cu[n], row_end = p.cu[n + 1];
        const size_t state_off = ((size_t)n * p.Hv + h) * DK * DV;

        float S[R];
        if (p.init_state) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int d = part * 4 + (r >> 2) * 4 * TPR + (r & 3);
                S[r] = p.init_state[state_off + (size_t)d * DV + j];
            }
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r) S[r] = 0.f;
        }

        for (int64_t row0 = row_begin; row0 < row_end; row0 += kTokBlock) {
            const int nvalid = (int)min((int64_t)kTokBlock, row_end - row0);
            // stage q, k, v, decay and beta of this token block
            for (int idx = tid; idx < kTokBlock * DK; idx += NT) {
                const int t = idx / DK, d = idx % DK;
                float kv = 0.f, qv = 0.f;
                if (t < nvalid) {
                    const size_t off = ((size_t)(row0 + t) * p.Hq + hq) * DK + d;
                    kv = to_f32<T>(kg[off]);
                    qv = to_f32<T>(qg[off]);
                }
                ks[t][d] = kv;
                qs[t][d] = qv;
            }
            for (int idx = tid; idx < kTokBlock * DV; idx += NT) {
                const int t = idx / DV, d = idx % DV;
                vs[t][d] = (t < nvalid) ? to_f32<T>(vg[((size_t)(row0 + t) * p.Hv + h) * DV + d]) : 0.f;
            }
            if (tid < kTokBlock) {
                const bool ok = tid < nvalid;
                const float gin = ok ? p.g[(size_t)(row0 + tid) * p.Hv + h] : 0.f;
                const float bin = ok ? p.beta[(size_t)(row0 + tid) * p.Hv + h] : 0.f;
                if (p.input_raw) {
                    // fused input stage: alpha = sigmoid(gate), beta = sigmoid(pre-activation)
                    as[tid] = ok ? 1.f / (1.f + expf(-gin)) : 1.f;
                    bs[tid] = ok ? 1.f / (1.f + expf(-bin)) : 0.f;
                } else {
                    as[tid] = ok ? expf(gin) : 1.f;
                    bs[tid] = bin;
                }
            }
            __syncthreads();
            if (p.input_raw) {
                // fused input stage: q and k rows L2-normalised, x / sqrt(sum x^2 + eps)
                for (int t = warp; t < kTokBlock; t += NT / 32) {
                    float sk = 0.f, sq = 0.f;
                    for (int d = lane; d < DK; d += 32) { sk = fmaf(ks[t][d], ks[t][d], sk); sq = fmaf(qs[t][d], qs[t][d], sq); }
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) {
                        sk += __shfl_xor_sync(0xffffffffu, sk, off);
                        sq += __shfl_xor_sync(0xffffffffu, sq, off);
                    }
                    const float rk = rsqrtf(sk + kNormEps), rq = rsqrtf(sq + kNormEps);
                    for (int d = lane; d < DK; d += 32) { ks[t][d] *= rk; qs[t][d] *= rq; }
                }
                __syncthreads();
            }
            for (int t = warp; t < kTokBlock; t += NT / 32) {
                float acc = 0.f;
                for (int d = lane; d < DK; d += 32) acc = fmaf(ks[t][d], qs[t][d], acc);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
                if (lane == 0) kqs[t] = acc;
            }
            __syncthreads();

            for (int tt = 0; tt < nvalid; ++tt) {
                const float a = as[tt], b = bs[tt];
                float r = 0.f, pq = 0.f;
#pragma unroll
                for (int i = 0; i < R / 4; ++i) {
                    const float4 k4 = *reinterpret_cast<const float4*>(&ks[tt][part * 4 + i * 4 * TPR]);
                    const float4 q4 = *reinterpret_cast<const float4*>(&qs[tt][part * 4 + i * 4 * TPR]);
                    r = fmaf(S[4 * i + 0], k4.x, r); pq = fmaf(S[4 * i + 0], q4.x, pq);
                    r = fmaf(S[4 * i + 1], k4.y, r); pq = fmaf(S[4 * i + 1], q4.y, pq);
                    r = fmaf(S[4 * i + 2], k4.z, r); pq = fmaf(S[4 * i + 2], q4.z, pq);
                    r = fmaf(S[4 * i + 3], k4.w, r); pq = fmaf(S[4 * i + 3], q4.w, pq);
                }
#pragma unroll
                for (int off = 1; off < TPR; off <<= 1) {
                    r += __shfl_xor_sync(0xffffffffu, r, off);
                    pq += __shfl_xor_sync(0xffffffffu, pq, off);
                }
                const float delta = b * (vs[tt][j] - a * r);
#pragma unroll
                for (int i = 0; i < R / 4; ++i) {
                    const float4 k4 = *reinterpret_cast<const float4*>(&ks[tt][part * 4 + i * 4 * TPR]);
                    S[4 * i + 0] = fmaf(a, S[4 * i + 0], delta * k4.x);
                    S[4 * i + 1] = fmaf(a, S[4 * i + 1], delta * k4.y);
                    S[4 * i + 2] = fmaf(a, S[4 * i + 2], delta * k4.z);
                    S[4 * i + 3] = fmaf(a, S[4 * i + 3], delta * k4.w);
                }
                if (part == 0) os[tt][j] = fmaf(a, pq, delta * kqs[tt]);
            }
            __syncthreads();
            if (og) {
                for (int idx = tid; idx < nvalid * DV; idx += NT) {
                    const int t = idx / DV, d = idx % DV;
                    og[((size_t)(row0 + t) * p.Hv + h) * DV + d] = from_f32<T>(os[t][d]);
                }
            }
            __syncthreads();
        }

        if (p.out_state) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int d = part * 4 + (r >> 2) * 4 * TPR + (r & 3);
                p.out_state[state_off + (size_t)d * DV + j] = S[r];
            }
        }
    }
}

template <int DK, int DV, typename T>
static cudaError_t launch_one(const Problem& p, const Sched& s, cudaStream_t stream)
{
    constexpr int NT = DV * (DK / 32);
    int dev = 0, sms = 0, per_sm = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gdn_simt_kernel<DK, DV, T>, NT, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const long long items = (long long)p.num_seqs * p.Hv;
    long long grid = (long long)sms * per_sm;
    if (grid > items) grid = items;
    if (grid < 1) grid = 1;
    gdn_simt_kernel<DK, DV, T><<<(unsigned)grid, NT, 0, stream>>>(p, s);
    return cudaGetLastError();
}

cudaError_t launch_simt(const Problem& p, const Sched& s, int io_dtype, cudaStream_t stream, int* launches)
{
    cudaError_t e = cudaErrorNotSupported;
#define GDN_SIMT_CASE(DKV, DVV)                                                           \
    if (p.dk == DKV && p.dv == DVV)                                                       \
        e = (io_dtype == GDN_BF16) ? launch_one<DKV, DVV, __nv_bfloat16>(p, s, stream)    \
                                   : launch_one<DKV, DVV, float>(p, s, stream);
    GDN_SIMT_CASE(64, 64)
    GDN_SIMT_CASE(64, 128)
    GDN_SIMT_CASE(128, 64)
    GDN_SIMT_CASE(128, 128)
#undef GDN_SIMT_CASE
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}

}  // namespace gdn

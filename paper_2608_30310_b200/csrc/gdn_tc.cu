// Tensor-core path of the GDN forward: chunkwise WY (UT-transform) evaluation of Eq. 1 on
// tcgen05 MMAs with TMEM accumulators and TMA-staged bf16 tiles.  bf16 io, dk = dv = 128, chunk 64.
//
// Everything is kept in the transposed orientation so that every MMA has M = 128 (one TMEM lane
// per value-dimension index i, or per key-dimension index for W): the carried state is
// S (dv x dk, fp32, TMEM-resident), and per chunk of C = 64 tokens with start state S0:
//
//   G_t   = cumsum(g) inside the chunk;  Gam[t,s] = exp(G_t - G_s) (t >= s)
//   Gram  = [K;Q] K^T                        (MMA, 128 x 64: rows 0-63 K K^T, rows 64-127 Q K^T)
//   A     = strict_lower(beta_t Gam (K K^T)),  P = lower_incl(Gam (Q K^T))
//   X     = (I + A)^-1                        (fp32, shared memory, blocked forward substitution)
//   T'    = X diag(beta),  T'' = X diag(beta e^G)
//   W^T   = K^T T''^T                         (MMA, 128(dk) x 64)
//   Dl^T  = V^T T'^T - S0 W^T                 (two MMAs into one accumulator, second negated)
//   O^T   = (S0 Q^T) diag(e^G) + Dl^T P^T     (two MMAs, combined in the epilogue)
//   S     = e^{G_C} S0 + (Dl diag(e^{G_C - G}))^T K    (MMA accumulating onto the pre-scaled state)
//
// One CTA walks one chain (request, v-head) at a time, chains handed out longest-first through an
// atomic counter.  Padding rows of a ragged last chunk get g = 0 and beta = 0, which makes them
// inert (their rows of A, W, U and Delta vanish); their outputs are not stored.
#include <cuda.h>
#include "common.cuh"
#include "ptx.cuh"

namespace gdn {
namespace {

using namespace ptx;

constexpr int LDF = 68;                       // fp32 row stride of the A / X scratch (floats)
constexpr float kLog2e = 1.4426950408889634f;

// ---- shared memory map (bytes from a 1024-aligned base) ---------------------------------------
constexpr uint32_t SM_KQ = 0;                 // 2 halves x [128 rows: K 0-63, Q 64-127] x 128 B   32 KB
constexpr uint32_t SM_V = 32768;              // 2 halves x [64 rows] x 128 B                       16 KB
constexpr uint32_t SM_W = 49152;              // W [t][dk] bf16, 2 halves x 64 rows x 128 B         16 KB
constexpr uint32_t SM_TP = 65536;             // T'  [t][s] bf16                                     8 KB
constexpr uint32_t SM_TPP = 73728;            // T'' [t][s] bf16                                     8 KB
constexpr uint32_t SM_P = 81920;              // P   [t][s] bf16                                     8 KB
constexpr uint32_t SM_AF = 90112;             // A fp32 [64][LDF]
constexpr uint32_t SM_XF = SM_AF + 64 * LDF * 4;   // X fp32 [64][LDF]
constexpr uint32_t SM_MF = SM_XF + 64 * LDF * 4;   // 16 x 64 fp32 scratch of the blocked solve
constexpr uint32_t SM_MISC = SM_MF + 16 * 64 * 4;
constexpr uint32_t SM_TOTAL = SM_MISC + 2048;
constexpr uint32_t SMEM_BYTES = SM_TOTAL + 1024;   // slack for the manual 1024-byte alignment

struct Misc {
    float g[64], beta[64], G[64], eG[64], eRest[64];
    unsigned long long bar_tma, bar_mma;
    uint32_t tmem_base, item, abort;
    float eGC;
};
static_assert(sizeof(Misc) <= 2048, "misc block");

// ---- TMEM column map (512 columns x 128 lanes x 32 bit) ----------------------------------------
constexpr uint32_t TM_S32 = 0;      // fp32 state S (dv x dk), 128 columns
constexpr uint32_t TM_SBF = 128;    // bf16 copy of the chunk-start state, 64 columns
constexpr uint32_t TM_ACC1 = 192;   // Delta^T accumulator (U^T - S0 W^T), 64 columns
constexpr uint32_t TM_ACC2 = 256;   // S0 Q^T, 64 columns
constexpr uint32_t TM_ACC3 = 320;   // Delta^T P^T, 64 columns
constexpr uint32_t TM_DBF = 384;    // Delta^T bf16, 32 columns
constexpr uint32_t TM_DPBF = 416;   // (Delta diag(e^{G_C - G}))^T bf16, 32 columns
constexpr uint32_t TM_GRAM = 448;   // Gram accumulator, later W^T accumulator, 64 columns

constexpr uint32_t ID_GRAM = idesc_bf16(128, 64, 0, 0, 0);    // [K;Q] (K-major) x K (K-major)
constexpr uint32_t ID_WU = idesc_bf16(128, 64, 1, 0, 0);      // K^T or V^T (M-major) x T (K-major)
constexpr uint32_t ID_SW = idesc_bf16(128, 64, 0, 0, 1);      // -S0 (TMEM) x W (K-major)
constexpr uint32_t ID_SQ = idesc_bf16(128, 64, 0, 0, 0);      // S0 (TMEM) x Q (K-major)
constexpr uint32_t ID_DP = idesc_bf16(128, 64, 0, 0, 0);      // Delta^T (TMEM) x P (K-major)
constexpr uint32_t ID_DK = idesc_bf16(128, 128, 0, 1, 0);     // Delta'^T (TMEM) x K (N-major)

struct TcParams {
    Problem p;
    Sched s;
    float* debug;     // debug builds only: intermediates of the first chain's first two chunks
};

#ifdef GDN_TC_DEBUG
constexpr int DBG_STRIDE = 61440;
#endif

__global__ void __launch_bounds__(128, 1)
gdn_tc_kernel(const TcParams prm, const __grid_constant__ CUtensorMap tm_q,
              const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v)
{
    extern __shared__ uint8_t smem_raw[];
    const Problem& p = prm.p;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t sb = (raw + 1023u) & ~1023u;           // shared-space address of the aligned base
    uint8_t* sm = smem_raw + (sb - raw);                  // generic pointer to the same place
    Misc* misc = reinterpret_cast<Misc*>(sm + SM_MISC);
    float* AF = reinterpret_cast<float*>(sm + SM_AF);
    float* XF = reinterpret_cast<float*>(sm + SM_XF);
    float* MF = reinterpret_cast<float*>(sm + SM_MF);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t bar_tma = sb + SM_MISC + offsetof(Misc, bar_tma);
    const uint32_t bar_mma = sb + SM_MISC + offsetof(Misc, bar_mma);

    if (warp == 0) {
        tmem_alloc(sb + SM_MISC + offsetof(Misc, tmem_base), 512);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
        misc->abort = 0;
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc->tmem_base;
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);     // this warp's lane window
    uint32_t ph_tma = 0, ph_mma = 0;
    bool aborted = false;

    const int G = p.Hv / p.Hq;
    const uint32_t num_items = (uint32_t)p.num_seqs * (uint32_t)p.Hv;
    __nv_bfloat16* __restrict__ og = reinterpret_cast<__nv_bfloat16*>(p.out_o);

    // Waits (bounded) on an mbarrier with all threads, then agrees on success across the CTA.
    auto wait_all = [&](uint32_t bar, uint32_t& phase) -> bool {
        if (!mbar_wait_bounded(bar, phase)) misc->abort = 1;
        phase ^= 1u;
        __syncthreads();
        return misc->abort == 0;
    };

    for (;;) {
        if (tid == 0) misc->item = atomicAdd(&prm.s.header->next_item, 1u);
        __syncthreads();
        const uint32_t item = misc->item;
        if (item >= num_items) break;
        const int n = prm.s.order[item / p.Hv];
        const int h = item % p.Hv;
        const int hq = h / G;
        const int row_begin = p.cu[n], row_end = p.cu[n + 1];
        const int nchunks = (row_end - row_begin + 63) >> 6;
        float* st_out = p.out_state ? p.out_state + ((size_t)n * p.Hv + h) * 128 * 128 : nullptr;

        for (int c = 0; c < nchunks; ++c) {
            const int row0 = row_begin + c * 64;
            const int nvalid = min(64, row_end - row0);

            // ---- A. TMA loads of the K, Q, V tiles of this chunk --------------------------------
            if (tid == 0) {
                mbar_arrive_expect_tx(bar_tma, 49152u);
                tma_load_2d(sb + SM_KQ, &tm_k, hq * 128, row0, bar_tma);
                tma_load_2d(sb + SM_KQ + 16384, &tm_k, hq * 128 + 64, row0, bar_tma);
                tma_load_2d(sb + SM_KQ + 8192, &tm_q, hq * 128, row0, bar_tma);
                tma_load_2d(sb + SM_KQ + 24576, &tm_q, hq * 128 + 64, row0, bar_tma);
                tma_load_2d(sb + SM_V, &tm_v, h * 128, row0, bar_tma);
                tma_load_2d(sb + SM_V + 8192, &tm_v, h * 128 + 64, row0, bar_tma);
            }
            // ---- B. log-decay cumsum and the decay factors ---------------------------------------
            if (tid < 64) {
                const bool ok = tid < nvalid;
                misc->g[tid] = ok ? p.g[(size_t)(row0 + tid) * p.Hv + h] : 0.f;
                misc->beta[tid] = ok ? p.beta[(size_t)(row0 + tid) * p.Hv + h] : 0.f;
            }
            __syncthreads();
            if (tid < 64) {
                float acc = 0.f;
                for (int s2 = 0; s2 <= tid; ++s2) acc += misc->g[s2];
                misc->G[tid] = acc;
            }
            __syncthreads();
            const float GC = misc->G[63];
            if (tid < 64) {
                const float Gt = misc->G[tid];
                misc->eG[tid] = ex2_approx(Gt * kLog2e);
                misc->eRest[tid] = ex2_approx((GC - Gt) * kLog2e);
            }
            const float eGC = ex2_approx(GC * kLog2e);

            // ---- C. chunk-start state: bf16 copy for the MMAs, fp32 master pre-scaled by e^{G_C} ----
            if (c > 0) {
                tc_fence_after();
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t r0[32], r1[32], pk[32];
                    tmem_ld32(tl + TM_S32 + hf * 64, r0);
                    tmem_ld32(tl + TM_S32 + hf * 64 + 32, r1);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        pk[i] = pack_bf16x2(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
                        pk[16 + i] = pack_bf16x2(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        r0[i] = __float_as_uint(__uint_as_float(r0[i]) * eGC);
                        r1[i] = __float_as_uint(__uint_as_float(r1[i]) * eGC);
                    }
                    tmem_st32(tl + TM_SBF + hf * 32, pk);
                    tmem_st32(tl + TM_S32 + hf * 64, r0);
                    tmem_st32(tl + TM_S32 + hf * 64 + 32, r1);
                }
                tmem_st_wait();
                tc_fence_before();
            }

            // ---- D. Gram MMA: [K;Q] K^T -> TM_GRAM ----------------------------------------------------
            if (!wait_all(bar_tma, ph_tma)) { aborted = true; break; }
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t a = sb + SM_KQ + (ks >> 2) * 16384 + (ks & 3) * 32;
                    mma_ss(tmem + TM_GRAM, smem_desc_sw128(a, 16, 1024), smem_desc_sw128(a, 16, 1024), ID_GRAM, ks > 0);
                }
                mma_commit(bar_mma);
            }
            if (!wait_all(bar_mma, ph_mma)) { aborted = true; break; }
            tc_fence_after();

            // ---- E. A (fp32, shared) and P (bf16 operand) from the Gram tile ---------------------------
            {
                uint32_t r0[32], r1[32];
                tmem_ld32(tl + TM_GRAM, r0);
                tmem_ld32(tl + TM_GRAM + 32, r1);
                tmem_ld_wait();
                const int t = tid & 63;
                const float Gt = misc->G[t];
                if (tid < 64) {
                    const float bt = misc->beta[t];
#pragma unroll
                    for (int s2 = 0; s2 < 64; ++s2) {
                        const float acc = __uint_as_float(s2 < 32 ? r0[s2 & 31] : r1[s2 & 31]);
                        const float arg = (s2 < t) ? (Gt - misc->G[s2]) * kLog2e : 0.f;
                        AF[t * LDF + s2] = (s2 < t) ? bt * ex2_approx(arg) * acc : 0.f;
                    }
                } else {
                    uint8_t* prow = sm + SM_P + t * 128;
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float v2[2];
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int s2 = ch * 8 + e * 2 + u;
                                const float acc = __uint_as_float(s2 < 32 ? r0[s2 & 31] : r1[s2 & 31]);
                                const float arg = (s2 <= t) ? (Gt - misc->G[s2]) * kLog2e : 0.f;
                                v2[u] = (s2 <= t) ? ex2_approx(arg) * acc : 0.f;
                            }
                            w[e] = pack_bf16x2(v2[0], v2[1]);
                        }
                        *reinterpret_cast<uint4*>(prow + ((ch ^ (t & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
#ifdef GDN_TC_DEBUG
            if (prm.debug && item == 0 && c < 2) {
                uint32_t r0[32], r1[32];
                tmem_ld32(tl + TM_GRAM, r0); tmem_ld32(tl + TM_GRAM + 32, r1); tmem_ld_wait();
                float* d = prm.debug + c * DBG_STRIDE;
                for (int i = 0; i < 32; ++i) { d[tid * 64 + i] = __uint_as_float(r0[i]); d[tid * 64 + 32 + i] = __uint_as_float(r1[i]); }
            }
#endif
            tc_fence_before();
            __syncthreads();

            // ---- F. X = (I + A)^-1: 16 x 16 diagonal blocks by substitution, then block rows ----------
            if (lane < 16) {
                const int b = warp * 16, j = lane;
                float x[16];
#pragma unroll
                for (int r = 0; r < 16; ++r) x[r] = (r == j) ? 1.f : 0.f;
#pragma unroll
                for (int r = 1; r < 16; ++r) {
                    float acc = 0.f;
#pragma unroll
                    for (int s2 = 0; s2 < r; ++s2) acc = fmaf(AF[(b + r) * LDF + b + s2], x[s2], acc);
                    x[r] = (r > j) ? -acc : x[r];
                }
#pragma unroll
                for (int r = 0; r < 16; ++r) XF[(b + r) * LDF + b + j] = x[r];
            }
            __syncthreads();
            for (int I = 1; I < 4; ++I) {
                const int ncol = 16 * I;
                for (int e = tid; e < 16 * ncol; e += 128) {
                    const int r = e / ncol, cc = e % ncol;
                    float acc = 0.f;
                    for (int m = cc & ~15; m < ncol; ++m) acc = fmaf(AF[(ncol + r) * LDF + m], XF[m * LDF + cc], acc);
                    MF[r * 64 + cc] = acc;
                }
                __syncthreads();
                for (int e = tid; e < 16 * ncol; e += 128) {
                    const int r = e / ncol, cc = e % ncol;
                    float acc = 0.f;
#pragma unroll
                    for (int m = 0; m < 16; ++m) acc = fmaf(XF[(ncol + r) * LDF + ncol + m], MF[m * 64 + cc], acc);
                    XF[(ncol + r) * LDF + cc] = -acc;
                }
                __syncthreads();
            }
            // T' = X diag(beta), T'' = X diag(beta e^G) as bf16 K-major operands
            {
                const int t = tid >> 1, hf = tid & 1;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t w1[4], w2[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float a1[2], a2[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int s2 = hf * 32 + ch * 8 + e * 2 + u;
                            const float x = (s2 <= t) ? XF[t * LDF + s2] : 0.f;
                            a1[u] = x * misc->beta[s2];
                            a2[u] = a1[u] * misc->eG[s2];
                        }
                        w1[e] = pack_bf16x2(a1[0], a1[1]);
                        w2[e] = pack_bf16x2(a2[0], a2[1]);
                    }
                    const int chunk16 = hf * 4 + ch;
                    const uint32_t off = t * 128 + ((chunk16 ^ (t & 7)) << 4);
                    *reinterpret_cast<uint4*>(sm + SM_TP + off) = make_uint4(w1[0], w1[1], w1[2], w1[3]);
                    *reinterpret_cast<uint4*>(sm + SM_TPP + off) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
                }
            }
#ifdef GDN_TC_DEBUG
            if (prm.debug && item == 0 && c < 2) {
                float* d = prm.debug + c * DBG_STRIDE + 8192;
                for (int e = tid; e < 4096; e += 128) d[e] = ((e & 63) <= (e >> 6)) ? XF[(e >> 6) * LDF + (e & 63)] : 0.f;
            }
#endif
            fence_proxy_async_smem();
            __syncthreads();

            // ---- G. W^T = K^T T''^T -> TM_GRAM,  U^T = V^T T'^T -> TM_ACC1 -----------------------------
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    mma_ss(tmem + TM_GRAM, smem_desc_sw128(sb + SM_KQ + ks * 2048, 16384, 1024),
                           smem_desc_sw128(sb + SM_TPP + ks * 32, 16, 1024), ID_WU, ks > 0);
                }
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    mma_ss(tmem + TM_ACC1, smem_desc_sw128(sb + SM_V + ks * 2048, 8192, 1024),
                           smem_desc_sw128(sb + SM_TP + ks * 32, 16, 1024), ID_WU, ks > 0);
                }
                mma_commit(bar_mma);
            }
            if (!wait_all(bar_mma, ph_mma)) { aborted = true; break; }
            tc_fence_after();

            // ---- H. W epilogue: W[t][dk] bf16 into shared memory as a K-major operand ------------------
            {
                uint32_t r0[32], r1[32];
                tmem_ld32(tl + TM_GRAM, r0);
                tmem_ld32(tl + TM_GRAM + 32, r1);
                tmem_ld_wait();
#ifdef GDN_TC_DEBUG
                if (prm.debug && item == 0 && c < 2) {
                    float* d = prm.debug + c * DBG_STRIDE + 12288;
                    for (int i = 0; i < 32; ++i) { d[tid * 64 + i] = __uint_as_float(r0[i]); d[tid * 64 + 32 + i] = __uint_as_float(r1[i]); }
                }
#endif
                const int dd = tid & 63;
                uint8_t* wbase = sm + SM_W + (tid >> 6) * 8192 + (dd & 7) * 2;
#pragma unroll
                for (int t = 0; t < 64; ++t) {
                    const float wv = __uint_as_float(t < 32 ? r0[t & 31] : r1[t & 31]);
                    *reinterpret_cast<__nv_bfloat16*>(wbase + t * 128 + (((dd >> 3) ^ (t & 7)) << 4)) = __float2bfloat16_rn(wv);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();

            // ---- I. Delta^T = U^T - S0 W^T (onto TM_ACC1),  S0 Q^T -> TM_ACC2 -------------------------
            if (c > 0) {
                if (tid == 0) {
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        mma_ts(tmem + TM_ACC1, tmem + TM_SBF + ks * 8,
                               smem_desc_sw128(sb + SM_W + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024), ID_SW, 1u);
                    }
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        mma_ts(tmem + TM_ACC2, tmem + TM_SBF + ks * 8,
                               smem_desc_sw128(sb + SM_KQ + 8192 + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024), ID_SQ, ks > 0);
                    }
                    mma_commit(bar_mma);
                }
                if (!wait_all(bar_mma, ph_mma)) { aborted = true; break; }
                tc_fence_after();
            }

            // ---- J. Delta epilogue: bf16 Delta^T and decayed Delta'^T as TMEM A operands ----------------
            {
                uint32_t r0[32], r1[32], d1[32], d2[32];
                tmem_ld32(tl + TM_ACC1, r0);
                tmem_ld32(tl + TM_ACC1 + 32, r1);
                tmem_ld_wait();
#ifdef GDN_TC_DEBUG
                if (prm.debug && item == 0 && c < 2) {
                    float* d = prm.debug + c * DBG_STRIDE + 20480;
                    for (int i = 0; i < 32; ++i) { d[tid * 64 + i] = __uint_as_float(r0[i]); d[tid * 64 + 32 + i] = __uint_as_float(r1[i]); }
                }
#endif
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float a0 = __uint_as_float(r0[2 * i]), a1 = __uint_as_float(r0[2 * i + 1]);
                    const float b0 = __uint_as_float(r1[2 * i]), b1 = __uint_as_float(r1[2 * i + 1]);
                    d1[i] = pack_bf16x2(a0, a1);
                    d1[16 + i] = pack_bf16x2(b0, b1);
                    d2[i] = pack_bf16x2(a0 * misc->eRest[2 * i], a1 * misc->eRest[2 * i + 1]);
                    d2[16 + i] = pack_bf16x2(b0 * misc->eRest[32 + 2 * i], b1 * misc->eRest[32 + 2 * i + 1]);
                }
                tmem_st32(tl + TM_DBF, d1);
                tmem_st32(tl + TM_DPBF, d2);
                tmem_st_wait();
            }
            tc_fence_before();
            __syncthreads();

            // ---- K. Delta^T P^T -> TM_ACC3,  S += Delta'^T K (onto the pre-scaled TM_S32) --------------
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    mma_ts(tmem + TM_ACC3, tmem + TM_DBF + ks * 8,
                           smem_desc_sw128(sb + SM_P + ks * 32, 16, 1024), ID_DP, ks > 0);
                }
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    mma_ts(tmem + TM_S32, tmem + TM_DPBF + ks * 8,
                           smem_desc_sw128(sb + SM_KQ + ks * 2048, 16384, 1024), ID_DK, (c > 0 || ks > 0) ? 1u : 0u);
                }
                mma_commit(bar_mma);
            }
            if (!wait_all(bar_mma, ph_mma)) { aborted = true; break; }
            tc_fence_after();

            // ---- L. output epilogue: O^T = diag(e^G) (S0 Q^T) + Delta^T P^T, stored for valid rows -----
            if (og) {
                uint32_t r0[32], r1[32], q0[32], q1[32];
                tmem_ld32(tl + TM_ACC3, r0);
                tmem_ld32(tl + TM_ACC3 + 32, r1);
                if (c > 0) {
                    tmem_ld32(tl + TM_ACC2, q0);
                    tmem_ld32(tl + TM_ACC2 + 32, q1);
                }
                tmem_ld_wait();
#ifdef GDN_TC_DEBUG
                if (prm.debug && item == 0 && c < 2) {
                    float* d = prm.debug + c * DBG_STRIDE;
                    for (int i = 0; i < 32; ++i) {
                        d[36864 + tid * 64 + i] = __uint_as_float(r0[i]); d[36864 + tid * 64 + 32 + i] = __uint_as_float(r1[i]);
                        d[28672 + tid * 64 + i] = c > 0 ? __uint_as_float(q0[i]) : 0.f;
                        d[28672 + tid * 64 + 32 + i] = c > 0 ? __uint_as_float(q1[i]) : 0.f;
                    }
                }
#endif
                __nv_bfloat16* orow = og + ((size_t)row0 * p.Hv + h) * 128 + tid;
#pragma unroll
                for (int t = 0; t < 64; ++t) {
                    float o = __uint_as_float(t < 32 ? r0[t & 31] : r1[t & 31]);
                    if (c > 0) o = fmaf(misc->eG[t], __uint_as_float(t < 32 ? q0[t & 31] : q1[t & 31]), o);
                    if (t < nvalid) orow[(size_t)t * p.Hv * 128] = __float2bfloat16_rn(o);
                }
            }
#ifdef GDN_TC_DEBUG
            if (prm.debug && item == 0 && c < 2) {
                float* d = prm.debug + c * DBG_STRIDE + 45056;
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t r0[32];
                    tmem_ld32(tl + TM_S32 + q4 * 32, r0); tmem_ld_wait();
                    for (int i = 0; i < 32; ++i) d[tid * 128 + q4 * 32 + i] = __uint_as_float(r0[i]);
                }
            }
#endif
            tc_fence_before();
            __syncthreads();
        }
        if (aborted) break;

        // ---- final state: out_state[n, h, a, b] = S[b][a] --------------------------------------------
        if (st_out) {
            if (nchunks == 0) {
                for (int a = 0; a < 128; ++a) st_out[a * 128 + tid] = 0.f;
            } else {
                tc_fence_after();
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t r0[32];
                    tmem_ld32(tl + TM_S32 + q4 * 32, r0);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) st_out[(q4 * 32 + i) * 128 + tid] = __uint_as_float(r0[i]);
                }
                tc_fence_before();
            }
        }
        __syncthreads();
    }

    if (aborted) {
        if (tid == 0 && p.status_word) *p.status_word = GDN_ERR_TIMEOUT;
        // give copies that may still be in flight a bounded chance to land before the CTA retires
        if (tid == 0) mbar_wait_bounded(bar_tma, ph_tma ^ 1u, 200000000ull);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// [rows][cols] bf16 row-major viewed as a 2-D tensor; boxes of 64 columns (128 bytes) x 64 rows,
// 128-byte swizzle; rows past the end read as zero.
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols)
{
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, 64};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

float* g_debug_buffer = nullptr;

}  // namespace

#ifdef GDN_TC_DEBUG
extern "C" GDN_API void gdn_debug_set_buffer(float* dev_ptr) { g_debug_buffer = dev_ptr; }
#endif

cudaError_t launch_tcgen05(const Problem& p, const Sched& s, cudaStream_t stream, int* launches)
{
    if (p.dk != 128 || p.dv != 128 || p.init_state != nullptr || p.total_tokens <= 0) return cudaErrorNotSupported;
    CUtensorMap tq, tk, tv;
    if (!make_map(&tq, p.q, (uint64_t)p.total_tokens, (uint64_t)p.Hq * 128) ||
        !make_map(&tk, p.k, (uint64_t)p.total_tokens, (uint64_t)p.Hq * 128) ||
        !make_map(&tv, p.v, (uint64_t)p.total_tokens, (uint64_t)p.Hv * 128))
        return cudaErrorUnknown;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    static bool attr_set[64] = {};
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(gdn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    long long grid = (long long)p.num_seqs * p.Hv;
    if (grid > sms) grid = sms;
    TcParams prm;
    prm.p = p; prm.s = s; prm.debug = g_debug_buffer;
    gdn_tc_kernel<<<(unsigned)grid, 128, SMEM_BYTES, stream>>>(prm, tq, tk, tv);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}

}  // namespace gdn

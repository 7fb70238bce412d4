// Tensor-core chunkwise Gated DeltaNet (Section 3, chunkwise equations, specialised to the gated
// delta rule of Section 4.3; decay applied on every token, state update only for linear tokens)
// for bf16 storage on sm_100a: a chunk-parallel "prepare" kernel and a sequential "scan" kernel.
//
// Notation per chunk of C = 64 tokens: beta~ = (1 - route) beta, G_i = inclusive cumulative log
// decay, gamma_i = exp(G_i), Gamma_ij = exp(G_i - G_j) (j <= i):
//   A_ij = beta~_i Gamma_ij (k_i.k_j) (j < i),  T = (I + A)^-1,
//   U = T diag(beta~) V,  W = T diag(beta~ gamma) K,  P_ij = scale_la Gamma_ij (q_i.k_j) (j <= i)
//   U~ = U - W S;  O = scale_la diag(gamma) Q S + P U~;  S <- gamma_C S + (diag(gamma_C/gamma) K)^T U~
// Block-level routing (Section 4.1: both operations compute the inner-chunk correlations) uses the
// same kernels with beta~ = beta for every token and the state update of a softmax block left
// out (S <- gamma_C S), so that its chunk sees the delta rule but the later ones do not.
//
// Precision.  q, k, v are exact bf16 inputs, but T, W, U~, P and S are computed quantities: an
// 8-bit significand on them puts the layer output 1.4-2e-2 x RMS off (the whole error budget), so
// every tensor-core operand here is fp16 (11-bit significand; the inputs convert exactly, all
// magnitudes are O(1) and decay factors only shrink them).  The 16x16 diagonal blocks of T are
// inverted in fp32, its blocks below the diagonal come from fp16 products with fp32 accumulation
// (their error stays at the level of the fp16 rounding T gets as an operand anyway), and U, which
// is only ever added to an accumulator, stays fp32.
//
// All products are laid out "transposed", with the head dimension on the MMA's M axis
// (M = 128 rows = TMEM lanes = one thread each) and the 64 tokens of a chunk on N or K, so that
// every operand a thread has to produce is one contiguous 128-byte row of a swizzled tile.
#include "common.cuh"
#include "natsl_internal.h"
#include "tc_common.cuh"

namespace natsl {

namespace {

using namespace tc;

constexpr int kRowThreads = 128;

// bf16 -> fp16, 8 values in place
__device__ __forceinline__ uint4 bf16x8_to_f16x8(uint4 u) {
    const uint32_t wv[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        o[i] = pack_half2(__uint_as_float(wv[i] << 16), __uint_as_float(wv[i] & 0xffff0000u));
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// ==========================================================================================
// Prepare: one CTA per chunk of one (batch, head).  One MMA group with M = 128 stacks [Q ; K] on
// the rows against K: TMEM rows 0-63 then hold Q K^T (-> P) and rows 64-127 K K^T (-> A).  Warps 0-1
// (rows 0-63) compute the gates, P and the decay factors; warps 2-3 (rows 64-127) build A, form
// T = (I + A)^-1 blockwise (16x16 diagonal blocks by substitution through warp shuffles, the rest as
// a handful of warp-level MMAs), and write the fp16 operands T beta~ and T beta~ gamma; then all
// 128 threads (one head-dimension row each) store U^T and W^T.  Warp 4 issues TMA and MMAs.
// 128 TMEM columns and ~50 KB of shared memory per CTA keep four CTAs on an SM, so that one chunk's
// dependent phases overlap with other chunks' loads and stores.
// ==========================================================================================
constexpr int kPrepThreads = 160;
constexpr int kPrepMisc = 2048;

template <int D> struct PrepLayout {
    static constexpr int KB = D / 64;
    static constexpr int oV = 0;                           // V: KB sub-tiles of 64 tokens x 64
    static constexpr int oQK = KB * 8192;                  // per 64-column block: [Q 8 KB][K 8 KB]
    static constexpr int oX = oQK + KB * 16384;            // d = 64 only: A^T, then the T operands
    static constexpr int kX = D == 64 ? 16384 : 0;
    static constexpr int oMisc = oX + kX;
    static constexpr int kTotal = oMisc + kPrepMisc;
    static constexpr int kLoadBytes = KB * 24576;
};

struct PrepMisc {
    uint64_t barLoad, barConv, barM, barXfree, barT, barUW;
    uint32_t tmem_base;
    int abort_flag, wait_kcycles;   // in this order: the waits read the limit as abort_flag[1]
    alignas(16) float G[64], bt[64], btg[64], wsum[2];   // cumulative log decay, beta~, beta~ gamma (read in pairs)
};
static_assert(sizeof(PrepMisc) <= kPrepMisc, "misc page too small");

template <int D>
__global__ void __launch_bounds__(kPrepThreads, 4)
gdn_prepare_tc_kernel(const __grid_constant__ CUtensorMap map_q,
                      const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v,
                      const __grid_constant__ CUtensorMap map_qh,
                      const __grid_constant__ CUtensorMap map_kh, const float *__restrict__ g,
                      const float *__restrict__ beta, const uint8_t *__restrict__ route,
                      float scale_la, __half *__restrict__ Wt, float *__restrict__ Ut,
                      __half *__restrict__ Ph, float *__restrict__ Gd, GdnTcExport ex,
                      int32_t *status, int L, int H, float norm_eps, int wait_kcycles) {
    using PL = PrepLayout<D>;
    constexpr int KB = PL::KB;
    extern __shared__ __align__(1024) uint8_t smem[];
    PrepMisc &ms = *reinterpret_cast<PrepMisc *>(smem + PL::oMisc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NC = L / kC;
    // (chunk fastest: a head-fastest order, whole rows of [B,L,H,d] read by neighbouring CTAs, and L2
    // prefetches of the next wave's tiles were both measured slower)
    const int c = (int)(blockIdx.x % NC), bh = (int)(blockIdx.x / NC), b = bh / H, h = bh % H;
    const int tok0 = c * kC;
    const size_t chunk = (size_t)bh * NC + c;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        mbar_init(&ms.barLoad, 1);
        mbar_init(&ms.barConv, kRowThreads);
        mbar_init(&ms.barM, 1);
        mbar_init(&ms.barXfree, 1);
        mbar_init(&ms.barT, kRowThreads);
        mbar_init(&ms.barUW, 1);
        ms.abort_flag = 0;
        ms.wait_kcycles = wait_kcycles;
        fence_mbar_init();
    }
    if (warp == 4) tmem_alloc(&ms.tmem_base, 128);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ms.tmem_base;
    volatile int *abort_flag = &ms.abort_flag;
    uint8_t *sV = smem + PL::oV, *sQK = smem + PL::oQK;
    // The fp16 tiles of A and T during the inversion, and afterwards the two fp16 operands: in the two Q blocks
    // once K K^T / Q K^T and the q copy are done with them (d = 128), or in their own region (d = 64).
    uint8_t *xLo = D == 128 ? sQK : smem + PL::oX;
    uint8_t *xHi = D == 128 ? sQK + 16384 : smem + PL::oX + 8192;

    if (warp == 4) {
        if (lane == 0) {
            mbar_arrive_expect_tx(&ms.barLoad, PL::kLoadBytes);
            for (int kb = 0; kb < KB; ++kb) {
                tma_load_4d(sQK + kb * 16384 + 8192, &map_k, &ms.barLoad, kb * 64, h, tok0, b);
                tma_load_4d(sQK + kb * 16384, &map_q, &ms.barLoad, kb * 64, h, tok0, b);
                tma_load_4d(sV + kb * 8192, &map_v, &ms.barLoad, kb * 64, h, tok0, b);
            }
            bool ok = mbar_wait(&ms.barConv, 0, abort_flag);       // tiles converted to fp16
            if (ok) {
                // ---- fp16 copies of q and k for the scan kernel; [Q ; K] K^T ----
                for (int kb = 0; kb < KB; ++kb) {
                    tma_store_2d(&map_qh, sQK + kb * 16384, kb * 64, bh * L + tok0);
                    tma_store_2d(&map_kh, sQK + kb * 16384 + 8192, kb * 64, bh * L + tok0);
                }
                tma_store_commit();
                tc_fence_after_sync();
                constexpr uint32_t idesc = make_idesc(kFmtF16, 128, 64, false, false);
                const uint32_t aQK = smem_u32(sQK);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16)
                        mma_ss(tmem, desc_kmajor(aQK + kb * 16384 + k16 * 32),
                               desc_kmajor(aQK + kb * 16384 + 8192 + k16 * 32), idesc, (kb | k16) != 0);
                mma_commit(&ms.barM);
                tma_store_wait_read();                    // the q copy has left its blocks
                ok = mbar_wait(&ms.barM, 0, abort_flag);  // and the MMAs have read them
                mbar_arrive(&ms.barXfree);
            }
            if (ok) ok = mbar_wait(&ms.barT, 0, abort_flag);
            if (ok) {
                // ---- U^T = V^T (T beta~)^T,  W^T = K^T (T beta~ gamma)^T ----
                tc_fence_after_sync();
                const uint32_t aV = smem_u32(sV), aK = smem_u32(sQK) + 8192, aTb = smem_u32(xLo),
                               aTg = smem_u32(xHi);
                if (D == 128) {
                    constexpr uint32_t idesc = make_idesc(kFmtF16, 128, 64, true, false);
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        mma_ss(tmem, desc_mnmajor(aV + k16 * 2048, 8192), desc_kmajor(aTb + k16 * 32),
                               idesc, k16 != 0);
                        mma_ss(tmem + 64, desc_mnmajor(aK + k16 * 2048, 16384),
                               desc_kmajor(aTg + k16 * 32), idesc, k16 != 0);
                    }
                } else {
                    // d = 64: rows 0-63 of M are V^T, rows 64-127 are K^T (16 KB further on);
                    // N = 128 = [T beta~ ; T beta~ gamma] (adjacent).
                    constexpr uint32_t idesc = make_idesc(kFmtF16, 128, 128, true, false);
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16)
                        mma_ss(tmem, desc_mnmajor(aV + k16 * 2048, 16384), desc_kmajor(aTb + k16 * 32),
                               idesc, k16 != 0);
                }
                mma_commit(&ms.barUW);
            }
            tma_store_wait_all();
        }
    } else {
        const int r = tid, i = r & 63;
        const bool solver = r >= 64;                       // rows 64-127: K K^T
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        // ---- gates (warps 0-1): beta~, inclusive cumulative log decay within the chunk ----
        if (!solver) {
            const size_t t = ((size_t)b * L + tok0 + i) * H + h;
            float G = g[t];
            const float btv = route && route[t] ? 0.f : beta[t];   // route == nullptr: beta~ = beta
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float y = __shfl_up_sync(0xffffffffu, G, o);
                if (lane >= o) G += y;
            }
            if (lane == 31) ms.wsum[warp] = G;
            named_barrier_sync(1, 64);
            if (warp == 1) G += ms.wsum[0];
            ms.G[i] = G;
            ms.bt[i] = btv;
            ms.btg[i] = btv * exp_ftz(G);
        }
        // ---- tiles to fp16, in place ----
        bool ok = mbar_wait(&ms.barLoad, 0, abort_flag);
        if (ok && norm_eps >= 0.f) {
            // L2-normalised q and k for the linear operation (Section 4.3): thread r owns row r of
            // [Q ; K] (all KB blocks of it), takes its 16-byte pieces in an order that spreads the warp
            // over the banks, and scales while it converts.  V is converted as below.
            static_assert(PL::oV == 0 && PL::oQK == KB * 8192, "V tile first, [Q ; K] blocks behind it");
            for (int idx = r; idx < KB * 8192 / 16; idx += kRowThreads) {
                uint4 *pp = reinterpret_cast<uint4 *>(smem) + idx;
                *pp = bf16x8_to_f16x8(*pp);
            }
            uint8_t *rowp = sQK + (solver ? 8192 : 0) + i * 128;
            float ss = 0.f;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 a = *reinterpret_cast<const uint4 *>(rowp + kb * 16384 + ((c ^ (i & 7)) << 4));
                    const uint32_t wd[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float lo = __uint_as_float(wd[e] << 16), hi = __uint_as_float(wd[e] & 0xffff0000u);
                        ss = fmaf(lo, lo, fmaf(hi, hi, ss));
                    }
                }
            const float rn = rsqrtf(ss + norm_eps);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint4 *pp = reinterpret_cast<uint4 *>(rowp + kb * 16384 + ((c ^ (i & 7)) << 4));
                    const uint4 a = *pp;
                    const uint32_t wd[4] = {a.x, a.y, a.z, a.w};
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        o[e] = pack_half2(__uint_as_float(wd[e] << 16) * rn, __uint_as_float(wd[e] & 0xffff0000u) * rn);
                    *pp = make_uint4(o[0], o[1], o[2], o[3]);
                }
        } else if (ok) {
            for (int idx = r; idx < PL::kLoadBytes / 16; idx += kRowThreads) {
                uint4 *pp = reinterpret_cast<uint4 *>(smem) + idx;   // V and [Q ; K] are contiguous
                *pp = bf16x8_to_f16x8(*pp);
            }
        }
        if (ok) {
            fence_proxy_async_smem();
            mbar_arrive(&ms.barConv);
            ok = mbar_wait(&ms.barXfree, 0, abort_flag);
        }
        if (ok) {
            tc_fence_after_sync();
            const float G = ms.G[i];
            if (!solver) {
                // ---- decay factors for the scan, P (lower triangle).  A real loop over 8-column
                // pieces: straight-line code that runs once per CTA is bound by instruction fetch. ----
                float *gd = Gd + chunk * 128;
                gd[i] = exp_ftz(G);
                gd[64 + i] = exp_ftz(ms.G[63] - G);
                if (ex.Gcum) ex.Gcum[(size_t)bh * L + tok0 + i] = G;
                uint4 *prow = reinterpret_cast<uint4 *>(Ph + (chunk * 64 + i) * 64);
#pragma unroll 1
                for (int pc = 0; pc < 8; ++pc) {
                    uint32_t d8[8];
                    tmem_ld8(tmem + lane_base + 8 * pc, d8);
                    tmem_wait_ld();
                    float x[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int j = 8 * pc + e;
                        // the mask goes on the exponent (exp(-inf) = 0): a conditional around the whole
                        // expression compiles to one divergent branch per element
                        x[e] = scale_la * exp_ftz(j <= i ? G - ms.G[j] : -INFINITY) * __uint_as_float(d8[e]);
                    }
                    prow[pc] = make_uint4(pack_half2(x[0], x[1]), pack_half2(x[2], x[3]),
                                          pack_half2(x[4], x[5]), pack_half2(x[6], x[7]));
                    if (ex.P) {
                        float4 *pf = reinterpret_cast<float4 *>(ex.P + (chunk * 64 + i) * 64 + 8 * pc);
                        pf[0] = make_float4(x[0], x[1], x[2], x[3]);
                        pf[1] = make_float4(x[4], x[5], x[6], x[7]);
                    }
                }
                tc_fence_before_sync();
                mbar_arrive(&ms.barT);
            } else {
                // ---- T = (I + A)^-1 with 16x16 blocks (T_bb = (I + A_bb)^-1 in fp32 registers; below the
                // diagonal T_10 = -T_11 A_10 T_00, T_32 likewise, then the 32x32 block
                // T_[23][01] = -T_[23][23] A_[23][01] T_[01][01], all as warp-level fp16 MMAs) ----
                uint32_t dd[2][32];
                tmem_ld32(tmem + lane_base, dd[0]);
                tmem_ld32(tmem + lane_base + 32, dd[1]);
                tmem_wait_ld();
                tc_fence_before_sync();
                const int sw = warp - 2;                   // solver warp: block rows 2 sw and 2 sw + 1
                const int bk = i >> 4, il = i & 15;        // this thread's block row, its row inside it
                const int g8 = lane >> 2, t4 = lane & 3;   // fragment coordinates
                const float btv = ms.bt[i];
                const uint32_t aA = smem_u32(xLo), aT = smem_u32(xHi);
                // A_ij = beta~_i Gamma_ij (k_i.k_j), j < i: blocks left of the diagonal as fp16 rows of
                // the A tile (xLo), the row of the diagonal block in registers.
                float ablk[16];
#pragma unroll
                for (int jb = 0; jb < 4; ++jb) {
                    if (jb <= bk) {
                        float a[16];
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            const int j = 16 * jb + jj;
                            a[jj] = btv * exp_ftz(j < i ? G - ms.G[j] : -INFINITY) * __uint_as_float(dd[j >> 5][j & 31]);
                        }
                        if (jb < bk) {
#pragma unroll
                            for (int hp = 0; hp < 2; ++hp)
                                *reinterpret_cast<uint4 *>(xLo + sw128_offset(i, 2 * jb + hp)) = make_uint4(
                                    pack_half2(a[8 * hp], a[8 * hp + 1]), pack_half2(a[8 * hp + 2], a[8 * hp + 3]),
                                    pack_half2(a[8 * hp + 4], a[8 * hp + 5]), pack_half2(a[8 * hp + 6], a[8 * hp + 7]));
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 16; ++jj) ablk[jj] = a[jj];
                        }
                    }
                }
                // Row il of the diagonal block's inverse: t_j = [j = il] - sum_{m > j} t_m A_mj, from the
                // right; A_mj sits in the registers of the thread that owns row m of the block.
                float td[16];
                {
                    float sacc[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) sacc[j] = 0.f;
                    const int grp = lane & 16;
#pragma unroll
                    for (int m = 15; m >= 0; --m) {
                        td[m] = (m == il ? 1.f : 0.f) - sacc[m];
#pragma unroll
                        for (int j = 0; j < m; ++j)
                            sacc[j] = fmaf(td[m], __shfl_sync(0xffffffffu, ablk[j], grp + m), sacc[j]);
                    }
                }
#pragma unroll
                for (int hp = 0; hp < 2; ++hp)              // fp16 copy for the products: T tile (xHi)
                    *reinterpret_cast<uint4 *>(xHi + sw128_offset(i, 2 * bk + hp)) = make_uint4(
                        pack_half2(td[8 * hp], td[8 * hp + 1]), pack_half2(td[8 * hp + 2], td[8 * hp + 3]),
                        pack_half2(td[8 * hp + 4], td[8 * hp + 5]), pack_half2(td[8 * hp + 6], td[8 * hp + 7]));
                __syncwarp();
                // Address this lane supplies to a 16x16 ldmatrix.x4 whose corner is (row0, 16-byte piece pc0).
                const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8, lpc = lane >> 4;
                auto frag_addr = [&](uint32_t base, int row0, int pc0) {
                    return base + sw128_offset(row0 + lrow, pc0 + lpc);
                };
                auto pack_a = [](const float (&lo)[4], const float (&hi)[4], uint32_t (&o)[4]) {
                    o[0] = pack_half2(lo[0], lo[1]); o[1] = pack_half2(lo[2], lo[3]);
                    o[2] = pack_half2(hi[0], hi[1]); o[3] = pack_half2(hi[2], hi[3]);
                };
                const int b0 = 2 * sw, b1 = b0 + 1, br = 2 + sw;
                float t10[2][4] = {};                       // this warp's T_{b1,b0} (sign applied below)
                {
                    uint32_t fa[4], fb[4], xa[4];
                    float x[2][4] = {};
                    ldmatrix_x4(frag_addr(aT, 16 * b1, 2 * b1), fa);            // T_{b1,b1}
                    ldmatrix_x4_trans(frag_addr(aA, 16 * b1, 2 * b0), fb);      // A_{b1,b0}
                    mma_m16n8k16(x[0], fa, fb[0], fb[1]);
                    mma_m16n8k16(x[1], fa, fb[2], fb[3]);
                    pack_a(x[0], x[1], xa);
                    ldmatrix_x4_trans(frag_addr(aT, 16 * b0, 2 * b0), fb);      // T_{b0,b0}
                    mma_m16n8k16(t10[0], xa, fb[0], fb[1]);
                    mma_m16n8k16(t10[1], xa, fb[2], fb[3]);
                }
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) t10[nt][e] = -t10[nt][e];
                    *reinterpret_cast<uint32_t *>(xHi + sw128_offset(16 * b1 + g8, 2 * b0 + nt) + 4 * t4) =
                        pack_half2(t10[nt][0], t10[nt][1]);
                    *reinterpret_cast<uint32_t *>(xHi + sw128_offset(16 * b1 + g8 + 8, 2 * b0 + nt) + 4 * t4) =
                        pack_half2(t10[nt][2], t10[nt][3]);
                }
                named_barrier_sync(2, 64);                  // both warps' A rows and T blocks are in place
                float r2[4][4] = {};                        // block row br of T_[23][01]
                {
                    uint32_t fa[4], fb[4], fc[4], ya[2][4];
                    float y[4][4] = {};                     // T_{br,[23]} A_[23][01]
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        if (ks <= sw) {                     // T_23 = 0
                            ldmatrix_x4(frag_addr(aT, 16 * br, 2 * (2 + ks)), fa);
                            ldmatrix_x4_trans(frag_addr(aA, 16 * (2 + ks), 0), fb);
                            ldmatrix_x4_trans(frag_addr(aA, 16 * (2 + ks), 2), fc);
                            mma_m16n8k16(y[0], fa, fb[0], fb[1]);
                            mma_m16n8k16(y[1], fa, fb[2], fb[3]);
                            mma_m16n8k16(y[2], fa, fc[0], fc[1]);
                            mma_m16n8k16(y[3], fa, fc[2], fc[3]);
                        }
                    }
                    pack_a(y[0], y[1], ya[0]);
                    pack_a(y[2], y[3], ya[1]);
                    ldmatrix_x4_trans(frag_addr(aT, 0, 0), fb);                 // T_00
                    mma_m16n8k16(r2[0], ya[0], fb[0], fb[1]);
                    mma_m16n8k16(r2[1], ya[0], fb[2], fb[3]);
                    ldmatrix_x4_trans(frag_addr(aT, 16, 0), fb);                // T_10
                    mma_m16n8k16(r2[0], ya[1], fb[0], fb[1]);
                    mma_m16n8k16(r2[1], ya[1], fb[2], fb[3]);
                    ldmatrix_x4_trans(frag_addr(aT, 16, 2), fb);                // T_11 (T_01 = 0)
                    mma_m16n8k16(r2[2], ya[1], fb[0], fb[1]);
                    mma_m16n8k16(r2[3], ya[1], fb[2], fb[3]);
                }
                named_barrier_sync(2, 64);                  // both tiles have been read: reuse them
                // ---- operands T diag(beta~) (xLo) and T diag(beta~ gamma) (xHi), fp16 K-major rows ----
                float *Trow = ex.T ? ex.T + chunk * 4096 : nullptr;
                auto put2 = [&](int row, int col, float v0, float v1) {
                    const float2 fb = *reinterpret_cast<const float2 *>(&ms.bt[col]);
                    const float2 fg = *reinterpret_cast<const float2 *>(&ms.btg[col]);
                    const uint32_t off = sw128_offset(row, col >> 3) + (col & 7) * 2;
                    *reinterpret_cast<uint32_t *>(xLo + off) = pack_half2(v0 * fb.x, v1 * fb.y);
                    *reinterpret_cast<uint32_t *>(xHi + off) = pack_half2(v0 * fg.x, v1 * fg.y);
                    if (Trow) *reinterpret_cast<float2 *>(Trow + row * 64 + col) = make_float2(v0, v1);
                };
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    put2(16 * b1 + g8, 16 * b0 + 8 * nt + 2 * t4, t10[nt][0], t10[nt][1]);
                    put2(16 * b1 + g8 + 8, 16 * b0 + 8 * nt + 2 * t4, t10[nt][2], t10[nt][3]);
                }
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    put2(16 * br + g8, 8 * nt + 2 * t4, -r2[nt][0], -r2[nt][1]);
                    put2(16 * br + g8 + 8, 8 * nt + 2 * t4, -r2[nt][2], -r2[nt][3]);
                }
#pragma unroll
                for (int hp = 0; hp < 2; ++hp) {            // own row of the diagonal block
                    float xb[8], xg[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        xb[e] = td[8 * hp + e] * ms.bt[16 * bk + 8 * hp + e];
                        xg[e] = td[8 * hp + e] * ms.btg[16 * bk + 8 * hp + e];
                    }
                    *reinterpret_cast<uint4 *>(xLo + sw128_offset(i, 2 * bk + hp)) =
                        make_uint4(pack_half2(xb[0], xb[1]), pack_half2(xb[2], xb[3]),
                                   pack_half2(xb[4], xb[5]), pack_half2(xb[6], xb[7]));
                    *reinterpret_cast<uint4 *>(xHi + sw128_offset(i, 2 * bk + hp)) =
                        make_uint4(pack_half2(xg[0], xg[1]), pack_half2(xg[2], xg[3]),
                                   pack_half2(xg[4], xg[5]), pack_half2(xg[6], xg[7]));
                    if (Trow) {
                        float4 *tr = reinterpret_cast<float4 *>(Trow + i * 64 + 16 * bk + 8 * hp);
                        tr[0] = make_float4(td[8 * hp], td[8 * hp + 1], td[8 * hp + 2], td[8 * hp + 3]);
                        tr[1] = make_float4(td[8 * hp + 4], td[8 * hp + 5], td[8 * hp + 6], td[8 * hp + 7]);
                    }
                }
                for (int pc = 2 * bk + 2; pc < 8; ++pc) {   // right of the diagonal block: zero
                    *reinterpret_cast<uint4 *>(xLo + sw128_offset(i, pc)) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4 *>(xHi + sw128_offset(i, pc)) = make_uint4(0, 0, 0, 0);
                    if (Trow) {
                        float4 *tr = reinterpret_cast<float4 *>(Trow + i * 64 + 8 * pc);
                        tr[0] = tr[1] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
                fence_proxy_async_smem();
                mbar_arrive(&ms.barT);
            }
            ok = mbar_wait(&ms.barUW, 0, abort_flag);
        }
        if (ok) {
            // ---- U^T (fp32) and W^T (fp16) rows to global; thread r <-> head-dimension row ----
            tc_fence_after_sync();
            const bool do_u = D == 128 || r < 64, do_w = D == 128 || r >= 64;
            const int row = D == 128 ? r : i;
            uint32_t x[2][32];
            if (do_u) {                                     // warp-uniform
                tmem_ld32(tmem + lane_base, x[0]);
                tmem_ld32(tmem + lane_base + 32, x[1]);
                tmem_wait_ld();
                // piece-major: 16-byte piece pc (4 tokens) of all D rows is contiguous, so that a
                // warp's stores here and its loads in the scan are fully coalesced
                uint4 *dst = reinterpret_cast<uint4 *>(Ut + chunk * D * 64) + row;
#pragma unroll
                for (int pc = 0; pc < 16; ++pc)
                    dst[pc * D] = make_uint4(x[pc >> 3][(4 * pc) & 31], x[pc >> 3][(4 * pc + 1) & 31],
                                             x[pc >> 3][(4 * pc + 2) & 31], x[pc >> 3][(4 * pc + 3) & 31]);
                if (ex.U) {      // token-major fp32 copy
                    float *uf = ex.U + (((size_t)b * L + tok0) * H + h) * D + row;
#pragma unroll
                    for (int j = 0; j < 64; ++j) uf[(size_t)j * H * D] = __uint_as_float(x[j >> 5][j & 31]);
                }
            }
            if (do_w) {
                tmem_ld32(tmem + lane_base + 64, x[0]);
                tmem_ld32(tmem + lane_base + 96, x[1]);
                tmem_wait_ld();
                if (ex.W) {
                    float *wf = ex.W + (((size_t)b * L + tok0) * H + h) * D + row;
#pragma unroll
                    for (int j = 0; j < 64; ++j) wf[(size_t)j * H * D] = __uint_as_float(x[j >> 5][j & 31]);
                }
                uint4 *dst = reinterpret_cast<uint4 *>(Wt + (chunk * D + row) * 64);
#pragma unroll
                for (int pc = 0; pc < 8; ++pc) {
                    const uint32_t *xx = &x[pc >> 2][(8 * pc) & 31];
                    dst[pc] = make_uint4(pack_half2(__uint_as_float(xx[0]), __uint_as_float(xx[1])),
                                         pack_half2(__uint_as_float(xx[2]), __uint_as_float(xx[3])),
                                         pack_half2(__uint_as_float(xx[4]), __uint_as_float(xx[5])),
                                         pack_half2(__uint_as_float(xx[6]), __uint_as_float(xx[7])));
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 128);
    }
    if (tid == 0 && ms.abort_flag) atomicMin(status, (int)NATSL_ERR_TIMEOUT);
}

// ==========================================================================================
// Scan: one CTA per (batch, head) -- or per segment of its chunks, see ScanSegments --, sequential
// over chunks.  Value column r of the state (row r of
// S^T, TMEM lane r) belongs to the two threads (r, half 0) and (r, half 1) of warps q and q + 4,
// which split every row between them; warp 8 issues MMAs, warp 9 issues TMA.  The fp32 state
// lives in the registers of its two threads (half a row each); per chunk c:
//   (a) S_c (fp16 operand) -> TMEM;                          MMA: WS = S^T W^T, QS = S^T Q^T
//   (b) U~^T = U^T - WS  -> operands U~ and U~ diag(gamma_C/gamma);
//                                      MMA: dS = (U~ diag(gamma_C/gamma))^T-rows x K,  D3 = U~^T P^T
//   (c) [for chunk c-1, behind the MMAs of (b)]  o_la^T = scale_la diag(gamma) QS + D3
//   next chunk: S_{c+1} = gamma_C S_c + dS
// QS and D3 are double-buffered in TMEM so that (c) of chunk c-1 runs behind the MMAs of chunk c.
// The read-out leaves the kernel as fp16 in the orientation the row threads hold it in, one tile
// per chunk in 16-byte pieces of 8 tokens: o_laT [B,H,L/C,8 pieces,d,8 tokens], row r of piece p at
// slot r ^ p.  A thread then stores four 16-byte pieces per chunk and a warp's store is 512
// contiguous bytes, where token-major rows took one narrow store per token (the load/store unit's
// instruction rate, not its bytes, bounded that version).  The softmax kernel's epilogue copies the
// 16 KB tile into shared memory as it is and reads it transposed; the slot permutation keeps
// those reads free of bank conflicts.  Warp 10 publishes the per-chunk completion counters for a kernel that
// consumes o_laT beside this one: the release fence costs a few thousand cycles and must not sit
// on the row threads' chain.
// ==========================================================================================
constexpr int kScanRowThreads = 256;
constexpr int kScanThreads = 352;
constexpr int kScanStages = 3;
constexpr int kScanMisc = 1024;
constexpr int kDecaySlots = 8;                             // ring of per-chunk decay factors

template <int D> struct ScanLayout {
    static constexpr int KB = D / 64;
    static constexpr int kW = D * 128;                     // W^T tile: D rows x 64 tokens (fp16)
    static constexpr int kQ = KB * 8192;                   // Q tile: 64 tokens x D
    static constexpr int kK = KB * 8192;
    static constexpr int kP = 8192;
    static constexpr int kG = 512;                         // gamma_i and gamma_C / gamma_i, 64 each
    static constexpr int oW = 0, oQ = oW + kW, oK = oQ + kQ, oP = oK + kK;
    static constexpr int kStage = oP + kP;
    static constexpr int kTx = kStage + kG;
    static constexpr int oG = kScanStages * kStage;        // decay ring
    static constexpr int oMisc = oG + kDecaySlots * kG;
    static constexpr int kTotal = oMisc + kScanMisc;
    static constexpr int kTmemCols = 512;
    // TMEM columns.  dS: fp32 state increment [D].  WS: fp32 W S [64], overwritten by each thread
    // with its fp16 operands (U~ | U~ diag(gamma_C/gamma), 16 + 16 packed columns per 32 tokens).
    // A: the fp16 state operand [D/2 packed].  QS, D3: double-buffered fp32 [64] each.
    static constexpr int cS = 0, cWS = D, cA = D + 64, cQS = cA + D / 2, cD3 = cQS + 128;
    static_assert(cD3 + 128 <= 512, "TMEM budget");
};

struct ScanMisc {
    uint64_t full[kScanStages], empty[kScanStages], barA, barWS, barQS[2], barB, barSU, barD3[2];
    uint32_t tmem_base;
    int abort_flag, wait_kcycles;   // in this order: the waits read the limit as abort_flag[1]
    int emit_count;                 // row warps x chunks whose read-out rows have been stored
};
static_assert(sizeof(ScanMisc) <= kScanMisc, "misc page too small");

template <int D, bool kBlock>      // kBlock: block-level routing (softmax blocks are not committed)
__global__ void __launch_bounds__(kScanThreads, 1)
gdn_scan_tc_kernel(const __grid_constant__ CUtensorMap map_wt,
                   const __grid_constant__ CUtensorMap map_qh,
                   const __grid_constant__ CUtensorMap map_kh,
                   const __grid_constant__ CUtensorMap map_ph, const float *__restrict__ Ut,
                   const float *__restrict__ Gd, float scale_la,
                   const float *__restrict__ state_in, float *__restrict__ state_out,
                   __half *__restrict__ o_la16, float *__restrict__ o_la32, int32_t *emit_flags,
                   GdnTcExport ex, ScanSegments sg,
                   const uint8_t *__restrict__ block_route, int32_t *status, int L, int H, int wait_kcycles) {
    using SL = ScanLayout<D>;
    // A kernel launched behind this one as a programmatic dependent (the softmax branch) may start
    // as soon as every CTA of this grid is resident; it reads o_la chunk by chunk behind emit_flags.
    launch_dependents();
    constexpr int KB = SL::KB;
    constexpr int kHalfCols = D / 2;                       // state columns per thread
    extern __shared__ __align__(1024) uint8_t smem[];
    ScanMisc &ms = *reinterpret_cast<ScanMisc *>(smem + SL::oMisc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NC = L / kC;
    // Which (batch, head), which segment of its chunks, and which of the two segment runs (see
    // ScanSegments): c below counts the chunks of the segment, c0 + c is the chunk's index.
    const int var = sg.mode == 1 ? (int)(blockIdx.x & 1) : 0;
    const int slot = sg.mode == 1 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;    // bh * nseg + seg
    const int seg = sg.mode == 0 ? 0 : slot % sg.nseg;
    const int bh = sg.mode == 0 ? slot : slot / sg.nseg, b = bh / H, h = bh % H;
    const int ncs = sg.mode == 0 ? NC : sg.ncs, c0 = seg * ncs;
    const bool emit_out = sg.mode != 1, zero_u = sg.mode == 1 && var == 1;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kScanStages; ++s) { mbar_init(&ms.full[s], 1); mbar_init(&ms.empty[s], 1); }
        mbar_init(&ms.barA, kScanRowThreads);
        mbar_init(&ms.barB, kScanRowThreads);
        mbar_init(&ms.barWS, 1);
        mbar_init(&ms.barSU, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(&ms.barQS[s], 1); mbar_init(&ms.barD3[s], 1); }
        ms.abort_flag = 0;
        ms.wait_kcycles = wait_kcycles;
        ms.emit_count = 0;
        fence_mbar_init();
    }
    if (warp == 8) tmem_alloc(&ms.tmem_base, SL::kTmemCols);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ms.tmem_base;
    volatile int *abort_flag = &ms.abort_flag;

    if (warp == 9) {
        if (lane == 0) {
            int c = 0;
            for (; c < ncs; ++c) {
                const int s = c % kScanStages;
                if (!mbar_wait(&ms.empty[s], ((c / kScanStages) & 1) ^ 1, abort_flag)) break;
                uint8_t *st = smem + s * SL::kStage;
                mbar_arrive_expect_tx(&ms.full[s], SL::kTx);
                tma_load_2d(st + SL::oW, &map_wt, &ms.full[s], 0, (bh * NC + c0 + c) * D);
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(st + SL::oQ + kb * 8192, &map_qh, &ms.full[s], kb * 64, bh * L + (c0 + c) * 64);
                    tma_load_2d(st + SL::oK + kb * 8192, &map_kh, &ms.full[s], kb * 64, bh * L + (c0 + c) * 64);
                }
                tma_load_2d(st + SL::oP, &map_ph, &ms.full[s], 0, (bh * NC + c0 + c) * 64);
                // A decay slot is reused kDecaySlots chunks later, i.e. only after the stages of the
                // chunks up to c + kDecaySlots - kScanStages have been released, which every row
                // thread's work on chunk c precedes.
                bulk_load_1d(smem + SL::oG + (c % kDecaySlots) * SL::kG,
                             Gd + ((size_t)bh * NC + c0 + c) * 128, SL::kG, &ms.full[s]);
            }
            // No copy may be in flight when the CTA retires: the copies issued last are waited for
            // here, with a bound of their own and whatever the abort flag says.
            for (int u = max(0, c - kScanStages); u < c; ++u)
                mbar_wait_drain(&ms.full[u % kScanStages], (u / kScanStages) & 1);
        }
    } else if (warp == 8) {
        if (lane == 0) {
            constexpr uint32_t id_ws = make_idesc(kFmtF16, 128, 64, false, true);    // B = W^T (MN-major)
            constexpr uint32_t id_qs = make_idesc(kFmtF16, 128, 64, false, false);   // B = Q
            constexpr uint32_t id_su = make_idesc(kFmtF16, 128, D, false, true);     // B = K (MN-major)
            constexpr uint32_t id_pu = make_idesc(kFmtF16, 128, 64, false, false);   // B = P
            for (int c = 0; c < ncs; ++c) {
                const int s = c % kScanStages;
                const uint32_t st = smem_u32(smem + s * SL::kStage);
                if (!mbar_wait(&ms.full[s], (c / kScanStages) & 1, abort_flag)) break;
                if (!mbar_wait(&ms.barA, c & 1, abort_flag)) break;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    mma_ts(tmem + SL::cWS, tmem + SL::cA + kk * 8,
                           desc_mnmajor(st + SL::oW + kk * 2048, 0), id_ws, kk != 0);
                mma_commit(&ms.barWS);
                if (emit_out) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ts(tmem + SL::cQS + 64 * (c & 1), tmem + SL::cA + kk * 8,
                               desc_kmajor(st + SL::oQ + (kk >> 2) * 8192 + (kk & 3) * 32), id_qs, kk != 0);
                    mma_commit(&ms.barQS[c & 1]);
                }
                if (!mbar_wait(&ms.barB, c & 1, abort_flag)) break;
                tc_fence_after_sync();
                // The state update first: it is on the chain between the chunks.  The output product
                // behind it still reads its operand from the WS columns after barSU has fired; the
                // next writer of those columns is the next chunk's W S product, issued behind it by
                // this thread, and MMAs of one thread execute in issue order.
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16)
                    mma_ts(tmem + SL::cS, tmem + SL::cWS + (k16 >> 1) * 32 + 16 + (k16 & 1) * 8,
                           desc_mnmajor(st + SL::oK + k16 * 2048, 8192), id_su, k16 != 0);
                mma_commit(&ms.barSU);
                if (emit_out) {
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16)
                        mma_ts(tmem + SL::cD3 + 64 * (c & 1), tmem + SL::cWS + (k16 >> 1) * 32 + (k16 & 1) * 8,
                               desc_kmajor(st + SL::oP + k16 * 32), id_pu, k16 != 0);
                    mma_commit(&ms.barD3[c & 1]);
                }
                mma_commit(&ms.empty[s]);
            }
        }
    } else if (warp == 10) {
        // Publisher: raises the per-chunk counters once all eight row warps have stored a chunk's
        // rows.  The row warps count in shared memory (after a block-scope fence); the gpu-scope
        // fence here then covers their stores, as in the usual "barrier, one thread fences and
        // sets the flag" hand-over.  Several chunks are published behind one fence when it lags.
        if (lane == 0 && emit_flags && emit_out) {
            volatile int *cnt = &ms.emit_count;
            const long long limit = wait_limit(abort_flag);
            long long t0 = clock64();
            int published = 0;
            while (published < ncs) {
                const int done = *cnt / kScanRowWarps;
                if (done > published) {
                    __threadfence();
                    for (int c = published; c < done; ++c)
                        red_release_add(emit_flags + (size_t)bh * NC + c0 + c, kScanRowWarps);
                    published = done;
                    t0 = clock64();
                } else {
                    if (*abort_flag) break;
                    if (clock64() - t0 > limit) { *abort_flag = 1; break; }
                    __nanosleep(128);
                }
            }
        }
    } else {
        const int q = warp & 3, half = warp >> 2;
        const int r = q * 32 + lane;                      // value column / TMEM lane
        const bool active = r < D;                        // d = 64: rows 64-127 are zero padding
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const int col0 = half * kHalfCols;                // this thread's state columns (key dim)
        const int tk0 = half * 32;                        // ... and its tokens of every chunk
        float S[kHalfCols];                               // fp32 state at the entry of the current chunk
#pragma unroll
        for (int x = 0; x < kHalfCols; ++x)
            S[x] = !active ? 0.f
                   : sg.mode == 1 ? (var == 1 && col0 + x == r ? 1.f : 0.f)
                   : sg.mode == 2 ? sg.start[((size_t)slot * D + col0 + x) * D + r]
                   : state_in     ? state_in[((size_t)bh * D + col0 + x) * D + r]
                                  : 0.f;
        // This thread's 8 pieces (4 tokens each) of row r of U^T of chunk c.
        auto u_src = [&](int c) {
            return reinterpret_cast<const float4 *>(Ut + ((size_t)bh * NC + c0 + c) * D * 64) + (tk0 / 4) * D + r;
        };
        // The U row of the next chunk is only pulled into L2 ahead of time and loaded into registers
        // right before it is used: a global load left in flight across TMEM loads makes their
        // consumers wait for it as well.
        auto prefetch_u = [&](int c) {
            if (active && !zero_u) {
                const float4 *src = u_src(c);
#pragma unroll
                for (int x = 0; x < 8; ++x) prefetch_l2(src + x * D);
            }
        };
        // (c): output rows of chunk c (its QS / D3 buffers and decay slot are still intact)
        auto emit = [&](int c) -> bool {
            const float *e1 = reinterpret_cast<const float *>(smem + SL::oG + (c % kDecaySlots) * SL::kG);
            if (!mbar_wait(&ms.barQS[c & 1], (c >> 1) & 1, abort_flag)) return false;
            if (!mbar_wait(&ms.barD3[c & 1], (c >> 1) & 1, abort_flag)) return false;
            tc_fence_after_sync();
            const size_t off = (((size_t)b * L + (size_t)(c0 + c) * 64 + tk0) * H + h) * D + r;
            uint32_t pk[16];                               // this thread's 32 tokens of row r, fp16 pairs
#pragma unroll
            for (int part = 0; part < 2; ++part) {        // 16 tokens at a time keeps registers low
                uint32_t x[16], y[16];
                tmem_ld16(tmem + SL::cQS + 64 * (c & 1) + tk0 + 16 * part + lane_base, x);
                tmem_ld16(tmem + SL::cD3 + 64 * (c & 1) + tk0 + 16 * part + lane_base, y);
                tmem_wait_ld();
                float o[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    o[i] = fmaf(scale_la * e1[tk0 + 16 * part + i], __uint_as_float(x[i]), __uint_as_float(y[i]));
#pragma unroll
                for (int i = 0; i < 8; ++i) pk[8 * part + i] = pack_half2(o[2 * i], o[2 * i + 1]);
                if (o_la32 && active) {                    // fp32 token-major copy (tests, backward)
#pragma unroll
                    for (int i = 0; i < 16; ++i) o_la32[off + (size_t)(16 * part + i) * H * D] = o[i];
                }
            }
            if (active) {
                uint4 *dst = reinterpret_cast<uint4 *>(o_la16 + ((size_t)bh * NC + c0 + c) * D * 64);
#pragma unroll
                for (int x4 = 0; x4 < 4; ++x4) {
                    const int pc = tk0 / 8 + x4;
                    dst[pc * D + (r ^ pc)] = make_uint4(pk[4 * x4], pk[4 * x4 + 1], pk[4 * x4 + 2], pk[4 * x4 + 3]);
                }
            }
            tc_fence_before_sync();
            // this warp's rows of the chunk are stored: count it for the publisher
            if (emit_flags) {
                __syncwarp();
                if (lane == 0) {
                    __threadfence_block();
                    atomicAdd(&ms.emit_count, 1);
                }
            }
            return true;
        };
        prefetch_u(0);
        bool ok = true;
        for (int c = 0; c < ncs && ok; ++c) {
            const int s = c % kScanStages;
            const float *e1 = reinterpret_cast<const float *>(smem + SL::oG + (c % kDecaySlots) * SL::kG);
            const float *e2 = e1 + 64;
            // Block-level routing: the delta rule runs over every block, but a softmax block's
            // update is not committed -- its state increment is multiplied by zero, so that the
            // state only decays across it (Section 4.3, the decay-always equation).
            const float commit =
                kBlock && block_route[((size_t)b * L + (size_t)(c0 + c) * 64) * H + h] ? 0.f : 1.f;
            ok = mbar_wait(&ms.full[s], (c / kScanStages) & 1, abort_flag);
            if (!ok) break;
            if (c > 0) {                                   // S_c = gamma_C S_{c-1} + dS_{c-1}
                ok = mbar_wait(&ms.barSU, (c - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                // decay across the previous chunk and its increment in one pass over the row
                const float gC = reinterpret_cast<const float *>(smem + SL::oG + ((c - 1) % kDecaySlots) * SL::kG)[63];
#pragma unroll
                for (int cb = 0; cb < kHalfCols / 32; ++cb) {
                    uint32_t ds[32];
                    tmem_ld32(tmem + SL::cS + col0 + cb * 32 + lane_base, ds);
                    tmem_wait_ld();
#pragma unroll
                    for (int x = 0; x < 32; ++x) S[cb * 32 + x] = fmaf(S[cb * 32 + x], gC, __uint_as_float(ds[x]));
                }
                tc_fence_before_sync();
            }
            // ---- (a) state row -> fp16 operand in TMEM; decay the register copy afterwards ----
            {
                uint32_t pk[kHalfCols / 2];
#pragma unroll
                for (int x = 0; x < kHalfCols / 2; ++x) pk[x] = pack_half2(S[2 * x], S[2 * x + 1]);
                if (kHalfCols == 64)
                    tmem_st32(tmem + SL::cA + half * (kHalfCols / 2) + lane_base,
                              reinterpret_cast<const uint32_t (&)[32]>(pk));
                else
                    tmem_st16(tmem + SL::cA + half * (kHalfCols / 2) + lane_base,
                              reinterpret_cast<const uint32_t (&)[16]>(pk));
                tmem_wait_st();
            }
            tc_fence_before_sync();
            mbar_arrive(&ms.barA);
            // (exports for the backward go behind the arrivals, off the chain between the chunks)
            if (ex.S_c && active) {      // chunk-entry state, [B,H,L/C,dk,dv]
                float *sc = ex.S_c + (((size_t)bh * NC + c0 + c) * D + col0) * D + r;
#pragma unroll
                for (int x = 0; x < kHalfCols; ++x) sc[(size_t)x * D] = S[x];
            }
            float u[32];                                   // from L2; lands while W S is computed
            if (active && !zero_u) {
                const float4 *src = u_src(c);
#pragma unroll
                for (int x = 0; x < 8; ++x) {
                    const float4 a = __ldg(src + x * D);
                    u[4 * x] = a.x; u[4 * x + 1] = a.y; u[4 * x + 2] = a.z; u[4 * x + 3] = a.w;
                }
            } else {
#pragma unroll
                for (int x = 0; x < 32; ++x) u[x] = 0.f;
            }
            // ---- (b) U~ = U - W S for this thread's 32 tokens ----
            ok = mbar_wait(&ms.barWS, c & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            {
                uint32_t ws[32];
                tmem_ld32(tmem + SL::cWS + tk0 + lane_base, ws);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) u[j] -= __uint_as_float(ws[j]);
            }
            {
                uint32_t pk[32];     // [0,16): U~ of this thread's 32 tokens, [16,32): U~ gamma_C/gamma
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    pk[x] = pack_half2(u[2 * x], u[2 * x + 1]);
                    const float f0 = kBlock ? commit * e2[tk0 + 2 * x] : e2[tk0 + 2 * x];
                    const float f1 = kBlock ? commit * e2[tk0 + 2 * x + 1] : e2[tk0 + 2 * x + 1];
                    pk[16 + x] = pack_half2(u[2 * x] * f0, u[2 * x + 1] * f1);
                }
                tmem_st32(tmem + SL::cWS + tk0 + lane_base, pk);   // over this thread's own W S columns
                tmem_wait_st();
            }
            tc_fence_before_sync();
            mbar_arrive(&ms.barB);
            if (ex.Ut && active) {       // U~, token-major
                float *ut = ex.Ut + (((size_t)b * L + (size_t)(c0 + c) * 64 + tk0) * H + h) * D + r;
#pragma unroll
                for (int j = 0; j < 32; ++j) ut[(size_t)j * H * D] = u[j];
            }
            // ---- behind the MMAs just released: next U row towards L2, previous chunk's output ----
            if (c + 1 < ncs) prefetch_u(c + 1);
            if (c > 0 && emit_out) ok = emit(c - 1);
        }
        if (ok && emit_out) ok = emit(ncs - 1);
        // where the state after the segment's last chunk goes
        float *final_state = sg.mode == 1 ? (var ? sg.trans : sg.incr) + (size_t)slot * D * D
                             : state_out && (sg.mode == 0 || seg == sg.nseg - 1) ? state_out + (size_t)bh * D * D
                                                                                   : nullptr;
        if (ok && final_state) {
            ok = mbar_wait(&ms.barSU, (ncs - 1) & 1, abort_flag);
            if (ok) {
                tc_fence_after_sync();
                const float gC_last =
                    reinterpret_cast<const float *>(smem + SL::oG + ((ncs - 1) % kDecaySlots) * SL::kG)[63];
#pragma unroll
                for (int cb = 0; cb < kHalfCols / 32; ++cb) {
                    uint32_t ds[32];
                    tmem_ld32(tmem + SL::cS + col0 + cb * 32 + lane_base, ds);
                    tmem_wait_ld();
                    if (active) {
#pragma unroll
                        for (int x = 0; x < 32; ++x)
                            final_state[(size_t)(col0 + cb * 32 + x) * D + r] =
                                fmaf(S[cb * 32 + x], gC_last, __uint_as_float(ds[x]));
                    }
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 8) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, SL::kTmemCols);
    }
    if (tid == 0 && ms.abort_flag) atomicMin(status, (int)NATSL_ERR_TIMEOUT);
}

// start[0] = state_in (or 0); start[s+1] = M_s start[s] + B_s.  The value columns are independent:
// one CTA per (batch, head) and 8 of them; thread (ag, v) owns key rows ag, ag + 32, ... of column v.
// M_s is staged through shared memory in tiles of 32 columns (coalesced 128-byte rows).
template <int D>
__global__ void __launch_bounds__(256)
scan_combine_kernel(const float *__restrict__ state_in, const float *__restrict__ incr,
                    const float *__restrict__ trans, float *__restrict__ start, int nseg) {
    constexpr int kV = 8, kRows = D / 32;
    __shared__ float Ss[D][kV + 1];
    __shared__ float Ms[D][33];
    const int bh = blockIdx.y, v0 = blockIdx.x * kV, v = threadIdx.x & (kV - 1), ag = threadIdx.x >> 3;
    for (int i = 0; i < kRows; ++i) {
        const int a = ag + 32 * i;
        Ss[a][v] = state_in ? state_in[((size_t)bh * D + a) * D + v0 + v] : 0.f;
    }
    __syncthreads();
    // The tiles of M are fetched one step ahead into registers, so that the chain over the segments
    // pays one global-memory latency per segment rather than one per tile.
    constexpr int kTileRegs = D * 32 / 256;
    float tile[kTileRegs];
    auto fetch = [&](int sgi, int b0) {
        const float *src = trans + ((size_t)bh * nseg + sgi) * D * D + b0;
#pragma unroll
        for (int i = 0; i < kTileRegs; ++i) {
            const int idx = threadIdx.x + 256 * i;
            tile[i] = src[(size_t)(idx >> 5) * D + (idx & 31)];
        }
    };
    if (nseg > 1) fetch(0, 0);
    for (int sgi = 0; sgi < nseg; ++sgi) {
        const size_t base = ((size_t)bh * nseg + sgi) * D * D;
        for (int i = 0; i < kRows; ++i) start[base + (size_t)(ag + 32 * i) * D + v0 + v] = Ss[ag + 32 * i][v];
        if (sgi + 1 == nseg) break;
        float acc[kRows];
#pragma unroll
        for (int i = 0; i < kRows; ++i) acc[i] = incr[base + (size_t)(ag + 32 * i) * D + v0 + v];
        for (int b0 = 0; b0 < D; b0 += 32) {
#pragma unroll
            for (int i = 0; i < kTileRegs; ++i) {                         // M[a][b0 .. b0+31]
                const int idx = threadIdx.x + 256 * i;
                Ms[idx >> 5][idx & 31] = tile[i];
            }
            __syncthreads();
            if (b0 + 32 < D) fetch(sgi, b0 + 32);
            else if (sgi + 2 < nseg) fetch(sgi + 1, 0);
#pragma unroll
            for (int i = 0; i < kRows; ++i) {
                const float *mr = Ms[ag + 32 * i];
#pragma unroll 8
                for (int bb = 0; bb < 32; ++bb) acc[i] = fmaf(mr[bb], Ss[b0 + bb][v], acc[i]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int i = 0; i < kRows; ++i) Ss[ag + 32 * i][v] = acc[i];
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_scan_combine(const float *state_in, const ScanSegments &sg, Shape s, cudaStream_t st) {
    dim3 grid(s.d / 8, s.B * s.H);
    if (s.d == 128) scan_combine_kernel<128><<<grid, 256, 0, st>>>(state_in, sg.incr, sg.trans, sg.start, sg.nseg);
    else scan_combine_kernel<64><<<grid, 256, 0, st>>>(state_in, sg.incr, sg.trans, sg.start, sg.nseg);
    count_launch();
    return cudaGetLastError();
}

template <int D>
static cudaError_t prepare_tc_impl(const void *q, const void *k, const void *v, const float *g,
                                   const float *beta, const uint8_t *route, float scale_la,
                                   const GdnTcWs &ws, const GdnTcExport &ex, int32_t *status,
                                   float norm_eps, Shape s, cudaStream_t st) {
    const int NC = s.L / kC;
    const uint64_t BH = (uint64_t)s.B * s.H;
    CUtensorMap mq, mk, mv, mqh, mkh;
    if (!tch::make_map_blhd(&mq, q, s.B, s.L, s.H, D, 64) ||
        !tch::make_map_blhd(&mk, k, s.B, s.L, s.H, D, 64) ||
        !tch::make_map_blhd(&mv, v, s.B, s.L, s.H, D, 64) ||
        !tch::make_map_2d(&mqh, ws.Qh, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mkh, ws.Kh, BH * s.L, D, 64))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(gdn_prepare_tc_kernel<D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         PrepLayout<D>::kTotal);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)NC * (unsigned)BH);
    gdn_prepare_tc_kernel<D><<<grid, kPrepThreads, PrepLayout<D>::kTotal, st>>>(
        mq, mk, mv, mqh, mkh, g, beta, route, scale_la, (__half *)ws.Wt, ws.Ut, (__half *)ws.Ph, ws.Gd, ex,
        status, s.L, s.H, norm_eps, debug_wait_kcycles());
    count_launch();
    return cudaGetLastError();
}

template <int D>
static cudaError_t scan_tc_impl(const GdnTcWs &ws, float scale_la, const float *state_in,
                                float *state_out, const ScanOut &out, const GdnTcExport &ex,
                                const ScanSegments &sg, const uint8_t *block_route, int32_t *status,
                                Shape s, cudaStream_t st) {
    const int NC = s.L / kC;
    const uint64_t BH = (uint64_t)s.B * s.H;
    CUtensorMap mwt, mqh, mkh, mph;
    if (!tch::make_map_2d(&mwt, ws.Wt, BH * NC * D, 64, D) ||
        !tch::make_map_2d(&mqh, ws.Qh, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mkh, ws.Kh, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mph, ws.Ph, BH * NC * 64, 64, 64))
        return cudaErrorInvalidValue;
    auto kernel = block_route ? gdn_scan_tc_kernel<D, true> : gdn_scan_tc_kernel<D, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ScanLayout<D>::kTotal);
    if (e != cudaSuccess) return e;
    const int ctas = s.B * s.H * (sg.mode == 0 ? 1 : sg.nseg) * (sg.mode == 1 ? 2 : 1);
    kernel<<<ctas, kScanThreads, ScanLayout<D>::kTotal, st>>>(
        mwt, mqh, mkh, mph, ws.Ut, ws.Gd, scale_la, state_in, state_out, (__half *)out.o_la16, out.o_la32,
        out.emit_flags, ex, sg, block_route, status, s.L, s.H, debug_wait_kcycles());
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_prepare_tc(const void *q, const void *k, const void *v, const float *g,
                                  const float *beta, const uint8_t *route, float scale_la,
                                  const GdnTcWs &ws, const GdnTcExport &ex, int32_t *status, Shape s,
                                  cudaStream_t st, float norm_eps) {
    if (s.d == 128) return prepare_tc_impl<128>(q, k, v, g, beta, route, scale_la, ws, ex, status, norm_eps, s, st);
    return prepare_tc_impl<64>(q, k, v, g, beta, route, scale_la, ws, ex, status, norm_eps, s, st);
}

cudaError_t launch_gdn_scan_tc(const GdnTcWs &ws, float scale_la, const float *state_in,
                               float *state_out, const ScanOut &out, const GdnTcExport &ex,
                               const ScanSegments &sg, const uint8_t *block_route, int32_t *status,
                               Shape s, cudaStream_t st) {
    if (s.d == 128)
        return scan_tc_impl<128>(ws, scale_la, state_in, state_out, out, ex, sg, block_route, status, s, st);
    return scan_tc_impl<64>(ws, scale_la, state_in, state_out, out, ex, sg, block_route, status, s, st);
}

}  // namespace natsl

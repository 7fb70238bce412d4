// Tensor-core reverse scan of the chunkwise Gated DeltaNet backward (bf16 storage, sm_100a).
//
// With the notation of gdn_tc.cu and, per chunk, S0 = entry state, dS1 = gradient w.r.t. the exit
// state, dO = gradient of the linear read-out:
//   dU~ = P^T dO + diag(gamma_C / gamma) K dS1
//   dS0 = (scale_la diag(gamma) Q)^T dO + gamma_C dS1 - W^T dU~
// One CTA per (batch, head) walks the chunks backwards.  As in the forward scan the head dimension
// sits on the MMA's M axis: value column r of dS (row r of dS^T, TMEM lane r) belongs to the two
// threads (r, half 0 / 1) of warps q and q + 4, the fp32 gradient state lives in their registers,
// and the operands a thread produces (dS1, dU~ as fp16) are written to its own TMEM lane:
//   X1 = dO^T P            X2 = dS1^T K^T                       (both [d, 64 tokens])
//   dU~^T = X1 + X2 diag(gamma_C / gamma)        -> global (fp32, token-major) and fp16 operand
//   Y  = (diag(scale_la gamma) dO)^T Q - dU~^T W                ([d, d], second product negated)
//   dS0^T = gamma_C dS1^T + Y
// dO and scale_la gamma dO arrive as fp16 tiles [B,H,L,d]; P, W^T and the fp16 q, k copies are the
// forward's own intermediates.  The chunk-exit gradients dS1 are stored for the later products.
#include "common.cuh"
#include "natsl_internal.h"
#include "tc_common.cuh"

namespace natsl {

namespace {

using namespace tc;

constexpr int kRsRowThreads = 256;
constexpr int kRsThreads = 320;
constexpr int kRsStages = 2;
constexpr int kRsMisc = 1024;
constexpr int kRsDecaySlots = 4;

template <int D> struct RsLayout {
    static constexpr int KB = D / 64;
    static constexpr int kT = KB * 8192;                   // a 64-token x D fp16 tile
    static constexpr int oDO = 0, oDOg = kT, oQ = 2 * kT, oK = 3 * kT, oW = 4 * kT;   // W^T: D rows x 64
    static constexpr int oP = oW + D * 128;
    static constexpr int kStage = oP + 8192;
    static constexpr int kG = 512;
    static constexpr int kTx = kStage + kG;
    static constexpr int oG = kRsStages * kStage;
    static constexpr int oMisc = oG + kRsDecaySlots * kG;
    static constexpr int kTotal = oMisc + kRsMisc;
    // TMEM columns: X1 [64], X2 [64] (X2's columns are then reused for the fp16 dU~ operand),
    // Y [D], A = fp16 dS1 operand [D/2 packed].
    static constexpr int cX1 = 0, cX2 = 64, cY = 128, cA = 128 + D;
    static constexpr int kTmemCols = D == 128 ? 512 : 256;
};

struct RsMisc {
    uint64_t full[kRsStages], empty[kRsStages], barA, barX, barB, barY;
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(RsMisc) <= kRsMisc, "misc page too small");

template <int D>
__global__ void __launch_bounds__(kRsThreads, 1)
gdn_rscan_tc_kernel(const __grid_constant__ CUtensorMap map_do,    // dO (fp16) [B*H*L][D], box 64
                    const __grid_constant__ CUtensorMap map_dog,   // scale_la gamma dO (fp16), box 64
                    const __grid_constant__ CUtensorMap map_qh, const __grid_constant__ CUtensorMap map_kh,
                    const __grid_constant__ CUtensorMap map_wt,    // W^T [B*H*NC*D][64], box D
                    const __grid_constant__ CUtensorMap map_ph,    // P [B*H*NC*64][64], box 64
                    const float *__restrict__ Gd, float *__restrict__ dUt, float *__restrict__ dS_c,
                    int32_t *status, int L, int H) {
    using SL = RsLayout<D>;
    constexpr int KB = SL::KB;
    constexpr int kHalfCols = D / 2;
    extern __shared__ __align__(1024) uint8_t smem[];
    RsMisc &ms = *reinterpret_cast<RsMisc *>(smem + SL::oMisc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NC = L / kC;
    const int bh = blockIdx.x, b = bh / H, h = bh % H;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kRsStages; ++s) { mbar_init(&ms.full[s], 1); mbar_init(&ms.empty[s], 1); }
        mbar_init(&ms.barA, kRsRowThreads);
        mbar_init(&ms.barB, kRsRowThreads);
        mbar_init(&ms.barX, 1);
        mbar_init(&ms.barY, 1);
        ms.abort_flag = 0;
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
            int n = 0;                                      // n-th chunk processed = chunk NC - 1 - n
            for (; n < NC; ++n) {
                const int c = NC - 1 - n, s = n % kRsStages;
                if (!mbar_wait(&ms.empty[s], ((n / kRsStages) & 1) ^ 1, abort_flag)) break;
                uint8_t *st = smem + s * SL::kStage;
                mbar_arrive_expect_tx(&ms.full[s], SL::kTx);
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(st + SL::oDO + kb * 8192, &map_do, &ms.full[s], kb * 64, bh * L + c * 64);
                    tma_load_2d(st + SL::oDOg + kb * 8192, &map_dog, &ms.full[s], kb * 64, bh * L + c * 64);
                    tma_load_2d(st + SL::oQ + kb * 8192, &map_qh, &ms.full[s], kb * 64, bh * L + c * 64);
                    tma_load_2d(st + SL::oK + kb * 8192, &map_kh, &ms.full[s], kb * 64, bh * L + c * 64);
                }
                tma_load_2d(st + SL::oW, &map_wt, &ms.full[s], 0, (bh * NC + c) * D);
                tma_load_2d(st + SL::oP, &map_ph, &ms.full[s], 0, (bh * NC + c) * 64);
                bulk_load_1d(smem + SL::oG + (n % kRsDecaySlots) * SL::kG, Gd + ((size_t)bh * NC + c) * 128,
                             SL::kG, &ms.full[s]);
            }
            if (*abort_flag)
                for (int u = max(0, n - kRsStages); u < n; ++u)
                    mbar_wait(&ms.full[u % kRsStages], (u / kRsStages) & 1, abort_flag);
        }
    } else if (warp == 8) {
        if (lane == 0) {
            constexpr uint32_t id_x1 = make_idesc(kFmtF16, 128, 64, true, true);    // A = dO (MN), B = P (MN)
            constexpr uint32_t id_x2 = make_idesc(kFmtF16, 128, 64, false, false);  // A = dS1 (TMEM), B = K
            constexpr uint32_t id_y1 = make_idesc(kFmtF16, 128, D, true, true);     // A = dOg (MN), B = Q (MN)
            constexpr uint32_t id_y2 = make_idesc(kFmtF16, 128, D, false, false, true);   // -dU~ (TMEM) x W^T
            for (int n = 0; n < NC; ++n) {
                const int s = n % kRsStages;
                const uint32_t st = smem_u32(smem + s * SL::kStage);
                if (!mbar_wait(&ms.full[s], (n / kRsStages) & 1, abort_flag)) break;
                tc_fence_after_sync();
                // X1 does not involve the gradient state and its columns are free (every row thread
                // read them before its barB arrival of the previous chunk): issue it ahead.
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16)
                    mma_ss(tmem + SL::cX1, desc_mnmajor(st + SL::oDO + k16 * 2048, 8192),
                           desc_mnmajor(st + SL::oP + k16 * 2048, 0), id_x1, k16 != 0);
                // barA: the row threads have consumed the previous chunk's Y and written dS1.
                if (!mbar_wait(&ms.barA, n & 1, abort_flag)) break;
                tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    mma_ts(tmem + SL::cX2, tmem + SL::cA + kk * 8,
                           desc_kmajor(st + SL::oK + (kk >> 2) * 8192 + (kk & 3) * 32), id_x2, kk != 0);
                mma_commit(&ms.barX);
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16)
                    mma_ss(tmem + SL::cY, desc_mnmajor(st + SL::oDOg + k16 * 2048, 8192),
                           desc_mnmajor(st + SL::oQ + k16 * 2048, 8192), id_y1, k16 != 0);
                if (!mbar_wait(&ms.barB, n & 1, abort_flag)) break;
                tc_fence_after_sync();
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16)
                    mma_ts(tmem + SL::cY, tmem + SL::cX2 + (k16 >> 1) * 32 + (k16 & 1) * 8,
                           desc_kmajor(st + SL::oW + k16 * 32), id_y2, true);
                mma_commit(&ms.barY);
                mma_commit(&ms.empty[s]);
            }
        }
    } else {
        const int q = warp & 3, half = warp >> 2;
        const int r = q * 32 + lane;
        const bool active = r < D;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const int col0 = half * kHalfCols, tk0 = half * 32;
        float G[kHalfCols];                                 // dS^T row r, key columns col0..
#pragma unroll
        for (int x = 0; x < kHalfCols; ++x) G[x] = 0.f;
        bool ok = true;
        for (int n = 0; n < NC && ok; ++n) {
            const int c = NC - 1 - n, s = n % kRsStages;
            const float *e1 = reinterpret_cast<const float *>(smem + SL::oG + (n % kRsDecaySlots) * SL::kG);
            const float *e2 = e1 + 64;
            // ---- dS1 (exit-state gradient of chunk c): store, and fp16 operand into TMEM ----
            if (active) {
                float *dst = dS_c + (((size_t)bh * NC + c) * D + col0) * D + r;
#pragma unroll
                for (int x = 0; x < kHalfCols; ++x) dst[(size_t)x * D] = G[x];
            }
            {
                uint32_t pk[kHalfCols / 2];
#pragma unroll
                for (int x = 0; x < kHalfCols / 2; ++x) pk[x] = pack_half2(G[2 * x], G[2 * x + 1]);
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
            ok = mbar_wait(&ms.full[s], (n / kRsStages) & 1, abort_flag);   // decay factors of the chunk
            if (!ok) break;
            {
                const float gC = e1[63];
#pragma unroll
                for (int x = 0; x < kHalfCols; ++x) G[x] *= gC;
            }
            // ---- dU~ for this thread's 32 tokens ----
            ok = mbar_wait(&ms.barX, n & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            {
                uint32_t x1[32], x2[32];
                tmem_ld32(tmem + SL::cX1 + tk0 + lane_base, x1);
                tmem_ld32(tmem + SL::cX2 + tk0 + lane_base, x2);
                tmem_wait_ld();
                float du[32];
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    du[j] = fmaf(e2[tk0 + j], __uint_as_float(x2[j]), __uint_as_float(x1[j]));
                if (active) {
                    float *dst = dUt + (((size_t)b * L + (size_t)c * 64 + tk0) * H + h) * D + r;
#pragma unroll
                    for (int j = 0; j < 32; ++j) dst[(size_t)j * H * D] = du[j];
                }
                uint32_t pk[16];
#pragma unroll
                for (int x = 0; x < 16; ++x) pk[x] = pack_half2(du[2 * x], du[2 * x + 1]);
                // into this thread's own X2 columns: 16 packed columns per 32 tokens
                tmem_st16(tmem + SL::cX2 + tk0 + lane_base, pk);
                tmem_wait_st();
            }
            tc_fence_before_sync();
            mbar_arrive(&ms.barB);
            // ---- dS0 = gamma_C dS1 + Y ----
            ok = mbar_wait(&ms.barY, n & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int cb = 0; cb < kHalfCols / 32; ++cb) {
                uint32_t y[32];
                tmem_ld32(tmem + SL::cY + col0 + cb * 32 + lane_base, y);
                tmem_wait_ld();
#pragma unroll
                for (int x = 0; x < 32; ++x) G[cb * 32 + x] += __uint_as_float(y[x]);
            }
            tc_fence_before_sync();
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

// gS[chunk] = <dS1[chunk], S0[chunk]> (first slot of the row; the other slots are zeroed).
__global__ void __launch_bounds__(256)
state_dot_kernel(const float *__restrict__ dS_c, const float *__restrict__ S_c, float *__restrict__ gS,
                 int n_slices, int dd) {
    __shared__ float red[8];
    const size_t chunk = blockIdx.x;
    const float4 *a = reinterpret_cast<const float4 *>(dS_c + chunk * dd);
    const float4 *bq = reinterpret_cast<const float4 *>(S_c + chunk * dd);
    float acc = 0.f;
    for (int i = threadIdx.x; i < dd / 4; i += 256) {
        const float4 x = a[i], y = bq[i];
        acc = fmaf(x.x, y.x, fmaf(x.y, y.y, fmaf(x.z, y.z, fmaf(x.w, y.w, acc))));
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int wv = 0; wv < 8; ++wv) t += red[wv];
        gS[chunk * n_slices] = t;
        for (int sl = 1; sl < n_slices; ++sl) gS[chunk * n_slices + sl] = 0.f;
    }
}

}  // namespace

template <int D>
static cudaError_t rscan_tc_impl(const void *dO16, const void *dOg16, const GdnTcWs &ws,
                                 const float *S_c, float *dUt, float *dS_c, float *gS,
                                 int32_t *status, Shape s, cudaStream_t st) {
    const int NC = s.L / kC;
    const uint64_t BH = (uint64_t)s.B * s.H;
    CUtensorMap mdo, mdog, mqh, mkh, mwt, mph;
    if (!tch::make_map_2d(&mdo, dO16, BH * s.L, D, 64) || !tch::make_map_2d(&mdog, dOg16, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mqh, ws.Qh, BH * s.L, D, 64) || !tch::make_map_2d(&mkh, ws.Kh, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mwt, ws.Wt, BH * NC * D, 64, D) || !tch::make_map_2d(&mph, ws.Ph, BH * NC * 64, 64, 64))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(gdn_rscan_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         RsLayout<D>::kTotal);
    if (e != cudaSuccess) return e;
    gdn_rscan_tc_kernel<D><<<s.B * s.H, kRsThreads, RsLayout<D>::kTotal, st>>>(
        mdo, mdog, mqh, mkh, mwt, mph, ws.Gd, dUt, dS_c, status, s.L, s.H);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    state_dot_kernel<<<(unsigned)(BH * NC), 256, 0, st>>>(dS_c, S_c, gS, D / 32, D * D);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_rscan_tc(const void *dO16, const void *dOg16, const GdnTcWs &ws,
                                const float *S_c, float *dUt, float *dS_c, float *gS,
                                int32_t *status, Shape s, cudaStream_t st) {
    if (s.d == 128) return rscan_tc_impl<128>(dO16, dOg16, ws, S_c, dUt, dS_c, gS, status, s, st);
    return rscan_tc_impl<64>(dO16, dOg16, ws, S_c, dUt, dS_c, gS, status, s, st);
}

}  // namespace natsl

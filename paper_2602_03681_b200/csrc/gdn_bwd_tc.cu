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
    int abort_flag, wait_kcycles;   // in this order: the waits read the limit as abort_flag[1]
};
static_assert(sizeof(RsMisc) <= kRsMisc, "misc page too small");

template <int D, bool kBlock>      // kBlock: block-level routing (softmax blocks were not committed)
__global__ void __launch_bounds__(kRsThreads, 1)
gdn_rscan_tc_kernel(const __grid_constant__ CUtensorMap map_do,    // dO (fp16) [B*H*L][D], box 64
                    const __grid_constant__ CUtensorMap map_dog,   // scale_la gamma dO (fp16), box 64
                    const __grid_constant__ CUtensorMap map_qh, const __grid_constant__ CUtensorMap map_kh,
                    const __grid_constant__ CUtensorMap map_wt,    // W^T [B*H*NC*D][64], box D
                    const __grid_constant__ CUtensorMap map_ph,    // P [B*H*NC*64][64], box 64
                    const float *__restrict__ Gd, float *__restrict__ dUt, float *__restrict__ dS_c,
                    const float *__restrict__ dstate_out, float *__restrict__ dstate_in,
                    const uint8_t *__restrict__ block_route, int32_t *status, int L, int H, int wait_kcycles) {
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
        ms.wait_kcycles = wait_kcycles;
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
            for (int u = max(0, n - kRsStages); u < n; ++u)      // no copy in flight at retirement
                mbar_wait_drain(&ms.full[u % kRsStages], (u / kRsStages) & 1);
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
        // The read-out gradients arrive times the power of two gsc.x (grad_scale): the gradient
        // state is carried in those units, and what leaves the kernel is multiplied by gsc.y = 1 / gsc.x.
        const float2 gsc = grad_scale(status);
        float G[kHalfCols];                                 // dS^T row r, key columns col0..
#pragma unroll
        for (int x = 0; x < kHalfCols; ++x)     // gradient arriving at the final state, if any
            G[x] = active && dstate_out ? gsc.x * dstate_out[((size_t)bh * D + col0 + x) * D + r] : 0.f;
        bool ok = true;
        for (int n = 0; n < NC && ok; ++n) {
            const int c = NC - 1 - n, s = n % kRsStages;
            const float *e1 = reinterpret_cast<const float *>(smem + SL::oG + (n % kRsDecaySlots) * SL::kG);
            const float *e2 = e1 + 64;
            // block-level routing: the update K~^T U~ of a softmax block never reached the state,
            // so the exit-state gradient does not flow into its dU~ (it still decays into dS0)
            const float commit = kBlock && block_route[((size_t)b * L + (size_t)c * 64) * H + h] ? 0.f : 1.f;
            // ---- dS1 (exit-state gradient of chunk c): fp16 operand into TMEM, then (behind the
            // arrival, off the chain) the fp32 copy the later products read ----
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
            if (active) {
                float *dst = dS_c + (((size_t)bh * NC + c) * D + col0) * D + r;
#pragma unroll
                for (int x = 0; x < kHalfCols; ++x) dst[(size_t)x * D] = gsc.y * G[x];
            }
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
            float du[32];
            {
                uint32_t x1[32], x2[32];
                tmem_ld32(tmem + SL::cX1 + tk0 + lane_base, x1);
                tmem_ld32(tmem + SL::cX2 + tk0 + lane_base, x2);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    du[j] = fmaf(kBlock ? commit * e2[tk0 + j] : e2[tk0 + j], __uint_as_float(x2[j]),
                                 __uint_as_float(x1[j]));
                uint32_t pk[16];
#pragma unroll
                for (int x = 0; x < 16; ++x) pk[x] = pack_half2(du[2 * x], du[2 * x + 1]);
                // into this thread's own X2 columns: 16 packed columns per 32 tokens
                tmem_st16(tmem + SL::cX2 + tk0 + lane_base, pk);
                tmem_wait_st();
            }
            tc_fence_before_sync();
            mbar_arrive(&ms.barB);
            if (active) {                                   // the fp32 copy, behind the arrival
                float *dst = dUt + (((size_t)b * L + (size_t)c * 64 + tk0) * H + h) * D + r;
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[(size_t)j * H * D] = gsc.y * du[j];
            }
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
        if (ok && active && dstate_in) {                    // what is left is the gradient of the initial state
#pragma unroll
            for (int x = 0; x < kHalfCols; ++x) dstate_in[((size_t)bh * D + col0 + x) * D + r] = gsc.y * G[x];
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
// Block-level routing (block_route given): the exit-state gradient of a softmax block, whose update
// was not committed, is then cleared, so that the dK~ product that reads it next yields zero.
__global__ void __launch_bounds__(256)
state_dot_kernel(float *__restrict__ dS_c, const float *__restrict__ S_c, float *__restrict__ gS,
                 int n_slices, int dd, const uint8_t *__restrict__ block_route, int L, int H) {
    __shared__ float red[8];
    const size_t chunk = blockIdx.x;
    float4 *a = reinterpret_cast<float4 *>(dS_c + chunk * dd);
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
    if (block_route) {
        const int NC = L / kC;
        const size_t bh = chunk / NC;
        const int c = (int)(chunk % NC), b = (int)(bh / H), h = (int)(bh % H);
        if (block_route[((size_t)b * L + (size_t)c * kC) * H + h])       // (every thread has read its part above)
            for (int i = threadIdx.x; i < dd / 4; i += 256) a[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}


// ==========================================================================================
// Chunk-parallel part of the backward for d = 64: everything that follows the reverse scan, one
// CTA per chunk, all operands of the chunk staged once in shared memory as fp16 tiles and every
// product (64x64x64) a set of warp-level MMAs fed by ldmatrix:
//   dQg = dO S0^T        dW = -dU~ S0^T        dK~ = U~ dS1^T        N = dO U~^T
//   dKb = T^T dW         dVb = T^T dU~         M = -(dKb W^T + dVb U^T)
//   Ns = scale_la (N . Gamma) [j <= i]    Mg = M . Gamma [j < i]    Ms = diag(beta~) Mg
//   dq = scale_la gamma dQg + Ns K + dq_softmax
//   dk = beta~ gamma dKb + (gamma_C/gamma) dK~ + beta~ Mg K + Ms^T K + Ns^T Q      (linear tokens)
//   dv = beta~ dVb                                                                  (linear tokens)
// and the per-token sums the gate gradients need (dG, kappa, dbeta).
// Range.  The forward quantities (U~, S0, T, W, U, q, k) are O(1) like every fp16 operand of the
// forward kernels; the three gradient tiles are not (their size follows the incoming gradient), so
// each of dO, dU~, dS1 is scaled by a power of two that brings its largest element of the chunk to
// (0.5, 1].  Every result is linear in exactly one of the three, and the factor is taken out again
// where the result is folded into dq, dk, dv and the sums.
// Each of the 8 warps owns a 16 x 32 block of every 64 x 64 result; dq, dk, dv accumulate in
// registers across the products.
// ==========================================================================================
constexpr int kCkThreads = 256;
constexpr int kLdH = 72;                       // row stride of a staged 64x64 fp16 tile, elements
constexpr int kTileH = 64 * kLdH;
constexpr int kCkSlots = 12;
constexpr int kCkSmem = kCkSlots * kTileH * 2 + 5 * 64 * 4 + 40 * 4;

struct ChunkBwdArgs {
    const __nv_bfloat16 *q, *k, *v;
    const float *dO, *dUt, *Ut, *S_c, *dS_c, *Tinv, *Up, *Gcum, *beta, *dq_sm;   // Up: U^T in 4-token pieces
    const __half *Wt;                                                            // W^T [chunk][d][64]
    const uint8_t *route;
    float scale_la;
    __nv_bfloat16 *dq, *dk, *dv;
    float *dg, *dbeta;
    int L, H;
    // Block-level routing (kernel instantiated with kBlock): every token takes part in the delta rule (beta~ = beta), a
    // softmax block's update was not committed (its exit-state gradient reaches nothing but the
    // decay), and every token's dk, dv also has a softmax-branch part, given in dk_x, dv_x
    // (fp32, token-major).
    const float *dk_x, *dv_x;
    float *kap_c;    // [B,H,L/C] or nullptr: sum over the chunk of kappa = <dS1, K~^T U~>, the gradient
                     // of a mask on the update this chunk commits to the state (Section 4.2, d score^la)
};

// acc (16 x 32 block at (row0, n0) of a 64 x 64 result) += A B over k = 0..63, fp16 tiles.
// AT: A is stored [k][m] (else [m][k]);  BNK: B is stored [n][k] (else [k][n]).
template <bool AT, bool BNK>
__device__ __forceinline__ void mma64(const __half *A, const __half *B, int row0, int n0, int lane,
                                      float (&acc)[4][4]) {
    const int l7 = lane & 7, m1 = (lane >> 3) & 1, m2 = lane >> 4;
    const uint32_t sa = smem_u32(A), sb = smem_u32(B);
#pragma unroll
    for (int k0 = 0; k0 < 64; k0 += 16) {
        uint32_t a[4], b[4];
        if (!AT) ldmatrix_x4(sa + 2 * ((row0 + l7 + 8 * m1) * kLdH + k0 + 8 * m2), a);
        else ldmatrix_x4_trans(sa + 2 * ((k0 + l7 + 8 * m2) * kLdH + row0 + 8 * m1), a);
#pragma unroll
        for (int np = 0; np < 2; ++np) {       // two 8-column tiles per load
            const int nb = n0 + 16 * np;
            if (BNK) ldmatrix_x4(sb + 2 * ((nb + l7 + 8 * m2) * kLdH + k0 + 8 * m1), b);
            else ldmatrix_x4_trans(sb + 2 * ((k0 + l7 + 8 * m1) * kLdH + nb + 8 * m2), b);
            mma_m16n8k16(acc[2 * np], a, b[0], b[1]);
            mma_m16n8k16(acc[2 * np + 1], a, b[2], b[3]);
        }
    }
}

__device__ __forceinline__ float pow2_scale(float amax) {   // power of two s with s * amax in (0.5, 1]
    if (!(amax > 0.f) || !isfinite(amax)) return 1.f;
    int e;
    frexpf(amax, &e);                                       // amax = m 2^e, m in [0.5, 1)
    return ldexpf(1.f, -min(max(e, -100), 100));
}

template <bool kBlock>   // kBlock: block-level routing (see ChunkBwdArgs)
__global__ void __launch_bounds__(kCkThreads, 2) gdn_bwd_chunk_kernel(ChunkBwdArgs p) {
    constexpr int D = 64;
    extern __shared__ __align__(16) uint8_t smraw[];
    __half *sm = reinterpret_cast<__half *>(smraw);
    __half *sDO = sm, *sDU = sm + kTileH, *sUt = sm + 2 * kTileH, *sS0 = sm + 3 * kTileH,
           *sDS1 = sm + 4 * kTileH, *sT = sm + 5 * kTileH, *sW = sm + 6 * kTileH, *sU = sm + 7 * kTileH,
           *sK = sm + 8 * kTileH, *sQ = sm + 9 * kTileH, *sX = sm + 10 * kTileH, *sY = sm + 11 * kTileH;
    float *sG = reinterpret_cast<float *>(sm + kCkSlots * kTileH), *sBt = sG + 64, *rG = sBt + 64,
          *rK = rG + 64, *rB = rK + 64, *sMax = rB + 64;   // sMax: 3 tiles x 8 warp maxima, 8 partial <dS1, S0>, 4 scan totals

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / p.H, h = bh % p.H, NC = p.L / kC;
    const size_t ts = (size_t)p.H * D;                              // token stride, elements
    const size_t tok0 = (((size_t)b * p.L + (size_t)c * kC) * p.H + h) * D;   // element offset of the chunk
    const size_t chunk = (size_t)bh * NC + c;

    // ---- stage the chunk.  Thread -> rows r0 + 16 it (it < 4), columns c4..c4+3 of every tile ----
    const int r0 = tid >> 4, c4 = (tid & 15) * 4;
    auto ld_tile = [&](float4 (&x)[4], const float *src, size_t row_stride) {
#pragma unroll
        for (int it = 0; it < 4; ++it)
            x[it] = *reinterpret_cast<const float4 *>(src + (size_t)(r0 + 16 * it) * row_stride + c4);
    };
    auto st_tile = [&](__half *dst, const float4 (&x)[4], float f) {
#pragma unroll
        for (int it = 0; it < 4; ++it)
            *reinterpret_cast<uint2 *>(dst + (r0 + 16 * it) * kLdH + c4) =
                make_uint2(pack_half2(f * x[it].x, f * x[it].y), pack_half2(f * x[it].z, f * x[it].w));
    };
    auto amax4 = [](const float4 (&x)[4]) {
        float m = 0.f;
#pragma unroll
        for (int it = 0; it < 4; ++it)
            m = fmaxf(m, fmaxf(fmaxf(fabsf(x[it].x), fabsf(x[it].y)), fmaxf(fabsf(x[it].z), fabsf(x[it].w))));
        return m;
    };
    float scO, scU, scS;
    {
        // Two batches of tiles are in flight at a time: the loads of the next batch are issued
        // before the previous one is converted and stored.
        float4 xo[4], xu[4], xs[4], y0[4], y1[4], y2[4];
        ld_tile(xo, p.dO + tok0, ts);
        ld_tile(xu, p.dUt + tok0, ts);
        ld_tile(xs, p.dS_c + chunk * D * D, D);
        ld_tile(y0, p.Ut + tok0, ts);
        ld_tile(y1, p.S_c + chunk * D * D, D);
        ld_tile(y2, p.Tinv + chunk * 4096, 64);
        if (tid < 64) {
            const size_t tk = ((size_t)b * p.L + (size_t)c * kC + tid) * p.H + h;
            sG[tid] = p.Gcum[(size_t)bh * p.L + c * kC + tid];
            sBt[tid] = !kBlock && p.route[tk] ? 0.f : p.beta[tk];
            rG[tid] = 0.f; rK[tid] = 0.f; rB[tid] = 0.f;
        }
        const float mo = warp_max(amax4(xo)), mu = warp_max(amax4(xu)), msx = warp_max(amax4(xs));
        // <dS1, S0> of the chunk (both tiles are in registers, element for element): the decay of the
        // entry state contributes gamma_C times it to every dg of the chunk
        float dot = 0.f;
#pragma unroll
        for (int it = 0; it < 4; ++it)
            dot = fmaf(xs[it].x, y1[it].x, fmaf(xs[it].y, y1[it].y, fmaf(xs[it].z, y1[it].z, fmaf(xs[it].w, y1[it].w, dot))));
        dot = warp_sum(dot);
        if (lane == 0) { sMax[warp] = mo; sMax[8 + warp] = mu; sMax[16 + warp] = msx; sMax[24 + warp] = dot; }
        __syncthreads();
        float a0 = 0.f, a1 = 0.f, a2 = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) {
            a0 = fmaxf(a0, sMax[wv]); a1 = fmaxf(a1, sMax[8 + wv]); a2 = fmaxf(a2, sMax[16 + wv]);
        }
        scO = pow2_scale(a0); scU = pow2_scale(a1); scS = pow2_scale(a2);
        st_tile(sDO, xo, scO);
        st_tile(sDU, xu, scU);
        // (an uncommitted block: the tile is zero, so dK~ and kappa vanish; <dS1, S0> above does not)
        st_tile(sDS1, xs, kBlock && p.route[((size_t)b * p.L + (size_t)c * kC) * p.H + h] ? 0.f : scS);
        // next batch into the freed registers: W^T and U^T as the forward kernels keep them (fp16
        // [d][64] tile; fp32 in 4-token pieces [16][d][4]) -- both are [k][n] operands as they are
        uint4 wt[2];
#pragma unroll
        for (int it = 0; it < 2; ++it)
            wt[it] = reinterpret_cast<const uint4 *>(p.Wt + chunk * D * 64)[tid + it * kCkThreads];
#pragma unroll
        for (int it = 0; it < 4; ++it)
            xu[it] = reinterpret_cast<const float4 *>(p.Up + chunk * D * 64)[tid + it * kCkThreads];
        uint2 qk[2][4];
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const size_t off = tok0 + (size_t)(r0 + 16 * it) * ts + c4;
            qk[0][it] = *reinterpret_cast<const uint2 *>(p.q + off);
            qk[1][it] = *reinterpret_cast<const uint2 *>(p.k + off);
        }
        st_tile(sUt, y0, 1.f);
        st_tile(sS0, y1, 1.f);
        st_tile(sT, y2, 1.f);
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int idx = tid + it * kCkThreads;
            *reinterpret_cast<uint4 *>(sW + (idx >> 3) * kLdH + (idx & 7) * 8) = wt[it];
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int e = tid + it * kCkThreads, pc = e >> 6, vv = e & 63;
            *reinterpret_cast<uint2 *>(sU + vv * kLdH + 4 * pc) =
                make_uint2(pack_half2(xu[it].x, xu[it].y), pack_half2(xu[it].z, xu[it].w));
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {                           // bf16 -> fp16 (exact)
            auto cv = [](uint32_t w) {
                return pack_half2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
            };
            *reinterpret_cast<uint2 *>(sQ + (r0 + 16 * it) * kLdH + c4) = make_uint2(cv(qk[0][it].x), cv(qk[0][it].y));
            *reinterpret_cast<uint2 *>(sK + (r0 + 16 * it) * kLdH + c4) = make_uint2(cv(qk[1][it].x), cv(qk[1][it].y));
        }
    }
    __syncthreads();

    const float iO = 1.f / scO, iU = 1.f / scU, iS = 1.f / scS;   // powers of two: exact
    const int row0 = 16 * (warp & 3), n0 = 32 * (warp >> 2);
    const int iA = row0 + g, iB = iA + 8;                          // this lane's two rows (tokens)
    const float GA = sG[iA], GB = sG[iB], GC = sG[63];
    const float gamA = exp_ftz(GA), gamB = exp_ftz(GB), ktA = exp_ftz(GC - GA), ktB = exp_ftz(GC - GB);
    const float btA = sBt[iA], btB = sBt[iB];
    float dq[4][4], dk[4][4], dv[4][4], acc[4][4];
    float dGA = 0.f, dGB = 0.f, kapA = 0.f, kapB = 0.f, dbA = 0.f, dbB = 0.f;
    auto zero = [&]() {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
    };
    // <row of X, row of acc> over this lane's columns, for its two rows
    auto rowdot = [&](const __half *X, float &sA, float &sB) {
        sA = 0.f; sB = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float2 xa = __half22float2(*reinterpret_cast<const __half2 *>(X + iA * kLdH + n0 + 8 * nt + 2 * t));
            const float2 xb = __half22float2(*reinterpret_cast<const __half2 *>(X + iB * kLdH + n0 + 8 * nt + 2 * t));
            sA = fmaf(xa.x, acc[nt][0], fmaf(xa.y, acc[nt][1], sA));
            sB = fmaf(xb.x, acc[nt][2], fmaf(xb.y, acc[nt][3], sB));
        }
    };
    // acc (scaled per row) -> a staged tile
    auto put = [&](__half *X, float fA, float fB) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            *reinterpret_cast<uint32_t *>(X + iA * kLdH + n0 + 8 * nt + 2 * t) = pack_half2(fA * acc[nt][0], fA * acc[nt][1]);
            *reinterpret_cast<uint32_t *>(X + iB * kLdH + n0 + 8 * nt + 2 * t) = pack_half2(fB * acc[nt][2], fB * acc[nt][3]);
        }
    };
    // dst += (fA | fB) acc
    auto fold = [&](float (&dst)[4][4], float fA, float fB, bool init) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            dst[nt][0] = fmaf(fA, acc[nt][0], init ? 0.f : dst[nt][0]);
            dst[nt][1] = fmaf(fA, acc[nt][1], init ? 0.f : dst[nt][1]);
            dst[nt][2] = fmaf(fB, acc[nt][2], init ? 0.f : dst[nt][2]);
            dst[nt][3] = fmaf(fB, acc[nt][3], init ? 0.f : dst[nt][3]);
        }
    };
    float sA, sB;

    // ---- dQg = dO S0^T ----
    zero();
    mma64<false, true>(sDO, sS0, row0, n0, lane, acc);
    rowdot(sQ, sA, sB);
    dGA = fmaf(iO * p.scale_la * gamA, sA, dGA); dGB = fmaf(iO * p.scale_la * gamB, sB, dGB);
    fold(dq, iO * p.scale_la * gamA, iO * p.scale_la * gamB, true);
    // ---- dW = -dU~ S0^T  -> X ----
    zero();
    mma64<false, true>(sDU, sS0, row0, n0, lane, acc);
    put(sX, -1.f, -1.f);
    // ---- dK~ = U~ dS1^T ----
    zero();
    mma64<false, true>(sUt, sDS1, row0, n0, lane, acc);
    rowdot(sK, sA, sB);
    kapA = iS * ktA * sA; kapB = iS * ktB * sB;
    dGA -= kapA; dGB -= kapB;
    fold(dk, iS * ktA, iS * ktB, true);
    // ---- N = dO U~^T;  Ns = scale_la (N . Gamma), j <= i  -> Y ----
    zero();
    mma64<false, true>(sDO, sUt, row0, n0, lane, acc);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = n0 + 8 * nt + 2 * t + (e & 1), i = e < 2 ? iA : iB;
            acc[nt][e] *= p.scale_la * exp_ftz(j <= i ? (e < 2 ? GA : GB) - sG[j] : -INFINITY);   // branch-free mask
        }
    put(sY, 1.f, 1.f);
    __syncthreads();                    // X = dW, Y = Ns; dO, S0, dS1 are free

    // ---- dKb = T^T dW  -> slot of dO ----
    zero();
    mma64<true, false>(sT, sX, row0, n0, lane, acc);
    rowdot(sK, sA, sB);
    dGA = fmaf(iU * btA * gamA, sA, dGA); dGB = fmaf(iU * btB * gamB, sB, dGB);
    dbA = fmaf(iU * gamA, sA, dbA); dbB = fmaf(iU * gamB, sB, dbB);
    fold(dk, iU * btA * gamA, iU * btB * gamB, false);
    put(sDO, 1.f, 1.f);
    // ---- dVb = T^T dU~  -> slot of S0 ----
    zero();
    mma64<true, false>(sT, sDU, row0, n0, lane, acc);
    {   // <v, dVb>: v straight from global memory
        sA = 0.f; sB = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float2 xa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(
                p.v + tok0 + (size_t)iA * ts + n0 + 8 * nt + 2 * t));
            const float2 xb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(
                p.v + tok0 + (size_t)iB * ts + n0 + 8 * nt + 2 * t));
            sA = fmaf(xa.x, acc[nt][0], fmaf(xa.y, acc[nt][1], sA));
            sB = fmaf(xb.x, acc[nt][2], fmaf(xb.y, acc[nt][3], sB));
        }
    }
    dbA = fmaf(iU, sA, dbA); dbB = fmaf(iU, sB, dbB);
    fold(dv, iU * btA, iU * btB, true);
    put(sS0, 1.f, 1.f);
    __syncthreads();                    // dKb, dVb in place; T, X, dU~ are free

    // ---- M = -(dKb W^T + dVb U^T);  Mg = M . Gamma, j < i -> X;  Ms = diag(beta~) Mg -> slot of T ----
    zero();
    mma64<false, false>(sDO, sW, row0, n0, lane, acc);      // sW, sU hold W^T, U^T: [k][n] operands
    mma64<false, false>(sS0, sU, row0, n0, lane, acc);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = n0 + 8 * nt + 2 * t + (e & 1), i = e < 2 ? iA : iB;
            acc[nt][e] *= -exp_ftz(j < i ? (e < 2 ? GA : GB) - sG[j] : -INFINITY);
        }
    put(sX, 1.f, 1.f);
    put(sT, btA, btB);
    __syncthreads();

    // ---- beta~ Mg K ----
    zero();
    mma64<false, false>(sX, sK, row0, n0, lane, acc);
    rowdot(sK, sA, sB);
    dGA = fmaf(iU * btA, sA, dGA); dGB = fmaf(iU * btB, sB, dGB);
    dbA = fmaf(iU, sA, dbA); dbB = fmaf(iU, sB, dbB);
    fold(dk, iU * btA, iU * btB, false);
    // ---- Ms^T K ----
    zero();
    mma64<true, false>(sT, sK, row0, n0, lane, acc);
    rowdot(sK, sA, sB);
    dGA = fmaf(-iU, sA, dGA); dGB = fmaf(-iU, sB, dGB);
    fold(dk, iU, iU, false);
    // ---- Ns K ----
    zero();
    mma64<false, false>(sY, sK, row0, n0, lane, acc);
    rowdot(sQ, sA, sB);
    dGA = fmaf(iO, sA, dGA); dGB = fmaf(iO, sB, dGB);
    fold(dq, iO, iO, false);
    // ---- Ns^T Q ----
    zero();
    mma64<true, false>(sY, sQ, row0, n0, lane, acc);
    rowdot(sK, sA, sB);
    dGA = fmaf(-iO, sA, dGA); dGB = fmaf(-iO, sB, dGB);
    fold(dk, iO, iO, false);

    // ---- per-token sums: over the 4 lanes of a row, then over the two column halves ----
    auto quad = [](float x) {
        x += __shfl_xor_sync(0xffffffffu, x, 1);
        return x + __shfl_xor_sync(0xffffffffu, x, 2);
    };
    dGA = quad(dGA); dGB = quad(dGB); kapA = quad(kapA); kapB = quad(kapB); dbA = quad(dbA); dbB = quad(dbB);
    if (t == 0) {
        atomicAdd(rG + iA, dGA); atomicAdd(rG + iB, dGB);
        atomicAdd(rK + iA, kapA); atomicAdd(rK + iB, kapB);
        atomicAdd(rB + iA, dbA); atomicAdd(rB + iB, dbB);
    }
    // ---- dq, dk, dv: through fp32 tiles in the (now free) operand slots, so that every global
    // access of the epilogue is a contiguous 64-byte piece of a row instead of a scattered pair ----
    constexpr int kLdF = 68;                                       // row stride of the fp32 tiles
    float *fDQ = reinterpret_cast<float *>(smraw), *fDK = fDQ + 64 * kLdF, *fDV = fDK + 64 * kLdF;
    static_assert(3 * 64 * kLdF * 4 <= 6 * kTileH * 2, "the three result tiles must fit in the first six slots");
    const int er = tid >> 2, ec = (tid & 3) * 16;                  // epilogue: row, first of 16 columns
    const size_t eoff = tok0 + (size_t)er * ts + ec;
    float4 dqs[4];                                                 // softmax-branch dq, on its way early
#pragma unroll
    for (int x = 0; x < 4; ++x) dqs[x] = *reinterpret_cast<const float4 *>(p.dq_sm + eoff + 4 * x);
    const bool lin = kBlock || p.route[((size_t)b * p.L + (size_t)c * kC + er) * p.H + h] == 0;

    __syncthreads();                                               // all products have read their operands
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const int cc = n0 + 8 * nt + 2 * t;
        *reinterpret_cast<float2 *>(fDQ + iA * kLdF + cc) = make_float2(dq[nt][0], dq[nt][1]);
        *reinterpret_cast<float2 *>(fDQ + iB * kLdF + cc) = make_float2(dq[nt][2], dq[nt][3]);
        *reinterpret_cast<float2 *>(fDK + iA * kLdF + cc) = make_float2(dk[nt][0], dk[nt][1]);
        *reinterpret_cast<float2 *>(fDK + iB * kLdF + cc) = make_float2(dk[nt][2], dk[nt][3]);
        *reinterpret_cast<float2 *>(fDV + iA * kLdF + cc) = make_float2(dv[nt][0], dv[nt][1]);
        *reinterpret_cast<float2 *>(fDV + iB * kLdF + cc) = make_float2(dv[nt][2], dv[nt][3]);
    }
    __syncthreads();
    {
        // add: values already in registers; gadd: fp32 token-major tensor read here (block routing)
        auto row16 = [&](const float *tile, const float4 *add, const float *gadd, __nv_bfloat16 *dst) {
            uint32_t o[8];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                float4 v4 = *reinterpret_cast<const float4 *>(tile + er * kLdF + ec + 4 * x);
                if (add) { v4.x += add[x].x; v4.y += add[x].y; v4.z += add[x].z; v4.w += add[x].w; }
                if (gadd) {
                    const float4 y = *reinterpret_cast<const float4 *>(gadd + eoff + 4 * x);
                    v4.x += y.x; v4.y += y.y; v4.z += y.z; v4.w += y.w;
                }
                o[2 * x] = pack_bf162(v4.x, v4.y);
                o[2 * x + 1] = pack_bf162(v4.z, v4.w);
            }
            uint4 *d4 = reinterpret_cast<uint4 *>(dst + eoff);
            d4[0] = make_uint4(o[0], o[1], o[2], o[3]);
            d4[1] = make_uint4(o[4], o[5], o[6], o[7]);
        };
        row16(fDQ, dqs, nullptr, p.dq);
        if (lin) {
            row16(fDK, nullptr, kBlock ? p.dk_x : nullptr, p.dk);
            row16(fDV, nullptr, kBlock ? p.dv_x : nullptr, p.dv);
        }
    }
    __syncthreads();
    if (tid < 64) {
        // dg_j = sum_{i >= j} dG_i + sum_i kappa_i + gamma_C <dS1, S0>  (i, j: tokens of the chunk)
        float suf = rG[tid], kap = rK[tid];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float y = __shfl_down_sync(0xffffffffu, suf, o);
            if (lane + o < 32) suf += y;
        }
        kap = warp_sum(kap);
        if (lane == 0) { sMax[32 + warp] = suf; sMax[34 + warp] = kap; }
        named_barrier_sync(1, 64);
        float gs = 0.f;
#pragma unroll
        for (int wv = 0; wv < 8; ++wv) gs += sMax[24 + wv];
        const float extra = sMax[34] + sMax[35] + exp_ftz(sG[63]) * gs + (warp == 0 ? sMax[33] : 0.f);
        if (kBlock && p.kap_c && tid == 0) p.kap_c[chunk] = sMax[34] + sMax[35];
        const size_t tk = ((size_t)b * p.L + (size_t)c * kC + tid) * p.H + h;
        p.dg[tk] = suf + extra;
        p.dbeta[tk] = !kBlock && p.route[tk] ? 0.f : rB[tid];
    }
}

// ------------------------------------------------------------------------------------------
// Backward of the softmax branch through a query's own block under block-level routing
// (Section 4.1: both operations compute the inner-chunk correlations; Section 4.2: ds = p (dp -
// <do, o>)).  A query in a linear block reads, besides the retained tokens of earlier softmax
// blocks (the kernels over the compacted K/V handle those), the causal part of its own block of
// 64 tokens.  One CTA per linear block adds that part, five 64 x 64 x 64 products on the
// warp-level tensor-core path of the chunk kernel above (fp16 tiles, fp32 accumulation):
//   S = Q K^T, dP = dO V^T;  p_ij = exp(scale s_ij - lse_i), ds_ij = scale p_ij (dp_ij - D_i), j <= i
//   dq += dS K  (added to the query-side result of the compacted kernels)
//   dk  = dS^T Q,  dv = P^T dO  (written: the tokens of a linear block have no other
//                                 softmax-branch gradient)
// with lse_i and D_i = <do_i, o_i> of the whole softmax row.  Softmax heads of 64 KB columns: KB = 1 for
// d = 64 or kG = 2 heads per linear head of d = 128 (Section 4.3; the head is then a column slice of rows
// of 128 columns, lse / Dsm are [B,H,kG,L]), KB = 2 for d = 128 (two tiles per operand: the logit products
// add over them, the three results are formed half by half).  kNormSrc: q and k come from the fp32 copies
// that hold the softmax operation's normalised rows (qn, kn) instead of the bf16 inputs.
template <int KB> constexpr int own_smem() { return (4 * KB + 2) * kTileH * 2; }

template <int kG, bool kNormSrc, int KB>
__global__ void __launch_bounds__(kCkThreads, KB == 1 ? 3 : 2)
softmax_bwd_own_block_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k,
                             const __nv_bfloat16 *__restrict__ v, const float *__restrict__ qn,
                             const float *__restrict__ kn, const __half *__restrict__ do16,
                             const float *__restrict__ lse, const float *__restrict__ Dsm,
                             const uint8_t *__restrict__ route, float scale_sm,
                             float *__restrict__ dq_sm, float *__restrict__ dk_x,
                             float *__restrict__ dv_x, const int32_t *gsc_status, int L, int H) {
    static_assert(KB == 1 || kG == 1, "grouped heads have 64 columns");
    constexpr int D = 64 * KB, DL = D * kG;
    const float ginv = grad_scale(gsc_status).y;   // do16 and Dsm arrive times the gradient scale
    extern __shared__ __align__(16) uint8_t smraw[];
    __half *sQ = reinterpret_cast<__half *>(smraw), *sK = sQ + KB * kTileH, *sV = sK + KB * kTileH,
           *sDO = sV + KB * kTileH, *sP = sDO + KB * kTileH, *sDS = sP + kTileH;      // KB tiles per operand
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int c = blockIdx.x, bhg = blockIdx.y, bh = bhg / kG, col0 = (bhg % kG) * D, b = bh / H, h = bh % H;
    const size_t ts = (size_t)H * DL;
    const size_t tok0 = (((size_t)b * L + (size_t)c * kC) * H + h) * DL + col0;
    if (route[((size_t)b * L + (size_t)c * kC) * H + h]) return;   // a softmax block: its tokens are retained ones
    {
        const int r0 = tid >> 4, c4 = (tid & 15) * 4;
        auto cv = [](uint32_t w) {                                  // bf16 pair -> fp16 pair (exact)
            return pack_half2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
        };
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int r = r0 + 16 * it, tl = kb * kTileH + r * kLdH + c4;
            const size_t off = tok0 + (size_t)r * ts + kb * 64 + c4;
            const uint2 xv = *reinterpret_cast<const uint2 *>(v + off);
            const uint2 xo = *reinterpret_cast<const uint2 *>(do16 + ((size_t)bh * L + (size_t)c * kC + r) * DL + col0 + kb * 64 + c4);
            if (kNormSrc) {
                const float4 fq = *reinterpret_cast<const float4 *>(qn + off), fk = *reinterpret_cast<const float4 *>(kn + off);
                *reinterpret_cast<uint2 *>(sQ + tl) = make_uint2(pack_half2(fq.x, fq.y), pack_half2(fq.z, fq.w));
                *reinterpret_cast<uint2 *>(sK + tl) = make_uint2(pack_half2(fk.x, fk.y), pack_half2(fk.z, fk.w));
            } else {
                const uint2 xq = *reinterpret_cast<const uint2 *>(q + off), xk = *reinterpret_cast<const uint2 *>(k + off);
                *reinterpret_cast<uint2 *>(sQ + tl) = make_uint2(cv(xq.x), cv(xq.y));
                *reinterpret_cast<uint2 *>(sK + tl) = make_uint2(cv(xk.x), cv(xk.y));
            }
            *reinterpret_cast<uint2 *>(sV + tl) = make_uint2(cv(xv.x), cv(xv.y));
            *reinterpret_cast<uint2 *>(sDO + tl) = xo;
        }
    }
    __syncthreads();
    const int row0 = 16 * (warp & 3), n0 = 32 * (warp >> 2);
    const int iA = row0 + g, iB = iA + 8;
    const size_t rowA = (size_t)bhg * L + (size_t)c * kC + iA;
    const float l2e = 1.4426950408889634f;
    const float lseA = lse[rowA] * l2e, lseB = lse[rowA + 8] * l2e, DA = Dsm[rowA], DB = Dsm[rowA + 8];
    float pr[4][4], acc[4][4];
    auto zero = [](float (&a)[4][4]) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) a[nt][e] = 0.f;
    };
    auto put = [&](__half *X, const float (&a)[4][4]) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            *reinterpret_cast<uint32_t *>(X + iA * kLdH + n0 + 8 * nt + 2 * t) = pack_half2(a[nt][0], a[nt][1]);
            *reinterpret_cast<uint32_t *>(X + iB * kLdH + n0 + 8 * nt + 2 * t) = pack_half2(a[nt][2], a[nt][3]);
        }
    };
    // p = exp(scale s - lse), causal inside the block (mask on the exponent: no branch per element)
    zero(pr);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) mma64<false, true>(sQ + kb * kTileH, sK + kb * kTileH, row0, n0, lane, pr);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = n0 + 8 * nt + 2 * t + (e & 1), i = e < 2 ? iA : iB;
            pr[nt][e] = ex2_ftz(j <= i ? fmaf(pr[nt][e], scale_sm * l2e, -(e < 2 ? lseA : lseB)) : -INFINITY);
        }
    put(sP, pr);
    // ds = scale p (dp - D)
    zero(acc);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) mma64<false, true>(sDO + kb * kTileH, sV + kb * kTileH, row0, n0, lane, acc);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nt][e] = scale_sm * pr[nt][e] * (acc[nt][e] - (e < 2 ? DA : DB));
    put(sDS, acc);
    __syncthreads();
    auto out2 = [&](float *dst, const float (&a)[4][4], bool add, int kb) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            float2 *pa = reinterpret_cast<float2 *>(dst + tok0 + (size_t)iA * ts + kb * 64 + n0 + 8 * nt + 2 * t);
            float2 *pb = reinterpret_cast<float2 *>(dst + tok0 + (size_t)iB * ts + kb * 64 + n0 + 8 * nt + 2 * t);
            float2 va = make_float2(ginv * a[nt][0], ginv * a[nt][1]), vb = make_float2(ginv * a[nt][2], ginv * a[nt][3]);
            if (add) {
                const float2 ca = *pa, cb = *pb;
                va.x += ca.x; va.y += ca.y; vb.x += cb.x; vb.y += cb.y;
            }
            *pa = va;
            *pb = vb;
        }
    };
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
        zero(acc);
        mma64<false, false>(sDS, sK + kb * kTileH, row0, n0, lane, acc);          // dq += dS K
        out2(dq_sm, acc, true, kb);
        zero(acc);
        mma64<true, false>(sDS, sQ + kb * kTileH, row0, n0, lane, acc);           // dk = dS^T Q
        out2(dk_x, acc, false, kb);
        zero(acc);
        mma64<true, false>(sP, sDO + kb * kTileH, row0, n0, lane, acc);           // dv = P^T dO
        out2(dv_x, acc, false, kb);
    }
}

}  // namespace

template <int D>
static cudaError_t rscan_tc_impl(const void *dO16, const void *dOg16, const GdnTcWs &ws,
                                 const float *S_c, float *dUt, float *dS_c, float *gS,
                                 const float *dstate_out, float *dstate_in,
                                 const uint8_t *block_route, int32_t *status, Shape s, cudaStream_t st) {
    const int NC = s.L / kC;
    const uint64_t BH = (uint64_t)s.B * s.H;
    CUtensorMap mdo, mdog, mqh, mkh, mwt, mph;
    if (!tch::make_map_2d(&mdo, dO16, BH * s.L, D, 64) || !tch::make_map_2d(&mdog, dOg16, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mqh, ws.Qh, BH * s.L, D, 64) || !tch::make_map_2d(&mkh, ws.Kh, BH * s.L, D, 64) ||
        !tch::make_map_2d(&mwt, ws.Wt, BH * NC * D, 64, D) || !tch::make_map_2d(&mph, ws.Ph, BH * NC * 64, 64, 64))
        return cudaErrorInvalidValue;
    auto kernel = block_route ? gdn_rscan_tc_kernel<D, true> : gdn_rscan_tc_kernel<D, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         RsLayout<D>::kTotal);
    if (e != cudaSuccess) return e;
    kernel<<<s.B * s.H, kRsThreads, RsLayout<D>::kTotal, st>>>(
        mdo, mdog, mqh, mkh, mwt, mph, ws.Gd, dUt, dS_c, dstate_out, dstate_in, block_route, status, s.L, s.H,
        debug_wait_kcycles());
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (gS) {     // (the fused chunk kernel forms <dS1, S0> itself)
        state_dot_kernel<<<(unsigned)(BH * NC), 256, 0, st>>>(dS_c, S_c, gS, D / 32, D * D, block_route, s.L, s.H);
        count_launch();
    }
    return cudaGetLastError();
}

cudaError_t launch_gdn_rscan_tc(const void *dO16, const void *dOg16, const GdnTcWs &ws,
                                const float *S_c, float *dUt, float *dS_c, float *gS,
                                const float *dstate_out, float *dstate_in,
                                const uint8_t *block_route, int32_t *status, Shape s, cudaStream_t st) {
    if (s.d == 128)
        return rscan_tc_impl<128>(dO16, dOg16, ws, S_c, dUt, dS_c, gS, dstate_out, dstate_in, block_route, status, s, st);
    return rscan_tc_impl<64>(dO16, dOg16, ws, S_c, dUt, dS_c, gS, dstate_out, dstate_in, block_route, status, s, st);
}


cudaError_t launch_gdn_bwd_chunk(const void *q, const void *k, const void *v, const float *dO,
                                 const float *dUt, const float *Ut, const float *S_c, const float *dS_c,
                                 const float *Tinv, const void *Wt, const float *Up, const float *Gcum,
                                 const float *beta, const uint8_t *route, const float *dq_sm,
                                 float scale_la, void *dq, void *dk, void *dv, float *dg,
                                 float *dbeta, bool block, const float *dk_x, const float *dv_x,
                                 float *kap_c, Shape s, cudaStream_t st) {
    if (s.d != 64 || !s.bf16) return cudaErrorInvalidValue;
    auto kernel = block ? gdn_bwd_chunk_kernel<true> : gdn_bwd_chunk_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kCkSmem);
    if (e != cudaSuccess) return e;
    ChunkBwdArgs a{(const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, dO, dUt, Ut,
                   S_c, dS_c, Tinv, Up, Gcum, beta, dq_sm, (const __half *)Wt, route, scale_la, (__nv_bfloat16 *)dq,
                   (__nv_bfloat16 *)dk, (__nv_bfloat16 *)dv, dg, dbeta, s.L, s.H, dk_x, dv_x, kap_c};
    dim3 grid(s.L / kC, s.B * s.H);
    kernel<<<grid, kCkThreads, kCkSmem, st>>>(a);
    count_launch();
    return cudaGetLastError();
}

// d score per block and head (Section 4.2), for the active operation only: a softmax block sums the
// mask gradients of its 64 keys (contiguous in the compacted order), a linear block takes the kappa
// sum of its chunk; the other entry is zero.  dscore [B, L/C, H, 2] = (linear, softmax).
namespace {
__global__ void __launch_bounds__(64)
dscore_kernel(const uint8_t *__restrict__ route, const int32_t *__restrict__ sm_chunk_prefix,
              const float *__restrict__ dmask, const float *__restrict__ kap_c,
              const float *__restrict__ kappa_tok, int cap, float *__restrict__ dscore, int L, int H, int G) {
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H, NC = L / kC;
    float *dst = dscore + (((size_t)b * NC + c) * H + h) * 2;
    if (route[((size_t)b * L + (size_t)c * kC) * H + h]) {
        // (grouped heads: dmask is [B,H,G,cap]; the softmax heads of a group share the block's mask)
        const int row = sm_chunk_prefix[(size_t)bh * (NC + 1) + c] + (int)threadIdx.x;
        float x = 0.f;
        for (int gg = 0; gg < G; ++gg) x += row < cap ? dmask[((size_t)bh * G + gg) * cap + row] : 0.f;
        x = warp_sum(x);
        __shared__ float part[2];
        if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = x;
        __syncthreads();
        if (threadIdx.x == 0) { dst[0] = 0.f; dst[1] = part[0] + part[1]; }
    } else if (kappa_tok) {
        float x = warp_sum(kappa_tok[(size_t)bh * L + (size_t)c * kC + threadIdx.x]);
        __shared__ float part2[2];
        if ((threadIdx.x & 31) == 0) part2[threadIdx.x >> 5] = x;
        __syncthreads();
        if (threadIdx.x == 0) { dst[0] = part2[0] + part2[1]; dst[1] = 0.f; }
    } else if (threadIdx.x == 0) {
        dst[0] = kap_c[(size_t)bh * NC + c];
        dst[1] = 0.f;
    }
}
}  // namespace

cudaError_t launch_dscore(const uint8_t *route, const int32_t *sm_chunk_prefix, const float *dmask,
                          const float *kap_c, const float *kappa_tok, int cap, float *dscore, Shape s,
                          cudaStream_t st, int G) {
    dim3 grid(s.L / kC, s.B * s.H);
    dscore_kernel<<<grid, 64, 0, st>>>(route, sm_chunk_prefix, dmask, kap_c, kappa_tok, cap, dscore, s.L, s.H,
                                       G > 1 ? G : 1);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_softmax_bwd_own_block(const void *q, const void *k, const void *v,
                                         const void *do16, const float *lse, const float *Dsm,
                                         const uint8_t *route, float scale_sm, float *dq_sm,
                                         float *dk_x, float *dv_x, const int32_t *gsc, Shape s,
                                         cudaStream_t st, int G, const float *qn, const float *kn) {
    if (!s.bf16 || !((s.d == 64 && G <= 1) || (s.d == 128 && G <= 2))) return cudaErrorInvalidValue;
    auto kernel = softmax_bwd_own_block_kernel<1, false, 1>;
    int smem = own_smem<1>();
    if (s.d == 64 && qn) kernel = softmax_bwd_own_block_kernel<1, true, 1>;
    if (s.d == 128 && G == 2) kernel = qn ? softmax_bwd_own_block_kernel<2, true, 1> : softmax_bwd_own_block_kernel<2, false, 1>;
    if (s.d == 128 && G <= 1) {
        kernel = qn ? softmax_bwd_own_block_kernel<1, true, 2> : softmax_bwd_own_block_kernel<1, false, 2>;
        smem = own_smem<2>();
    }
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(s.L / kC, s.B * s.H * (G == 2 ? 2 : 1));
    kernel<<<grid, kCkThreads, smem, st>>>(
        (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, qn, kn, (const __half *)do16,
        lse, Dsm, route, scale_sm, dq_sm, dk_x, dv_x, gsc, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

}  // namespace natsl

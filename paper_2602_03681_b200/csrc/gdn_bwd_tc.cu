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


// ==========================================================================================
// Chunk-parallel part of the backward for d = 64: everything that follows the reverse scan, one
// CTA per chunk, all operands of the chunk staged once in shared memory (fp32, padded rows) and
// every product a warp-level tf32 MMA (64x64x64; fp32 range, so no operand can under- or overflow):
//   dQg = dO S0^T        dW = -dU~ S0^T        dK~ = U~ dS1^T        N = dO U~^T
//   dKb = T^T dW         dVb = T^T dU~         M = -(dKb W^T + dVb U^T)
//   Ns = scale_la (N . Gamma) [j <= i]    Mg = M . Gamma [j < i]    Ms = diag(beta~) Mg
//   dq = scale_la gamma dQg + Ns K + dq_softmax
//   dk = beta~ gamma dKb + (gamma_C/gamma) dK~ + beta~ Mg K + Ms^T K + Ns^T Q      (linear tokens)
//   dv = beta~ dVb                                                                  (linear tokens)
// and the per-token sums the gate gradients need (dG, kappa, dbeta).  Each of the 8 warps owns a
// 16 x 32 block of every 64 x 64 result; dq, dk, dv accumulate in registers across the products.
// ==========================================================================================
constexpr int kCkThreads = 256;
constexpr int kLd = 68;                        // row stride of a staged 64x64 tile, floats
constexpr int kTileFloats = 64 * kLd;
constexpr int kCkSlots = 13;
constexpr int kCkSmem = kCkSlots * kTileFloats * 4 + 5 * 64 * 4;

struct ChunkBwdArgs {
    const __nv_bfloat16 *q, *k, *v;
    const float *dO, *dUt, *Ut, *S_c, *dS_c, *Tinv, *W, *U, *Gcum, *beta, *dq_sm;
    const uint8_t *route;
    float scale_la;
    __nv_bfloat16 *dq, *dk, *dv;
    float *dGrow, *kappa, *dbeta;
    int L, H;
};

__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
        "{%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp_async16(void *dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// acc (16 x 32 block at (row0, n0) of a 64 x 64 result) += A B over k = 0..63.
// AT: A is stored [k][m] (else [m][k]);  BNK: B is stored [n][k] (else [k][n]).
// Fragment coordinates of a lane: g = lane / 4, t = lane % 4.
template <bool AT, bool BNK>
__device__ __forceinline__ void mma64(const float *__restrict__ A, const float *__restrict__ B, int row0,
                                      int n0, int g, int t, float (&acc)[4][4]) {
#pragma unroll
    for (int k0 = 0; k0 < 64; k0 += 8) {
        uint32_t a[4];
        if (!AT) {
            a[0] = to_tf32(A[(row0 + g) * kLd + k0 + t]);
            a[1] = to_tf32(A[(row0 + g + 8) * kLd + k0 + t]);
            a[2] = to_tf32(A[(row0 + g) * kLd + k0 + t + 4]);
            a[3] = to_tf32(A[(row0 + g + 8) * kLd + k0 + t + 4]);
        } else {
            a[0] = to_tf32(A[(k0 + t) * kLd + row0 + g]);
            a[1] = to_tf32(A[(k0 + t) * kLd + row0 + g + 8]);
            a[2] = to_tf32(A[(k0 + t + 4) * kLd + row0 + g]);
            a[3] = to_tf32(A[(k0 + t + 4) * kLd + row0 + g + 8]);
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const int n = n0 + 8 * nt + g;
            const float b0 = BNK ? B[n * kLd + k0 + t] : B[(k0 + t) * kLd + n];
            const float b1 = BNK ? B[n * kLd + k0 + t + 4] : B[(k0 + t + 4) * kLd + n];
            mma_tf32(acc[nt], a, to_tf32(b0), to_tf32(b1));
        }
    }
}

__device__ __forceinline__ bool sBtLin(const ChunkBwdArgs &p, int b, int c, int i, int h) {
    return p.route[((size_t)b * p.L + (size_t)c * kC + i) * p.H + h] == 0;
}

__global__ void __launch_bounds__(kCkThreads, 1) gdn_bwd_chunk_kernel(ChunkBwdArgs p) {
    constexpr int D = 64;
    extern __shared__ __align__(16) float sm[];
    float *sDO = sm, *sDU = sm + kTileFloats, *sUt = sm + 2 * kTileFloats, *sS0 = sm + 3 * kTileFloats,
          *sDS1 = sm + 4 * kTileFloats, *sT = sm + 5 * kTileFloats, *sW = sm + 6 * kTileFloats,
          *sU = sm + 7 * kTileFloats, *sK = sm + 8 * kTileFloats, *sQ = sm + 9 * kTileFloats,
          *sV = sm + 10 * kTileFloats, *sX = sm + 11 * kTileFloats, *sY = sm + 12 * kTileFloats;
    float *sG = sm + kCkSlots * kTileFloats, *sBt = sG + 64, *rG = sBt + 64, *rK = rG + 64, *rB = rK + 64;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / p.H, h = bh % p.H, NC = p.L / kC;
    const size_t ts = (size_t)p.H * D;                              // token stride, elements
    const size_t tok0 = (((size_t)b * p.L + (size_t)c * kC) * p.H + h) * D;   // element offset of the chunk
    const size_t chunk = (size_t)bh * NC + c;

    // ---- stage the chunk: fp32 tiles asynchronously in the order the products need them ----
    auto stage = [&](float *dst, const float *src, size_t row_stride) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int idx = tid + it * kCkThreads, r = idx >> 4, c4 = (idx & 15) * 4;
            cp_async16(dst + r * kLd + c4, src + (size_t)r * row_stride + c4);
        }
    };
    stage(sDO, p.dO + tok0, ts);
    stage(sDU, p.dUt + tok0, ts);
    stage(sUt, p.Ut + tok0, ts);
    stage(sS0, p.S_c + chunk * D * D, D);
    stage(sDS1, p.dS_c + chunk * D * D, D);
    cp_async_commit();
    stage(sT, p.Tinv + chunk * 4096, 64);
    cp_async_commit();
    stage(sW, p.W + tok0, ts);
    stage(sU, p.U + tok0, ts);
    cp_async_commit();
    if (tid < 64) {
        const size_t tk = ((size_t)b * p.L + (size_t)c * kC + tid) * p.H + h;
        sG[tid] = p.Gcum[(size_t)bh * p.L + c * kC + tid];
        sBt[tid] = p.route[tk] ? 0.f : p.beta[tk];
        rG[tid] = 0.f; rK[tid] = 0.f; rB[tid] = 0.f;
    }
#pragma unroll
    for (int it = 0; it < 4; ++it) {                               // q, k, v: bf16 -> fp32
        const int idx = tid + it * kCkThreads, r = idx >> 4, c4 = (idx & 15) * 4;
        const size_t off = tok0 + (size_t)r * ts + c4;
        store4(sQ + r * kLd + c4, load4(p.q + off));
        store4(sK + r * kLd + c4, load4(p.k + off));
        store4(sV + r * kLd + c4, load4(p.v + off));
    }
    cp_async_wait<2>();
    __syncthreads();

    const int row0 = 16 * (warp & 3), n0 = 32 * (warp >> 2);
    const int iA = row0 + g, iB = iA + 8;                          // this lane's two rows (tokens)
    const float GA = sG[iA], GB = sG[iB], GC = sG[63];
    const float gamA = __expf(GA), gamB = __expf(GB), ktA = __expf(GC - GA), ktB = __expf(GC - GB);
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
    auto rowdot = [&](const float *X, float &sA, float &sB) {
        sA = 0.f; sB = 0.f;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float2 xa = *reinterpret_cast<const float2 *>(X + iA * kLd + n0 + 8 * nt + 2 * t);
            const float2 xb = *reinterpret_cast<const float2 *>(X + iB * kLd + n0 + 8 * nt + 2 * t);
            sA = fmaf(xa.x, acc[nt][0], fmaf(xa.y, acc[nt][1], sA));
            sB = fmaf(xb.x, acc[nt][2], fmaf(xb.y, acc[nt][3], sB));
        }
    };
    // acc (scaled per row) -> a staged tile
    auto put = [&](float *X, float fA, float fB) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            *reinterpret_cast<float2 *>(X + iA * kLd + n0 + 8 * nt + 2 * t) = make_float2(fA * acc[nt][0], fA * acc[nt][1]);
            *reinterpret_cast<float2 *>(X + iB * kLd + n0 + 8 * nt + 2 * t) = make_float2(fB * acc[nt][2], fB * acc[nt][3]);
        }
    };
    float sA, sB;

    // ---- dQg = dO S0^T ----
    zero();
    mma64<false, true>(sDO, sS0, row0, n0, g, t, acc);
    rowdot(sQ, sA, sB);
    dGA = fmaf(p.scale_la * gamA, sA, dGA); dGB = fmaf(p.scale_la * gamB, sB, dGB);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        dq[nt][0] = p.scale_la * gamA * acc[nt][0]; dq[nt][1] = p.scale_la * gamA * acc[nt][1];
        dq[nt][2] = p.scale_la * gamB * acc[nt][2]; dq[nt][3] = p.scale_la * gamB * acc[nt][3];
    }
    // ---- dW = -dU~ S0^T  -> X ----
    zero();
    mma64<false, true>(sDU, sS0, row0, n0, g, t, acc);
    put(sX, -1.f, -1.f);
    // ---- dK~ = U~ dS1^T ----
    zero();
    mma64<false, true>(sUt, sDS1, row0, n0, g, t, acc);
    rowdot(sK, sA, sB);
    kapA = ktA * sA; kapB = ktB * sB;
    dGA -= kapA; dGB -= kapB;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        dk[nt][0] = ktA * acc[nt][0]; dk[nt][1] = ktA * acc[nt][1];
        dk[nt][2] = ktB * acc[nt][2]; dk[nt][3] = ktB * acc[nt][3];
    }
    // ---- N = dO U~^T;  Ns = scale_la (N . Gamma), j <= i  -> Y ----
    zero();
    mma64<false, true>(sDO, sUt, row0, n0, g, t, acc);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = n0 + 8 * nt + 2 * t + (e & 1), i = e < 2 ? iA : iB;
            acc[nt][e] = j <= i ? p.scale_la * __expf((e < 2 ? GA : GB) - sG[j]) * acc[nt][e] : 0.f;
        }
    put(sY, 1.f, 1.f);
    cp_async_wait<1>();
    __syncthreads();                    // X = dW, Y = Ns, T staged; dO, S0, dS1 are free

    // ---- dKb = T^T dW  -> slot of dO ----
    zero();
    mma64<true, false>(sT, sX, row0, n0, g, t, acc);
    rowdot(sK, sA, sB);
    dGA = fmaf(btA * gamA, sA, dGA); dGB = fmaf(btB * gamB, sB, dGB);
    dbA = fmaf(gamA, sA, dbA); dbB = fmaf(gamB, sB, dbB);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        dk[nt][0] = fmaf(btA * gamA, acc[nt][0], dk[nt][0]); dk[nt][1] = fmaf(btA * gamA, acc[nt][1], dk[nt][1]);
        dk[nt][2] = fmaf(btB * gamB, acc[nt][2], dk[nt][2]); dk[nt][3] = fmaf(btB * gamB, acc[nt][3], dk[nt][3]);
    }
    put(sDO, 1.f, 1.f);
    // ---- dVb = T^T dU~  -> slot of S0 ----
    zero();
    mma64<true, false>(sT, sDU, row0, n0, g, t, acc);
    rowdot(sV, sA, sB);
    dbA += sA; dbB += sB;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        dv[nt][0] = btA * acc[nt][0]; dv[nt][1] = btA * acc[nt][1];
        dv[nt][2] = btB * acc[nt][2]; dv[nt][3] = btB * acc[nt][3];
    }
    put(sS0, 1.f, 1.f);
    cp_async_wait<0>();
    __syncthreads();                    // dKb, dVb, W, U staged; T, X, dU~ are free

    // ---- M = -(dKb W^T + dVb U^T);  Mg = M . Gamma, j < i -> X;  Ms = diag(beta~) Mg -> slot of T ----
    zero();
    mma64<false, true>(sDO, sW, row0, n0, g, t, acc);
    mma64<false, true>(sS0, sU, row0, n0, g, t, acc);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int j = n0 + 8 * nt + 2 * t + (e & 1), i = e < 2 ? iA : iB;
            acc[nt][e] = j < i ? -__expf((e < 2 ? GA : GB) - sG[j]) * acc[nt][e] : 0.f;
        }
    put(sX, 1.f, 1.f);
    put(sT, btA, btB);
    __syncthreads();

    // ---- beta~ Mg K ----
    zero();
    mma64<false, false>(sX, sK, row0, n0, g, t, acc);
    rowdot(sK, sA, sB);
    dGA = fmaf(btA, sA, dGA); dGB = fmaf(btB, sB, dGB);
    dbA += sA; dbB += sB;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        dk[nt][0] = fmaf(btA, acc[nt][0], dk[nt][0]); dk[nt][1] = fmaf(btA, acc[nt][1], dk[nt][1]);
        dk[nt][2] = fmaf(btB, acc[nt][2], dk[nt][2]); dk[nt][3] = fmaf(btB, acc[nt][3], dk[nt][3]);
    }
    // ---- Ms^T K ----
    zero();
    mma64<true, false>(sT, sK, row0, n0, g, t, acc);
    rowdot(sK, sA, sB);
    dGA -= sA; dGB -= sB;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) dk[nt][e] += acc[nt][e];
    // ---- Ns K ----
    zero();
    mma64<false, false>(sY, sK, row0, n0, g, t, acc);
    rowdot(sQ, sA, sB);
    dGA += sA; dGB += sB;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) dq[nt][e] += acc[nt][e];
    // ---- Ns^T Q ----
    zero();
    mma64<true, false>(sY, sQ, row0, n0, g, t, acc);
    rowdot(sK, sA, sB);
    dGA -= sA; dGB -= sB;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) dk[nt][e] += acc[nt][e];

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
    // ---- dq, dk, dv ----
    const bool linA = sBtLin(p, b, c, iA, h), linB = sBtLin(p, b, c, iB, h);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const size_t oA = tok0 + (size_t)iA * ts + n0 + 8 * nt + 2 * t, oB = tok0 + (size_t)iB * ts + n0 + 8 * nt + 2 * t;
        const float2 sa = *reinterpret_cast<const float2 *>(p.dq_sm + oA);
        const float2 sb = *reinterpret_cast<const float2 *>(p.dq_sm + oB);
        *reinterpret_cast<__nv_bfloat162 *>(p.dq + oA) = __floats2bfloat162_rn(dq[nt][0] + sa.x, dq[nt][1] + sa.y);
        *reinterpret_cast<__nv_bfloat162 *>(p.dq + oB) = __floats2bfloat162_rn(dq[nt][2] + sb.x, dq[nt][3] + sb.y);
        if (linA) {
            *reinterpret_cast<__nv_bfloat162 *>(p.dk + oA) = __floats2bfloat162_rn(dk[nt][0], dk[nt][1]);
            *reinterpret_cast<__nv_bfloat162 *>(p.dv + oA) = __floats2bfloat162_rn(dv[nt][0], dv[nt][1]);
        }
        if (linB) {
            *reinterpret_cast<__nv_bfloat162 *>(p.dk + oB) = __floats2bfloat162_rn(dk[nt][2], dk[nt][3]);
            *reinterpret_cast<__nv_bfloat162 *>(p.dv + oB) = __floats2bfloat162_rn(dv[nt][2], dv[nt][3]);
        }
    }
    __syncthreads();
    if (tid < 64) {
        const size_t tk = ((size_t)b * p.L + (size_t)c * kC + tid) * p.H + h;
        p.dGrow[(size_t)bh * p.L + c * kC + tid] = rG[tid];
        p.kappa[(size_t)bh * p.L + c * kC + tid] = rK[tid];
        p.dbeta[tk] = p.route[tk] ? 0.f : rB[tid];
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


cudaError_t launch_gdn_bwd_chunk(const void *q, const void *k, const void *v, const float *dO,
                                 const float *dUt, const float *Ut, const float *S_c, const float *dS_c,
                                 const float *Tinv, const float *W, const float *U, const float *Gcum,
                                 const float *beta, const uint8_t *route, const float *dq_sm,
                                 float scale_la, void *dq, void *dk, void *dv, float *dGrow,
                                 float *kappa, float *dbeta, Shape s, cudaStream_t st) {
    if (s.d != 64 || !s.bf16) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(gdn_bwd_chunk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kCkSmem);
    if (e != cudaSuccess) return e;
    ChunkBwdArgs a{(const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, dO, dUt, Ut,
                   S_c, dS_c, Tinv, W, U, Gcum, beta, dq_sm, route, scale_la, (__nv_bfloat16 *)dq,
                   (__nv_bfloat16 *)dk, (__nv_bfloat16 *)dv, dGrow, kappa, dbeta, s.L, s.H};
    dim3 grid(s.L / kC, s.B * s.H);
    gdn_bwd_chunk_kernel<<<grid, kCkThreads, kCkSmem, st>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace natsl

// Tensor-core backward of the softmax branch over the retained tokens (Section 4.2: the logit
// gradient is p (dp - <do, o>); k, v gradients exist only for retained tokens), bf16 storage,
// sm_100a.  With p_ij = exp(scale q_i.k_j - lse_i) over the retained keys j <= i:
//   dv_j = sum_i p_ij do_i,   dp_ij = do_i.v_j,   ds_ij = scale p_ij (dp_ij - D_i),
//   dq_i = sum_j ds_ij k_j,   dk_j = sum_i ds_ij q_i           (D_i = <do_i, o_i>)
// Two kernels, both recomputing p from the saved log-sum-exp:
//   * query side: one CTA per 128 queries walks the compacted K/V in tiles of 64 keys
//     (S = Q K^T and dP = dO V^T into TMEM, ds rows by one thread per query, dQ += dS K);
//   * key side: one CTA per 128 retained keys walks the query tiles that can see them
//     (S^T = K Q^T and dP^T = V dO^T, rows owned by one thread per key, dV += P^T dO, dK += dS^T Q).
// Every operand is fp16 (q, k, v convert exactly; p, ds, do are computed values that need more
// than bf16's 8 significant bits to keep the gradients within tolerance); accumulation is fp32.
#include "common.cuh"
#include "natsl_internal.h"
#include "tc_common.cuh"

namespace natsl {

namespace {

using namespace tc;

constexpr int kThreadsB = 192;       // warps 0-3 rows, warp 4 MMA issue, warp 5 TMA
constexpr int kRowsB = 128;
constexpr int kMiscB = 2048;
constexpr float kLog2e = 1.4426950408889634f;

struct MiscB {
    uint64_t barQ, full[3], empty[3], barS, barSfree, barP, barAcc;
    uint32_t tmem_base;
    int abort_flag, wait_kcycles;   // in this order: the waits read the limit as abort_flag[1]
    alignas(16) int pos[kRowsB];
    alignas(16) float lse2[2][64], dsum[2][64];   // key side: per query of the tile in flight (double-buffered)
};
static_assert(sizeof(MiscB) <= kMiscB, "misc page too small");

// ==========================================================================================
// Query side
// ==========================================================================================
template <int D> struct QLayout {
    static constexpr int KB = D / 64;
    static constexpr int kQ = KB * 128 * 128;             // 128 queries x D fp16
    static constexpr int kKV = KB * 64 * 128;             // 64 keys x D fp16
    static constexpr int kStages = 3;
    static constexpr int oQ = 0, oDO = kQ, oK = 2 * kQ, oV = oK + kStages * kKV, oDS = oV + kStages * kKV;
    static constexpr int oMisc = oDS + 128 * 128;
    static constexpr int kTotal = oMisc + kMiscB;
    static constexpr int kTmem = D == 64 ? 256 : 512;     // S 64 + dP 64 + dQ D
};

// kG softmax heads per linear head (Section 4.3, grouped heads): a CTA's head is then one slice of D
// columns of rows of kG D columns -- the x coordinate of every copy and the column offset of every
// store --, the lists of retained tokens are the linear head's, lse and Dsm are [B,H,kG,L].
template <int D, int kG>
__global__ void __launch_bounds__(kThreadsB)
softmax_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap map_q,    // Qh  [B*H*L][D] fp16, box 128
                         const __grid_constant__ CUtensorMap map_do,   // dO16 [B*H*L][D] fp16, box 128
                         const __grid_constant__ CUtensorMap map_k,    // k16 [B*H*cap][D], box 64
                         const __grid_constant__ CUtensorMap map_v,    // v16 [B*H*cap][D], box 64
                         int cap, const int32_t *__restrict__ sm_idx,
                         const int32_t *__restrict__ sm_chunk_prefix, const float *__restrict__ lse,
                         const float *__restrict__ Dsm, float scale_sm, float *__restrict__ dq_sm,
                         int32_t *status, int L, int H, int wait_kcycles) {
    using SL = QLayout<D>;
    constexpr int KB = SL::KB;
    extern __shared__ __align__(1024) uint8_t smem[];
    MiscB &ms = *reinterpret_cast<MiscB *>(smem + SL::oMisc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NP = (L + 127) / 128, NC = L / kC;
    const int p = NP - 1 - (int)blockIdx.x;
    const int bhg = blockIdx.y, bh = bhg / kG, x0 = (bhg % kG) * D, b = bh / H, h = bh % H;
    const int32_t *pre = sm_chunk_prefix + (size_t)bh * (NC + 1);
    const int n_full = min(pre[2 * p], cap), n_end = min(pre[min(2 * p + 2, NC)], cap);
    const int T = (n_end + 63) / 64;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        mbar_init(&ms.barQ, 1);
        for (int s = 0; s < SL::kStages; ++s) { mbar_init(&ms.full[s], 1); mbar_init(&ms.empty[s], 1); }
        mbar_init(&ms.barS, 1);
        mbar_init(&ms.barSfree, kRowsB);
        mbar_init(&ms.barP, kRowsB);
        mbar_init(&ms.barAcc, 1);
        ms.abort_flag = 0;
        ms.wait_kcycles = wait_kcycles;
        fence_mbar_init();
    }
    if (tid < kRowsB) {
        const int jj = n_full + tid;
        ms.pos[tid] = jj < n_end ? sm_idx[(size_t)bh * L + jj] : 0x7fffffff;
    }
    if (warp == 4) tmem_alloc(&ms.tmem_base, SL::kTmem);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ms.tmem_base;
    const uint32_t tS = tmem, tDP = tmem + 64, tDQ = tmem + 128;
    volatile int *abort_flag = &ms.abort_flag;

    if (warp == 5) {
        if (lane == 0 && T > 0) {      // nothing is loaded for a tile that sees no retained key
            mbar_arrive_expect_tx(&ms.barQ, 2 * SL::kQ);
            for (int kb = 0; kb < KB; ++kb) {
                tma_load_2d(smem + SL::oQ + kb * 16384, &map_q, &ms.barQ, x0 + kb * 64, bh * L + p * 128);
                tma_load_2d(smem + SL::oDO + kb * 16384, &map_do, &ms.barQ, x0 + kb * 64, bh * L + p * 128);
            }
            int t = 0;
            for (; t < T; ++t) {
                const int s = t % SL::kStages;
                if (!mbar_wait(&ms.empty[s], ((t / SL::kStages) & 1) ^ 1, abort_flag)) break;
                mbar_arrive_expect_tx(&ms.full[s], 2 * SL::kKV);
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(smem + SL::oK + s * SL::kKV + kb * 8192, &map_k, &ms.full[s], x0 + kb * 64,
                                bh * cap + t * 64);
                    tma_load_2d(smem + SL::oV + s * SL::kKV + kb * 8192, &map_v, &ms.full[s], x0 + kb * 64,
                                bh * cap + t * 64);
                }
            }
            for (int u = max(0, t - SL::kStages); u < t; ++u)    // no copy in flight at retirement
                mbar_wait_drain(&ms.full[u % SL::kStages], (u / SL::kStages) & 1);
            mbar_wait_drain(&ms.barQ, 0);
        }
    } else if (warp == 4) {
        if (lane == 0 && T > 0) {
            constexpr uint32_t id_s = make_idesc(kFmtF16, 128, 64, false, false);
            constexpr uint32_t id_dq = make_idesc(kFmtF16, 128, D, false, true);
            const uint32_t aQ = smem_u32(smem + SL::oQ), aDO = smem_u32(smem + SL::oDO),
                           aDS = smem_u32(smem + SL::oDS);
            auto issue_s = [&](int t) {
                const uint32_t aK = smem_u32(smem + SL::oK + (t % SL::kStages) * SL::kKV);
                const uint32_t aV = smem_u32(smem + SL::oV + (t % SL::kStages) * SL::kKV);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        mma_ss(tS, desc_kmajor(aQ + kb * 16384 + k16 * 32),
                               desc_kmajor(aK + kb * 8192 + k16 * 32), id_s, (kb | k16) != 0);
                        mma_ss(tDP, desc_kmajor(aDO + kb * 16384 + k16 * 32),
                               desc_kmajor(aV + kb * 8192 + k16 * 32), id_s, (kb | k16) != 0);
                    }
                mma_commit(&ms.barS);
            };
            bool ok = mbar_wait(&ms.barQ, 0, abort_flag) && mbar_wait(&ms.full[0], 0, abort_flag);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0);
            }
            for (int t = 0; ok && t < T; ++t) {
                // S and dP of the next tile go into the same TMEM columns as soon as the row threads
                // have read this tile's out of them (barSfree), i.e. while they still compute dS.
                if (t + 1 < T) {
                    ok = mbar_wait(&ms.full[(t + 1) % SL::kStages], ((t + 1) / SL::kStages) & 1, abort_flag) &&
                         mbar_wait(&ms.barSfree, t & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_s(t + 1);
                }
                ok = mbar_wait(&ms.barP, t & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t aK = smem_u32(smem + SL::oK + (t % SL::kStages) * SL::kKV);
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16)
                    mma_ss(tDQ, desc_kmajor(aDS + k16 * 32), desc_mnmajor(aK + k16 * 2048, 8192), id_dq,
                           (t | k16) != 0);
                mma_commit(&ms.barAcc);
                mma_commit(&ms.empty[t % SL::kStages]);     // K/V stage t is free after dQ(t)
            }
        }
    } else {
        const int r = tid, i_abs = p * 128 + r;
        const bool row_ok = i_abs < L;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float sl2 = scale_sm * kLog2e;
        const float lse2 = row_ok ? lse[(size_t)bhg * L + i_abs] * kLog2e : 0.f;
        const float Di = row_ok ? Dsm[(size_t)bhg * L + i_abs] : 0.f;
        bool ok = true;
        // The compacted keys are in position order, so row i sees exactly the first `cnt` of them
        // (a per-element look-up of the key's position costs a divergent branch per element).
        int cnt = 0;
        if (row_ok) {
            cnt = n_full;
            for (int kq = 0; kq < n_end - n_full; ++kq) cnt += ms.pos[kq] <= i_abs ? 1 : 0;
        }
        for (int t = 0; t < T; ++t) {
            ok = mbar_wait(&ms.barS, t & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            float ds[64];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t sv[32], dv[32];
                tmem_ld32(tS + lane_base + 32 * half, sv);
                tmem_ld32(tDP + lane_base + 32 * half, dv);
                tmem_wait_ld();
                if (half == 1) {                            // both halves are in registers
                    tc_fence_before_sync();
                    mbar_arrive(&ms.barSfree);
                }
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int jj = t * 64 + 32 * half + c;
                    const bool vis = jj < cnt;
                    // mask on the exponent (exp2(-inf) = 0), not around the expression: no branch
                    const float pr = ex2_ftz(vis ? fmaf(__uint_as_float(sv[c]), sl2, -lse2) : -INFINITY);
                    ds[32 * half + c] = scale_sm * pr * (__uint_as_float(dv[c]) - Di);
                }
            }
            if (t > 0) {
                ok = mbar_wait(&ms.barAcc, (t - 1) & 1, abort_flag);   // dS buffer consumed
                if (!ok) break;
            }
#pragma unroll
            for (int pc = 0; pc < 8; ++pc)
                *reinterpret_cast<uint4 *>(smem + SL::oDS + sw128_offset(r, pc)) =
                    make_uint4(pack_half2(ds[8 * pc], ds[8 * pc + 1]), pack_half2(ds[8 * pc + 2], ds[8 * pc + 3]),
                               pack_half2(ds[8 * pc + 4], ds[8 * pc + 5]), pack_half2(ds[8 * pc + 6], ds[8 * pc + 7]));
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&ms.barP);
        }
        if (ok && T > 0) {
            ok = mbar_wait(&ms.barAcc, (T - 1) & 1, abort_flag);
            tc_fence_after_sync();
        }
        if (ok) {
            const float gi = grad_scale(status).y;          // dO and Dsm arrive times the gradient scale
            float4 *dst = reinterpret_cast<float4 *>(dq_sm + (((size_t)b * L + i_abs) * H + h) * (D * kG) + x0);
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                uint32_t x[32];
                if (T > 0) {
                    tmem_ld32(tDQ + lane_base + cb * 32, x);
                    tmem_wait_ld();
                }
                if (!row_ok) continue;
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4)
                    dst[cb * 8 + c4] = T > 0 ? make_float4(gi * __uint_as_float(x[4 * c4]), gi * __uint_as_float(x[4 * c4 + 1]),
                                                           gi * __uint_as_float(x[4 * c4 + 2]), gi * __uint_as_float(x[4 * c4 + 3]))
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, SL::kTmem);
    }
    if (tid == 0 && ms.abort_flag) atomicMin(status, (int)NATSL_ERR_TIMEOUT);
}

// ==========================================================================================
// Key side
// ==========================================================================================
template <int D> struct KLayout {
    static constexpr int KB = D / 64;
    static constexpr int kKV = KB * 128 * 128;            // 128 keys x D fp16
    static constexpr int kQ = KB * 64 * 128;              // 64 queries x D fp16
    static constexpr int oK = 0, oV = kKV, oQ = 2 * kKV, oDO = oQ + 2 * kQ, oP = oDO + 2 * kQ,
                         oDS = oP + 128 * 128;
    static constexpr int oMisc = oDS + 128 * 128;
    static constexpr int kTotal = oMisc + kMiscB;
    static constexpr int kTmem = D == 64 ? 256 : 512;     // S^T 64 + dP^T 64 + dV D + dK D
};

template <int D, bool kMask, int kG>   // kMask: also the per-key sums of the mask gradient (dmask); kG: as above
__global__ void __launch_bounds__(kThreadsB)
softmax_bwd_dkv_tc_kernel(const __grid_constant__ CUtensorMap map_q,    // Qh [B*H*L][D], box 64
                          const __grid_constant__ CUtensorMap map_do,   // dO16, box 64
                          const __grid_constant__ CUtensorMap map_k,    // k16 [B*H*cap][D], box 128
                          const __grid_constant__ CUtensorMap map_v,    // v16, box 128
                          int cap, const int32_t *__restrict__ sm_idx,
                          const int32_t *__restrict__ sm_chunk_prefix,
                          const float *__restrict__ lse, const float *__restrict__ Dsm,
                          float scale_sm, float *__restrict__ dk_sm, float *__restrict__ dv_sm,
                          float *__restrict__ dmask,     // [B*H*cap]: sum_i p_ij (dp_ij - D_i) per key j
                          int32_t *status, int L, int H, int wait_kcycles) {
    using SL = KLayout<D>;
    constexpr int KB = SL::KB;
    extern __shared__ __align__(1024) uint8_t smem[];
    MiscB &ms = *reinterpret_cast<MiscB *>(smem + SL::oMisc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NC = L / kC;
    const int kt = blockIdx.x, bhg = blockIdx.y, bh = bhg / kG, x0 = (bhg % kG) * D;
    const int n_sm = min(sm_chunk_prefix[(size_t)bh * (NC + 1) + NC], cap);
    if (kt * 128 >= n_sm) return;                        // uniform: no retained key in this tile
    const int first_pos = sm_idx[(size_t)bh * L + kt * 128];
    const int qt0 = first_pos / 64;                       // first query tile that sees a key of the tile
    const int T = NC - qt0;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        mbar_init(&ms.barQ, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(&ms.full[s], 1); mbar_init(&ms.empty[s], 1 + kRowsB); }
        mbar_init(&ms.barS, 1);
        mbar_init(&ms.barSfree, kRowsB);
        mbar_init(&ms.barP, kRowsB);
        mbar_init(&ms.barAcc, 1);
        ms.abort_flag = 0;
        ms.wait_kcycles = wait_kcycles;
        fence_mbar_init();
    }
    if (warp == 4) tmem_alloc(&ms.tmem_base, SL::kTmem);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ms.tmem_base;
    const uint32_t tS = tmem, tDP = tmem + 64, tDV = tmem + 128, tDK = tmem + 128 + D;
    volatile int *abort_flag = &ms.abort_flag;

    if (warp == 5) {
        if (lane == 0) {
            mbar_arrive_expect_tx(&ms.barQ, 2 * SL::kKV);
            for (int kb = 0; kb < KB; ++kb) {
                tma_load_2d(smem + SL::oK + kb * 16384, &map_k, &ms.barQ, x0 + kb * 64, bh * cap + kt * 128);
                tma_load_2d(smem + SL::oV + kb * 16384, &map_v, &ms.barQ, x0 + kb * 64, bh * cap + kt * 128);
            }
            int t = 0;
            for (; t < T; ++t) {
                const int s = t & 1;
                if (!mbar_wait(&ms.empty[s], ((t >> 1) & 1) ^ 1, abort_flag)) break;
                mbar_arrive_expect_tx(&ms.full[s], 2 * SL::kQ);
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(smem + SL::oQ + s * SL::kQ + kb * 8192, &map_q, &ms.full[s], x0 + kb * 64,
                                bh * L + (qt0 + t) * 64);
                    tma_load_2d(smem + SL::oDO + s * SL::kQ + kb * 8192, &map_do, &ms.full[s], x0 + kb * 64,
                                bh * L + (qt0 + t) * 64);
                }
            }
            for (int u = max(0, t - 2); u < t; ++u) mbar_wait_drain(&ms.full[u & 1], (u >> 1) & 1);
            mbar_wait_drain(&ms.barQ, 0);
        }
    } else if (warp == 4) {
        if (lane == 0) {
            constexpr uint32_t id_s = make_idesc(kFmtF16, 128, 64, false, false);
            constexpr uint32_t id_acc = make_idesc(kFmtF16, 128, D, false, true);
            const uint32_t aK = smem_u32(smem + SL::oK), aV = smem_u32(smem + SL::oV),
                           aP = smem_u32(smem + SL::oP), aDS = smem_u32(smem + SL::oDS);
            auto issue_s = [&](int t) {
                const uint32_t aQ = smem_u32(smem + SL::oQ + (t & 1) * SL::kQ);
                const uint32_t aDO = smem_u32(smem + SL::oDO + (t & 1) * SL::kQ);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        mma_ss(tS, desc_kmajor(aK + kb * 16384 + k16 * 32),
                               desc_kmajor(aQ + kb * 8192 + k16 * 32), id_s, (kb | k16) != 0);
                        mma_ss(tDP, desc_kmajor(aV + kb * 16384 + k16 * 32),
                               desc_kmajor(aDO + kb * 8192 + k16 * 32), id_s, (kb | k16) != 0);
                    }
                mma_commit(&ms.barS);
            };
            bool ok = mbar_wait(&ms.barQ, 0, abort_flag) && mbar_wait(&ms.full[0], 0, abort_flag);
            if (ok) {
                tc_fence_after_sync();
                issue_s(0);
            }
            for (int t = 0; ok && t < T; ++t) {
                // S^T and dP^T of the next query tile go into the same TMEM columns as soon as the row
                // threads have read this tile's out of them, i.e. while they still compute P^T, dS^T.
                if (t + 1 < T) {
                    ok = mbar_wait(&ms.full[(t + 1) & 1], ((t + 1) >> 1) & 1, abort_flag) &&
                         mbar_wait(&ms.barSfree, t & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_s(t + 1);
                }
                ok = mbar_wait(&ms.barP, t & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t aQ = smem_u32(smem + SL::oQ + (t & 1) * SL::kQ);
                const uint32_t aDO = smem_u32(smem + SL::oDO + (t & 1) * SL::kQ);
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16) {
                    mma_ss(tDV, desc_kmajor(aP + k16 * 32), desc_mnmajor(aDO + k16 * 2048, 8192), id_acc,
                           (t | k16) != 0);
                    mma_ss(tDK, desc_kmajor(aDS + k16 * 32), desc_mnmajor(aQ + k16 * 2048, 8192), id_acc,
                           (t | k16) != 0);
                }
                mma_commit(&ms.barAcc);
                mma_commit(&ms.empty[t & 1]);
            }
        }
    } else {
        const int r = tid, j = kt * 128 + r;              // this thread's retained key
        const bool key_ok = j < n_sm;
        const int pos_j = key_ok ? sm_idx[(size_t)bh * L + j] : 0x7fffffff;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float sl2 = scale_sm * kLog2e;
        float msum = 0.f;                                   // mask gradient of this key, over all queries
        bool ok = true;
        for (int t = 0; t < T; ++t) {
            const int i0 = (qt0 + t) * 64;
            // per-query log-sum-exp and D of this tile; two buffers, so that a thread still reading
            // the previous tile's values is not overtaken (the barrier below separates t from t + 2)
            float *lse2 = ms.lse2[t & 1], *dsum = ms.dsum[t & 1];
            if (r < 64) {
                lse2[r] = lse[(size_t)bhg * L + i0 + r] * kLog2e;
                dsum[r] = Dsm[(size_t)bhg * L + i0 + r];
            }
            named_barrier_sync(1, kRowsB);
            ok = mbar_wait(&ms.barS, t & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            float pv[64], ds[64];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t sv[32], dv[32];
                tmem_ld32(tS + lane_base + 32 * half, sv);
                tmem_ld32(tDP + lane_base + 32 * half, dv);
                tmem_wait_ld();
                if (half == 1) {                            // both halves are in registers
                    tc_fence_before_sync();
                    mbar_arrive(&ms.barSfree);
                }
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    const int cc = 32 * half + c;
                    const bool vis = pos_j <= i0 + cc;
                    const float pr = ex2_ftz(vis ? fmaf(__uint_as_float(sv[c]), sl2, -lse2[cc]) : -INFINITY);
                    pv[cc] = pr;
                    const float dm = pr * (__uint_as_float(dv[c]) - dsum[cc]);   // dM_ij (Section 4.2)
                    if (kMask) msum += dm;
                    ds[cc] = scale_sm * dm;
                }
            }
            if (t > 0) {
                ok = mbar_wait(&ms.barAcc, (t - 1) & 1, abort_flag);   // P^T / dS^T buffers consumed
                if (!ok) break;
            }
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
                *reinterpret_cast<uint4 *>(smem + SL::oP + sw128_offset(r, pc)) =
                    make_uint4(pack_half2(pv[8 * pc], pv[8 * pc + 1]), pack_half2(pv[8 * pc + 2], pv[8 * pc + 3]),
                               pack_half2(pv[8 * pc + 4], pv[8 * pc + 5]), pack_half2(pv[8 * pc + 6], pv[8 * pc + 7]));
                *reinterpret_cast<uint4 *>(smem + SL::oDS + sw128_offset(r, pc)) =
                    make_uint4(pack_half2(ds[8 * pc], ds[8 * pc + 1]), pack_half2(ds[8 * pc + 2], ds[8 * pc + 3]),
                               pack_half2(ds[8 * pc + 4], ds[8 * pc + 5]), pack_half2(ds[8 * pc + 6], ds[8 * pc + 7]));
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&ms.barP);
            mbar_arrive(&ms.empty[t & 1]);     // (the stage's release also waits for the MMAs' commit)
        }
        if (ok) {
            ok = mbar_wait(&ms.barAcc, (T - 1) & 1, abort_flag);
            tc_fence_after_sync();
        }
        if (ok) {      // the TMEM loads are warp-wide: only the stores depend on the key being real
            float4 *dv_dst = reinterpret_cast<float4 *>(dv_sm + ((size_t)bh * cap + j) * (D * kG) + x0);
            float4 *dk_dst = reinterpret_cast<float4 *>(dk_sm + ((size_t)bh * cap + j) * (D * kG) + x0);
            const float gi = grad_scale(status).y;          // dO and Dsm arrive times the gradient scale
            if (kMask && key_ok) dmask[(size_t)bhg * cap + j] = gi * msum;
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                uint32_t x[32], y[32];
                tmem_ld32(tDV + lane_base + cb * 32, x);
                tmem_ld32(tDK + lane_base + cb * 32, y);
                tmem_wait_ld();
                if (!key_ok) continue;
#pragma unroll
                for (int c4 = 0; c4 < 8; ++c4) {
                    dv_dst[cb * 8 + c4] = make_float4(gi * __uint_as_float(x[4 * c4]), gi * __uint_as_float(x[4 * c4 + 1]),
                                                      gi * __uint_as_float(x[4 * c4 + 2]), gi * __uint_as_float(x[4 * c4 + 3]));
                    dk_dst[cb * 8 + c4] = make_float4(gi * __uint_as_float(y[4 * c4]), gi * __uint_as_float(y[4 * c4 + 1]),
                                                      gi * __uint_as_float(y[4 * c4 + 2]), gi * __uint_as_float(y[4 * c4 + 3]));
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, SL::kTmem);
    }
    if (tid == 0 && ms.abort_flag) atomicMin(status, (int)NATSL_ERR_TIMEOUT);
}

// q (bf16, [B,L,H,d]) -> fp16 [B,H,L,d]; 8 values per thread.  norm_eps >= 0: each of the `groups` slices
// of a row RMS-normalised on the way (Section 4.3: the softmax operation's q; a slice's pieces sit in
// neighbouring lanes).
template <int D>
__global__ void __launch_bounds__(256)
to_f16_bhld_kernel(const __nv_bfloat16 *__restrict__ q, __half *__restrict__ qh, int B, int L, int H,
                   int groups, float norm_eps) {
    constexpr int kPieces = D / 8;
    const size_t idx = (size_t)blockIdx.x * 256 + threadIdx.x;
    const size_t total = (size_t)B * L * H * kPieces;
    if (idx >= total) return;
    const int pc = idx % kPieces;
    const size_t row = idx / kPieces;          // (b, l, h)
    const int h = row % H;
    const size_t bl = row / H;
    const int l = bl % L, b = bl / L;
    const uint4 u = reinterpret_cast<const uint4 *>(q)[idx];
    const uint32_t wv[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
    float rq = 1.f;
    if (norm_eps >= 0.f) {         // (the grid covers whole rows, so all lanes of a row are here)
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(wv[i] << 16), hi = __uint_as_float(wv[i] & 0xffff0000u);
            ss = fmaf(lo, lo, fmaf(hi, hi, ss));
        }
        const int lanes = kPieces / groups;
        const unsigned row_mask = ((1u << kPieces) - 1u) << ((threadIdx.x & 31) & ~(kPieces - 1));
        for (int off = 1; off < lanes; off <<= 1) ss += __shfl_xor_sync(row_mask, ss, off);
        rq = rsqrtf(ss * groups / D + norm_eps);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
        o[i] = pack_half2(__uint_as_float(wv[i] << 16) * rq, __uint_as_float(wv[i] & 0xffff0000u) * rq);
    reinterpret_cast<uint4 *>(qh)[(((size_t)b * H + h) * L + l) * kPieces + pc] =
        make_uint4(o[0], o[1], o[2], o[3]);
}

}  // namespace

template <int D, int G>      // D: columns of a softmax head, G of them per linear head (s.d = D G)
static cudaError_t softmax_bwd_tc_impl(const void *q, void *Qh, const void *dO16, const void *k16,
                                       const void *v16, int cap, const int32_t *sm_idx,
                                       const int32_t *pre, const float *lse, const float *Dsm,
                                       float scale_sm, float *dq_sm, float *dk_sm, float *dv_sm,
                                       float *dmask, bool qh_ready, int32_t *status, Shape s,
                                       cudaStream_t st, cudaStream_t st_kv, float norm_eps) {
    const uint64_t BH = (uint64_t)s.B * s.H;
    constexpr int DL = D * G;
    if (!qh_ready) {      // (the linear branch's prepare kernel leaves the same fp16 copy of q behind --
                          //  unless q is normalised, differently for the two operations)
        const size_t pieces = (size_t)s.B * s.L * s.H * (DL / 8);
        to_f16_bhld_kernel<DL><<<(unsigned)((pieces + 255) / 256), 256, 0, st>>>(
            (const __nv_bfloat16 *)q, (__half *)Qh, s.B, s.L, s.H, G, norm_eps);
        count_launch();
    }
    CUtensorMap mq128, mdo128, mk64, mv64, mq64, mdo64, mk128, mv128;
    if (!tch::make_map_2d(&mq128, Qh, BH * s.L, DL, 128) || !tch::make_map_2d(&mdo128, dO16, BH * s.L, DL, 128) ||
        !tch::make_map_2d(&mk64, k16, BH * cap, DL, 64) || !tch::make_map_2d(&mv64, v16, BH * cap, DL, 64) ||
        !tch::make_map_2d(&mq64, Qh, BH * s.L, DL, 64) || !tch::make_map_2d(&mdo64, dO16, BH * s.L, DL, 64) ||
        !tch::make_map_2d(&mk128, k16, BH * cap, DL, 128) || !tch::make_map_2d(&mv128, v16, BH * cap, DL, 128))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(softmax_bwd_dq_tc_kernel<D, G>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, QLayout<D>::kTotal);
    if (e != cudaSuccess) return e;
    auto dkv = dmask ? softmax_bwd_dkv_tc_kernel<D, true, G> : softmax_bwd_dkv_tc_kernel<D, false, G>;
    e = cudaFuncSetAttribute(dkv, cudaFuncAttributeMaxDynamicSharedMemorySize, KLayout<D>::kTotal);
    if (e != cudaSuccess) return e;
    dim3 gq((s.L + 127) / 128, s.B * s.H * G);
    softmax_bwd_dq_tc_kernel<D, G><<<gq, kThreadsB, QLayout<D>::kTotal, st>>>(
        mq128, mdo128, mk64, mv64, cap, sm_idx, pre, lse, Dsm, scale_sm, dq_sm, status, s.L, s.H, debug_wait_kcycles());
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    dim3 gk((s.L + 127) / 128, s.B * s.H * G);
    dkv<<<gk, kThreadsB, KLayout<D>::kTotal, st_kv>>>(
        mq64, mdo64, mk128, mv128, cap, sm_idx, pre, lse, Dsm, scale_sm, dk_sm, dv_sm, dmask, status, s.L, s.H, debug_wait_kcycles());
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_softmax_bwd_tc(const void *q, void *Qh, const void *dO16, const void *k16,
                                  const void *v16, int cap, const int32_t *sm_idx,
                                  const int32_t *sm_chunk_prefix, const float *lse, const float *Dsm,
                                  float scale_sm, float *dq_sm, float *dk_sm, float *dv_sm,
                                  float *dmask, bool qh_ready, int32_t *status, Shape s,
                                  cudaStream_t st, cudaStream_t st_kv, HeadGroups hg) {
    if (hg.norm_eps >= 0.f && qh_ready) return cudaErrorInvalidValue;   // (the copy at hand is the linear operation's)
    if (hg.G == 2 && s.d == 128)
        return softmax_bwd_tc_impl<64, 2>(q, Qh, dO16, k16, v16, cap, sm_idx, sm_chunk_prefix, lse, Dsm, scale_sm,
                                          dq_sm, dk_sm, dv_sm, dmask, qh_ready, status, s, st, st_kv, hg.norm_eps);
    if (hg.G > 1) return cudaErrorInvalidValue;
    if (s.d == 128)
        return softmax_bwd_tc_impl<128, 1>(q, Qh, dO16, k16, v16, cap, sm_idx, sm_chunk_prefix, lse, Dsm, scale_sm,
                                           dq_sm, dk_sm, dv_sm, dmask, qh_ready, status, s, st, st_kv, hg.norm_eps);
    return softmax_bwd_tc_impl<64, 1>(q, Qh, dO16, k16, v16, cap, sm_idx, sm_chunk_prefix, lse, Dsm, scale_sm,
                                      dq_sm, dk_sm, dv_sm, dmask, qh_ready, status, s, st, st_kv, hg.norm_eps);
}

}  // namespace natsl

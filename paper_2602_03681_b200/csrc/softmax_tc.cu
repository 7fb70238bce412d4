// Tensor-core softmax branch over the retained tokens (Section 4.1, O_nla with mask M^nla) with
// the RMS-norm / weighted combination (Section 4.3, Norm equation) as its epilogue, for bf16
// storage on sm_100a.
//
// One CTA owns 128 consecutive queries of one (batch, head) and walks the compacted K/V of that
// head in tiles of 64 retained tokens: logits = Q K^T as a bf16 tcgen05 MMA into TMEM (q and k
// are exact bf16 inputs), online softmax in registers (one thread per query row), probabilities
// written as fp16 into the TMEM columns their logits came from and P V as an fp16 MMA with A in
// TMEM (V is gathered as fp16: the bf16 inputs convert exactly, and an 11-bit probability keeps the
// branch output within ~2e-3 of its RMS where an 8-bit one would not).  The logits are
// double-buffered in TMEM, so the probabilities of tile t + 1 never wait for the product of tile
// t; with P in a single shared-memory tile every tile paid that product's latency.  K and V
// tiles arrive by TMA into two-stage rings.
// Epilogue: o_la arrives as the scan leaves it, fp16 and transposed per chunk (o_laT, one 16 KB tile
// per chunk: [8 pieces][d][8 tokens], row r of piece p at slot r ^ p); the CTA's two tiles come in
// by bulk copies (into the Q tile, free once the last Q K^T has run) while the last K/V tile is still
// being processed, and each thread reads its query's column out of them (the slot permutation
// spreads a warp's four pieces over the banks), normalises
// its own row of both branches, combines them and writes its row of `out` into a swizzled
// shared-memory tile that one bulk tensor store sends out, so that no global access of the
// epilogue is issued per thread and row.
// The kernel may run beside the scan that produces o_la (launched behind it as a programmatic
// dependent): nothing before the epilogue needs o_la, and the epilogue's load waits, bounded, for
// the per-chunk counters the scan raises (emit_flags); CTAs are then ordered by query tile first,
// so that the tiles whose chunks the scan finishes first are also scheduled first.
// Warp roles: warps 0-3 softmax/epilogue (thread r <-> query row r <-> TMEM lane r), warp 4 issues
// the MMAs, warp 5 issues the TMA loads.
// Block-level routing (template flag): after the retained tiles, one more tile per linear block of
// the CTA's two, holding that block's own 64 tokens (Section 4.1, inner-chunk correlations).
// Grouped softmax heads (template count kG; Section 4.3, several softmax heads under one linear head's
// mask): the kG softmax heads of linear head h are the kG column slices of D columns of its q, k, v.
// A CTA then serves one softmax head: its Q, K, V tiles are the slice's columns of the same tensors
// ([B,L,H,kG D] read as [B,L,H kG,D]), the retained-token lists, the counters and the weights are the
// linear head's, the softmax output is normalised over the slice and the linear read-out over its
// whole row of kG D columns, of which the CTA writes its slice.  With norm_eps >= 0 the logits are
// those of RMS-normalised q and k rows (Section 4.3), both as fp16: the K rows were normalised when
// they were gathered, the softmax threads normalise the Q tile in place before the first product.
#include "common.cuh"
#include "natsl_internal.h"
#include "tc_common.cuh"

namespace natsl {

namespace {

using namespace tc;

constexpr int kBM = 128;        // queries per CTA
constexpr int kBN = 64;         // retained tokens per K/V tile
constexpr int kStages = 2;
constexpr int kSoftmaxThreads = 128;
constexpr int kThreadsTc = 192;
constexpr int kMiscBytes = 1024;

template <int D> struct SmLayout {
    static constexpr int KB = D / 64;                    // 64-column blocks of the head dimension
    static constexpr int kQBytes = KB * kBM * 128;
    static constexpr int kKStage = KB * kBN * 128;
    static constexpr int kVStage = KB * kBN * 128;
    static constexpr int oQ = 0;
    static constexpr int oK = oQ + kQBytes;
    static constexpr int oV = oK + kStages * kKStage;
    static constexpr int oMisc = oV + kStages * kVStage;
    static constexpr int kTotal = oMisc + kMiscBytes;
};

struct Misc {                    // lives in the last kMiscBytes of the CTA's shared memory
    uint64_t barQ, barQn, barKn[2], fullK[kStages], emptyK[kStages], fullV[kStages], emptyV[kStages], barS[2], barP, barO, barE;
    uint32_t tmem_base;
    int abort_flag, wait_kcycles;   // in this order: the waits read the limit as abort_flag[1]
    alignas(16) int pos[kBM];    // positions of the retained tokens inside the CTA's own chunks
};
static_assert(sizeof(Misc) <= kMiscBytes, "misc page too small");

// kBlock: block-level routing (own-block tiles after the retained ones); kG: softmax heads per linear
// head; kNorm: RMS-normalised q and k (norm_eps is read only then)
template <int D, bool kBlock, int kG, bool kNorm>
__global__ void __launch_bounds__(kThreadsTc)
softmax_combine_tc_kernel(const __grid_constant__ CUtensorMap map_q,
                          const __grid_constant__ CUtensorMap map_k,
                          const __grid_constant__ CUtensorMap map_v,
                          const __grid_constant__ CUtensorMap map_out,    // out [B,L,H,D] bf16, box 128 x 64, if has_out
                          const __grid_constant__ CUtensorMap map_kd,     // the layer's k, v [B,L,H,D] bf16, box
                          const __grid_constant__ CUtensorMap map_vd,     //   64 x 64: own-block tiles (block routing)
                          const uint8_t *__restrict__ block_route, int appending, int cap, int capv, const int32_t *__restrict__ sm_idx,
                          const int32_t *__restrict__ sm_chunk_prefix,
                          const __half *__restrict__ o_laT, const int32_t *emit_flags,
                          const float *__restrict__ w,
                          float scale_sm, float eps, float norm_eps, int has_out, float *__restrict__ o_nla,
                          float *__restrict__ lse, int32_t *status, int L, int H, int wait_kcycles) {
    using SL = SmLayout<D>;
    constexpr int KB = SL::KB;
    constexpr int DL = D * kG;                            // columns of the linear head
    // the two o_laT tiles of the epilogue land in the Q tile and, for grouped heads, the K ring behind it
    static_assert(2 * DL * 128 <= SL::kQBytes + (kG > 1 ? kStages * SL::kKStage : 0), "o_laT tiles do not fit");
    static_assert(kG == 1 || SL::oK == SL::oQ + SL::kQBytes, "K ring must follow the Q tile");
    extern __shared__ __align__(1024) uint8_t smem[];
    Misc &ms = *reinterpret_cast<Misc *>(smem + SL::oMisc);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int NP = (L + kBM - 1) / kBM, NC = L / kC;
    // grid = (B*H, NP).  Beside the scan: tiles in ascending order, all (batch, head) pairs of a tile
    // before the next tile.  Otherwise: long rows first.
    const int p = emit_flags ? (int)blockIdx.y : NP - 1 - (int)blockIdx.y;
    // blockIdx.x = (batch, linear head, softmax head of the group); H counts linear heads
    const int bhg = blockIdx.x, bh = bhg / kG, sg = bhg % kG, b = bh / H, h = bh % H;
    const int hq = h * kG + sg;                           // head index in the [B,L,H kG,D] view
    const int c0 = 2 * p, c1 = min(2 * p + 2, NC);
    const int32_t *pre = sm_chunk_prefix + (size_t)bh * (NC + 1);
    const int n_full = min(pre[c0], cap);             // retained tokens before the CTA's chunks
    const int n_end = min(pre[c1], cap);              // ... up to the end of the CTA's chunks
    const int T = (n_end + kBN - 1) / kBN;
    // Block-level routing (Section 4.1, intra-chunk correlations of both operations): a query in a
    // linear block also reads the causal part of its own block, whose tokens are not among the
    // retained ones.  Each linear block of the CTA's two adds one tile, taken from the layer's
    // own k and v after the retained tiles (the softmax threads turn its V tile into fp16 in
    // place, exactly as the gather does for the retained rows).
    int nx = 0, xc0 = 0;                                // number of own-block tiles; block of the first
    if (kBlock)
        for (int e = 0; e < c1 - c0; ++e)
            if (block_route[((size_t)b * L + (size_t)(c0 + e) * kC) * H + h] == 0) {
                if (nx == 0) xc0 = e;
                ++nx;
            }
    const int T2 = kBlock ? T + nx : T;
    auto own_block = [&](int t) { return t == T ? xc0 : 1; };   // block (0 or 1) of own-block tile t >= T

    if ((smem_u32(smem) & 1023u) != 0) {              // operand tiles need 1024-byte alignment
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        mbar_init(&ms.barQ, 1);
        mbar_init(&ms.barQn, kSoftmaxThreads);       // normalised queries written (NATSL_QK_NORM)
        mbar_init(&ms.barKn[0], 1);                  // ... and the keys of an own-block tile: one barrier per tile,
        mbar_init(&ms.barKn[1], 1);                  //     each completing once
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&ms.fullK[s], 1); mbar_init(&ms.emptyK[s], 1);
            mbar_init(&ms.fullV[s], 1); mbar_init(&ms.emptyV[s], 1);
        }
        mbar_init(&ms.barS[0], 1);
        mbar_init(&ms.barS[1], 1);
        mbar_init(&ms.barP, kSoftmaxThreads);
        mbar_init(&ms.barO, 1);
        mbar_init(&ms.barE, 1);
        ms.abort_flag = 0;
        ms.wait_kcycles = wait_kcycles;
        fence_mbar_init();
    }
    if (tid < kBM) {    // sm_idx lists this call's retained tokens; when the call appends to a
        const int jj = n_full + tid - (appending ? pre[0] : 0);   // cache, pre[0] were there before
        ms.pos[tid] = n_full + tid < n_end ? sm_idx[(size_t)bh * L + jj] : 0x7fffffff;
    }
    if (warp == 4) tmem_alloc(&ms.tmem_base, 256);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = ms.tmem_base;
    const uint32_t tS[2] = {tmem, tmem + 64}, tO = tmem + 128;
    volatile int *abort_flag = &ms.abort_flag;

    if (warp == 5) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int nk = 0, nv = 0;                 // K / V tiles requested so far
            bool ok = true;
            if (T2 > 0) {                       // nothing is loaded for a tile that sees no key at all
                prefetch_tmap(&map_q); prefetch_tmap(&map_k); prefetch_tmap(&map_v);
                mbar_arrive_expect_tx(&ms.barQ, SL::kQBytes);
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_4d(smem + SL::oQ + kb * kBM * 128, &map_q, &ms.barQ, kb * 64, hq, p * kBM, b);
                // K and V tiles have their own rings: a K tile is free as soon as its Q K^T has run
                // (early), a V tile only after its P V; K(u) is therefore requested before V(u-1).
                for (int u = 0; u <= T2 && ok; ++u) {
                    if (u < T2) {
                        const int s = u % kStages;
                        ok = mbar_wait(&ms.emptyK[s], ((u / kStages) & 1) ^ 1, abort_flag);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&ms.fullK[s], SL::kKStage);
                        for (int kb = 0; kb < KB; ++kb) {
                            uint8_t *dst = smem + SL::oK + s * SL::kKStage + kb * kBN * 128;
                            if (!kBlock || u < T) tma_load_2d(dst, &map_k, &ms.fullK[s], sg * D + kb * 64, bh * cap + u * kBN);
                            else tma_load_4d(dst, &map_kd, &ms.fullK[s], kb * 64, hq, (c0 + own_block(u)) * kC, b);
                        }
                        nk = u + 1;
                    }
                    if (u >= 1) {
                        const int t = u - 1, s = t % kStages;
                        ok = mbar_wait(&ms.emptyV[s], ((t / kStages) & 1) ^ 1, abort_flag);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&ms.fullV[s], SL::kVStage);
                        for (int kb = 0; kb < KB; ++kb) {
                            uint8_t *dst = smem + SL::oV + s * SL::kVStage + kb * kBN * 128;
                            if (!kBlock || t < T) tma_load_2d(dst, &map_v, &ms.fullV[s], sg * D + kb * 64, bh * capv + t * kBN);
                            else tma_load_4d(dst, &map_vd, &ms.fullV[s], kb * 64, hq, (c0 + own_block(t)) * kC, b);
                        }
                        nv = t + 1;
                    }
                }
                // the Q tile and the K ring are free once the last Q K^T has run
                if (ok) ok = mbar_wait(&ms.emptyK[(T2 - 1) % kStages], ((T2 - 1) / kStages) & 1, abort_flag);
            }
            // beside the scan: the tile's chunks of o_la are complete once all row warps of the scan
            // CTA have raised the chunk's counter
            if (emit_flags) {
                for (int c = c0; c < c1 && ok; ++c)
                    ok = wait_counter_ge(emit_flags + (size_t)bh * NC + c, kScanRowWarps, abort_flag);
                fence_proxy_async_all();
            }
            bool e_issued = false;
            if (ok) {                           // the o_laT tiles of the CTA's one or two chunks
                mbar_arrive_expect_tx(&ms.barE, (c1 - c0) * DL * 128);
                for (int e = 0; e < c1 - c0; ++e)
                    bulk_load_1d(smem + SL::oQ + e * (DL * 128), o_laT + ((size_t)bh * NC + c0 + e) * DL * 64,
                                 DL * 128, &ms.barE);
                e_issued = true;
            }
            // No copy may be in flight when the CTA retires, aborted or not: wait (with a bound of
            // their own) for the copies issued last.
            if (T2 > 0) mbar_wait_drain(&ms.barQ, 0);
            for (int u = max(0, nk - kStages); u < nk; ++u)
                mbar_wait_drain(&ms.fullK[u % kStages], (u / kStages) & 1);
            for (int u = max(0, nv - kStages); u < nv; ++u)
                mbar_wait_drain(&ms.fullV[u % kStages], (u / kStages) & 1);
            if (e_issued) mbar_wait_drain(&ms.barE, 0);
        }
    } else if (warp == 4) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0 && T2 > 0) {
            // logits: q and k as given are bf16; normalised ones are fp16 (see the softmax threads)
            constexpr uint32_t idesc_qk = make_idesc(kNorm ? kFmtF16 : kFmtBF16, kBM, kBN, false, false);
            constexpr uint32_t idesc_pv = make_idesc(kFmtF16, kBM, D, false, true);
            const uint32_t aQ = smem_u32(smem + SL::oQ);
            auto issue_qk = [&](int t) {
                const uint32_t aK = smem_u32(smem + SL::oK + (t % kStages) * SL::kKStage);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16)
                        mma_ss(tS[t & 1], desc_kmajor(aQ + kb * kBM * 128 + k16 * 32),
                               desc_kmajor(aK + kb * kBN * 128 + k16 * 32), idesc_qk,
                               (kb | k16) != 0);
                mma_commit(&ms.emptyK[t % kStages]);
                mma_commit(&ms.barS[t & 1]);
            };
            // (normalisation with block-level routing: an own-block tile's keys arrive raw and are
            // normalised in place by the softmax threads first.  One single-phase barrier per own-block
            // tile, of which a CTA has at most two: with one barrier and a phase per tile, nothing kept the
            // softmax threads from completing the second phase before this thread had looked at the
            // first -- a parity wait then never returns -- and a late enough start of this thread, as in
            // the first wave of a launch, did let that happen.)
            auto own_keys_ready = [&](int t) {
                return !(kBlock && kNorm) || t < T || mbar_wait(&ms.barKn[t - T], 0, abort_flag);
            };
            bool ok = mbar_wait(&ms.barQ, 0, abort_flag) && (!kNorm || mbar_wait(&ms.barQn, 0, abort_flag)) &&
                      mbar_wait(&ms.fullK[0], 0, abort_flag) && own_keys_ready(0);
            if (ok) {
                tc_fence_after_sync();
                issue_qk(0);
            }
            for (int t = 0; ok && t < T2; ++t) {
                if (t + 1 < T2) {
                    ok = mbar_wait(&ms.fullK[(t + 1) % kStages], ((t + 1) / kStages) & 1, abort_flag) &&
                         own_keys_ready(t + 1);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_qk(t + 1);
                }
                ok = mbar_wait(&ms.barP, t & 1, abort_flag) &&
                     mbar_wait(&ms.fullV[t % kStages], (t / kStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t aV = smem_u32(smem + SL::oV + (t % kStages) * SL::kVStage);
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16)      // A = P(t): fp16 pairs in the first 32 columns of S(t)
                    mma_ts(tO, tS[t & 1] + k16 * 8, desc_mnmajor(aV + k16 * 2048, kBN * 128),
                           idesc_pv, (t | k16) != 0);
                mma_commit(&ms.emptyV[t % kStages]);
                mma_commit(&ms.barO);
            }
        }
    } else {
        // ------------------------------ softmax + epilogue ------------------------------
        const int r = tid;                              // query row inside the tile, TMEM lane
        const int i_abs = p * kBM + r;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float sl2 = scale_sm * 1.4426950408889634f;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        if (kNorm && T2 > 0) {
            // RMS-normalised queries (Section 4.3): thread r rewrites row r of the Q tile (bf16, as loaded)
            // as fp16 of the normalised row, over the D columns of its softmax head; the keys were
            // normalised and stored as fp16 when they were gathered, so the logit product is an fp16
            // MMA (bf16 keeps 8 bits: rounding the normalised keys to it alone costs 2.8e-2 of the
            // branch output's RMS).  Eight 16-byte pieces per row and block, taken in an order that
            // spreads the warp over the banks.
            ok = mbar_wait(&ms.barQ, 0, abort_flag);
            if (ok) {
                uint8_t *rowp = smem + SL::oQ + tid * 128;
                float ss = 0.f;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 a = *reinterpret_cast<const uint4 *>(rowp + kb * kBM * 128 + ((c ^ (tid & 7)) << 4));
                        const uint32_t wd[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float lo = __uint_as_float(wd[e] << 16), hi = __uint_as_float(wd[e] & 0xffff0000u);
                            ss = fmaf(lo, lo, fmaf(hi, hi, ss));
                        }
                    }
                const float rq = rsqrtf(ss / D + norm_eps);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint4 *pp = reinterpret_cast<uint4 *>(rowp + kb * kBM * 128 + ((c ^ (tid & 7)) << 4));
                        const uint4 a = *pp;
                        const uint32_t wd[4] = {a.x, a.y, a.z, a.w};
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            o[e] = pack_half2(__uint_as_float(wd[e] << 16) * rq, __uint_as_float(wd[e] & 0xffff0000u) * rq);
                        *pp = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                fence_proxy_async_smem();
                mbar_arrive(&ms.barQn);
            }
        }
        float2 wv = make_float2(0.5f, 0.5f);             // (w_nla, w_la) of this row
        if (w && i_abs < L) wv = __ldg(reinterpret_cast<const float2 *>(w + (((size_t)b * L + i_abs) * H + h) * 2));
        // The compacted keys are in position order, so row i sees exactly the first `cnt` of them:
        // all n_full earlier ones plus those of the CTA's own chunks at positions <= i.
        int cnt = n_full;
        for (int kq = 0; kq < n_end - n_full; ++kq) cnt += ms.pos[kq] <= i_abs ? 1 : 0;
        // Keys of own-block tile u (block-level routing with normalisation): raw bf16 rows from the layer's
        // k; threads 0-63 rewrite one row each as fp16 of the RMS-normalised row.
        auto normalise_own_keys = [&](int u) -> bool {
            if (!mbar_wait(&ms.fullK[u % kStages], (u / kStages) & 1, abort_flag)) return false;
            if (tid < kBN) {
                uint8_t *rowp = smem + SL::oK + (u % kStages) * SL::kKStage + tid * 128;
                float ss = 0.f;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const uint4 a = *reinterpret_cast<const uint4 *>(rowp + kb * kBN * 128 + ((c ^ (tid & 7)) << 4));
                        const uint32_t wd[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float lo = __uint_as_float(wd[e] << 16), hi = __uint_as_float(wd[e] & 0xffff0000u);
                            ss = fmaf(lo, lo, fmaf(hi, hi, ss));
                        }
                    }
                const float rk = rsqrtf(ss / D + norm_eps);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint4 *pp = reinterpret_cast<uint4 *>(rowp + kb * kBN * 128 + ((c ^ (tid & 7)) << 4));
                        const uint4 a = *pp;
                        const uint32_t wd[4] = {a.x, a.y, a.z, a.w};
                        uint32_t o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            o[e] = pack_half2(__uint_as_float(wd[e] << 16) * rk, __uint_as_float(wd[e] & 0xffff0000u) * rk);
                        *pp = make_uint4(o[0], o[1], o[2], o[3]);
                    }
            }
            // One arrival per tile, after all rows are written.  (With one arrival per thread, the threads
            // that have no row to write reached the next tile's arrival while the others were still
            // writing this tile's rows, and completed this tile's phase for them.)
            fence_proxy_async_smem();
            named_barrier_sync(2, kSoftmaxThreads);
            if (tid == 0) mbar_arrive(&ms.barKn[u - T]);
            return true;
        };
        if (kBlock && kNorm && ok && T2 > 0 && T == 0) ok = normalise_own_keys(0);
        for (int t = 0; ok && t < T2; ++t) {
            if (kBlock && kNorm && t + 1 < T2 && t + 1 >= T) {      // (before this tile's logits are waited for)
                ok = normalise_own_keys(t + 1);
                if (!ok) break;
            }
            ok = mbar_wait(&ms.barS[t & 1], (t >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sv[2][32];
            tmem_ld32(tS[t & 1] + lane_base, sv[0]);
            tmem_ld32(tS[t & 1] + lane_base + 32, sv[1]);
            tmem_wait_ld();
            float x[kBN];
#pragma unroll
            for (int c = 0; c < kBN; ++c) x[c] = __uint_as_float(sv[c >> 5][c & 31]);   // raw logits: the scale
                                                                                        // goes into the exponent's FMA
            const int j0 = t * kBN;
            if (kBlock && t >= T) {
                // own-block tile: row r sees keys 0 .. r % 64 if it is in that block
                const int vis = (r >> 6) == own_block(t) ? (r & 63) + 1 : 0;
#pragma unroll
                for (int c = 0; c < kBN; ++c) x[c] = c < vis ? x[c] : -INFINITY;
            } else if (!__all_sync(0xffffffffu, j0 + kBN <= cnt)) {   // some row of the warp is cut off here
#pragma unroll
                for (int c = 0; c < kBN; ++c) x[c] = j0 + c < cnt ? x[c] : -INFINITY;
            }
            float mx4[4] = {x[0], x[1], x[2], x[3]};      // four independent chains, not one of 63
#pragma unroll
            for (int c = 4; c < kBN; ++c) mx4[c & 3] = fmaxf(mx4[c & 3], x[c]);
            // (scale_sm > 0, checked on the host: the maximum of the raw logits is the maximum logit)
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * sl2;
            // The running maximum only has to bound the exponents, not equal the true maximum: it
            // is raised (and O rescaled) only when a logit exceeds it by more than 8 (base 2), so
            // probabilities stay below 2^8 and, for inputs whose logits vary little, the accumulator
            // is never touched between the tiles.  lse = m + log2(l) holds for any such m.
            const float m_new = (mx > m + 8.f || m == -INFINITY) ? fmaxf(m, mx) : m;
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            const float corr = exp2f(m - m_use);        // m = -inf -> 0; unchanged m -> 1
            float ps4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < kBN; ++c) {
                x[c] = ex2_ftz(fmaf(x[c], sl2, -m_use));
                ps4[c & 3] += x[c];
            }
            l = l * corr + ((ps4[0] + ps4[1]) + (ps4[2] + ps4[3]));
            m = m_new;
            // barO's phases are consumed strictly in order, one per tile (a parity wait cannot skip a
            // phase): before the accumulator is touched when it has to be rescaled, otherwise at the
            // end of the tile, when the previous tile's product has had the whole tile to finish.
            bool waited_o = false;
            if (t > 0 && __any_sync(0xffffffffu, corr != 1.f)) {
                waited_o = true;
                ok = mbar_wait(&ms.barO, (t - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                {
#pragma unroll
                    for (int cb = 0; cb < D / 32; ++cb) {
                        uint32_t ov[32];
                        tmem_ld32(tO + lane_base + cb * 32, ov);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * corr);
                        tmem_st32(tO + lane_base + cb * 32, ov);
                    }
                    tmem_wait_st();
                }
            }
            {
                uint32_t pk[32];                        // P(t), over the logits this thread has consumed
#pragma unroll
                for (int c = 0; c < 32; ++c) pk[c] = pack_half2(x[2 * c], x[2 * c + 1]);
                tmem_st32(tS[t & 1] + lane_base, pk);
                tmem_wait_st();
            }
            if (kBlock && t >= T) {   // own-block tile: its V rows arrived as bf16; fp16 in place (exact)
                ok = mbar_wait(&ms.fullV[t % kStages], (t / kStages) & 1, abort_flag);
                if (!ok) break;
                uint4 *vt = reinterpret_cast<uint4 *>(smem + SL::oV + (t % kStages) * SL::kVStage);
                for (int i = r; i < SL::kVStage / 16; i += kSoftmaxThreads) {
                    const uint4 a = vt[i];
                    auto cv = [](uint32_t wd) {
                        return pack_half2(__uint_as_float(wd << 16), __uint_as_float(wd & 0xffff0000u));
                    };
                    vt[i] = make_uint4(cv(a.x), cv(a.y), cv(a.z), cv(a.w));
                }
            }
            // (before the arrival below, not after it: once this thread has arrived, the MMA warp may
            // complete the next phase of barO too, and a parity wait two phases behind never returns)
            if (t > 0 && !waited_o) {
                ok = mbar_wait(&ms.barO, (t - 1) & 1, abort_flag);
                if (!ok) break;
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&ms.barP);
        }
        if (ok && T2 > 0) {
            ok = mbar_wait(&ms.barO, (T2 - 1) & 1, abort_flag);
            tc_fence_after_sync();
        }
        if (ok) ok = mbar_wait(&ms.barE, 0, abort_flag);        // the tile's rows of o_la have landed
        if (ok) {
            // o_laT tiles (fp16): chunk e of the CTA at oQ + e * D * 128; piece p (tokens 8 p ..) of
            // head-dimension row `row` at 16-byte slot p * D + (row ^ p).
            // out tile (bf16): box kb (columns 64 kb ..) at oV + kb * 16 KB, row r, piece j at j ^ (r & 7).
            const float inv = l > 0.f ? 1.f / l : 0.f;       // l = 0 (no visible key): o_nla = 0
            float ssn4[4] = {0.f, 0.f, 0.f, 0.f}, ssl4[4] = {0.f, 0.f, 0.f, 0.f};
            const int tok = r & 63, tp = tok >> 3;
            const uint8_t *la_col = smem + SL::oQ + (r >> 6) * (DL * 128) + tp * (DL * 16) + (tok & 7) * 2;
            if (kG > 1) {        // the other softmax heads' columns of the linear row: mean square only
#pragma unroll 4
                for (int row = 0; row < DL; row += 2) {
                    if (row / D == sg) continue;
                    const float a0 = __half2float(*reinterpret_cast<const __half *>(la_col + ((row ^ tp) << 4)));
                    const float a1 = __half2float(*reinterpret_cast<const __half *>(la_col + (((row + 1) ^ tp) << 4)));
                    ssl4[(row >> 1) & 3] = fmaf(a0, a0, fmaf(a1, a1, ssl4[(row >> 1) & 3]));
                }
            }
            // This query's column of o_la is read once, kept as fp16 pairs (D / 2 registers: the logits of
            // the main loop are dead by now) and used twice: for its mean square and for the output.
            uint32_t la2[D / 2];
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                uint32_t ov[32];
                if (T2 > 0) {
                    tmem_ld32(tO + lane_base + cb * 32, ov);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) ov[e] = 0u;
                }
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const int row = sg * D + 32 * cb + e;
                    const __half a0 = *reinterpret_cast<const __half *>(la_col + ((row ^ tp) << 4));
                    const __half a1 = *reinterpret_cast<const __half *>(la_col + (((row + 1) ^ tp) << 4));
                    const __half2 ap = __halves2half2(a0, a1);
                    la2[(32 * cb + e) / 2] = *reinterpret_cast<const uint32_t *>(&ap);
                    const float2 af = __half22float2(ap);
                    ssl4[(e >> 1) & 3] = fmaf(af.x, af.x, fmaf(af.y, af.y, ssl4[(e >> 1) & 3]));
                    const float o0 = __uint_as_float(ov[e]), o1 = __uint_as_float(ov[e + 1]);
                    ssn4[(e >> 1) & 3] = fmaf(o0, o0, fmaf(o1, o1, ssn4[(e >> 1) & 3]));
                }
            }
            // mean square of the normalised row = inv^2 * mean square of the accumulator row
            const float msn = inv * inv * ((ssn4[0] + ssn4[1]) + (ssn4[2] + ssn4[3])) / D;
            const float wn = wv.x * rsqrtf(msn + eps) * inv;          // applies to the raw accumulator
            const float wl = wv.y * rsqrtf(((ssl4[0] + ssl4[1]) + (ssl4[2] + ssl4[3])) / DL + eps);
            float *onla_row = o_nla && i_abs < L ? o_nla + (((size_t)b * L + i_abs) * H + h) * DL + sg * D : nullptr;
#pragma unroll
            for (int cb = 0; cb < D / 32; ++cb) {
                uint32_t ov[32];
                if (T2 > 0) {
                    tmem_ld32(tO + lane_base + cb * 32, ov);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) ov[e] = 0u;
                }
#pragma unroll
                for (int j2 = 0; j2 < 4; ++j2) {
                    float y[8];
#pragma unroll
                    for (int e = 0; e < 8; e += 2) {
                        const float2 af = __half22float2(*reinterpret_cast<const __half2 *>(&la2[(32 * cb + 8 * j2 + e) / 2]));
                        y[e] = fmaf(wn, __uint_as_float(ov[8 * j2 + e]), wl * af.x);
                        y[e + 1] = fmaf(wn, __uint_as_float(ov[8 * j2 + e + 1]), wl * af.y);
                    }
                    if (has_out)
                        *reinterpret_cast<uint4 *>(smem + SL::oV + (cb >> 1) * (kBM * 128) +
                                                   sw128_offset(r, (cb & 1) * 4 + j2)) =
                            make_uint4(pack_bf162(y[0], y[1]), pack_bf162(y[2], y[3]), pack_bf162(y[4], y[5]),
                                       pack_bf162(y[6], y[7]));
                    if (onla_row) {         // the raw branch output (fp32), straight from the registers
                        float4 *dst = reinterpret_cast<float4 *>(onla_row + cb * 32 + j2 * 8);
                        dst[0] = make_float4(__uint_as_float(ov[8 * j2]) * inv, __uint_as_float(ov[8 * j2 + 1]) * inv,
                                             __uint_as_float(ov[8 * j2 + 2]) * inv, __uint_as_float(ov[8 * j2 + 3]) * inv);
                        dst[1] = make_float4(__uint_as_float(ov[8 * j2 + 4]) * inv, __uint_as_float(ov[8 * j2 + 5]) * inv,
                                             __uint_as_float(ov[8 * j2 + 6]) * inv, __uint_as_float(ov[8 * j2 + 7]) * inv);
                    }
                }
            }
            if (lse && i_abs < L)
                lse[(size_t)bhg * L + i_abs] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
            fence_proxy_async_smem();
            named_barrier_sync(1, kSoftmaxThreads);
            if (tid == 0) {
                if (has_out)
                    for (int kb = 0; kb < KB; ++kb)
                        tma_store_4d(&map_out, smem + SL::oV + kb * (kBM * 128), kb * 64, hq, p * kBM, b);
                tma_store_commit();
                tma_store_wait_read();                      // shared memory may go once it has been read
            }
        }
    }
    // ------------------------------ teardown ------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 256);
    }
    if (tid == 0 && ms.abort_flag) atomicMin(status, (int)NATSL_ERR_TIMEOUT);
}

// Copy the retained tokens' K rows (bf16) and V rows (as fp16) into the compacted layouts
// [B,H,cap,d] / [B,H,capv,d] (optionally K as fp16 too, for the backward) and zero the fp16 rows
// up to the next multiple of 128, so that a K/V tile never multiplies a zero probability or a
// zero logit gradient with an uninitialised value.  grid = (row blocks, B*H).
template <int D>
__global__ void __launch_bounds__(256)
gather_kv_tc_kernel(const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                    const int32_t *__restrict__ sm_idx, const int32_t *__restrict__ sm_chunk_prefix,
                    __nv_bfloat16 *__restrict__ k_sm, __nv_bfloat16 *__restrict__ v_sm,
                    __half *__restrict__ v16, __half *__restrict__ k16, int cap, int capv, int appending,
                    int groups, float norm_eps, int raw_k_sm, int32_t *status, int L, int H) {
    // raw_k_sm (with the normalisation): k_sm is a cache that keeps the keys as given; the normalised
    // fp16 keys then go to k16 only
    constexpr int kVecPerRow = D * 2 / 16;
    constexpr int kRows = 256 / kVecPerRow;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int n_sm = sm_chunk_prefix[(size_t)bh * (NC + 1) + NC];
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_sm > cap) atomicMin(status, (int)NATSL_ERR_CACHE_FULL);
    const int n = min(n_sm, cap);
    const int n_pad = min((n + 127) / 128 * 128, capv);
    const int n_prev = appending ? sm_chunk_prefix[(size_t)bh * (NC + 1)] : 0;   // rows of earlier calls
    const int piece = threadIdx.x % kVecPerRow;
    // RMS-normalised keys of the softmax operation (Section 4.3), per softmax head = per slice of D / groups
    // columns, as fp16 (the softmax kernel's logit product is an fp16 MMA in this mode): the slice's pieces
    // sit in neighbouring lanes of the row's lanes.  bf16 pieces in, fp16 pieces out.
    auto rms_fp16 = [&](uint4 kk) {
        const uint32_t kw[4] = {kk.x, kk.y, kk.z, kk.w};
        float f[8], ss = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(kw[i] << 16);
            f[2 * i + 1] = __uint_as_float(kw[i] & 0xffff0000u);
            ss = fmaf(f[2 * i], f[2 * i], fmaf(f[2 * i + 1], f[2 * i + 1], ss));
        }
        const int lanes = kVecPerRow / groups;            // lanes per slice (a power of two)
        const unsigned row_mask = (kVecPerRow == 32 ? 0xffffffffu : ((1u << kVecPerRow) - 1u))
                                  << ((threadIdx.x & 31) & ~(kVecPerRow - 1));
        for (int o = 1; o < lanes; o <<= 1) ss += __shfl_xor_sync(row_mask, ss, o);
        const float rk = rsqrtf(ss * groups / D + norm_eps);
        return make_uint4(pack_half2(f[0] * rk, f[1] * rk), pack_half2(f[2] * rk, f[3] * rk),
                          pack_half2(f[4] * rk, f[5] * rk), pack_half2(f[6] * rk, f[7] * rk));
    };
    // the grid is sized for a typical retention rate; each CTA strides over the rows there are
    for (int row = blockIdx.x * kRows + threadIdx.x / kVecPerRow; row < n_pad; row += gridDim.x * kRows) {
        uint4 *dv16 = reinterpret_cast<uint4 *>(v16 + ((size_t)bh * capv + row) * D) + piece;
        uint4 *dk16 = k16 ? reinterpret_cast<uint4 *>(k16 + ((size_t)bh * capv + row) * D) + piece : nullptr;
        if (row >= n) {
            *dv16 = make_uint4(0u, 0u, 0u, 0u);
            if (dk16) *dk16 = make_uint4(0u, 0u, 0u, 0u);
            continue;
        }
        const size_t dst = ((size_t)bh * cap + row) * D;
        if (row < n_prev) {     // already in the cache: only the fp16 copy of its V row is made
            const uint4 vv = reinterpret_cast<const uint4 *>(v_sm + dst)[piece];
            const uint32_t wv[4] = {vv.x, vv.y, vv.z, vv.w};
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                o[i] = pack_half2(__uint_as_float(wv[i] << 16), __uint_as_float(wv[i] & 0xffff0000u));
            *dv16 = make_uint4(o[0], o[1], o[2], o[3]);
            // (and, with the normalisation, the normalised copy of its key, which the cache keeps as given)
            if (dk16 && norm_eps >= 0.f) *dk16 = rms_fp16(reinterpret_cast<const uint4 *>(k_sm + dst)[piece]);
            continue;
        }
        const int tok = sm_idx[(size_t)bh * L + row - n_prev];
        const size_t src = (((size_t)b * L + tok) * H + h) * D;
        uint4 kk = reinterpret_cast<const uint4 *>(k + src)[piece];
        if (norm_eps >= 0.f && raw_k_sm) reinterpret_cast<uint4 *>(k_sm + dst)[piece] = kk;
        if (norm_eps >= 0.f) kk = rms_fp16(kk);
        if (!(norm_eps >= 0.f && raw_k_sm)) reinterpret_cast<uint4 *>(k_sm + dst)[piece] = kk;
        if (dk16 && norm_eps >= 0.f) {
            *dk16 = kk;                                   // already fp16
        } else if (dk16) {
            const uint32_t kw[4] = {kk.x, kk.y, kk.z, kk.w};
            uint32_t ko[4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
                ko[i] = pack_half2(__uint_as_float(kw[i] << 16), __uint_as_float(kw[i] & 0xffff0000u));
            *dk16 = make_uint4(ko[0], ko[1], ko[2], ko[3]);
        }
        const uint4 vv = reinterpret_cast<const uint4 *>(v + src)[piece];
        if (v_sm) reinterpret_cast<uint4 *>(v_sm + dst)[piece] = vv;
        const uint32_t wv[4] = {vv.x, vv.y, vv.z, vv.w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            o[i] = pack_half2(__uint_as_float(wv[i] << 16), __uint_as_float(wv[i] & 0xffff0000u));
        *dv16 = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

}  // namespace

template <int D, int G>      // D: columns of a softmax head; G of them per linear head (s.d = D G)
static cudaError_t softmax_tc_impl(const void *q, const void *k_sm, const void *v16, int32_t cap,
                                   int32_t capv, const int32_t *sm_idx, const int32_t *pre,
                                   const void *o_la16, const int32_t *emit_flags, const float *w,
                                   float scale_sm, float eps, float norm_eps, void *out, float *o_nla, float *lse,
                                   BlockRouting br, bool appending, int32_t *status, Shape s,
                                   cudaStream_t st) {
    using SL = SmLayout<D>;
    CUtensorMap mq, mk, mv, mout, mkd, mvd;
    // q, out, k, v [B,L,H,G D] are read as [B,L,H G,D]; the compacted K/V rows keep all G D columns
    if (!tch::make_map_blhd(&mq, q, s.B, s.L, s.H * G, D, kBM) ||
        !tch::make_map_2d(&mk, k_sm, (uint64_t)s.B * s.H * cap, D * G, kBN) ||
        !tch::make_map_2d(&mv, v16, (uint64_t)s.B * s.H * capv, D * G, kBN))
        return cudaErrorInvalidValue;
    mout = mq;                                             // placeholder when `out` is not asked for
    if (out && !tch::make_map_blhd(&mout, out, s.B, s.L, s.H * G, D, kBM)) return cudaErrorInvalidValue;
    mkd = mq;
    mvd = mq;
    if (br.route && (!tch::make_map_blhd(&mkd, br.k, s.B, s.L, s.H * G, D, kBN) ||
                     !tch::make_map_blhd(&mvd, br.v, s.B, s.L, s.H * G, D, kBN)))
        return cudaErrorInvalidValue;
    auto kernel = softmax_combine_tc_kernel<D, false, G, false>;
    if (norm_eps >= 0.f) kernel = softmax_combine_tc_kernel<D, false, G, true>;
    if (br.route) kernel = norm_eps >= 0.f ? softmax_combine_tc_kernel<D, true, G, true>
                                          : softmax_combine_tc_kernel<D, true, G, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::kTotal);
    if (e != cudaSuccess) return e;
    // With emit_flags the kernel is launched as a programmatic dependent of the kernel before it in
    // the stream (the scan): it may start once all of the scan's CTAs are resident, and finds o_la
    // through the flags.  A launch the runtime serialises instead finds every flag already raised.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(s.B * s.H * G, (s.L + kBM - 1) / kBM);
    cfg.blockDim = dim3(kThreadsTc);
    cfg.dynamicSmemBytes = SL::kTotal;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = emit_flags ? 1 : 0;
    e = cudaLaunchKernelEx(&cfg, kernel, mq, mk, mv, mout, mkd, mvd, br.route, appending ? 1 : 0,
                           (int)cap, (int)capv, sm_idx, pre, (const __half *)o_la16, emit_flags, w, scale_sm, eps,
                           norm_eps, out ? 1 : 0, o_nla, lse, status, s.L, s.H, debug_wait_kcycles());
    count_launch();
    return e;
}

cudaError_t launch_softmax_combine_tc(const void *q, const void *k_sm, const void *v16, int32_t cap,
                                      int32_t capv, const int32_t *sm_idx,
                                      const int32_t *sm_chunk_prefix, const void *o_la16,
                                      const int32_t *emit_flags, const float *w, float scale_sm,
                                      float eps, void *out, float *o_nla, float *lse, BlockRouting br,
                                      bool appending, int32_t *status, Shape s, cudaStream_t st,
                                      HeadGroups hg) {
    if (hg.G == 2 && s.d == 128)
        return softmax_tc_impl<64, 2>(q, k_sm, v16, cap, capv, sm_idx, sm_chunk_prefix, o_la16, emit_flags,
                                      w, scale_sm, eps, hg.norm_eps, out, o_nla, lse, br, appending, status, s, st);
    if (hg.G > 1) return cudaErrorInvalidValue;
    if (s.d == 128)
        return softmax_tc_impl<128, 1>(q, k_sm, v16, cap, capv, sm_idx, sm_chunk_prefix, o_la16, emit_flags,
                                       w, scale_sm, eps, hg.norm_eps, out, o_nla, lse, br, appending, status, s, st);
    return softmax_tc_impl<64, 1>(q, k_sm, v16, cap, capv, sm_idx, sm_chunk_prefix, o_la16, emit_flags, w,
                                  scale_sm, eps, hg.norm_eps, out, o_nla, lse, br, appending, status, s, st);
}

template <int D>
static cudaError_t gather_tc_impl(const void *k, const void *v, const int32_t *sm_idx,
                                  const int32_t *pre, void *k_sm, void *v_sm, void *v16, void *k16,
                                  int cap, int capv, bool appending, int32_t *status, Shape s,
                                  cudaStream_t st, HeadGroups hg, bool raw_k_sm) {
    constexpr int kRows = 256 / (D * 2 / 16);
    const int max_rows = s.L < capv ? s.L : capv;
    const int blocks = (max_rows + kRows - 1) / kRows;
    dim3 grid(blocks < 48 ? blocks : 48, s.B * s.H);
    gather_kv_tc_kernel<D><<<grid, 256, 0, st>>>(
        (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, sm_idx, pre, (__nv_bfloat16 *)k_sm,
        (__nv_bfloat16 *)v_sm, (__half *)v16, (__half *)k16, cap, capv, appending ? 1 : 0, hg.G, hg.norm_eps,
        raw_k_sm ? 1 : 0, status, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gather_kv_tc(const void *k, const void *v, const int32_t *sm_idx,
                                const int32_t *sm_chunk_prefix, void *k_sm, void *v_sm, void *v16,
                                void *k16, int32_t cap, int32_t capv, bool appending, int32_t *status,
                                Shape s, cudaStream_t st, HeadGroups hg, bool raw_k_sm) {
    if (s.d == 128)
        return gather_tc_impl<128>(k, v, sm_idx, sm_chunk_prefix, k_sm, v_sm, v16, k16, cap, capv, appending, status, s, st, hg, raw_k_sm);
    return gather_tc_impl<64>(k, v, sm_idx, sm_chunk_prefix, k_sm, v_sm, v16, k16, cap, capv, appending, status, s, st, hg, raw_k_sm);
}

}  // namespace natsl

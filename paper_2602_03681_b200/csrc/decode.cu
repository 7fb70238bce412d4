// Decode step (Section 4.1, per-token generation): decay the fp32 d x d state, apply the gated
// delta rule (linear token) or retain the token's K/V (softmax token) -- or both, while the
// decision of the token's block is still open -- read both branches and combine their
// RMS-normalised outputs (Section 4.3, Norm equation).  decode_block_end_kernel rolls back the
// operation that was not chosen once a block is complete.
//
// HBM-bound: per (sequence, head) the state is read and written once (2 d^2 4 bytes) and the
// retained K/V are read once.  To keep enough bytes in flight and the SMs evenly loaded, each
// (sequence, head) is split over kDecodeParts + kStateParts CTAs: a "cache" CTA streams one slice
// of the retained K/V through a four-stage ring of bulk asynchronous copies (16 KB per stage in
// flight whatever the arithmetic is doing) and leaves a partial online-softmax result in the
// workspace; a "state" CTA streams half of the state's value columns through registers (the
// columns of the delta rule are independent) and leaves its part of the linear read-out there.
// Whichever CTA of the head finishes last (an atomic ticket, nobody waits) merges the partials,
// adds the new token's own term, normalises, combines, writes `out`, appends the token to the
// cache and bumps its length.
// Grouped softmax heads and per-operation q/k normalisation (Section 4.3; template flag, so that the
// plain instantiation is unchanged code): the G softmax heads of a linear head are the G slices of d / G
// columns -- the lanes that share a key row split into G groups, each with its own logit, running
// maximum and sum --, the state CTAs work on the L2-normalised q and k, and the cache keeps the keys as
// given: a cached key is RMS-normalised per slice as it is read (its sum of squares rides along with the
// logit's reduction), because normalised keys rounded to the cache's bf16 would cost 2.8e-2 of the
// branch output's RMS.
#include "common.cuh"
#include "natsl_internal.h"
#include "tc_common.cuh"

namespace natsl {

namespace {

using namespace tc;

constexpr int kWorkThreads = 256;
constexpr int kWarps = kWorkThreads / 32;
constexpr int kThreads = kWorkThreads + 32;      // + one warp that issues the bulk copies
constexpr int kTileKeys = 32;
constexpr int kStages = 4;
constexpr int kStateParts = 2;
constexpr int kCtasPerHead = kDecodeParts + kStateParts;

template <typename T> struct Vec16;   // 16 bytes of T as fp32 values
template <> struct Vec16<float> {
    static constexpr int kN = 4;
    __device__ static void unpack(const uint4 u, float (&x)[4]) {
        x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
        x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kN = 8;
    __device__ static void unpack(const uint4 u, float (&x)[8]) {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

// Workspace: [0,256) status word; then tickets [BH] i32; partials [BH][kDecodeParts][D+8] f32
// (m[G], z[G] in the first 8 with G <= 4, then acc[D]); o_la [BH][D] f32.
constexpr int kPartHead = 8;
__host__ __device__ inline size_t dec_off_tickets() { return 256; }
__host__ __device__ inline size_t dec_off_partials(size_t BH) {
    return (256 + BH * 4 + 255) / 256 * 256;
}
__host__ __device__ inline size_t dec_off_ola(size_t BH, int D) {
    return dec_off_partials(BH) + (BH * kDecodeParts * (D + kPartHead) * 4 + 255) / 256 * 256;
}

template <typename T, int D, bool kGrouped>
__global__ void __launch_bounds__(kThreads, 3)
decode_step_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                   const float *__restrict__ g, const float *__restrict__ beta,
                   const uint8_t *__restrict__ route, const float *__restrict__ w,
                   float *__restrict__ state, T *__restrict__ k_cache, T *__restrict__ v_cache,
                   int32_t *__restrict__ cache_len, int cap, T *__restrict__ out, float scale_la,
                   float scale_sm, float eps, uint8_t *__restrict__ ws, int BH, int Gin, float norm_eps) {
    const int G = kGrouped ? Gin : 1;              // softmax heads per linear head
    const int ds = D / G;                          // columns per softmax head
    const bool normed = kGrouped && norm_eps >= 0.f;
    constexpr int kE = Vec16<T>::kN;               // elements per 16-byte piece
    constexpr int kRowBytes = D * (int)sizeof(T);
    constexpr int kLpk = kRowBytes / 16;           // lanes per key row
    constexpr int kStreams = kWorkThreads / kLpk;  // independent online-softmax streams
    constexpr int kTileBytes = kTileKeys * kRowBytes;
    static_assert(kStreams <= kTileKeys && kTileKeys % kStreams == 0, "tile / stream mismatch");

    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ __align__(16) float qs[D], ks[D], vs[D];     // (normalised: the linear operation's q, k)
    __shared__ __align__(16) float qsm[kGrouped ? D : 4], ksm[kGrouped ? D : 4];   // the softmax operation's q, k
    __shared__ float sm_m[kTileKeys * (kGrouped ? 4 : 1)], sm_z[kTileKeys * (kGrouped ? 4 : 1)];
    __shared__ float norm_red[2][kWarps];
    __shared__ int s_last, s_abort[2];   // s_abort[1]: wait limit (see mbar_wait)

    const int part = blockIdx.x, bh = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int32_t *status = reinterpret_cast<int32_t *>(ws);
    int32_t *ticket = reinterpret_cast<int32_t *>(ws + dec_off_tickets()) + bh;
    float *partials =
        reinterpret_cast<float *>(ws + dec_off_partials(BH)) + (size_t)bh * kDecodeParts * (D + kPartHead);
    float *ola_ws = reinterpret_cast<float *>(ws + dec_off_ola(BH, D)) + (size_t)bh * D;

    // route 0: linear token (delta rule); 1: softmax token (appended to the cache); 2: token of a
    // block whose decision is still open -- both (Section 4.1, pseudo-update of both hidden states)
    const int rv = route[bh];
    const bool r = rv != 0;                        // append, and attend to itself
    const bool fold = rv != 1;                     // delta rule
    // A stored length outside [0, cap] (a prefill whose cache overflowed, a caller's mistake) is
    // clamped, so that no copy below can leave the head's rows, and reported.
    const int n_raw = cache_len[bh];
    const int n_old = min(max(n_raw, 0), cap);
    if (n_raw != n_old && tid == 0 && part == 0) atomicMin(status, (int)NATSL_ERR_CACHE_FULL);
    const bool cache_full = r && n_old >= cap;     // no room: the sequence is left untouched
    if (tid < D) {
        qs[tid] = to_f32(q[(size_t)bh * D + tid]);
        ks[tid] = to_f32(k[(size_t)bh * D + tid]);
        vs[tid] = to_f32(v[(size_t)bh * D + tid]);
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kWorkThreads); }
        s_abort[0] = 0;
        s_abort[1] = 0;
        fence_mbar_init();
    }
    __syncthreads();
    volatile int *abort_flag = s_abort;
    if (kGrouped && warp < kWarps) {     // (the work threads only: the copy warp goes straight to its ring)
        // q, k of the two operations: L2 over the row for the linear one (in place in qs, ks), RMS per slice
        // for the softmax one (qsm, ksm); without the normalisation both are the token's q, k.
        float sq = 0.f, sk = 0.f;
        if (tid < D) { sq = qs[tid] * qs[tid]; sk = ks[tid] * ks[tid]; }
        sq = warp_sum(sq);
        sk = warp_sum(sk);
        if (lane == 0 && warp < D / 32) { norm_red[0][warp] = sq; norm_red[1][warp] = sk; }
        named_barrier_sync(1, kWorkThreads);
        if (tid < D) {
            float aq = 0.f, ak = 0.f, gq = 0.f, gk = 0.f;
            for (int wv = 0; wv < D / 32; ++wv) {
                aq += norm_red[0][wv];
                ak += norm_red[1][wv];
                if ((32 * wv) / ds == tid / ds) { gq += norm_red[0][wv]; gk += norm_red[1][wv]; }
            }
            const float qv = qs[tid], kv = ks[tid];
            qsm[tid] = normed ? qv * rsqrtf(gq / ds + norm_eps) : qv;
            ksm[tid] = normed ? kv * rsqrtf(gk / ds + norm_eps) : kv;
            if (normed) { qs[tid] = qv * rsqrtf(aq + norm_eps); ks[tid] = kv * rsqrtf(ak + norm_eps); }
        }
        named_barrier_sync(1, kWorkThreads);
    }

    if (part < kDecodeParts) {
        // ---------------- cache CTA: one slice of the retained K/V ----------------
        const int tiles_total = cache_full ? 0 : (n_old + kTileKeys - 1) / kTileKeys;
        const int tpp = (tiles_total + kDecodeParts - 1) / kDecodeParts;
        const int t_begin = min(part * tpp, tiles_total), t_end = min(t_begin + tpp, tiles_total);
        const uint8_t *kc = reinterpret_cast<const uint8_t *>(k_cache + (size_t)bh * cap * D);
        const uint8_t *vc = reinterpret_cast<const uint8_t *>(v_cache + (size_t)bh * cap * D);
        if (warp == kWarps) {
            if (lane == 0) {
                int t = t_begin;
                for (; t < t_end; ++t) {
                    const int i = t - t_begin, s = i % kStages;
                    if (!mbar_wait(&empty[s], ((i / kStages) & 1) ^ 1, abort_flag)) break;
                    const int rows = min(kTileKeys, n_old - t * kTileKeys);
                    const uint32_t bytes = (uint32_t)rows * kRowBytes;
                    mbar_arrive_expect_tx(&full[s], 2 * bytes);
                    bulk_load_1d(smem + (2 * s) * kTileBytes, kc + (size_t)t * kTileBytes, bytes, &full[s]);
                    bulk_load_1d(smem + (2 * s + 1) * kTileBytes, vc + (size_t)t * kTileBytes, bytes,
                                 &full[s]);
                }
                if (*abort_flag)           // let the copies already issued land before the CTA retires
                    for (int u = max(t_begin, t - kStages); u < t; ++u)
                        mbar_wait_drain(&full[(u - t_begin) % kStages], ((u - t_begin) / kStages) & 1);
            }
        } else {
            const int stream = tid / kLpk, piece = tid % kLpk;
            float qf[kE];
#pragma unroll
            for (int x = 0; x < kE; ++x) qf[x] = (kGrouped ? qsm[piece * kE + x] : qs[piece * kE + x]) * scale_sm;
            const int lps = kLpk / G;              // lanes per softmax head within a key row
            const float inv_ds = 1.f / ds;
            float m = -INFINITY, z = 0.f, acc[kE];
#pragma unroll
            for (int x = 0; x < kE; ++x) acc[x] = 0.f;
            for (int t = t_begin; t < t_end; ++t) {
                const int i = t - t_begin, s = i % kStages;
                if (!mbar_wait(&full[s], (i / kStages) & 1, abort_flag)) break;
                const uint8_t *kt = smem + (2 * s) * kTileBytes, *vt = kt + kTileBytes;
                const int rows = min(kTileKeys, n_old - t * kTileKeys);
#pragma unroll
                for (int u = 0; u < kTileKeys / kStreams; ++u) {
                    const int j = u * kStreams + stream;       // trip count uniform over the warp
                    float kx[kE], vx[kE];
                    Vec16<T>::unpack(*reinterpret_cast<const uint4 *>(kt + j * kRowBytes + piece * 16), kx);
                    Vec16<T>::unpack(*reinterpret_cast<const uint4 *>(vt + j * kRowBytes + piece * 16), vx);
                    float sc = 0.f;
#pragma unroll
                    for (int x = 0; x < kE; ++x) sc = fmaf(qf[x], kx[x], sc);
                    if (!kGrouped) {
#pragma unroll
                        for (int o = kLpk / 2; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
                    } else {                     // per softmax head; the key's sum of squares rides along
                        float kk = 0.f;
#pragma unroll
                        for (int x = 0; x < kE; ++x) kk = fmaf(kx[x], kx[x], kk);
#pragma unroll
                        for (int o = kLpk / 2; o > 0; o >>= 1)
                            if (o < lps) {           // (uniform: the group count is the same for every lane)
                                sc += __shfl_xor_sync(0xffffffffu, sc, o);
                                kk += __shfl_xor_sync(0xffffffffu, kk, o);
                            }
                        if (normed) sc *= rsqrtf(fmaf(kk, inv_ds, norm_eps));
                    }
                    if (j < rows) {                            // rows past the slice hold stale bytes
                        const float m_new = fmaxf(m, sc);
                        const float corr = __expf(m - m_new), pj = __expf(sc - m_new);
                        z = fmaf(z, corr, pj);
                        m = m_new;
#pragma unroll
                        for (int x = 0; x < kE; ++x) acc[x] = fmaf(acc[x], corr, pj * vx[x]);
                    }
                }
                mbar_arrive(&empty[s]);
            }
            // merge the streams of this CTA -> one partial (m, z, acc[D]); the ring is free now
            float *stage_acc = reinterpret_cast<float *>(smem);   // [kStreams][D]
            named_barrier_sync(1, kWorkThreads);
            if (piece % lps == 0) { sm_m[stream * G + piece / lps] = m; sm_z[stream * G + piece / lps] = z; }
#pragma unroll
            for (int x = 0; x < kE; ++x) stage_acc[stream * D + piece * kE + x] = acc[x];
            named_barrier_sync(1, kWorkThreads);
            if (tid < D) {
                const int sg = tid / ds;             // this column's softmax head
                float M = -INFINITY;
                for (int st = 0; st < kStreams; ++st) M = fmaxf(M, sm_m[st * G + sg]);
                float Z = 0.f, o = 0.f;
                if (M > -INFINITY) {
                    for (int st = 0; st < kStreams; ++st) {
                        const float f = __expf(sm_m[st * G + sg] - M);
                        Z = fmaf(sm_z[st * G + sg], f, Z);
                        o = fmaf(stage_acc[st * D + tid], f, o);
                    }
                }
                float *pp = partials + (size_t)part * (D + kPartHead);
                pp[kPartHead + tid] = o;
                if (tid % ds == 0) { pp[sg] = M; pp[4 + sg] = Z; }
            }
        }
    } else if (warp < kWarps && !cache_full) {
        // ---------------- state CTA: half of the value columns, all rows ----------------
        constexpr int kCols = D / kStateParts;      // value columns of this CTA
        constexpr int kLpr = kCols / 4;             // lanes per (half) state row
        constexpr int kRpl = 32 / kLpr;             // rows per warp-wide access
        constexpr int kSlots = kWarps * kRpl;       // row slots in the CTA
        constexpr int kR = D / kSlots;              // rows per thread
        static_assert(kSlots <= 32, "reduction scratch too small");
        float (*redv)[kCols] = reinterpret_cast<float (*)[kCols]>(smem);   // [kSlots][kCols]
        const int c0 = (part - kDecodeParts) * kCols;
        const float alpha = __expf(g[bh]);
        const float bt = fold ? beta[bh] : 0.f;
        const int slot = warp * kRpl + lane / kLpr;
        const int col = (lane % kLpr) * 4;
        float *sp = state + (size_t)bh * D * D + c0;
        float4 s[kR];
#pragma unroll
        for (int rr = 0; rr < kR; ++rr)
            s[rr] = *reinterpret_cast<const float4 *>(sp + (size_t)(slot * kR + rr) * D + col);
#pragma unroll
        for (int rr = 0; rr < kR; ++rr) {
            s[rr].x *= alpha; s[rr].y *= alpha; s[rr].z *= alpha; s[rr].w *= alpha;
        }
        if (fold) {   // block-uniform
            float4 p = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int rr = 0; rr < kR; ++rr) {
                const float ka = ks[slot * kR + rr];
                p.x = fmaf(ka, s[rr].x, p.x); p.y = fmaf(ka, s[rr].y, p.y);
                p.z = fmaf(ka, s[rr].z, p.z); p.w = fmaf(ka, s[rr].w, p.w);
            }
            *reinterpret_cast<float4 *>(&redv[slot][col]) = p;
            named_barrier_sync(1, kWorkThreads);
            float4 e = *reinterpret_cast<const float4 *>(&vs[c0 + col]);
#pragma unroll
            for (int sl = 0; sl < kSlots; ++sl) {
                const float4 t = *reinterpret_cast<const float4 *>(&redv[sl][col]);
                e.x -= t.x; e.y -= t.y; e.z -= t.z; e.w -= t.w;
            }
#pragma unroll
            for (int rr = 0; rr < kR; ++rr) {
                const float bk = bt * ks[slot * kR + rr];
                s[rr].x = fmaf(bk, e.x, s[rr].x); s[rr].y = fmaf(bk, e.y, s[rr].y);
                s[rr].z = fmaf(bk, e.z, s[rr].z); s[rr].w = fmaf(bk, e.w, s[rr].w);
            }
            named_barrier_sync(1, kWorkThreads);   // redv is reused below
        }
        float4 p = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int rr = 0; rr < kR; ++rr) {
            const float qa = qs[slot * kR + rr];
            p.x = fmaf(qa, s[rr].x, p.x); p.y = fmaf(qa, s[rr].y, p.y);
            p.z = fmaf(qa, s[rr].z, p.z); p.w = fmaf(qa, s[rr].w, p.w);
            *reinterpret_cast<float4 *>(sp + (size_t)(slot * kR + rr) * D + col) = s[rr];
        }
        *reinterpret_cast<float4 *>(&redv[slot][col]) = p;
        named_barrier_sync(1, kWorkThreads);
        if (tid < kCols) {
            float a = 0.f;
#pragma unroll
            for (int sl = 0; sl < kSlots; ++sl) a += redv[sl][tid];
            ola_ws[c0 + tid] = scale_la * a;
        }
    }

    // -------- ticket: the last CTA of this (sequence, head) to get here finishes the step --------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int old = atomicAdd(ticket, 1);
        s_last = old == kCtasPerHead - 1;
        if (s_last) *ticket = 0;                      // ready for the next step
        if (s_abort[0]) atomicMin(status, (int)NATSL_ERR_TIMEOUT);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (cache_full) {
        if (tid < D) out[(size_t)bh * D + tid] = from_f32<T>(0.f);
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CACHE_FULL);
        return;
    }
    float on = 0.f, ol = 0.f;
    const int sg = tid < D ? tid / ds : 0;            // this column's softmax head
    if (tid < D) {
        const volatile float *pv = partials;
        constexpr int kPs = D + kPartHead;
        float M = -INFINITY;
        for (int pt = 0; pt < kDecodeParts; ++pt) M = fmaxf(M, pv[pt * kPs + sg]);
        float sc_self = 0.f;
        if (r) {                                       // the token attends to itself
            if (kGrouped)
                for (int x = sg * ds; x < (sg + 1) * ds; ++x) sc_self = fmaf(qsm[x] * scale_sm, ksm[x], sc_self);
            else
                for (int x = 0; x < D; ++x) sc_self = fmaf(qs[x] * scale_sm, ks[x], sc_self);
            M = fmaxf(M, sc_self);
        }
        float Z = 0.f;
        if (M > -INFINITY) {
            for (int pt = 0; pt < kDecodeParts; ++pt) {
                const float mp = pv[pt * kPs + sg];
                if (mp > -INFINITY) {
                    const float f = __expf(mp - M);
                    Z = fmaf(pv[pt * kPs + 4 + sg], f, Z);
                    on = fmaf(pv[pt * kPs + kPartHead + tid], f, on);
                }
            }
            if (r) {
                const float f = __expf(sc_self - M);
                Z += f;
                on = fmaf(vs[tid], f, on);
            }
            on /= Z;
        }
        ol = reinterpret_cast<const volatile float *>(ola_ws)[tid];
    }
    float ssn = warp_sum(on * on), ssl = warp_sum(ol * ol);
    if (lane == 0 && warp < kWarps) { norm_red[0][warp] = ssn; norm_red[1][warp] = ssl; }
    __syncthreads();
    if (tid < D) {
        float tn = 0.f, tl = 0.f;      // softmax output: over this column's softmax head; linear read-out: over the row
#pragma unroll
        for (int wv = 0; wv < kWarps; ++wv) {
            if (!kGrouped || (32 * wv) / ds == sg) tn += norm_red[0][wv];
            tl += norm_red[1][wv];
        }
        const float fn = rsqrtf(tn / ds + eps), fl = rsqrtf(tl / D + eps);
        const float wn = w ? w[(size_t)bh * 2] : 0.5f, wl = w ? w[(size_t)bh * 2 + 1] : 0.5f;
        out[(size_t)bh * D + tid] = from_f32<T>(wn * on * fn + wl * ol * fl);
        if (r) {   // retain the token: every reader of the old length has finished
            k_cache[((size_t)bh * cap + n_old) * D + tid] = k[(size_t)bh * D + tid];
            v_cache[((size_t)bh * cap + n_old) * D + tid] = v[(size_t)bh * D + tid];
        }
    }
    if (r && tid == 0) cache_len[bh] = n_old + 1;
}

// End of a block of R tokens decoded with the decision open: a softmax block resets the state to
// its value at the block's start times the block's decay (the block's K/V stay in the cache); a
// linear block keeps the state and drops its R cache entries.  state_start then holds the new
// state: the start of the next block.  One CTA per (sequence, head).
__global__ void __launch_bounds__(256)
decode_block_end_kernel(const uint8_t *__restrict__ route_block, const float *__restrict__ g_block,
                        float *__restrict__ state, float *__restrict__ state_start,
                        int32_t *__restrict__ cache_len, int R, int n4, int32_t *status) {
    const int bh = blockIdx.x;
    float4 *S = reinterpret_cast<float4 *>(state) + (size_t)bh * n4;
    float4 *S0 = reinterpret_cast<float4 *>(state_start) + (size_t)bh * n4;
    if (route_block[bh]) {
        const float decay = expf(g_block[bh]);
        for (int i = threadIdx.x; i < n4; i += blockDim.x) {
            float4 a = S0[i];
            a.x *= decay; a.y *= decay; a.z *= decay; a.w *= decay;
            S[i] = a;
            S0[i] = a;
        }
    } else {
        for (int i = threadIdx.x; i < n4; i += blockDim.x) S0[i] = S[i];
        if (threadIdx.x == 0) {
            const int n = cache_len[bh];
            if (n < R) atomicMin(status, (int)NATSL_ERR_ROUTE);   // the block's entries are not there
            else cache_len[bh] = n - R;
        }
    }
}

}  // namespace

cudaError_t launch_decode_block_end(const uint8_t *route_block, const float *g_block, float *state,
                                    float *state_start, int32_t *cache_len, int32_t block_len,
                                    void *ws, Shape s, cudaStream_t st) {
    decode_block_end_kernel<<<s.B * s.H, 256, 0, st>>>(route_block, g_block, state, state_start,
                                                       cache_len, block_len, s.d * s.d / 4,
                                                       reinterpret_cast<int32_t *>(ws));
    count_launch();
    return cudaGetLastError();
}

size_t decode_workspace_bytes(int B, int H, int d) {
    return dec_off_ola((size_t)B * H, d) + ((size_t)B * H * d * 4 + 255) / 256 * 256;
}

template <typename T, int D>
static cudaError_t decode_impl(const void *q, const void *k, const void *v, const float *g,
                               const float *beta, const uint8_t *route, const float *w,
                               float *state, void *k_cache, void *v_cache, int32_t *cache_len,
                               int32_t cap, void *out, float scale_la, float scale_sm, float eps,
                               void *ws, Shape s, cudaStream_t st, HeadGroups hg) {
    constexpr int kTileBytes = kTileKeys * D * (int)sizeof(T);
    constexpr int kRing = 2 * kStages * kTileBytes;
    constexpr int kRed = 32 * D * 4;               // per-stream / per-slot reduction scratch
    constexpr int kSmem = kRing > kRed ? kRing : kRed;
    const bool grouped = hg.G > 1 || hg.norm_eps >= 0.f;
    if (grouped && (hg.G > 4 || D % (32 * hg.G) != 0)) return cudaErrorInvalidValue;
    auto kernel = grouped ? decode_step_kernel<T, D, true> : decode_step_kernel<T, D, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    dim3 grid(kCtasPerHead, s.B * s.H);
    kernel<<<grid, kThreads, kSmem, st>>>(
        (const T *)q, (const T *)k, (const T *)v, g, beta, route, w, state, (T *)k_cache,
        (T *)v_cache, cache_len, cap, (T *)out, scale_la, scale_sm, eps, (uint8_t *)ws, s.B * s.H, hg.G,
        hg.norm_eps);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_decode_step(const void *q, const void *k, const void *v, const float *g,
                               const float *beta, const uint8_t *route, const float *w,
                               float *state, void *k_cache, void *v_cache, int32_t *cache_len,
                               int32_t cache_cap, void *out, float scale_la, float scale_sm,
                               float eps, void *ws, Shape s, cudaStream_t st, HeadGroups hg) {
#define ARGS q, k, v, g, beta, route, w, state, k_cache, v_cache, cache_len, cache_cap, out, \
             scale_la, scale_sm, eps, ws, s, st, hg
    if (s.bf16) {
        if (s.d == 128) return decode_impl<__nv_bfloat16, 128>(ARGS);
        return decode_impl<__nv_bfloat16, 64>(ARGS);
    }
    if (s.d == 128) return decode_impl<float, 128>(ARGS);
    return decode_impl<float, 64>(ARGS);
#undef ARGS
}

}  // namespace natsl

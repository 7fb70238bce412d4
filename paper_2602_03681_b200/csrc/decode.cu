// Decode step (Section 4.1, per-token generation): one CTA per (batch, head) streams the fp32
// d x d state once (decay, rank-1 gated delta update, read-out, write back) and the retained
// K/V cache once (online softmax), then RMS-normalises and combines both branch outputs
// (Section 4.3, Norm equation).  HBM-bound: every global access is a 16-byte vector, whole
// rows per warp instruction, with several independent loads in flight per thread.
#include "common.cuh"
#include "natsl_internal.h"

namespace natsl {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

template <typename T> struct Vec16;   // 16 bytes of T as fp32 values
template <> struct Vec16<float> {
    static constexpr int kN = 4;
    __device__ static void load(const float *p, float (&x)[4]) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kN = 8;
    __device__ static void load(const __nv_bfloat16 *p, float (&x)[8]) {
        const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
decode_step_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                   const float *__restrict__ g, const float *__restrict__ beta,
                   const uint8_t *__restrict__ route, const float *__restrict__ w,
                   float *__restrict__ state, T *__restrict__ k_cache, T *__restrict__ v_cache,
                   int32_t *__restrict__ cache_len, int cap, T *__restrict__ out, float scale_la,
                   float scale_sm, float eps, int32_t *status) {
    // state tiling: a lane owns 4 consecutive value columns; a warp instruction covers kRpl rows
    constexpr int kLpr = D / 4;                 // lanes per state row
    constexpr int kRpl = 32 / kLpr;             // rows per warp-wide load
    constexpr int kSlots = kWarps * kRpl;       // row slots in the CTA
    constexpr int kR = D / kSlots;              // rows per thread
    // cache tiling: 16-byte pieces, kLpk lanes per key row, kStreams independent softmax streams
    constexpr int kE = Vec16<T>::kN;
    constexpr int kLpk = D / kE;
    constexpr int kStreams = kThreads / kLpk;
    constexpr int kUnroll = 4;

    __shared__ float qs[D], ks[D], vs[D];
    __shared__ float red[kSlots][D];
    __shared__ float o_la_s[D], o_nla_s[D];
    __shared__ float sm_m[kStreams], sm_z[kStreams];
    __shared__ float sm_acc[kStreams][D];
    __shared__ float norm_red[2][kWarps];

    const int bh = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = route[bh] != 0;
    const int n_old = cache_len[bh];
    if (r && n_old >= cap) {   // no room: leave the sequence untouched, report
        if (tid < D) out[(size_t)bh * D + tid] = from_f32<T>(0.f);
        if (tid == 0) atomicMin(status, (int)NATSL_ERR_CACHE_FULL);
        return;
    }
    if (tid < D) {
        qs[tid] = to_f32(q[(size_t)bh * D + tid]);
        ks[tid] = to_f32(k[(size_t)bh * D + tid]);
        vs[tid] = to_f32(v[(size_t)bh * D + tid]);
    }
    const float alpha = __expf(g[bh]);
    const float bt = r ? 0.f : beta[bh];

    // ---------------- linear branch: state in registers ----------------
    const int slot = warp * kRpl + lane / kLpr;
    const int col = (lane % kLpr) * 4;
    float *sp = state + (size_t)bh * D * D;
    float4 s[kR];
#pragma unroll
    for (int rr = 0; rr < kR; ++rr)
        s[rr] = *reinterpret_cast<const float4 *>(sp + (size_t)(slot * kR + rr) * D + col);
    __syncthreads();   // qs/ks/vs visible
#pragma unroll
    for (int rr = 0; rr < kR; ++rr) {
        s[rr].x *= alpha; s[rr].y *= alpha; s[rr].z *= alpha; s[rr].w *= alpha;
    }
    if (!r) {   // block-uniform
        float4 p = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int rr = 0; rr < kR; ++rr) {
            const float ka = ks[slot * kR + rr];
            p.x = fmaf(ka, s[rr].x, p.x); p.y = fmaf(ka, s[rr].y, p.y);
            p.z = fmaf(ka, s[rr].z, p.z); p.w = fmaf(ka, s[rr].w, p.w);
        }
        *reinterpret_cast<float4 *>(&red[slot][col]) = p;
        __syncthreads();
        float4 e = *reinterpret_cast<const float4 *>(&vs[col]);
#pragma unroll
        for (int sl = 0; sl < kSlots; ++sl) {
            const float4 t = *reinterpret_cast<const float4 *>(&red[sl][col]);
            e.x -= t.x; e.y -= t.y; e.z -= t.z; e.w -= t.w;
        }
#pragma unroll
        for (int rr = 0; rr < kR; ++rr) {
            const float bk = bt * ks[slot * kR + rr];
            s[rr].x = fmaf(bk, e.x, s[rr].x); s[rr].y = fmaf(bk, e.y, s[rr].y);
            s[rr].z = fmaf(bk, e.z, s[rr].z); s[rr].w = fmaf(bk, e.w, s[rr].w);
        }
        __syncthreads();   // red is reused below
    }
    {
        float4 p = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int rr = 0; rr < kR; ++rr) {
            const float qa = qs[slot * kR + rr];
            p.x = fmaf(qa, s[rr].x, p.x); p.y = fmaf(qa, s[rr].y, p.y);
            p.z = fmaf(qa, s[rr].z, p.z); p.w = fmaf(qa, s[rr].w, p.w);
            *reinterpret_cast<float4 *>(sp + (size_t)(slot * kR + rr) * D + col) = s[rr];
        }
        *reinterpret_cast<float4 *>(&red[slot][col]) = p;
    }
    __syncthreads();
    if (tid < D) {
        float acc = 0.f;
#pragma unroll
        for (int sl = 0; sl < kSlots; ++sl) acc += red[sl][tid];
        o_la_s[tid] = scale_la * acc;
    }

    // ---------------- softmax branch: stream the retained K/V once ----------------
    if (r) {   // append the new token's K/V (the token attends to itself from shared memory)
        if (tid < D) {
            k_cache[((size_t)bh * cap + n_old) * D + tid] = k[(size_t)bh * D + tid];
            v_cache[((size_t)bh * cap + n_old) * D + tid] = v[(size_t)bh * D + tid];
        }
        if (tid == 0) cache_len[bh] = n_old + 1;
    }
    const int stream = tid / kLpk, piece = tid % kLpk;
    const T *kc = k_cache + (size_t)bh * cap * D + piece * kE;
    const T *vc = v_cache + (size_t)bh * cap * D + piece * kE;
    float qf[kE];
#pragma unroll
    for (int x = 0; x < kE; ++x) qf[x] = qs[piece * kE + x] * scale_sm;
    float m = -INFINITY, z = 0.f, acc[kE];
#pragma unroll
    for (int x = 0; x < kE; ++x) acc[x] = 0.f;

    // Trip count and shuffles are uniform over the CTA; only the state updates are predicated.
    for (int base = 0; base < n_old; base += kStreams * kUnroll) {
        float kx[kUnroll][kE], vx[kUnroll][kE];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int j = base + u * kStreams + stream;
            if (j < n_old) {
                Vec16<T>::load(kc + (size_t)j * D, kx[u]);
                Vec16<T>::load(vc + (size_t)j * D, vx[u]);
            } else {
#pragma unroll
                for (int x = 0; x < kE; ++x) { kx[u][x] = 0.f; vx[u][x] = 0.f; }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int j = base + u * kStreams + stream;
            float sc = 0.f;
#pragma unroll
            for (int x = 0; x < kE; ++x) sc = fmaf(qf[x], kx[u][x], sc);
#pragma unroll
            for (int o = kLpk / 2; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
            if (j < n_old) {
                const float m_new = fmaxf(m, sc);
                const float corr = __expf(m - m_new), pj = __expf(sc - m_new);
                z = fmaf(z, corr, pj);
                m = m_new;
#pragma unroll
                for (int x = 0; x < kE; ++x) acc[x] = fmaf(acc[x], corr, pj * vx[u][x]);
            }
        }
    }
    if (r && warp == 0) {   // the token itself, from shared memory; stream 0 takes it
        float sc = 0.f;
#pragma unroll
        for (int x = 0; x < kE; ++x) sc = fmaf(qf[x], ks[piece * kE + x], sc);
#pragma unroll
        for (int o = kLpk / 2; o > 0; o >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, o);
        if (stream == 0) {
            const float m_new = fmaxf(m, sc);
            const float corr = __expf(m - m_new), pj = __expf(sc - m_new);
            z = fmaf(z, corr, pj);
            m = m_new;
#pragma unroll
            for (int x = 0; x < kE; ++x) acc[x] = fmaf(acc[x], corr, pj * vs[piece * kE + x]);
        }
    }
    if (piece == 0) { sm_m[stream] = m; sm_z[stream] = z; }
#pragma unroll
    for (int x = 0; x < kE; ++x) sm_acc[stream][piece * kE + x] = acc[x];
    __syncthreads();
    if (tid < D) {
        float M = -INFINITY;
        for (int st = 0; st < kStreams; ++st) M = fmaxf(M, sm_m[st]);
        float Z = 0.f, o = 0.f;
        if (M > -INFINITY) {
            for (int st = 0; st < kStreams; ++st) {
                const float f = __expf(sm_m[st] - M);
                Z = fmaf(sm_z[st], f, Z);
                o = fmaf(sm_acc[st][tid], f, o);
            }
            o /= Z;
        }
        o_nla_s[tid] = o;
    }
    __syncthreads();
    // ---------------- combination ----------------
    float ssn = 0.f, ssl = 0.f;
    if (tid < D) { ssn = o_nla_s[tid] * o_nla_s[tid]; ssl = o_la_s[tid] * o_la_s[tid]; }
    ssn = warp_sum(ssn);
    ssl = warp_sum(ssl);
    if (lane == 0) { norm_red[0][warp] = ssn; norm_red[1][warp] = ssl; }
    __syncthreads();
    if (tid < D) {
        float tn = 0.f, tl = 0.f;
#pragma unroll
        for (int wv = 0; wv < kWarps; ++wv) { tn += norm_red[0][wv]; tl += norm_red[1][wv]; }
        const float fn = rsqrtf(tn / D + eps), fl = rsqrtf(tl / D + eps);
        const float wn = w ? w[(size_t)bh * 2] : 0.5f, wl = w ? w[(size_t)bh * 2 + 1] : 0.5f;
        out[(size_t)bh * D + tid] = from_f32<T>(wn * o_nla_s[tid] * fn + wl * o_la_s[tid] * fl);
    }
}

}  // namespace

template <typename T, int D>
static cudaError_t decode_impl(const void *q, const void *k, const void *v, const float *g,
                               const float *beta, const uint8_t *route, const float *w,
                               float *state, void *k_cache, void *v_cache, int32_t *cache_len,
                               int32_t cap, void *out, float scale_la, float scale_sm, float eps,
                               int32_t *status, Shape s, cudaStream_t st) {
    decode_step_kernel<T, D><<<s.B * s.H, kThreads, 0, st>>>(
        (const T *)q, (const T *)k, (const T *)v, g, beta, route, w, state, (T *)k_cache,
        (T *)v_cache, cache_len, cap, (T *)out, scale_la, scale_sm, eps, status);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_decode_step(const void *q, const void *k, const void *v, const float *g,
                               const float *beta, const uint8_t *route, const float *w,
                               float *state, void *k_cache, void *v_cache, int32_t *cache_len,
                               int32_t cache_cap, void *out, float scale_la, float scale_sm,
                               float eps, int32_t *status, Shape s, cudaStream_t st) {
#define ARGS q, k, v, g, beta, route, w, state, k_cache, v_cache, cache_len, cache_cap, out, \
             scale_la, scale_sm, eps, status, s, st
    if (s.bf16) {
        if (s.d == 128) return decode_impl<__nv_bfloat16, 128>(ARGS);
        return decode_impl<__nv_bfloat16, 64>(ARGS);
    }
    if (s.d == 128) return decode_impl<float, 128>(ARGS);
    return decode_impl<float, 64>(ARGS);
#undef ARGS
}

}  // namespace natsl

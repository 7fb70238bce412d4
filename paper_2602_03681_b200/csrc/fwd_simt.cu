// fp32 CUDA-core forward of the hybrid layer: the chunkwise Gated DeltaNet branch (prepare +
// scan), and the softmax branch over the retained tokens with the RMS-norm / weighted
// combination fused into its epilogue.  This is the exact-precision path (fp32 storage needs
// ~1e-6 relative error, which rules out bf16/tf32 tensor-core operands); it also accepts bf16
// storage and then serves as the in-library cross-check of the tensor-core kernels.
//
// Chunkwise form (Section 3, chunkwise equations, specialised to the gated delta rule of
// Section 4.3), per chunk of C = 64 tokens, beta~ = (1 - route) beta, G_i = inclusive
// cumulative log decay inside the chunk, gamma_i = exp(G_i), Gamma_ij = exp(G_i - G_j):
//   A_ij = beta~_i Gamma_ij (k_i.k_j) (j<i);  (I + A) W = diag(beta~ gamma) K;  (I + A) U = diag(beta~) V
//   P_ij = scale_la (q_i.k_j) Gamma_ij (j<=i)
//   U~ = U - W S;   O = scale_la diag(gamma) Q S + P U~;   S <- gamma_C S + (diag(gamma_C/gamma) K)^T U~
#include "common.cuh"
#include "natsl_internal.h"

namespace natsl {

namespace {

constexpr int kThreads = 256;

// Load a 64 x D tile (token stride `ts` elements) into padded fp32 shared memory [64][D+1].
template <typename T, int D>
__device__ __forceinline__ void load_tile(const T *__restrict__ src, size_t ts, float *dst) {
    for (int idx = threadIdx.x; idx < kC * D / 4; idx += kThreads) {
        const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
        const float4 x = load4(src + (size_t)r * ts + c4);
        float *p = dst + r * (D + 1) + c4;
        p[0] = x.x; p[1] = x.y; p[2] = x.z; p[3] = x.w;
    }
}

// ------------------------------------------------------------------------------------------
// Prepare: state-independent per-chunk quantities.  grid = (L/C, B*H).
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
gdn_prepare_simt_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                        const float *__restrict__ g, const float *__restrict__ beta,
                        const uint8_t *__restrict__ route, float scale_la, float *__restrict__ W,
                        float *__restrict__ U, float *__restrict__ P, float *__restrict__ Abar,
                        float *__restrict__ Gcum, int L, int H) {
    extern __shared__ float smem[];
    float *Ks = smem;                       // [64][D+1]
    float *Vs = Ks + kC * (D + 1);          // [64][D+1]  (V, later Q)
    float *As = Vs + kC * (D + 1);          // [64][64]
    float *Gs = As + kC * kC;               // [64] inclusive cumulative log decay
    float *bts = Gs + kC;                   // [64] beta~

    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const size_t ts = (size_t)H * D;
    const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;  // index of the chunk's first token

    load_tile<T, D>(k + tok0 * D, ts, Ks);
    load_tile<T, D>(v + tok0 * D, ts, Vs);
    if (threadIdx.x < kC) {
        const size_t t = tok0 + (size_t)threadIdx.x * H;
        bts[threadIdx.x] = route && route[t] ? 0.f : beta[t];   // route == nullptr: beta~ = beta
        Gs[threadIdx.x] = g[t];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int i = 0; i < kC; ++i) { acc += Gs[i]; Gs[i] = acc; }
    }
    __syncthreads();
    if (Gcum && threadIdx.x < kC) Gcum[(size_t)bh * L + c * kC + threadIdx.x] = Gs[threadIdx.x];
    // A (strictly lower); Abar = A without the beta~ row factor (the backward needs it)
    {
        const int i = threadIdx.x >> 2;
        float *Ab = Abar ? Abar + ((size_t)bh * (L / kC) + c) * kC * kC : nullptr;
        for (int m = 0; m < 16; ++m) {
            const int j = (threadIdx.x & 3) + 4 * m;
            float a = 0.f;
            if (j < i && (bts[i] != 0.f || Ab)) {
                float dot = 0.f;
                const float *ki = Ks + i * (D + 1), *kj = Ks + j * (D + 1);
#pragma unroll 8
                for (int x = 0; x < D; ++x) dot = fmaf(ki[x], kj[x], dot);
                a = __expf(Gs[i] - Gs[j]) * dot;
            }
            if (Ab) Ab[i * kC + j] = a;
            As[i * kC + j] = bts[i] * a;
        }
    }
    __syncthreads();
    // Forward substitution, one right-hand-side column per thread: columns [0,D) give W, [D,2D) U.
    if (threadIdx.x < 2 * D) {
        const bool isW = threadIdx.x < D;
        const int col = isW ? threadIdx.x : threadIdx.x - D;
        const float *src = isW ? Ks : Vs;
        float x[kC];
#pragma unroll
        for (int i = 0; i < kC; ++i) {
            float acc = bts[i] * (isW ? __expf(Gs[i]) : 1.f) * src[i * (D + 1) + col];
#pragma unroll
            for (int j = 0; j < i; ++j) acc = fmaf(-As[i * kC + j], x[j], acc);
            x[i] = acc;
        }
        float *dst = (isW ? W : U) + tok0 * D + col;
#pragma unroll
        for (int i = 0; i < kC; ++i) dst[(size_t)i * ts] = x[i];
    }
    __syncthreads();
    // P = scale_la (Q K^T) . Gamma, lower triangle including the diagonal
    load_tile<T, D>(q + tok0 * D, ts, Vs);
    __syncthreads();
    {
        const int i = threadIdx.x >> 2;
        float *Pc = P + ((size_t)bh * (L / kC) + c) * kC * kC;
        for (int m = 0; m < 16; ++m) {
            const int j = (threadIdx.x & 3) + 4 * m;
            float a = 0.f;
            if (j <= i) {
                float dot = 0.f;
                const float *qi = Vs + i * (D + 1), *kj = Ks + j * (D + 1);
#pragma unroll 8
                for (int x = 0; x < D; ++x) dot = fmaf(qi[x], kj[x], dot);
                a = scale_la * __expf(Gs[i] - Gs[j]) * dot;
            }
            Pc[i * kC + j] = a;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Scan: sequential over chunks, one CTA per (batch, head, slice of 32 value columns).
// grid = (D/32, B*H).
// ------------------------------------------------------------------------------------------
constexpr int kDvs = 32;

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
gdn_scan_simt_kernel(const T *__restrict__ q, const T *__restrict__ k, const float *__restrict__ g,
                     const float *__restrict__ W, const float *__restrict__ U,
                     const float *__restrict__ P, float scale_la, const float *__restrict__ state_in,
                     float *__restrict__ state_out, float *__restrict__ chunk_states,
                     float *__restrict__ Ut, float *__restrict__ o_la,
                     const uint8_t *__restrict__ block_route, int L, int H) {
    extern __shared__ float smem[];
    float *Ss = smem;                        // [D][32]
    float *Ws = Ss + D * kDvs;               // [64][D+1]
    float *Qs = Ws + kC * (D + 1);           // [64][D+1]
    float *Ks = Qs + kC * (D + 1);           // [64][D+1]
    float *Ps = Ks + kC * (D + 1);           // [64][65]
    float *Us = Ps + kC * (kC + 1);          // [64][33]
    float *Gs = Us + kC * (kDvs + 1);        // [64]

    const int slice = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const size_t ts = (size_t)H * D;
    const int c0 = slice * kDvs;

    for (int idx = threadIdx.x; idx < D * kDvs; idx += kThreads) {
        const int a = idx / kDvs, cc = idx % kDvs;
        Ss[idx] = state_in ? state_in[((size_t)bh * D + a) * D + c0 + cc] : 0.f;
    }

    for (int c = 0; c < NC; ++c) {
        const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
        __syncthreads();
        if (chunk_states) {  // state at chunk entry, [B,H,NC,D,D]
            for (int idx = threadIdx.x; idx < D * kDvs; idx += kThreads) {
                const int a = idx / kDvs, cc = idx % kDvs;
                chunk_states[(((size_t)bh * NC + c) * D + a) * D + c0 + cc] = Ss[idx];
            }
        }
        load_tile<float, D>(W + tok0 * D, ts, Ws);
        load_tile<T, D>(q + tok0 * D, ts, Qs);
        load_tile<T, D>(k + tok0 * D, ts, Ks);
        {
            const float *Pc = P + ((size_t)bh * NC + c) * kC * kC;
            for (int idx = threadIdx.x; idx < kC * kC; idx += kThreads)
                Ps[(idx >> 6) * (kC + 1) + (idx & 63)] = Pc[idx];
            for (int idx = threadIdx.x; idx < kC * kDvs; idx += kThreads) {
                const int r = idx / kDvs, cc = idx % kDvs;
                Us[r * (kDvs + 1) + cc] = U[(tok0 + (size_t)r * H) * D + c0 + cc];
            }
            if (threadIdx.x < kC) Gs[threadIdx.x] = g[tok0 + (size_t)threadIdx.x * H];
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float acc = 0.f;
            for (int i = 0; i < kC; ++i) { acc += Gs[i]; Gs[i] = acc; }
        }
        __syncthreads();
        const int r = threadIdx.x >> 2, cb = (threadIdx.x & 3) * 8;
        // U~ = U - W S
        {
            float acc[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] = Us[r * (kDvs + 1) + cb + x];
            const float *wr = Ws + r * (D + 1);
            for (int a = 0; a < D; ++a) {
                const float wv = wr[a];
                const float *sr = Ss + a * kDvs + cb;
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[x] = fmaf(-wv, sr[x], acc[x]);
            }
            __syncthreads();
#pragma unroll
            for (int x = 0; x < 8; ++x) Us[r * (kDvs + 1) + cb + x] = acc[x];
            if (Ut) {
                float *dst = Ut + (tok0 + (size_t)r * H) * D + c0 + cb;
                store4(dst, make_float4(acc[0], acc[1], acc[2], acc[3]));
                store4(dst + 4, make_float4(acc[4], acc[5], acc[6], acc[7]));
            }
        }
        __syncthreads();
        // O = scale_la gamma_r q_r S + sum_{j<=r} P_rj U~_j
        {
            float acc[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] = 0.f;
            const float *qr = Qs + r * (D + 1);
            for (int a = 0; a < D; ++a) {
                const float qv = qr[a];
                const float *sr = Ss + a * kDvs + cb;
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[x] = fmaf(qv, sr[x], acc[x]);
            }
            const float gs = scale_la * __expf(Gs[r]);
#pragma unroll
            for (int x = 0; x < 8; ++x) acc[x] *= gs;
            const float *pr = Ps + r * (kC + 1);
            for (int j = 0; j <= r; ++j) {
                const float pv = pr[j];
                const float *ur = Us + j * (kDvs + 1) + cb;
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[x] = fmaf(pv, ur[x], acc[x]);
            }
            float *dst = o_la + (tok0 + (size_t)r * H) * D + c0 + cb;
            store4(dst, make_float4(acc[0], acc[1], acc[2], acc[3]));
            store4(dst + 4, make_float4(acc[4], acc[5], acc[6], acc[7]));
        }
        __syncthreads();
        // S <- gamma_C S + (diag(gamma_C / gamma) K)^T U~
        {
            constexpr int kPer = D / 8;            // outputs per thread
            constexpr int kTpr = kDvs / kPer;      // threads per state row
            const int a = threadIdx.x / kTpr, cs = (threadIdx.x % kTpr) * kPer;
            const float gl = Gs[kC - 1];
            const float gC = __expf(gl);
            float acc[kPer];
#pragma unroll
            for (int x = 0; x < kPer; ++x) acc[x] = gC * Ss[a * kDvs + cs + x];
            // block-level routing: a softmax block's update is not committed, the state only decays
            const bool commit = !(block_route && block_route[tok0]);
            for (int j = 0; commit && j < kC; ++j) {
                const float kv = Ks[j * (D + 1) + a] * __expf(gl - Gs[j]);
                const float *ur = Us + j * (kDvs + 1) + cs;
#pragma unroll
                for (int x = 0; x < kPer; ++x) acc[x] = fmaf(kv, ur[x], acc[x]);
            }
#pragma unroll
            for (int x = 0; x < kPer; ++x) Ss[a * kDvs + cs + x] = acc[x];
        }
    }
    __syncthreads();
    if (state_out) {
        for (int idx = threadIdx.x; idx < D * kDvs; idx += kThreads) {
            const int a = idx / kDvs, cc = idx % kDvs;
            state_out[((size_t)bh * D + a) * D + c0 + cc] = Ss[idx];
        }
    }
}

// ------------------------------------------------------------------------------------------
// Softmax branch over the retained tokens (Section 4.1, O_nla with mask M^nla) with the
// combination (Section 4.3, Norm equation) as epilogue.  grid = (L/64, B*H*G); each warp owns
// 8 query rows, each lane one key of the current 32-key tile.
// G softmax heads per linear head (Section 4.3, grouped heads): softmax head (h, sg) works on the
// columns [sg D, (sg+1) D) of q, k, v rows of DL = G D columns; lists, weights and the linear read-out
// are those of linear head h; the softmax output is normalised over its D columns, the linear
// read-out over all DL, and the CTA writes its D columns of `out`.  lse is [B,H,G,L].
// ------------------------------------------------------------------------------------------
template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads)
softmax_combine_simt_kernel(const T *__restrict__ q, const T *__restrict__ k_sm,
                            const T *__restrict__ v_sm, int cap, const int32_t *__restrict__ sm_idx,
                            const int32_t *__restrict__ sm_chunk_prefix,
                            const float *__restrict__ o_la, const float *__restrict__ w,
                            float scale_sm, float eps, T *__restrict__ out,
                            float *__restrict__ o_nla, float *__restrict__ lse,
                            const uint8_t *__restrict__ block_route, const T *__restrict__ k_tok,
                            const T *__restrict__ v_tok, int L, int H) {
    extern __shared__ float smem[];
    float *Qs = smem;                      // [64][D]
    float *Kt = Qs + kC * D;               // [32][D+1]
    float *Vt = Kt + 32 * (D + 1);         // [32][D]
    int *pos = reinterpret_cast<int *>(Vt + 32 * D);  // [32]

    constexpr int DL = D * G;
    const int c = blockIdx.x, bhg = blockIdx.y, bh = bhg / G, sg = bhg % G, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t ts = (size_t)H * DL;
    const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
    const int n_end = min(sm_chunk_prefix[(size_t)bh * (NC + 1) + c + 1], cap);
    const int col0 = sg * D;                             // first column of this softmax head

    for (int idx = threadIdx.x; idx < kC * D / 4; idx += kThreads) {
        const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
        store4(Qs + r * D + c4, load4(q + tok0 * DL + (size_t)r * ts + col0 + c4));
    }
    constexpr int kQ = 8, kCols = D / 32;
    float m[kQ], z[kQ], acc[kQ][kCols];
#pragma unroll
    for (int r = 0; r < kQ; ++r) {
        m[r] = -INFINITY; z[r] = 0.f;
#pragma unroll
        for (int x = 0; x < kCols; ++x) acc[r][x] = 0.f;
    }
    const T *kb = k_sm + (size_t)bh * cap * DL + col0, *vb = v_sm + (size_t)bh * cap * DL + col0;

    // Block-level routing: a query in a linear block also reads the causal part of its own block
    // (two more tiles of 32 keys, taken from the layer's own k and v).
    const int n_ret = (n_end + 31) / 32 * 32;
    const int n_all = n_ret + (block_route && block_route[tok0] == 0 ? kC : 0);
    for (int j0 = 0; j0 < n_all; j0 += 32) {
        const bool own = j0 >= n_ret;
        __syncthreads();
        for (int idx = threadIdx.x; idx < 32 * D / 4; idx += kThreads) {
            const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
            float4 kx = make_float4(0.f, 0.f, 0.f, 0.f), vx = kx;
            if (own) {
                const size_t src = (tok0 + (size_t)(j0 - n_ret + r) * H) * DL + col0 + c4;
                kx = load4(k_tok + src);
                vx = load4(v_tok + src);
            } else if (j0 + r < n_end) {
                kx = load4(kb + (size_t)(j0 + r) * DL + c4);
                vx = load4(vb + (size_t)(j0 + r) * DL + c4);
            }
            float *kp = Kt + r * (D + 1) + c4;
            kp[0] = kx.x; kp[1] = kx.y; kp[2] = kx.z; kp[3] = kx.w;
            store4(Vt + r * D + c4, vx);
        }
        if (threadIdx.x < 32)
            pos[threadIdx.x] = own ? c * kC + (j0 - n_ret) + (int)threadIdx.x
                               : (j0 + threadIdx.x < n_end) ? sm_idx[(size_t)bh * L + j0 + threadIdx.x]
                                                            : 0x7fffffff;
        __syncthreads();
        const int my_pos = pos[lane];
        const float *kr = Kt + lane * (D + 1);
#pragma unroll
        for (int r = 0; r < kQ; ++r) {
            const int i = c * kC + warp * kQ + r;
            const float *qr = Qs + (warp * kQ + r) * D;
            float s = 0.f;
#pragma unroll 8
            for (int x = 0; x < D; ++x) s = fmaf(qr[x], kr[x], s);
            const bool valid = my_pos <= i;
            s = valid ? s * scale_sm : -INFINITY;
            const float m_new = fmaxf(m[r], warp_max(s));
            if (m_new == -INFINITY) continue;          // warp-uniform
            const float pj = valid ? __expf(s - m_new) : 0.f;
            const float corr = __expf(m[r] - m_new);   // exp(-inf) = 0 on the first tile
            z[r] = z[r] * corr + warp_sum(pj);
            m[r] = m_new;
#pragma unroll
            for (int x = 0; x < kCols; ++x) acc[r][x] *= corr;
            for (int j = 0; j < 32; ++j) {
                const float pb = __shfl_sync(0xffffffffu, pj, j);
#pragma unroll
                for (int x = 0; x < kCols; ++x) acc[r][x] = fmaf(pb, Vt[j * D + lane + 32 * x], acc[r][x]);
            }
        }
    }
    // epilogue: normalise both branches and combine
#pragma unroll
    for (int r = 0; r < kQ; ++r) {
        const int i = c * kC + warp * kQ + r;
        const size_t t = tok0 + (size_t)(warp * kQ + r) * H;
        const float inv = z[r] > 0.f ? 1.f / z[r] : 0.f;
        float on[kCols], ol[kCols], ssn = 0.f, ssl = 0.f;
#pragma unroll
        for (int x = 0; x < kCols; ++x) {
            on[x] = acc[r][x] * inv;
            ol[x] = o_la[t * DL + col0 + lane + 32 * x];
            ssn = fmaf(on[x], on[x], ssn);
            ssl = fmaf(ol[x], ol[x], ssl);
        }
        if (G > 1)        // the linear read-out is normalised over its whole row
            for (int x = 0; x < DL / 32; ++x) {
                if ((32 * x) / D == sg) continue;
                const float y = o_la[t * DL + lane + 32 * x];
                ssl = fmaf(y, y, ssl);
            }
        ssn = warp_sum(ssn);
        ssl = warp_sum(ssl);
        const float fn = rsqrtf(ssn / D + eps), fl = rsqrtf(ssl / DL + eps);
        const float wn = w ? w[t * 2] : 0.5f, wl = w ? w[t * 2 + 1] : 0.5f;
#pragma unroll
        for (int x = 0; x < kCols; ++x) {
            if (out) out[t * DL + col0 + lane + 32 * x] = from_f32<T>(wn * on[x] * fn + wl * ol[x] * fl);
            if (o_nla) o_nla[t * DL + col0 + lane + 32 * x] = on[x];
        }
        if (lse && lane == 0) lse[(size_t)bhg * L + i] = z[r] > 0.f ? m[r] + __logf(z[r]) : -INFINITY;
    }
}

// Per-operation normalisation of q and k for fp32 storage (Section 4.3): one warp per row of d
// columns writes the L2-normalised row (linear operation) and the row with each of its G slices
// RMS-normalised (softmax operation).  The tensor-core path does both inside its kernels instead.
// (qk_norm_f32_kernel, below the vector helpers.)

// Backward of that normalisation, in place on fp32 gradients, one warp per row.  On entry dq holds the
// gradient with respect to the L2-normalised q (linear operation) and dq_sm the one with respect to the
// slice-wise RMS-normalised q (softmax operation); dk holds, for a linear token, the gradient with
// respect to the L2-normalised k and, for a retained token, the one with respect to the RMS-normalised k
// (a token's k reaches only the operation the token was routed to).  x^ = x r, r = (sum x^2 + e)^-1/2:
// dx = r (g - x^ <x^, g>);  x~ = x r, r = (mean x^2 + e)^-1/2 over a slice of ds columns:
// dx = r (g - x~ <x~, g> / ds).
// (One warp per row; a lane owns D / 32 neighbouring columns, moved as one vector.  A slice is an aligned
// group of 32 / G lanes, so one xor butterfly yields a slice's sum on the way to the row's.)
template <int N> __device__ __forceinline__ void load_vec(const float *p, float (&x)[N]) {
    if (N == 4) { const float4 v = *reinterpret_cast<const float4 *>(p); x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
    else { const float2 v = *reinterpret_cast<const float2 *>(p); x[0] = v.x; x[1] = v.y; }
}
template <int N> __device__ __forceinline__ void load_vec(const __nv_bfloat16 *p, float (&x)[N]) {
    if (N == 4) {
        const uint2 v = *reinterpret_cast<const uint2 *>(p);
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    } else {
        const uint32_t v = *reinterpret_cast<const uint32_t *>(p);
        x[0] = __uint_as_float(v << 16); x[1] = __uint_as_float(v & 0xffff0000u);
    }
}
template <int N> __device__ __forceinline__ void store_vec(float *p, const float (&x)[N]) {
    if (N == 4) *reinterpret_cast<float4 *>(p) = make_float4(x[0], x[1], x[2], x[3]);
    else *reinterpret_cast<float2 *>(p) = make_float2(x[0], x[1]);
}
template <int N> __device__ __forceinline__ void store_vec(__nv_bfloat16 *p, const float (&x)[N]) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(x[0], x[1]);
    if (N == 4) {
        __nv_bfloat162 hi = __floats2bfloat162_rn(x[2], x[3]);
        *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
    } else {
        *reinterpret_cast<uint32_t *>(p) = *reinterpret_cast<uint32_t *>(&lo);
    }
}

// The forward normalisation with the same layout (d = 64 or 128, a slice an aligned group of 32 / G lanes).
template <typename T, int D>
__global__ void __launch_bounds__(256)
qk_norm_f32_kernel(const T *__restrict__ q, const T *__restrict__ k, float *__restrict__ q_la,
                       float *__restrict__ k_la, float *__restrict__ q_sm, float *__restrict__ k_sm,
                       size_t rows, int G, float norm_eps) {
    constexpr int N = D / 32;
    const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const int lps = 32 / G;
    const float inv_ds = (float)G / D;
    const size_t at = row * D + (size_t)lane * N;
    float x[2][N];
    load_vec<N>(q + at, x[0]);
    load_vec<N>(k + at, x[1]);
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        float ss = 0.f, ss_s = 0.f;
#pragma unroll
        for (int j = 0; j < N; ++j) ss = fmaf(x[which][j], x[which][j], ss);
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            if (o == lps) ss_s = ss;
            ss += __shfl_xor_sync(0xffffffffu, ss, o);
        }
        if (lps == 32) ss_s = ss;
        const float rl = rsqrtf(ss + norm_eps), rs = rsqrtf(fmaf(ss_s, inv_ds, norm_eps));
        float y[N];
#pragma unroll
        for (int j = 0; j < N; ++j) y[j] = x[which][j] * rl;
        store_vec<N>((which ? k_la : q_la) + at, y);
        if (q_sm) {
#pragma unroll
            for (int j = 0; j < N; ++j) y[j] = x[which][j] * rs;
            store_vec<N>((which ? k_sm : q_sm) + at, y);
        }
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(256)
qk_norm_bwd_f32_kernel(const T *__restrict__ q, const T *__restrict__ k,
                       const uint8_t *__restrict__ route, const float *dq_la,
                       const float *__restrict__ dq_sm, const float *dk_in, const float *dv_in,
                       T *dq, T *dk, T *dv, size_t rows, int G, float norm_eps,
                       const float *__restrict__ dk_sm) {
    constexpr int N = D / 32;
    const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    const int lps = 32 / G;                                  // lanes per slice
    const float inv_ds = (float)G / D;
    const bool retained = route[row] != 0;
    const size_t at = row * D + (size_t)lane * N;
    if (dv_in) {
        float t[N];
        load_vec<N>(dv_in + at, t);
        store_vec<N>(dv + at, t);
    }
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        const float *sm_in = which == 0 ? dq_sm : dk_sm;   // separate softmax-operation gradient, if any
        const bool l2_part = sm_in || !retained, rms_part = sm_in || retained;
        float x[N], g[N], gs[N], out[N];
        load_vec<N>((which ? k : q) + at, x);
        load_vec<N>((which ? dk_in : dq_la) + at, g);
        if (sm_in) load_vec<N>(sm_in + at, gs);
        float ss = 0.f, xg = 0.f, xs = 0.f;
#pragma unroll
        for (int j = 0; j < N; ++j) {
            if (!sm_in) gs[j] = g[j];
            ss = fmaf(x[j], x[j], ss);
            xg = fmaf(x[j], g[j], xg);
            xs = fmaf(x[j], gs[j], xs);
        }
        float ss_s = 0.f, xs_s = 0.f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            if (o == lps) { ss_s = ss; xs_s = xs; }
            ss += __shfl_xor_sync(0xffffffffu, ss, o);
            xg += __shfl_xor_sync(0xffffffffu, xg, o);
            xs += __shfl_xor_sync(0xffffffffu, xs, o);
        }
        if (lps == 32) { ss_s = ss; xs_s = xs; }
        const float rl = rsqrtf(ss + norm_eps), dot = rl * xg;
        const float rs = rsqrtf(fmaf(ss_s, inv_ds, norm_eps)), m = rs * xs_s * inv_ds;
#pragma unroll
        for (int j = 0; j < N; ++j) {
            out[j] = l2_part ? rl * (g[j] - x[j] * rl * dot) : 0.f;
            if (rms_part) out[j] += rs * (gs[j] - x[j] * rs * m);
        }
        store_vec<N>((which ? dk : dq) + at, out);
    }
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

size_t simt_prepare_smem(int d) { return sizeof(float) * (2 * kC * (d + 1) + kC * kC + 2 * kC); }
size_t simt_scan_smem(int d) {
    return sizeof(float) * (d * kDvs + 3 * kC * (d + 1) + kC * (kC + 1) + kC * (kDvs + 1) + kC);
}
static size_t simt_softmax_smem(int d) { return sizeof(float) * (kC * d + 32 * (d + 1) + 32 * d + 32); }

#define NATSL_DISPATCH(FN, ...)                                                   \
    do {                                                                          \
        if (s.bf16) {                                                             \
            if (s.d == 128) return FN<__nv_bfloat16, 128>(__VA_ARGS__);           \
            return FN<__nv_bfloat16, 64>(__VA_ARGS__);                            \
        }                                                                         \
        if (s.d == 128) return FN<float, 128>(__VA_ARGS__);                       \
        return FN<float, 64>(__VA_ARGS__);                                        \
    } while (0)

template <typename T, int D>
static cudaError_t prepare_impl(const void *q, const void *k, const void *v, const float *g,
                                const float *beta, const uint8_t *route, float scale_la, float *W,
                                float *U, float *P, float *Abar, float *Gcum, Shape s,
                                cudaStream_t st) {
    const size_t smem = simt_prepare_smem(D);
    cudaError_t e = set_smem(gdn_prepare_simt_kernel<T, D>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(s.L / kC, s.B * s.H);
    gdn_prepare_simt_kernel<T, D><<<grid, kThreads, smem, st>>>(
        (const T *)q, (const T *)k, (const T *)v, g, beta, route, scale_la, W, U, P, Abar, Gcum, s.L,
        s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_prepare_simt(const void *q, const void *k, const void *v, const float *g,
                                    const float *beta, const uint8_t *route, float scale_la,
                                    float *W, float *U, float *P, float *Abar, float *Gcum, Shape s,
                                    cudaStream_t st) {
    NATSL_DISPATCH(prepare_impl, q, k, v, g, beta, route, scale_la, W, U, P, Abar, Gcum, s, st);
}

template <typename T, int D>
static cudaError_t scan_impl(const void *q, const void *k, const float *g, const float *W,
                             const float *U, const float *P, float scale_la, const float *state_in,
                             float *state_out, float *chunk_states, float *Ut, float *o_la,
                             const uint8_t *block_route, Shape s, cudaStream_t st) {
    const size_t smem = simt_scan_smem(D);
    cudaError_t e = set_smem(gdn_scan_simt_kernel<T, D>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(D / kDvs, s.B * s.H);
    gdn_scan_simt_kernel<T, D><<<grid, kThreads, smem, st>>>(
        (const T *)q, (const T *)k, g, W, U, P, scale_la, state_in, state_out, chunk_states, Ut,
        o_la, block_route, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_scan_simt(const void *q, const void *k, const float *g, const float *W,
                                 const float *U, const float *P, float scale_la,
                                 const float *state_in, float *state_out, float *chunk_states,
                                 float *Ut, float *o_la, const uint8_t *block_route, Shape s,
                                 cudaStream_t st) {
    NATSL_DISPATCH(scan_impl, q, k, g, W, U, P, scale_la, state_in, state_out, chunk_states, Ut, o_la,
                   block_route, s, st);
}

template <typename T, int D, int G = 1>
static cudaError_t softmax_impl(const void *q, const void *k_sm, const void *v_sm, int32_t cap,
                                const int32_t *sm_idx, const int32_t *pre, const float *o_la,
                                const float *w, float scale_sm, float eps, void *out, float *o_nla,
                                float *lse, BlockRouting br, Shape s, cudaStream_t st) {
    const size_t smem = simt_softmax_smem(D);
    cudaError_t e = set_smem(softmax_combine_simt_kernel<T, D, G>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(s.L / kC, s.B * s.H * G);
    softmax_combine_simt_kernel<T, D, G><<<grid, kThreads, smem, st>>>(
        (const T *)q, (const T *)k_sm, (const T *)v_sm, cap, sm_idx, pre, o_la, w, scale_sm, eps,
        (T *)out, o_nla, lse, br.route, (const T *)br.k, (const T *)br.v, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_softmax_combine_simt(const void *q, const void *k_sm, const void *v_sm,
                                        int32_t cap, const int32_t *sm_idx,
                                        const int32_t *sm_chunk_prefix, const float *o_la,
                                        const float *w, float scale_sm, float eps, void *out,
                                        float *o_nla, float *lse, BlockRouting br, Shape s,
                                        cudaStream_t st, int G) {
    if (G > 1) {      // grouped softmax heads: fp32 storage, d / G in {32, 64}
        if (s.bf16) return cudaErrorInvalidValue;
#define NATSL_GROUPED(DS, GG)                                                                           \
        if (s.d == DS * GG && G == GG)                                                                  \
            return softmax_impl<float, DS, GG>(q, k_sm, v_sm, cap, sm_idx, sm_chunk_prefix, o_la, w,    \
                                               scale_sm, eps, out, o_nla, lse, br, s, st)
        NATSL_GROUPED(32, 2);
        NATSL_GROUPED(64, 2);
        NATSL_GROUPED(32, 4);
#undef NATSL_GROUPED
        return cudaErrorInvalidValue;
    }
    NATSL_DISPATCH(softmax_impl, q, k_sm, v_sm, cap, sm_idx, sm_chunk_prefix, o_la, w, scale_sm, eps,
                   out, o_nla, lse, br, s, st);
}

cudaError_t launch_qk_norm_f32(const void *q, const void *k, bool bf16, float *q_la, float *k_la, float *q_sm,
                               float *k_sm, size_t rows, int d, int G, float norm_eps, cudaStream_t st) {
    const unsigned blocks = (unsigned)((rows + 7) / 8);
    if ((d != 64 && d != 128) || G < 1 || 32 % G != 0 || !q_sm != !k_sm) return cudaErrorInvalidValue;
#define NATSL_NF(TT, DD)                                                                                  \
    qk_norm_f32_kernel<TT, DD><<<blocks, 256, 0, st>>>((const TT *)q, (const TT *)k, q_la, k_la, q_sm, k_sm, \
                                                      rows, G, norm_eps)
    if (bf16) { if (d == 128) NATSL_NF(__nv_bfloat16, 128); else NATSL_NF(__nv_bfloat16, 64); }
    else { if (d == 128) NATSL_NF(float, 128); else NATSL_NF(float, 64); }
#undef NATSL_NF
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_qk_norm_bwd_f32(const void *q, const void *k, bool bf16, const uint8_t *route,
                                   const float *dq_la, const float *dq_sm, const float *dk_in,
                                   const float *dv_in, void *dq, void *dk, void *dv, size_t rows, int d, int G,
                                   float norm_eps, cudaStream_t st, const float *dk_sm) {
    const unsigned blocks = (unsigned)((rows + 7) / 8);
    if ((d != 64 && d != 128) || G < 1 || 32 % G != 0) return cudaErrorInvalidValue;
#define NATSL_NB(TT, DD)                                                                                      \
    qk_norm_bwd_f32_kernel<TT, DD><<<blocks, 256, 0, st>>>((const TT *)q, (const TT *)k, route, dq_la, dq_sm,  \
                                                          dk_in, dv_in, (TT *)dq, (TT *)dk, (TT *)dv, rows, G, \
                                                          norm_eps, dk_sm)
    if (bf16) { if (d == 128) NATSL_NB(__nv_bfloat16, 128); else NATSL_NB(__nv_bfloat16, 64); }
    else { if (d == 128) NATSL_NB(float, 128); else NATSL_NB(float, 64); }
#undef NATSL_NB
    count_launch();
    return cudaGetLastError();
}

}  // namespace natsl

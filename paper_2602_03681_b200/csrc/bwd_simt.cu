// fp32 CUDA-core backward of the hybrid layer.
//
// The paper states the properties the backward must have (Section 4.2: the softmax logit
// gradient is P (dP - <do, o>); k, v gradients of an operation vanish for tokens inactive for
// it) but gives no backward of the gated delta rule.  This file differentiates the chunkwise
// forward of fwd_simt.cu.  Per chunk, with entry state S0, exit-state gradient dS1, output
// gradient dO and the forward quantities W, U, P, U~ (same notation as fwd_simt.cu):
//
//   dU~ = P^T dO + K~ dS1                       K~ = diag(gamma_C / gamma) K
//   dS0 = Qg^T dO + gamma_C dS1 - W^T dU~       Qg = scale_la diag(gamma) Q      (reverse scan)
//   dQg = dO S0^T     dW = -dU~ S0^T     dK~ = U~ dS1^T     N = lower(dO U~^T)
//   [dKb | dVb] = (I + A)^-T [dW | dU~]         Kb = diag(beta~ gamma) K, Vb = diag(beta~) V
//   M  = -strict_lower(dKb W^T + dVb U^T)       (gradient w.r.t. A)
//   dq = scale_la gamma dQg + (N . scale_la Gamma) K
//   dk = beta~ gamma dKb + (gamma_C/gamma) dK~ + (M . beta~ Gamma) K + (M . beta~ Gamma)^T K
//        + (N . scale_la Gamma)^T Q
//   dv = beta~ dVb
//   every gamma / Gamma factor contributes to dG_i (G = in-chunk cumulative log decay), and
//   dg_j = sum_{i >= j} dG_i;  dbeta = (1 - route) dbeta~.
//
// The dense products run through one generic batched tile-GEMM kernel over (batch, head,
// chunk); the sequential part is the reverse scan.  Softmax-branch gradients are formed over
// the compacted K/V list only and scattered back to the retained tokens.
#include <cuda_fp16.h>

#include "common.cuh"
#include "natsl_internal.h"

namespace natsl {

namespace {

constexpr int kThreads = 256;

// ------------------------------------------------------------------------------------------
// generic batched GEMM: C = alpha * op(A) op(B) (+ C), 64x64 output tiles, fp32.
// fp32 storage (1e-4 tolerance): fp32 FMAs (bgemm_kernel).  bf16 storage, whose tolerance it fits:
// the warp-level tensor-core path with tf32 operands (fp32 range, 11 significant bits) and fp32
// accumulation (bgemm_tf32_kernel, below) -- warp w owns rows 16 (w & 3) .. and columns 32 (w >> 2) ..
// of the tile, four m16n8k8 products per 8 values of k.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void mma_tf32_16x8x8(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ void store2(float *p, float a, float b) { *reinterpret_cast<float2 *>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16 *p, float a, float b) {
    *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(a, b);
}
__device__ __forceinline__ const float *mat_base(const BMat &m, int b, int h, int ch) {
    return m.p + (size_t)b * m.sb + (size_t)h * m.sh + (size_t)ch * m.sc;
}

template <bool TA, bool TB, int MASK>
__global__ void __launch_bounds__(kThreads)
bgemm_kernel(BMat A, BMat B, BMat Cm, int K, float alpha, int accumulate, int H, int NC) {
    constexpr int kLd = 68;
    __shared__ __align__(16) float As[16][kLd];
    __shared__ __align__(16) float Bs[16][kLd];
    const int z = blockIdx.z, ch = z % NC, bh = z / NC, b = bh / H, h = bh % H;
    const float *Ap = mat_base(A, b, h, ch), *Bp = mat_base(B, b, h, ch);
    float *Cp = const_cast<float *>(mat_base(Cm, b, h, ch));
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
    float acc[4][4];          // rows ty*4 + i, columns tx*4 + j
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < K; k0 += 16) {
        if (!TA) {   // A[m][k], k contiguous
            const int r = t >> 2, kk = (t & 3) * 4;
            const float4 x = *reinterpret_cast<const float4 *>(Ap + (size_t)(m0 + r) * A.ld + k0 + kk);
            As[kk][r] = x.x; As[kk + 1][r] = x.y; As[kk + 2][r] = x.z; As[kk + 3][r] = x.w;
        } else {     // A[k][m], m contiguous
            const int kk = t >> 4, r4 = (t & 15) * 4;
            *reinterpret_cast<float4 *>(&As[kk][r4]) =
                *reinterpret_cast<const float4 *>(Ap + (size_t)(k0 + kk) * A.ld + m0 + r4);
        }
        if (!TB) {   // B[k][n], n contiguous
            const int kk = t >> 4, c4 = (t & 15) * 4;
            *reinterpret_cast<float4 *>(&Bs[kk][c4]) =
                *reinterpret_cast<const float4 *>(Bp + (size_t)(k0 + kk) * B.ld + n0 + c4);
        } else {     // B[n][k], k contiguous
            const int c = t >> 2, kk = (t & 3) * 4;
            const float4 x = *reinterpret_cast<const float4 *>(Bp + (size_t)(n0 + c) * B.ld + k0 + kk);
            Bs[kk][c] = x.x; Bs[kk + 1][c] = x.y; Bs[kk + 2][c] = x.z; Bs[kk + 3][c] = x.w;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            const float4 a = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
            const float4 bb = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = m0 + ty * 4 + i;
        float *cr = Cp + (size_t)row * Cm.ld + n0 + tx * 4;
        float o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = n0 + tx * 4 + j;
            float val = alpha * acc[i][j];
            if (MASK == 1 && col > row) val = 0.f;
            if (MASK == 2 && col >= row) val = 0.f;
            o[j] = val;
        }
        if (accumulate) {
            const float4 old = *reinterpret_cast<const float4 *>(cr);
            o[0] += old.x; o[1] += old.y; o[2] += old.z; o[3] += old.w;
        }
        *reinterpret_cast<float4 *>(cr) = make_float4(o[0], o[1], o[2], o[3]);
    }
}

// The tf32 case as a pipeline: operands go to shared memory in the layout they have in global memory
// (16-byte asynchronous copies, three 32-wide steps of k in flight) and the fragment reads adapt to the
// layout instead -- rows of 36 floats for a k-contiguous operand, of 72 for an m- or n-contiguous one,
// both free of bank conflicts for the m16n8k8 fragments.  Operands are rounded to tf32 as they are
// read, products accumulated in fp32; k is a multiple of 32 (64 or the head dimension).
constexpr int kBgK = 32, kBgStages = 3;
constexpr int kBgTileFloats = 64 * (kBgK + 4);           // = kBgK * 72: either layout
constexpr size_t kBgSmem = (size_t)kBgStages * 2 * kBgTileFloats * sizeof(float);
__device__ __forceinline__ void cp_async16(float *dst, const float *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(
                     static_cast<uint32_t>(__cvta_generic_to_shared(dst))),
                 "l"(reinterpret_cast<uint64_t>(src))
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <bool TA, bool TB, int MASK>
__global__ void __launch_bounds__(kThreads)
bgemm_tf32_kernel(BMat A, BMat B, BMat Cm, int K, float alpha, int accumulate, int H, int NC) {
    extern __shared__ __align__(16) float bg_smem[];
    constexpr int kLdK = kBgK + 4, kLdMN = 72;
    const int z = blockIdx.z, ch = z % NC, bh = z / NC, b = bh / H, h = bh % H;
    const float *Ap = mat_base(A, b, h, ch), *Bp = mat_base(B, b, h, ch);
    float *Cp = const_cast<float *>(mat_base(Cm, b, h, ch));
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31, fg = lane >> 2, ft = lane & 3;
    const int wr = (warp & 3) * 16, wc = (warp >> 2) * 32;
    const int nk = K / kBgK;
    auto issue = [&](int kt) {
        if (kt < nk) {
            float *As = bg_smem + (size_t)(kt % kBgStages) * 2 * kBgTileFloats, *Bs = As + kBgTileFloats;
            const int k0 = kt * kBgK;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int f = t + kThreads * i;
                if (!TA) {   // A[m][k], k contiguous
                    const int r = f / (kBgK / 4), kq = (f % (kBgK / 4)) * 4;
                    cp_async16(As + r * kLdK + kq, Ap + (size_t)(m0 + r) * A.ld + k0 + kq);
                } else {     // A[k][m], m contiguous
                    const int kk = f / 16, r4 = (f % 16) * 4;
                    cp_async16(As + kk * kLdMN + r4, Ap + (size_t)(k0 + kk) * A.ld + m0 + r4);
                }
                if (TB) {    // B[n][k], k contiguous
                    const int c = f / (kBgK / 4), kq = (f % (kBgK / 4)) * 4;
                    cp_async16(Bs + c * kLdK + kq, Bp + (size_t)(n0 + c) * B.ld + k0 + kq);
                } else {     // B[k][n], n contiguous
                    const int kk = f / 16, c4 = (f % 16) * 4;
                    cp_async16(Bs + kk * kLdMN + c4, Bp + (size_t)(k0 + kk) * B.ld + n0 + c4);
                }
            }
        }
        cp_async_commit();       // (an empty group past the end keeps the count uniform)
    };
    float acc[4][4];             // n-tile i, fragment element j
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll
    for (int kt = 0; kt < kBgStages - 1; ++kt) issue(kt);
    for (int kt = 0; kt < nk; ++kt) {
        cp_async_wait<kBgStages - 2>();          // step kt has landed (this thread's copies) ...
        __syncthreads();                         // ... and everyone's; step kt - 1 has been read by all
        issue(kt + kBgStages - 1);               // into the slot of step kt - 1
        const float *As = bg_smem + (size_t)(kt % kBgStages) * 2 * kBgTileFloats, *Bs = As + kBgTileFloats;
        auto a_at = [&](int m, int k) { return to_tf32(TA ? As[k * kLdMN + m] : As[m * kLdK + k]); };
        auto b_at = [&](int k, int n) { return to_tf32(TB ? Bs[n * kLdK + k] : Bs[k * kLdMN + n]); };
#pragma unroll
        for (int k8 = 0; k8 < kBgK; k8 += 8) {
            const uint32_t a[4] = {a_at(wr + fg, k8 + ft), a_at(wr + fg + 8, k8 + ft),
                                   a_at(wr + fg, k8 + ft + 4), a_at(wr + fg + 8, k8 + ft + 4)};
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const uint32_t bfr[2] = {b_at(k8 + ft, wc + 8 * nt + fg), b_at(k8 + ft + 4, wc + 8 * nt + fg)};
                mma_tf32_16x8x8(acc[nt], a, bfr);
            }
        }
    }
    cp_async_wait<0>();
    // fragment layout: elements (0, 1) in row fg, (2, 3) in row fg + 8; columns 2 ft, 2 ft + 1
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = m0 + wr + fg + 8 * hh, col = n0 + wc + 8 * nt + 2 * ft;
            float o0 = alpha * acc[nt][2 * hh], o1 = alpha * acc[nt][2 * hh + 1];
            if (MASK == 1) { if (col > row) o0 = 0.f; if (col + 1 > row) o1 = 0.f; }
            if (MASK == 2) { if (col >= row) o0 = 0.f; if (col + 1 >= row) o1 = 0.f; }
            float2 *cr = reinterpret_cast<float2 *>(Cp + (size_t)row * Cm.ld + col);
            if (accumulate) { const float2 old = *cr; o0 += old.x; o1 += old.y; }
            *cr = make_float2(o0, o1);
        }
}

// ------------------------------------------------------------------------------------------
// storage type -> fp32 copies of q, k, v
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void to_f32_kernel(const T *__restrict__ a, const T *__restrict__ b, const T *__restrict__ c,
                              float *__restrict__ a32, float *__restrict__ b32,
                              float *__restrict__ c32, size_t n4) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4;
         i += (size_t)gridDim.x * blockDim.x) {
        if (a) store4(a32 + 4 * i, load4(a + 4 * i));      // (a, b: optional)
        if (b) store4(b32 + 4 * i, load4(b + 4 * i));
        store4(c32 + 4 * i, load4(c + 4 * i));
    }
}

// ------------------------------------------------------------------------------------------
// combination backward (row-local): do_la, do_nla, dw, Dsm = <do_nla, o_nla>
// ------------------------------------------------------------------------------------------
// max |dout| over the whole tensor, as the bit pattern of a non-negative float (ordered like an
// integer), into the status page; the word is zeroed by the caller beforehand.
template <typename T>
__global__ void __launch_bounds__(256)
dout_amax_kernel(const T *__restrict__ dout, size_t n4, int32_t *status) {
    float m = 0.f;
    const size_t stride = (size_t)gridDim.x * 256;
    size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {          // four loads in flight per thread
        float4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = load4(dout + 4 * (i + u * stride));
#pragma unroll
        for (int u = 0; u < 4; ++u)
            m = fmaxf(fmaxf(m, fmaxf(fabsf(x[u].x), fabsf(x[u].y))), fmaxf(fabsf(x[u].z), fabsf(x[u].w)));
    }
    for (; i < n4; i += stride) {
        const float4 x = load4(dout + 4 * i);
        m = fmaxf(fmaxf(m, fmaxf(fabsf(x.x), fabsf(x.y))), fmaxf(fabsf(x.z), fabsf(x.w)));
    }
    m = warp_max(m);
    if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(status + kGradAmaxWord, __float_as_int(m));
}

// Four neighbouring columns per lane (one vector per array and lane), D / 4 lanes per row, so a warp takes
// two rows at D = 64: the kernel sits at the head of the backward's dependency chain and is bound by how
// many bytes a warp has in flight.
// G > 1 (grouped softmax heads, Section 4.3): the softmax branch's output is normalised per slice of
// D / G columns, so its part of the backward (do_nla, dw_nla, D_i = <do_i, o_i>) is formed per slice;
// Dsm is then [B,H,G,L].  A slice is an aligned group of D / (4 G) lanes: one xor butterfly gives the
// slice's sum on its way to the row's.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
combine_bwd_kernel(const float *__restrict__ o_la, const float *__restrict__ o_nla,
                   const T *__restrict__ dout, const float *__restrict__ w, float eps,
                   float *__restrict__ do_la, float *__restrict__ do_nla, float *__restrict__ dw,
                   float *__restrict__ Dsm, __half *__restrict__ do16,
                   __half *__restrict__ dola16, __half *__restrict__ dolag16,
                   const float *__restrict__ Gd, float scale_la, const int32_t *gsc, int G, int B, int L, int H) {
    constexpr int kLpr = D / 4, kRpw = 32 / kLpr;           // lanes per row, rows per warp
    const float gs = grad_scale(gsc).x;      // scale of the fp16 operand copies (and of Dsm with them)
    const int lane = threadIdx.x & 31, sub = lane / kLpr, li = lane % kLpr;
    const int lps = kLpr / G;                               // lanes per slice
    const float inv_ds = (float)G / D;
    const size_t row = ((size_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5)) * kRpw + sub;
    const bool live = row < (size_t)B * L * H;              // (all lanes stay for the shuffles)
    const size_t rr = live ? row : 0;
    const int h = rr % H;
    const size_t bl = rr / H;
    const int l = bl % L, b = bl / L;
    const size_t at = rr * D + li * 4;
    const float4 a = *reinterpret_cast<const float4 *>(o_la + at), n = *reinterpret_cast<const float4 *>(o_nla + at);
    float dy[4];
    if (sizeof(T) == 2) {
        const uint2 u = *reinterpret_cast<const uint2 *>(dout + at);
        dy[0] = __uint_as_float(u.x << 16); dy[1] = __uint_as_float(u.x & 0xffff0000u);
        dy[2] = __uint_as_float(u.y << 16); dy[3] = __uint_as_float(u.y & 0xffff0000u);
    } else {
        const float4 u = *reinterpret_cast<const float4 *>(dout + at);
        dy[0] = u.x; dy[1] = u.y; dy[2] = u.z; dy[3] = u.w;
    }
    const float ol[4] = {a.x, a.y, a.z, a.w}, on[4] = {n.x, n.y, n.z, n.w};
    // returns the row's sum; slice = the sum over the lane's slice
    auto sums = [&](float v, float &slice) {
#pragma unroll
        for (int o = 1; o < kLpr; o <<= 1) {
            if (o == lps) slice = v;
            v += __shfl_xor_sync(0xffffffffu, v, o);
        }
        if (lps == kLpr) slice = v;
        return v;
    };
    float ssl = 0.f, ssn = 0.f, ssn_s, unused;
#pragma unroll
    for (int x = 0; x < 4; ++x) { ssl = fmaf(ol[x], ol[x], ssl); ssn = fmaf(on[x], on[x], ssn); }
    ssl = sums(ssl, unused);
    sums(ssn, ssn_s);
    const float fl = rsqrtf(ssl / D + eps), fn = rsqrtf(ssn_s * inv_ds + eps);   // fn: of the lane's slice
    const float wn = w ? w[rr * 2] : 0.5f, wl = w ? w[rr * 2 + 1] : 0.5f;
    // scale_la gamma_l of the token (decay from its chunk's entry), for the reverse scan's operand
    const float sg = dolag16 ? scale_la * Gd[((size_t)(b * H + h) * (L / kC) + l / kC) * 128 + l % kC] : 0.f;
    float dwl = 0.f, dwn = 0.f, dwn_s;
#pragma unroll
    for (int x = 0; x < 4; ++x) { dwl = fmaf(dy[x], ol[x] * fl, dwl); dwn = fmaf(dy[x], on[x] * fn, dwn); }
    dwl = sums(dwl, unused);
    dwn = sums(dwn, dwn_s);                  // <dy, y_nla> over the row and over the slice
    const float ml = wl * dwl / D, mn = wn * dwn_s * inv_ds;
    float dl[4], dn[4], dsm = 0.f, dsm_s;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        dl[x] = fl * (wl * dy[x] - ol[x] * fl * ml);
        dn[x] = fn * (wn * dy[x] - on[x] * fn * mn);
        dsm = fmaf(dn[x], on[x], dsm);
    }
    sums(dsm, dsm_s);
    if (!live) return;
    *reinterpret_cast<float4 *>(do_la + at) = make_float4(dl[0], dl[1], dl[2], dl[3]);
    // (the tensor-core softmax backward reads the fp16 copy only)
    if (do_nla) *reinterpret_cast<float4 *>(do_nla + at) = make_float4(dn[0], dn[1], dn[2], dn[3]);
    const size_t at16 = (((size_t)b * H + h) * L + l) * D + li * 4;
    auto h4 = [](float x0, float x1, float x2, float x3) {
        const __half2 p = __floats2half2_rn(x0, x1), q2 = __floats2half2_rn(x2, x3);
        return make_uint2(*reinterpret_cast<const uint32_t *>(&p), *reinterpret_cast<const uint32_t *>(&q2));
    };
    if (do16) *reinterpret_cast<uint2 *>(do16 + at16) = h4(gs * dn[0], gs * dn[1], gs * dn[2], gs * dn[3]);
    if (dolag16) {
        *reinterpret_cast<uint2 *>(dola16 + at16) = h4(gs * dl[0], gs * dl[1], gs * dl[2], gs * dl[3]);
        const float gg = gs * sg;
        *reinterpret_cast<uint2 *>(dolag16 + at16) = h4(gg * dl[0], gg * dl[1], gg * dl[2], gg * dl[3]);
    }
    if (li % lps == 0) Dsm[(((size_t)b * H + h) * G + li / lps) * L + l] = gs * dsm_s;
    if (li == 0 && dw) { dw[rr * 2] = dwn; dw[rr * 2 + 1] = dwl; }
}

// ------------------------------------------------------------------------------------------
// softmax backward, query side: dq_sm.  grid = (L/64, B*H), same tiling as the forward.
// ------------------------------------------------------------------------------------------
// G softmax heads per linear head (Section 4.3): the kernel's head is a slice of D columns of rows of
// DL = G D columns; lse and Dsm are [B,H,G,L].
template <int D, int G>
__global__ void __launch_bounds__(kThreads)
softmax_bwd_dq_kernel(const float *__restrict__ q32, const float *__restrict__ k_sm32,
                      const float *__restrict__ v_sm32, int cap, const int32_t *__restrict__ sm_idx,
                      const int32_t *__restrict__ sm_chunk_prefix,
                      const float *__restrict__ do_nla, const float *__restrict__ lse,
                      const float *__restrict__ Dsm, float scale_sm, float *__restrict__ dq_sm,
                      int L, int H) {
    extern __shared__ float smem[];
    float *Qs = smem;                      // [64][D]
    float *dOs = Qs + kC * D;              // [64][D]
    float *Kt = dOs + kC * D;              // [32][D+1]
    float *Vt = Kt + 32 * (D + 1);         // [32][D+1]
    int *pos = reinterpret_cast<int *>(Vt + 32 * (D + 1));

    constexpr int DL = D * G;
    const int c = blockIdx.x, bhg = blockIdx.y, bh = bhg / G, col0 = (bhg % G) * D, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t ts = (size_t)H * DL;
    const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
    const int n_end = min(sm_chunk_prefix[(size_t)bh * (NC + 1) + c + 1], cap);

    for (int idx = threadIdx.x; idx < kC * D / 4; idx += kThreads) {
        const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
        store4(Qs + r * D + c4, load4(q32 + tok0 * DL + (size_t)r * ts + col0 + c4));
        store4(dOs + r * D + c4, load4(do_nla + tok0 * DL + (size_t)r * ts + col0 + c4));
    }
    constexpr int kQ = 8, kCols = D / 32;
    float acc[kQ][kCols], lse_r[kQ], dsm_r[kQ];
#pragma unroll
    for (int r = 0; r < kQ; ++r) {
        const int i = c * kC + warp * kQ + r;
        lse_r[r] = lse[(size_t)bhg * L + i];
        dsm_r[r] = Dsm[(size_t)bhg * L + i];
#pragma unroll
        for (int x = 0; x < kCols; ++x) acc[r][x] = 0.f;
    }
    const float *kb = k_sm32 + (size_t)bh * cap * DL + col0, *vb = v_sm32 + (size_t)bh * cap * DL + col0;
    for (int j0 = 0; j0 < n_end; j0 += 32) {
        __syncthreads();
        for (int idx = threadIdx.x; idx < 32 * D / 4; idx += kThreads) {
            const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
            float4 kx = make_float4(0.f, 0.f, 0.f, 0.f), vx = kx;
            if (j0 + r < n_end) {
                kx = load4(kb + (size_t)(j0 + r) * DL + c4);
                vx = load4(vb + (size_t)(j0 + r) * DL + c4);
            }
            float *kp = Kt + r * (D + 1) + c4, *vp = Vt + r * (D + 1) + c4;
            kp[0] = kx.x; kp[1] = kx.y; kp[2] = kx.z; kp[3] = kx.w;
            vp[0] = vx.x; vp[1] = vx.y; vp[2] = vx.z; vp[3] = vx.w;
        }
        if (threadIdx.x < 32)
            pos[threadIdx.x] = (j0 + threadIdx.x < n_end) ? sm_idx[(size_t)bh * L + j0 + threadIdx.x]
                                                          : 0x7fffffff;
        __syncthreads();
        const int my_pos = pos[lane];
        const float *kr = Kt + lane * (D + 1), *vr = Vt + lane * (D + 1);
#pragma unroll
        for (int r = 0; r < kQ; ++r) {
            const int i = c * kC + warp * kQ + r;
            const float *qr = Qs + (warp * kQ + r) * D, *dor = dOs + (warp * kQ + r) * D;
            float s = 0.f, dp = 0.f;
#pragma unroll 8
            for (int x = 0; x < D; ++x) {
                s = fmaf(qr[x], kr[x], s);
                dp = fmaf(dor[x], vr[x], dp);
            }
            const float pj = (my_pos <= i) ? __expf(s * scale_sm - lse_r[r]) : 0.f;
            const float ds = pj * (dp - dsm_r[r]);
            for (int j = 0; j < 32; ++j) {
                const float db = __shfl_sync(0xffffffffu, ds, j);
#pragma unroll
                for (int x = 0; x < kCols; ++x)
                    acc[r][x] = fmaf(db, Kt[j * (D + 1) + lane + 32 * x], acc[r][x]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kQ; ++r) {
        const size_t t = tok0 + (size_t)(warp * kQ + r) * H;
#pragma unroll
        for (int x = 0; x < kCols; ++x) dq_sm[t * DL + col0 + lane + 32 * x] = scale_sm * acc[r][x];
    }
}

// ------------------------------------------------------------------------------------------
// softmax backward, key side: dk_sm, dv_sm per compacted key.  grid = (ceil(cap/32), B*H).
// ------------------------------------------------------------------------------------------
template <int D, int G>
__global__ void __launch_bounds__(kThreads)
softmax_bwd_dkv_kernel(const float *__restrict__ q32, const float *__restrict__ k_sm32,
                       const float *__restrict__ v_sm32, int cap, const int32_t *__restrict__ sm_idx,
                       const int32_t *__restrict__ sm_chunk_prefix,
                       const float *__restrict__ do_nla, const float *__restrict__ lse,
                       const float *__restrict__ Dsm, float scale_sm, float *__restrict__ dk_sm,
                       float *__restrict__ dv_sm, float *__restrict__ dmask, int L, int H) {
    // dmask [B,H,cap] (or nullptr): per retained key j the sum over its queries of
    // dM_ij = p_ij (dp_ij - <do_i, o_i>), the mask gradient of Section 4.2
    extern __shared__ float smem[];
    float *Kt = smem;                       // [32][D+1]
    float *Vt = Kt + 32 * (D + 1);          // [32][D+1]
    float *Qs = Vt + 32 * (D + 1);          // [64][D]
    float *dOs = Qs + kC * D;               // [64][D]
    float *Ps = dOs + kC * D;               // [64][33]
    float *Dss = Ps + kC * 33;              // [64][33]
    float *lse_s = Dss + kC * 33;           // [64]
    float *dsm_s = lse_s + kC;              // [64]
    int *pos = reinterpret_cast<int *>(dsm_s + kC);

    constexpr int DL = D * G;
    const int bhg = blockIdx.y, bh = bhg / G, col0 = (bhg % G) * D, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int n_sm = min(sm_chunk_prefix[(size_t)bh * (NC + 1) + NC], cap);
    const int j0 = blockIdx.x * 32;
    if (j0 >= n_sm) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t ts = (size_t)H * DL;
    const float *kb = k_sm32 + (size_t)bh * cap * DL + col0, *vb = v_sm32 + (size_t)bh * cap * DL + col0;

    for (int idx = threadIdx.x; idx < 32 * D / 4; idx += kThreads) {
        const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
        float4 kx = make_float4(0.f, 0.f, 0.f, 0.f), vx = kx;
        if (j0 + r < n_sm) {
            kx = load4(kb + (size_t)(j0 + r) * DL + c4);
            vx = load4(vb + (size_t)(j0 + r) * DL + c4);
        }
        float *kp = Kt + r * (D + 1) + c4, *vp = Vt + r * (D + 1) + c4;
        kp[0] = kx.x; kp[1] = kx.y; kp[2] = kx.z; kp[3] = kx.w;
        vp[0] = vx.x; vp[1] = vx.y; vp[2] = vx.z; vp[3] = vx.w;
    }
    if (threadIdx.x < 32)
        pos[threadIdx.x] = (j0 + threadIdx.x < n_sm) ? sm_idx[(size_t)bh * L + j0 + threadIdx.x]
                                                     : 0x7fffffff;
    __syncthreads();
    const int my_pos = pos[lane];
    const int c_first = pos[0] / kC;
    constexpr int kPer = D / 8;
    const int kj = threadIdx.x >> 3, cs = threadIdx.x & 7;
    float adk[kPer], adv[kPer], adm = 0.f;
#pragma unroll
    for (int x = 0; x < kPer; ++x) { adk[x] = 0.f; adv[x] = 0.f; }

    for (int c = c_first; c < NC; ++c) {
        const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
        __syncthreads();
        for (int idx = threadIdx.x; idx < kC * D / 4; idx += kThreads) {
            const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
            store4(Qs + r * D + c4, load4(q32 + tok0 * DL + (size_t)r * ts + col0 + c4));
            store4(dOs + r * D + c4, load4(do_nla + tok0 * DL + (size_t)r * ts + col0 + c4));
        }
        if (threadIdx.x < kC) {
            lse_s[threadIdx.x] = lse[(size_t)bhg * L + c * kC + threadIdx.x];
            dsm_s[threadIdx.x] = Dsm[(size_t)bhg * L + c * kC + threadIdx.x];
        }
        __syncthreads();
        const float *kr = Kt + lane * (D + 1), *vr = Vt + lane * (D + 1);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int il = warp * 8 + r, i = c * kC + il;
            const float *qr = Qs + il * D, *dor = dOs + il * D;
            float s = 0.f, dp = 0.f;
#pragma unroll 8
            for (int x = 0; x < D; ++x) {
                s = fmaf(qr[x], kr[x], s);
                dp = fmaf(dor[x], vr[x], dp);
            }
            const float pj = (my_pos <= i) ? __expf(s * scale_sm - lse_s[il]) : 0.f;
            Ps[il * 33 + lane] = pj;
            Dss[il * 33 + lane] = pj * (dp - dsm_s[il]);
        }
        __syncthreads();
        for (int il = 0; il < kC; ++il) {
            const float pj = Ps[il * 33 + kj], ds = Dss[il * 33 + kj];
            adm += ds;
            const float *dor = dOs + il * D + cs, *qr = Qs + il * D + cs;
#pragma unroll
            for (int x = 0; x < kPer; ++x) {
                adv[x] = fmaf(pj, dor[8 * x], adv[x]);
                adk[x] = fmaf(ds, qr[8 * x], adk[x]);
            }
        }
    }
    if (j0 + kj < n_sm) {
        float *dkr = dk_sm + ((size_t)bh * cap + j0 + kj) * DL + col0 + cs;
        float *dvr = dv_sm + ((size_t)bh * cap + j0 + kj) * DL + col0 + cs;
#pragma unroll
        for (int x = 0; x < kPer; ++x) { dkr[8 * x] = scale_sm * adk[x]; dvr[8 * x] = adv[x]; }
        if (dmask && cs == 0) dmask[(size_t)bhg * cap + j0 + kj] = adm;
    }
}

// ------------------------------------------------------------------------------------------
// Block-level routing (Section 4.1, inner-chunk correlations): a query in a linear block also reads
// the causal part of its own block, whose tokens are not among the retained ones.  One CTA per
// linear block adds that part of the softmax branch's backward in fp32:
//   p_ij = exp(scale s_ij - lse_i), ds_ij = p_ij (dp_ij - D_i), j <= i, with lse_i and
//   D_i = <do_i, o_i> of the whole softmax row;
//   dq_sm += scale dS K;  dk_x = scale dS^T Q,  dv_x = P^T dO  (written: the tokens of a linear
//   block have no other softmax-branch gradient).  grid = (L/64, B*H); softmax blocks return.
// Dsm arrives times the gradient scale of the tensor-core kernels (gsc; 1 without them).
// ------------------------------------------------------------------------------------------
// G softmax heads per linear head: a CTA's head is a slice of D columns of rows of DL = G D columns;
// lse and Dsm are [B,H,G,L]; q32, k32 are the softmax operation's copies of q and k.
template <int D, int G>
__global__ void __launch_bounds__(kThreads)
softmax_bwd_own_block_simt_kernel(const float *__restrict__ q32, const float *__restrict__ k32,
                                  const float *__restrict__ v32, const float *__restrict__ do_nla,
                                  const float *__restrict__ lse, const float *__restrict__ Dsm,
                                  const uint8_t *__restrict__ route, float scale_sm,
                                  float *__restrict__ dq_sm, float *__restrict__ dk_x,
                                  float *__restrict__ dv_x, const int32_t *gsc, int L, int H) {
    extern __shared__ float smem[];
    float *Qs = smem;                        // [64][D+1]
    float *Ks = Qs + kC * (D + 1);
    float *Vs = Ks + kC * (D + 1);
    float *dOs = Vs + kC * (D + 1);
    float *Ps = dOs + kC * (D + 1);          // [64][65]
    float *dSs = Ps + kC * (kC + 1);         // [64][65]
    constexpr int DL = D * G;
    const int c = blockIdx.x, bhg = blockIdx.y, bh = bhg / G, col0 = (bhg % G) * D, b = bh / H, h = bh % H;
    const size_t ts = (size_t)H * DL;
    const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
    if (route[tok0]) return;                 // a softmax block: its tokens are retained ones
    const float ginv = grad_scale(gsc).y;
    for (int idx = threadIdx.x; idx < kC * D / 4; idx += kThreads) {
        const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
        const size_t src = tok0 * DL + (size_t)r * ts + col0 + c4;
        const float4 a = load4(q32 + src), bb = load4(k32 + src), cc = load4(v32 + src), dd = load4(do_nla + src);
        float *p0 = Qs + r * (D + 1) + c4, *p1 = Ks + r * (D + 1) + c4, *p2 = Vs + r * (D + 1) + c4,
              *p3 = dOs + r * (D + 1) + c4;
        p0[0] = a.x; p0[1] = a.y; p0[2] = a.z; p0[3] = a.w;
        p1[0] = bb.x; p1[1] = bb.y; p1[2] = bb.z; p1[3] = bb.w;
        p2[0] = cc.x; p2[1] = cc.y; p2[2] = cc.z; p2[3] = cc.w;
        p3[0] = dd.x; p3[1] = dd.y; p3[2] = dd.z; p3[3] = dd.w;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < kC * kC; idx += kThreads) {
        const int i = idx >> 6, j = idx & 63;
        float pj = 0.f, ds = 0.f;
        if (j <= i) {
            const float *qr = Qs + i * (D + 1), *kr = Ks + j * (D + 1), *dor = dOs + i * (D + 1), *vr = Vs + j * (D + 1);
            float s = 0.f, dp = 0.f;
#pragma unroll 8
            for (int x = 0; x < D; ++x) {
                s = fmaf(qr[x], kr[x], s);
                dp = fmaf(dor[x], vr[x], dp);
            }
            const size_t row = (size_t)bhg * L + (size_t)c * kC + i;
            pj = __expf(s * scale_sm - lse[row]);
            ds = pj * (dp - ginv * Dsm[row]);
        }
        Ps[i * (kC + 1) + j] = pj;
        dSs[i * (kC + 1) + j] = ds;
    }
    __syncthreads();
    // thread (row r, column group cg): D / 4 columns cg, cg + 4, ... of dq_r, dk_r, dv_r
    const int r = threadIdx.x >> 2, cg = threadIdx.x & 3;
    for (int x = cg; x < D; x += 4) {
        float aq = 0.f, ak = 0.f, av = 0.f;
        for (int j = 0; j <= r; ++j) aq = fmaf(dSs[r * (kC + 1) + j], Ks[j * (D + 1) + x], aq);
        for (int i = r; i < kC; ++i) {
            ak = fmaf(dSs[i * (kC + 1) + r], Qs[i * (D + 1) + x], ak);
            av = fmaf(Ps[i * (kC + 1) + r], dOs[i * (D + 1) + x], av);
        }
        const size_t dst = tok0 * DL + (size_t)r * ts + col0 + x;
        dq_sm[dst] += scale_sm * aq;
        dk_x[dst] = scale_sm * ak;
        dv_x[dst] = av;
    }
}

// ------------------------------------------------------------------------------------------
// reverse scan over chunks: dU~ (stored), chunk-exit dS (stored), <dS1, S0> partials.
// grid = (D/32, B*H), mirrors gdn_scan_simt_kernel.
// ------------------------------------------------------------------------------------------
constexpr int kDvs = 32;

template <int D>
__global__ void __launch_bounds__(kThreads)
gdn_rscan_kernel(const float *__restrict__ q32, const float *__restrict__ k32,
                 const float *__restrict__ Gcum, const float *__restrict__ W,
                 const float *__restrict__ P, const float *__restrict__ do_la,
                 const float *__restrict__ chunk_states, float scale_la, float *__restrict__ dUt,
                 float *__restrict__ dS_c, float *__restrict__ gS, const float *__restrict__ dstate_out,
                 float *__restrict__ dstate_in, const uint8_t *__restrict__ block_route, int L, int H) {
    // block_route (block-level routing): a softmax block's update was not committed to the state, so
    // its exit-state gradient reaches the entry state through the decay only: no K~ dS term in dU~, and
    // the stored chunk-exit gradient (which the dK~ product reads) is zero; <dS1, S0> is not.
    extern __shared__ float smem[];
    float *dSs = smem;                       // [D][32]
    float *Ws = dSs + D * kDvs;              // [64][D+1]
    float *Qs = Ws + kC * (D + 1);           // [64][D+1]
    float *Ks = Qs + kC * (D + 1);           // [64][D+1]
    float *Ps = Ks + kC * (D + 1);           // [64][65]
    float *dOs = Ps + kC * (kC + 1);         // [64][33]
    float *dUs = dOs + kC * (kDvs + 1);      // [64][33]
    float *Gs = dUs + kC * (kDvs + 1);       // [64]
    float *red = Gs + kC;                    // [8]

    const int slice = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const size_t ts = (size_t)H * D;
    const int c0 = slice * kDvs;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int idx = threadIdx.x; idx < D * kDvs; idx += kThreads)     // gradient arriving at the final state
        dSs[idx] = dstate_out ? dstate_out[((size_t)bh * D + idx / kDvs) * D + c0 + idx % kDvs] : 0.f;

    for (int c = NC - 1; c >= 0; --c) {
        const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
        const float commit = block_route && block_route[tok0] ? 0.f : 1.f;
        __syncthreads();
        // store the chunk-exit gradient and the partial <dS1, S0>
        {
            float part = 0.f;
            for (int idx = threadIdx.x; idx < D * kDvs; idx += kThreads) {
                const int a = idx / kDvs, cc = idx % kDvs;
                const size_t gi = (((size_t)bh * NC + c) * D + a) * D + c0 + cc;
                dS_c[gi] = commit * dSs[idx];
                part = fmaf(dSs[idx], chunk_states[gi], part);
            }
            part = warp_sum(part);
            if (lane == 0) red[warp] = part;
        }
        for (int idx = threadIdx.x; idx < kC * D / 4; idx += kThreads) {
            const int r = idx / (D / 4), c4 = (idx % (D / 4)) * 4;
            const float4 wv = load4(W + tok0 * D + (size_t)r * ts + c4);
            const float4 qv = load4(q32 + tok0 * D + (size_t)r * ts + c4);
            const float4 kv = load4(k32 + tok0 * D + (size_t)r * ts + c4);
            float *wp = Ws + r * (D + 1) + c4, *qp = Qs + r * (D + 1) + c4, *kp = Ks + r * (D + 1) + c4;
            wp[0] = wv.x; wp[1] = wv.y; wp[2] = wv.z; wp[3] = wv.w;
            qp[0] = qv.x; qp[1] = qv.y; qp[2] = qv.z; qp[3] = qv.w;
            kp[0] = kv.x; kp[1] = kv.y; kp[2] = kv.z; kp[3] = kv.w;
        }
        {
            const float *Pc = P + ((size_t)bh * NC + c) * kC * kC;
            for (int idx = threadIdx.x; idx < kC * kC; idx += kThreads)
                Ps[(idx >> 6) * (kC + 1) + (idx & 63)] = Pc[idx];
            for (int idx = threadIdx.x; idx < kC * kDvs; idx += kThreads) {
                const int r = idx / kDvs, cc = idx % kDvs;
                dOs[r * (kDvs + 1) + cc] = do_la[(tok0 + (size_t)r * H) * D + c0 + cc];
            }
            if (threadIdx.x < kC) Gs[threadIdx.x] = Gcum[(size_t)bh * L + c * kC + threadIdx.x];
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            float tot = 0.f;
            for (int wv = 0; wv < kThreads / 32; ++wv) tot += red[wv];
            gS[((size_t)bh * NC + c) * (D / kDvs) + slice] = tot;
        }
        const float gl = Gs[kC - 1];
        const int r = threadIdx.x >> 2, cb = (threadIdx.x & 3) * 8;
        // dU~_r = sum_{i>=r} P[i][r] dO_i + (gamma_C/gamma_r) k_r dS
        {
            float acc[8], acc2[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) { acc[x] = 0.f; acc2[x] = 0.f; }
            for (int i = r; i < kC; ++i) {
                const float pv = Ps[i * (kC + 1) + r];
                const float *dr = dOs + i * (kDvs + 1) + cb;
#pragma unroll
                for (int x = 0; x < 8; ++x) acc[x] = fmaf(pv, dr[x], acc[x]);
            }
            const float *kr = Ks + r * (D + 1);
            for (int a = 0; a < D; ++a) {
                const float kv = kr[a];
                const float *sr = dSs + a * kDvs + cb;
#pragma unroll
                for (int x = 0; x < 8; ++x) acc2[x] = fmaf(kv, sr[x], acc2[x]);
            }
            const float kt = commit * __expf(gl - Gs[r]);
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                acc[x] = fmaf(kt, acc2[x], acc[x]);
                dUs[r * (kDvs + 1) + cb + x] = acc[x];
            }
            float *dst = dUt + (tok0 + (size_t)r * H) * D + c0 + cb;
            store4(dst, make_float4(acc[0], acc[1], acc[2], acc[3]));
            store4(dst + 4, make_float4(acc[4], acc[5], acc[6], acc[7]));
        }
        __syncthreads();
        // dS0 = Qg^T dO + gamma_C dS1 - W^T dU~
        {
            constexpr int kPer = D / 8, kTpr = kDvs / kPer;
            const int a = threadIdx.x / kTpr, cs = (threadIdx.x % kTpr) * kPer;
            const float gC = __expf(gl);
            float acc[kPer];
#pragma unroll
            for (int x = 0; x < kPer; ++x) acc[x] = gC * dSs[a * kDvs + cs + x];
            for (int i = 0; i < kC; ++i) {
                const float qg = scale_la * __expf(Gs[i]) * Qs[i * (D + 1) + a];
                const float wv = Ws[i * (D + 1) + a];
                const float *dor = dOs + i * (kDvs + 1) + cs, *dur = dUs + i * (kDvs + 1) + cs;
#pragma unroll
                for (int x = 0; x < kPer; ++x) acc[x] = fmaf(qg, dor[x], fmaf(-wv, dur[x], acc[x]));
            }
            __syncthreads();
#pragma unroll
            for (int x = 0; x < kPer; ++x) dSs[a * kDvs + cs + x] = acc[x];
            if (c == 0 && dstate_in) {      // what is left after the first chunk: the initial state's gradient
#pragma unroll
                for (int x = 0; x < kPer; ++x) dstate_in[((size_t)bh * D + a) * D + c0 + cs + x] = acc[x];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// transposed triangular solve: [dKb | dVb] = (I + A)^-T [dW | dU~], A = diag(beta~) Abar.
// grid = (L/C, B*H); one right-hand-side column per thread.
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kThreads)
gdn_tsolve_kernel(const float *__restrict__ Abar, const float *__restrict__ beta,
                  const uint8_t *__restrict__ route, const float *__restrict__ dW,
                  const float *__restrict__ dUt, float *__restrict__ dKb, float *__restrict__ dVb,
                  int L, int H) {
    __shared__ float As[kC * kC];
    __shared__ float bts[kC];
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const size_t ts = (size_t)H * D;
    const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
    if (threadIdx.x < kC) {
        const size_t t = tok0 + (size_t)threadIdx.x * H;
        bts[threadIdx.x] = route && route[t] ? 0.f : beta[t];   // route == nullptr: beta~ = beta
    }
    __syncthreads();
    const float *Ab = Abar + ((size_t)bh * (L / kC) + c) * kC * kC;
    for (int idx = threadIdx.x; idx < kC * kC; idx += kThreads) As[idx] = bts[idx >> 6] * Ab[idx];
    __syncthreads();
    if (threadIdx.x < 2 * D) {
        const bool first = threadIdx.x < D;
        const int col = first ? threadIdx.x : threadIdx.x - D;
        const float *src = (first ? dW : dUt) + tok0 * D + col;
        float x[kC];
#pragma unroll
        for (int i = kC - 1; i >= 0; --i) {
            float acc = src[(size_t)i * ts];
#pragma unroll
            for (int j = i + 1; j < kC; ++j) acc = fmaf(-As[j * kC + i], x[j], acc);
            x[i] = acc;
        }
        float *dst = (first ? dKb : dVb) + tok0 * D + col;
#pragma unroll
        for (int i = 0; i < kC; ++i) dst[(size_t)i * ts] = x[i];
    }
}

// ------------------------------------------------------------------------------------------
// Mg = M . Gamma, Ms = diag(beta~) Mg, Ns = scale_la N . Gamma    (all 64x64 per chunk)
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
mask_scale_kernel(const float *__restrict__ M, const float *__restrict__ N,
                  const float *__restrict__ Gcum, const float *__restrict__ beta,
                  const uint8_t *__restrict__ route, float scale_la, float *__restrict__ Mg,
                  float *__restrict__ Ms, float *__restrict__ Ns, int L, int H) {
    __shared__ float Gs[kC], bts[kC];
    const int NC = L / kC;
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    if (threadIdx.x < kC) {
        const size_t t = ((size_t)b * L + (size_t)c * kC + threadIdx.x) * H + h;
        bts[threadIdx.x] = route && route[t] ? 0.f : beta[t];
        Gs[threadIdx.x] = Gcum[(size_t)bh * L + c * kC + threadIdx.x];
    }
    __syncthreads();
    const size_t base = ((size_t)bh * NC + c) * kC * kC;
    for (int idx = threadIdx.x; idx < kC * kC; idx += kThreads) {
        const int i = idx >> 6, j = idx & 63;
        const float gam = j <= i ? __expf(Gs[i] - Gs[j]) : 0.f;
        const float mg = M[base + idx] * gam;
        Mg[base + idx] = mg;
        Ms[base + idx] = bts[i] * mg;
        Ns[base + idx] = scale_la * N[base + idx] * gam;
    }
}

// ------------------------------------------------------------------------------------------
// assembly: dq (all tokens), dk/dv (linear tokens), per-row dG, kappa, dbeta.
// one warp per (token, head) row.
// ------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
gdn_assemble_kernel(const float *__restrict__ q32, const float *__restrict__ k32,
                    const float *__restrict__ v32, const float *__restrict__ Gcum,
                    const float *__restrict__ beta, const uint8_t *__restrict__ route,
                    const float *__restrict__ dQg, const float *__restrict__ dKb,
                    const float *__restrict__ dVb, const float *__restrict__ dKt,
                    const float *__restrict__ X1p, const float *__restrict__ X2,
                    const float *__restrict__ X3, const float *__restrict__ X4,
                    const float *__restrict__ dq_sm, const float *__restrict__ dk_x,
                    const float *__restrict__ dv_x, float scale_la, T *__restrict__ dq,
                    T *__restrict__ dk, T *__restrict__ dv, float *__restrict__ dGrow,
                    float *__restrict__ kappa, float *__restrict__ dbeta, int B, int L, int H) {
    constexpr int kCols = D / 32;
    const int lane = threadIdx.x & 31;
    const size_t row = (size_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (row >= (size_t)B * L * H) return;
    const int h = row % H;
    const size_t bl = row / H;
    const int l = bl % L, b = bl / L;
    const size_t bhl = ((size_t)b * H + h) * L;
    const float Gi = Gcum[bhl + l], GC = Gcum[bhl + (l | (kC - 1))];
    // route == nullptr (block-level routing): every token takes part in the delta rule, and every
    // token's dk, dv also has a softmax-branch part, given in dk_x, dv_x (fp32, token-major)
    const bool lin = !route || route[row] == 0;
    const float bt = lin ? beta[row] : 0.f;
    const float gam = __expf(Gi), kt = __expf(GC - Gi);
    float kdKb = 0.f, qdQg = 0.f, kdKt = 0.f, kX1 = 0.f, kX2 = 0.f, qX3 = 0.f, kX4 = 0.f, vdVb = 0.f;
#pragma unroll
    for (int x = 0; x < kCols; ++x) {
        const size_t i = row * D + lane + 32 * x;
        const float qv = q32[i], kv = k32[i], vv = v32[i];
        const float a_dQg = dQg[i], a_dKb = dKb[i], a_dVb = dVb[i], a_dKt = dKt[i];
        const float x1 = X1p[i], x2 = X2[i], x3 = X3[i], x4 = X4[i];
        kdKb = fmaf(kv, a_dKb, kdKb); qdQg = fmaf(qv, a_dQg, qdQg); kdKt = fmaf(kv, a_dKt, kdKt);
        kX1 = fmaf(kv, x1, kX1); kX2 = fmaf(kv, x2, kX2); qX3 = fmaf(qv, x3, qX3);
        kX4 = fmaf(kv, x4, kX4); vdVb = fmaf(vv, a_dVb, vdVb);
        dq[i] = from_f32<T>(scale_la * gam * a_dQg + x3 + (dq_sm ? dq_sm[i] : 0.f));
        if (lin) {
            dk[i] = from_f32<T>(bt * gam * a_dKb + kt * a_dKt + bt * x1 + x2 + x4 + (dk_x ? dk_x[i] : 0.f));
            dv[i] = from_f32<T>(bt * a_dVb + (dv_x ? dv_x[i] : 0.f));
        }
    }
    kdKb = warp_sum(kdKb); qdQg = warp_sum(qdQg); kdKt = warp_sum(kdKt); kX1 = warp_sum(kX1);
    kX2 = warp_sum(kX2); qX3 = warp_sum(qX3); kX4 = warp_sum(kX4); vdVb = warp_sum(vdVb);
    if (lane == 0) {
        const float kap = kt * kdKt;
        dGrow[bhl + l] = bt * gam * kdKb + scale_la * gam * qdQg - kap + bt * kX1 - kX2 + qX3 - kX4;
        kappa[bhl + l] = kap;
        dbeta[row] = lin ? gam * kdKb + vdVb + kX1 : 0.f;
    }
}

// The middle of the chunk-level chain in one kernel per chunk (bf16 storage, tf32 products):
//   dKb = Tinv^T dW, dVb = Tinv^T dU~   (written out: the assembly reads them)
//   M = -strictly_lower(dKb W^T + dVb U^T),  N = lower(dO U~^T)
//   Mg = M . Gamma, Ms = diag(beta~) Mg, Ns = scale_la N . Gamma
// 64 columns of the head at a time: dKb, dVb of those columns go from the accumulators to shared memory as
// the next products' operands, and M, N add up in accumulators over the column blocks; the two 64 x 64
// intermediates never reach global memory.  Warp w owns rows 16 (w & 3) .. and columns 32 (w >> 2) ..
// of every 64 x 64 result.  Operand rows are 72 floats when read along the row index and 68 when read
// along k (both free of bank conflicts for the fragments).
constexpr size_t kTmSmem = sizeof(float) * (5 * kC * 72 + 2 * kC);

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
gdn_tm_kernel(const float *__restrict__ Tinv, const float *__restrict__ dW, const float *__restrict__ dUt,
              const float *__restrict__ W, const float *__restrict__ U, const float *__restrict__ dO,
              const float *__restrict__ Ut, const float *__restrict__ Gcum, const float *__restrict__ beta,
              const uint8_t *__restrict__ route, float scale_la, float *__restrict__ dKb,
              float *__restrict__ dVb, float *__restrict__ Mg, float *__restrict__ Ms, float *__restrict__ Ns,
              int L, int H) {
    extern __shared__ __align__(16) float tm_smem[];
    float *sT = tm_smem, *bufA = sT + kC * 72, *bufB = bufA + kC * 72, *bufC = bufB + kC * 72, *bufD = bufC + kC * 72;
    float *Gs = bufD + kC * 72, *bts = Gs + kC;
    const int NC = L / kC, ch = blockIdx.x % NC, bh = blockIdx.x / NC, b = bh / H, h = bh % H;
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31, fg = lane >> 2, ft = lane & 3;
    const int wr = (warp & 3) * 16, wc = (warp >> 2) * 32;
    const size_t tok0 = ((size_t)b * L + (size_t)ch * kC) * H + h;         // the chunk's first token (stride H)
    // 64 tokens x 64 columns [n0, n0 + 64) of a token-major array into rows of `ld` floats
    auto load_tile = [&](float *dst, int ld, const float *src, int n0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int f = t + kThreads * i, r = f >> 4, c4 = (f & 15) * 4;
            cp_async16(dst + r * ld + c4, src + (tok0 + (size_t)r * H) * D + n0 + c4);
        }
    };
    {
        const float *ti = Tinv + (size_t)blockIdx.x * kC * kC;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int f = t + kThreads * i, r = f >> 4, c4 = (f & 15) * 4;
            cp_async16(sT + r * 72 + c4, ti + r * kC + c4);
        }
    }
    if (t < kC) {
        const size_t tok = tok0 + (size_t)t * H;
        bts[t] = route && route[tok] ? 0.f : beta[tok];
        Gs[t] = Gcum[(size_t)bh * L + (size_t)ch * kC + t];
    }
    float Macc[4][4], Nacc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { Macc[i][j] = 0.f; Nacc[i][j] = 0.f; }
    const int m0 = wr + fg, m1 = wr + fg + 8;
    // acc += A B^T with both operands stored [row][k] in rows of 68 floats
    auto mma_abt = [&](float (&acc)[4][4], const float *A, const float *Bm) {
#pragma unroll 2
        for (int k8 = 0; k8 < kC; k8 += 8) {
            const int ka = k8 + ft, kb = k8 + ft + 4;
            const uint32_t a[4] = {to_tf32(A[m0 * 68 + ka]), to_tf32(A[m1 * 68 + ka]),
                                   to_tf32(A[m0 * 68 + kb]), to_tf32(A[m1 * 68 + kb])};
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int n = wc + 8 * nt + fg;
                const uint32_t bb[2] = {to_tf32(Bm[n * 68 + ka]), to_tf32(Bm[n * 68 + kb])};
                mma_tf32_16x8x8(acc[nt], a, bb);
            }
        }
    };
    // Per 64 columns: every group of loads is in flight while the previous product runs.
    for (int n0 = 0; n0 < D; n0 += 64) {
        load_tile(bufA, 68, dO, n0);
        load_tile(bufC, 68, Ut, n0);
        cp_async_commit();
        load_tile(bufB, 72, dW, n0);
        load_tile(bufD, 72, dUt, n0);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        mma_abt(Nacc, bufA, bufC);           // dO U~^T
        __syncthreads();                     // dO, U~ of these columns have been read by all
        load_tile(bufA, 68, W, n0);
        load_tile(bufC, 68, U, n0);
        cp_async_commit();
        cp_async_wait<1>();                  // dW, dU~ (and Tinv) have landed
        __syncthreads();
        float kb_[4][4], vb_[4][4];          // dKb, dVb of these 64 columns
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) { kb_[i][j] = 0.f; vb_[i][j] = 0.f; }
#pragma unroll 2
        for (int k8 = 0; k8 < kC; k8 += 8) {
            const int ka = k8 + ft, kb = k8 + ft + 4;
            const uint32_t a[4] = {to_tf32(sT[ka * 72 + m0]), to_tf32(sT[ka * 72 + m1]),
                                   to_tf32(sT[kb * 72 + m0]), to_tf32(sT[kb * 72 + m1])};
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int n = wc + 8 * nt + fg;
                const uint32_t b1[2] = {to_tf32(bufB[ka * 72 + n]), to_tf32(bufB[kb * 72 + n])};
                const uint32_t b2[2] = {to_tf32(bufD[ka * 72 + n]), to_tf32(bufD[kb * 72 + n])};
                mma_tf32_16x8x8(kb_[nt], a, b1);
                mma_tf32_16x8x8(vb_[nt], a, b2);
            }
        }
        __syncthreads();                     // dW, dU~ of these columns have been read by all
        // fragment layout: elements (0, 1) in row fg, (2, 3) in row fg + 8; columns 2 ft, 2 ft + 1
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int row = wr + fg + 8 * hh, cl = wc + 8 * nt + 2 * ft;
                const size_t i = (tok0 + (size_t)row * H) * D + n0 + cl;
                const float2 kv = make_float2(kb_[nt][2 * hh], kb_[nt][2 * hh + 1]);
                const float2 vv = make_float2(vb_[nt][2 * hh], vb_[nt][2 * hh + 1]);
                *reinterpret_cast<float2 *>(dKb + i) = kv;
                *reinterpret_cast<float2 *>(dVb + i) = vv;
                *reinterpret_cast<float2 *>(bufB + row * 68 + cl) = kv;
                *reinterpret_cast<float2 *>(bufD + row * 68 + cl) = vv;
            }
        cp_async_wait<0>();                  // W, U
        __syncthreads();
        mma_abt(Macc, bufB, bufA);           // dKb W^T
        mma_abt(Macc, bufD, bufC);           // + dVb U^T
        __syncthreads();
    }
    const size_t base = (size_t)blockIdx.x * kC * kC;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = wr + fg + 8 * hh, col = wc + 8 * nt + 2 * ft;
            float mg[2], ns[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int j = col + e;
                const float gam = j <= row ? __expf(Gs[row] - Gs[j]) : 0.f;
                mg[e] = j < row ? -Macc[nt][2 * hh + e] * gam : 0.f;
                ns[e] = scale_la * Nacc[nt][2 * hh + e] * gam;
            }
            const size_t o = base + (size_t)row * kC + col;
            *reinterpret_cast<float2 *>(Mg + o) = make_float2(mg[0], mg[1]);
            *reinterpret_cast<float2 *>(Ms + o) = make_float2(bts[row] * mg[0], bts[row] * mg[1]);
            *reinterpret_cast<float2 *>(Ns + o) = make_float2(ns[0], ns[1]);
        }
}

// The last four chunk-level products and the assembly in one kernel per chunk (bf16 storage, tf32
// products as in bgemm_tf32_kernel): X1 = Mg K, X2 = Ms^T K, X3 = Ns K, X4 = Ns^T Q stay in the
// accumulator fragments and meet the other terms of dq, dk, dv there, so the four [B,L,H,d] fp32
// arrays are neither written nor read back.  One CTA per chunk, 64 columns at a time; warp w owns rows
// 16 (w & 3) .. and columns 32 (w >> 2) .. of the 64; the eight per-row dot products are summed over a
// thread's columns, then over the four lanes that share a row, then over the two warps that do.
constexpr int kXaLdA = 68, kXaLdT = 72;                  // rows read along k / read transposed (and K, Q)
constexpr size_t kXaSmem = sizeof(float) * (2 * kC * kXaLdA + 3 * kC * kXaLdT + 4 * kC + 2 * kC * 8);

template <typename T, int D>
__global__ void __launch_bounds__(kThreads, 2)
gdn_xassemble_kernel(const float *__restrict__ q32, const float *__restrict__ k32,
                     const float *__restrict__ v32, const float *__restrict__ Gcum,
                     const float *__restrict__ beta, const uint8_t *__restrict__ route,
                     const float *__restrict__ dQg, const float *__restrict__ dKb,
                     const float *__restrict__ dVb, const float *__restrict__ dKt,
                     const float *__restrict__ Mg, const float *__restrict__ Ms,
                     const float *__restrict__ Ns, const float *__restrict__ dq_sm,
                     const float *__restrict__ dk_x, const float *__restrict__ dv_x, float scale_la,
                     T *__restrict__ dq, T *__restrict__ dk, T *__restrict__ dv, float *__restrict__ dGrow,
                     float *__restrict__ kappa, float *__restrict__ dbeta, int L, int H) {
    extern __shared__ __align__(16) float xa_smem[];
    float *sMg = xa_smem;                        // [i][j], ld 68
    float *sNs = sMg + kC * kXaLdA;              // [i][j], ld 68
    float *sMs = sNs + kC * kXaLdA;              // [i][j], ld 72 (read transposed only)
    float *sK = sMs + kC * kXaLdT;               // [token][64 columns], ld 72
    float *sQ = sK + kC * kXaLdT;
    float *sGam = sQ + kC * kXaLdT, *sKt = sGam + kC, *sBt = sKt + kC, *sLin = sBt + kC;
    float *sSum = sLin + kC;                     // [2 column warps][64 rows][8]
    const int NC = L / kC, ch = blockIdx.x % NC, bh = blockIdx.x / NC, b = bh / H, h = bh % H;
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31, fg = lane >> 2, ft = lane & 3;
    const int wr = (warp & 3) * 16, wcw = warp >> 2, wc = wcw * 32;
    const size_t tok0 = ((size_t)b * L + (size_t)ch * kC) * H + h;         // the chunk's first token (stride H)
    const size_t bhl = (size_t)bh * L + (size_t)ch * kC;
    {
        const float *mg = Mg + (size_t)blockIdx.x * kC * kC, *msrc = Ms + (size_t)blockIdx.x * kC * kC,
                    *ns = Ns + (size_t)blockIdx.x * kC * kC;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int f = t + kThreads * i, r = f >> 4, c4 = (f & 15) * 4;
            cp_async16(sMg + r * kXaLdA + c4, mg + r * kC + c4);
            cp_async16(sNs + r * kXaLdA + c4, ns + r * kC + c4);
            cp_async16(sMs + r * kXaLdT + c4, msrc + r * kC + c4);
        }
    }
    if (t < kC) {
        const size_t tok = tok0 + (size_t)t * H;
        const float Gi = Gcum[bhl + t], GC = Gcum[bhl + kC - 1];
        const bool lin = !route || route[tok] == 0;
        sGam[t] = __expf(Gi);
        sKt[t] = __expf(GC - Gi);
        sBt[t] = lin ? beta[tok] : 0.f;
        sLin[t] = lin ? 1.f : 0.f;
    }
    float sums[2][8];            // per row half: kdKb, qdQg, kdKt, kX1, kX2, qX3, kX4, vdVb
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int j = 0; j < 8; ++j) sums[hh][j] = 0.f;

    for (int n0 = 0; n0 < D; n0 += 64) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int f = t + kThreads * i, r = f >> 4, c4 = (f & 15) * 4;
            cp_async16(sK + r * kXaLdT + c4, k32 + (tok0 + (size_t)r * H) * D + n0 + c4);
            cp_async16(sQ + r * kXaLdT + c4, q32 + (tok0 + (size_t)r * H) * D + n0 + c4);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
        float x1[4][4], x2[4][4], x3[4][4], x4[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) { x1[i][j] = 0.f; x2[i][j] = 0.f; x3[i][j] = 0.f; x4[i][j] = 0.f; }
#pragma unroll 2
        for (int k8 = 0; k8 < kC; k8 += 8) {
            const int m0 = wr + fg, m1 = wr + fg + 8, ka = k8 + ft, kb = k8 + ft + 4;
            const uint32_t a1[4] = {to_tf32(sMg[m0 * kXaLdA + ka]), to_tf32(sMg[m1 * kXaLdA + ka]),
                                    to_tf32(sMg[m0 * kXaLdA + kb]), to_tf32(sMg[m1 * kXaLdA + kb])};
            const uint32_t a2[4] = {to_tf32(sMs[ka * kXaLdT + m0]), to_tf32(sMs[ka * kXaLdT + m1]),
                                    to_tf32(sMs[kb * kXaLdT + m0]), to_tf32(sMs[kb * kXaLdT + m1])};
            const uint32_t a3[4] = {to_tf32(sNs[m0 * kXaLdA + ka]), to_tf32(sNs[m1 * kXaLdA + ka]),
                                    to_tf32(sNs[m0 * kXaLdA + kb]), to_tf32(sNs[m1 * kXaLdA + kb])};
            const uint32_t a4[4] = {to_tf32(sNs[ka * kXaLdA + m0]), to_tf32(sNs[ka * kXaLdA + m1]),
                                    to_tf32(sNs[kb * kXaLdA + m0]), to_tf32(sNs[kb * kXaLdA + m1])};
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int n = wc + 8 * nt + fg;
                const uint32_t bk[2] = {to_tf32(sK[ka * kXaLdT + n]), to_tf32(sK[kb * kXaLdT + n])};
                const uint32_t bq[2] = {to_tf32(sQ[ka * kXaLdT + n]), to_tf32(sQ[kb * kXaLdT + n])};
                mma_tf32_16x8x8(x1[nt], a1, bk);
                mma_tf32_16x8x8(x2[nt], a2, bk);
                mma_tf32_16x8x8(x3[nt], a3, bk);
                mma_tf32_16x8x8(x4[nt], a4, bq);
            }
        }
        // fragment layout: elements (0, 1) in row fg, (2, 3) in row fg + 8; columns 2 ft, 2 ft + 1
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = wr + fg + 8 * hh;
            const float gam = sGam[row], kt = sKt[row], bt = sBt[row];
            const bool lin = sLin[row] != 0.f;
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int cl = wc + 8 * nt + 2 * ft;                     // column within the 64
                const size_t i = (tok0 + (size_t)row * H) * D + n0 + cl;
                const float2 a_dQg = *reinterpret_cast<const float2 *>(dQg + i), a_dKb = *reinterpret_cast<const float2 *>(dKb + i);
                const float2 a_dVb = *reinterpret_cast<const float2 *>(dVb + i), a_dKt = *reinterpret_cast<const float2 *>(dKt + i);
                const float2 vv = *reinterpret_cast<const float2 *>(v32 + i);
                const float2 qv = *reinterpret_cast<const float2 *>(sQ + row * kXaLdT + cl);
                const float2 kv = *reinterpret_cast<const float2 *>(sK + row * kXaLdT + cl);
                float2 e_dq = dq_sm ? *reinterpret_cast<const float2 *>(dq_sm + i) : make_float2(0.f, 0.f);
                float2 e_dk = dk_x ? *reinterpret_cast<const float2 *>(dk_x + i) : make_float2(0.f, 0.f);
                float2 e_dv = dv_x ? *reinterpret_cast<const float2 *>(dv_x + i) : make_float2(0.f, 0.f);
                const float x1a = x1[nt][2 * hh], x1b = x1[nt][2 * hh + 1], x2a = x2[nt][2 * hh], x2b = x2[nt][2 * hh + 1];
                const float x3a = x3[nt][2 * hh], x3b = x3[nt][2 * hh + 1], x4a = x4[nt][2 * hh], x4b = x4[nt][2 * hh + 1];
                float *sm = sums[hh];
                sm[0] = fmaf(kv.x, a_dKb.x, fmaf(kv.y, a_dKb.y, sm[0]));
                sm[1] = fmaf(qv.x, a_dQg.x, fmaf(qv.y, a_dQg.y, sm[1]));
                sm[2] = fmaf(kv.x, a_dKt.x, fmaf(kv.y, a_dKt.y, sm[2]));
                sm[3] = fmaf(kv.x, x1a, fmaf(kv.y, x1b, sm[3]));
                sm[4] = fmaf(kv.x, x2a, fmaf(kv.y, x2b, sm[4]));
                sm[5] = fmaf(qv.x, x3a, fmaf(qv.y, x3b, sm[5]));
                sm[6] = fmaf(kv.x, x4a, fmaf(kv.y, x4b, sm[6]));
                sm[7] = fmaf(vv.x, a_dVb.x, fmaf(vv.y, a_dVb.y, sm[7]));
                const float sgm = scale_la * gam;
                store2(dq + i, sgm * a_dQg.x + x3a + e_dq.x, sgm * a_dQg.y + x3b + e_dq.y);
                if (lin) {
                    const float bg = bt * gam;
                    store2(dk + i, bg * a_dKb.x + kt * a_dKt.x + bt * x1a + x2a + x4a + e_dk.x,
                           bg * a_dKb.y + kt * a_dKt.y + bt * x1b + x2b + x4b + e_dk.y);
                    store2(dv + i, bt * a_dVb.x + e_dv.x, bt * a_dVb.y + e_dv.y);
                }
            }
        }
        __syncthreads();         // K, Q of these columns have been read by all
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float v = sums[hh][j];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            if (ft == 0) sSum[(wcw * kC + wr + fg + 8 * hh) * 8 + j] = v;
        }
    __syncthreads();
    if (t < kC) {
        float r[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) r[j] = sSum[t * 8 + j] + sSum[(kC + t) * 8 + j];
        const float gam = sGam[t], kt = sKt[t], bt = sBt[t];
        const bool lin = sLin[t] != 0.f;
        const float kap = kt * r[2];
        dGrow[bhl + t] = bt * gam * r[0] + scale_la * gam * r[1] - kap + bt * r[3] - r[4] + r[5] - r[6];
        kappa[bhl + t] = kap;
        dbeta[tok0 + (size_t)t * H] = lin ? gam * r[0] + r[7] + r[3] : 0.f;
    }
}

// dg_j = sum_{i>=j in chunk} dG_i, with the chunk-end extras added to the last row.
__global__ void dg_kernel(const float *__restrict__ dGrow, const float *__restrict__ kappa,
                          const float *__restrict__ gS, const float *__restrict__ Gcum, int n_slices,
                          float *__restrict__ dg, int B, int L, int H) {
    const int NC = L / kC;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)B * H * NC) return;
    const int c = idx % NC;
    const size_t bh = idx / NC;
    const int h = bh % H, b = bh / H;
    const size_t base = bh * L + (size_t)c * kC;
    float extra = 0.f;
    for (int i = 0; i < kC; ++i) extra += kappa[base + i];
    float gs = 0.f;
    for (int s = 0; s < n_slices; ++s) gs += gS[idx * n_slices + s];
    extra += __expf(Gcum[base + kC - 1]) * gs;
    float run = extra;
    for (int i = kC - 1; i >= 0; --i) {
        run += dGrow[base + i];
        dg[((size_t)b * L + (size_t)c * kC + i) * H + h] = run;
    }
}

// dk, dv of the retained tokens: scatter the compacted softmax-branch gradients.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
scatter_sm_kernel(const float *__restrict__ dk_sm, const float *__restrict__ dv_sm, int cap,
                  const int32_t *__restrict__ sm_idx, const int32_t *__restrict__ sm_chunk_prefix,
                  T *__restrict__ dk, T *__restrict__ dv, int L, int H) {
    constexpr int kVec = D / 4, kRows = kThreads / kVec;
    const int bh = blockIdx.y, b = bh / H, h = bh % H;
    const int NC = L / kC;
    const int n = min(sm_chunk_prefix[(size_t)bh * (NC + 1) + NC], cap);
    const int row = blockIdx.x * kRows + threadIdx.x / kVec, c4 = (threadIdx.x % kVec) * 4;
    if (row >= n) return;
    const int tok = sm_idx[(size_t)bh * L + row];
    const size_t dst = (((size_t)b * L + tok) * H + h) * D + c4;
    const size_t src = ((size_t)bh * cap + row) * D + c4;
    store4(dk + dst, load4(dk_sm + src));
    store4(dv + dst, load4(dv_sm + src));
}

template <typename Kn>
cudaError_t set_smem(Kn kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host launchers
// ------------------------------------------------------------------------------------------
cudaError_t launch_bgemm(bool ta, bool tb, int mask, BMat A, BMat B, BMat C, int m, int n, int k,
                         float alpha, bool accumulate, Shape s, cudaStream_t st) {
    const int NC = s.L / kC;
    if (m % 64 || n % 64 || k % kBgK) return cudaErrorInvalidValue;
    dim3 grid(n / 64, m / 64, s.B * s.H * NC);
#define NATSL_BG(TA, TB, MK)                                                                                   \
    do {                                                                                                        \
        if (s.bf16) {                                                                                           \
            cudaError_t e = cudaFuncSetAttribute(bgemm_tf32_kernel<TA, TB, MK>,                                 \
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBgSmem);    \
            if (e != cudaSuccess) return e;                                                                     \
            bgemm_tf32_kernel<TA, TB, MK><<<grid, kThreads, kBgSmem, st>>>(A, B, C, k, alpha, accumulate ? 1 : 0, s.H, NC); \
        } else bgemm_kernel<TA, TB, MK><<<grid, kThreads, 0, st>>>(A, B, C, k, alpha, accumulate ? 1 : 0, s.H, NC); \
    } while (0)
    if (!ta && !tb && mask == 0) NATSL_BG(false, false, 0);
    else if (!ta && tb && mask == 0) NATSL_BG(false, true, 0);
    else if (ta && !tb && mask == 0) NATSL_BG(true, false, 0);
    else if (!ta && tb && mask == 1) NATSL_BG(false, true, 1);
    else if (!ta && tb && mask == 2) NATSL_BG(false, true, 2);
    else return cudaErrorInvalidValue;
#undef NATSL_BG
    count_launch();
    return cudaGetLastError();
}

template <typename T>
static cudaError_t to_f32_impl(const void *a, const void *b, const void *c, float *a32, float *b32,
                               float *c32, size_t n, cudaStream_t st) {
    to_f32_kernel<T><<<1184, 256, 0, st>>>((const T *)a, (const T *)b, (const T *)c, a32, b32, c32,
                                           n / 4);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_to_f32(const void *a, const void *b, const void *c, float *a32, float *b32,
                          float *c32, size_t n, bool bf16, cudaStream_t st) {
    return bf16 ? to_f32_impl<__nv_bfloat16>(a, b, c, a32, b32, c32, n, st)
                : to_f32_impl<float>(a, b, c, a32, b32, c32, n, st);
}

template <typename T, int D>
static cudaError_t combine_bwd_impl(const float *o_la, const float *o_nla, const void *dout,
                                    const float *w, float eps, float *do_la, float *do_nla,
                                    float *dw, float *Dsm, void *do16, void *dola16, void *dolag16,
                                    const float *Gd, float scale_la, const int32_t *gsc, Shape s,
                                    cudaStream_t st, int G) {
    const size_t rows = (size_t)s.B * s.L * s.H;
    constexpr int kRowsPerBlock = (kThreads / 32) * (32 / (D / 4));
    combine_bwd_kernel<T, D><<<(unsigned)((rows + kRowsPerBlock - 1) / kRowsPerBlock), kThreads, 0, st>>>(
        o_la, o_nla, (const T *)dout, w, eps, do_la, do_nla, dw, Dsm, (__half *)do16, (__half *)dola16,
        (__half *)dolag16, Gd, scale_la, gsc, G, s.B, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_dout_amax(const void *dout, size_t n, bool bf16, int32_t *status, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(status + kGradAmaxWord, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return e;
    const size_t n4 = n / 4;
    const unsigned blocks = (unsigned)((n4 + 255) / 256 < 1184 ? (n4 + 255) / 256 : 1184);
    if (bf16) dout_amax_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16 *)dout, n4, status);
    else dout_amax_kernel<float><<<blocks, 256, 0, st>>>((const float *)dout, n4, status);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_combine_bwd(const float *o_la, const float *o_nla, const void *dout,
                               const float *w, float eps, float *do_la, float *do_nla, float *dw,
                               float *Dsm, void *do16, void *dola16, void *dolag16, const float *Gd,
                               float scale_la, const int32_t *gsc, Shape s, cudaStream_t st, int G) {
    if (G < 1 || s.d % (32 * G) != 0) return cudaErrorInvalidValue;
    if (s.bf16) {
        if (s.d == 128) return combine_bwd_impl<__nv_bfloat16, 128>(o_la, o_nla, dout, w, eps, do_la, do_nla, dw, Dsm, do16, dola16, dolag16, Gd, scale_la, gsc, s, st, G);
        return combine_bwd_impl<__nv_bfloat16, 64>(o_la, o_nla, dout, w, eps, do_la, do_nla, dw, Dsm, do16, dola16, dolag16, Gd, scale_la, gsc, s, st, G);
    }
    if (s.d == 128) return combine_bwd_impl<float, 128>(o_la, o_nla, dout, w, eps, do_la, do_nla, dw, Dsm, do16, dola16, dolag16, Gd, scale_la, gsc, s, st, G);
    return combine_bwd_impl<float, 64>(o_la, o_nla, dout, w, eps, do_la, do_nla, dw, Dsm, do16, dola16, dolag16, Gd, scale_la, gsc, s, st, G);
}

template <int D, int G = 1>
static cudaError_t softmax_bwd_impl(const float *q32, const float *k_sm32, const float *v_sm32,
                                    int cap, const int32_t *sm_idx, const int32_t *pre,
                                    const float *do_nla, const float *lse, const float *Dsm,
                                    float scale_sm, float *dq_sm, float *dk_sm, float *dv_sm,
                                    float *dmask, Shape s, cudaStream_t st) {
    const size_t smem_q = sizeof(float) * (2 * kC * D + 2 * 32 * (D + 1) + 32);
    const size_t smem_k = sizeof(float) * (2 * 32 * (D + 1) + 2 * kC * D + 2 * kC * 33 + 2 * kC + 32);
    cudaError_t e = set_smem(softmax_bwd_dq_kernel<D, G>, smem_q);
    if (e != cudaSuccess) return e;
    e = set_smem(softmax_bwd_dkv_kernel<D, G>, smem_k);
    if (e != cudaSuccess) return e;
    dim3 gq(s.L / kC, s.B * s.H * G);
    softmax_bwd_dq_kernel<D, G><<<gq, kThreads, smem_q, st>>>(q32, k_sm32, v_sm32, cap, sm_idx, pre,
                                                           do_nla, lse, Dsm, scale_sm, dq_sm, s.L, s.H);
    count_launch();
    dim3 gk((cap + 31) / 32, s.B * s.H * G);
    softmax_bwd_dkv_kernel<D, G><<<gk, kThreads, smem_k, st>>>(q32, k_sm32, v_sm32, cap, sm_idx, pre,
                                                            do_nla, lse, Dsm, scale_sm, dk_sm, dv_sm,
                                                            dmask, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_softmax_bwd(const float *q32, const float *k_sm32, const float *v_sm32, int cap,
                               const int32_t *sm_idx, const int32_t *sm_chunk_prefix,
                               const float *do_nla, const float *lse, const float *Dsm,
                               float scale_sm, float *dq_sm, float *dk_sm, float *dv_sm, Shape s,
                               cudaStream_t st, float *dmask, int G) {
    if (G > 1) {      // grouped softmax heads: slices of 32 or 64 columns
#define NATSL_GROUPED(DS, GG)                                                                                 \
        if (s.d == DS * GG && G == GG)                                                                        \
            return softmax_bwd_impl<DS, GG>(q32, k_sm32, v_sm32, cap, sm_idx, sm_chunk_prefix, do_nla, lse, Dsm, \
                                            scale_sm, dq_sm, dk_sm, dv_sm, dmask, s, st)
        NATSL_GROUPED(32, 2);
        NATSL_GROUPED(64, 2);
        NATSL_GROUPED(32, 4);
#undef NATSL_GROUPED
        return cudaErrorInvalidValue;
    }
    if (s.d == 128) return softmax_bwd_impl<128>(q32, k_sm32, v_sm32, cap, sm_idx, sm_chunk_prefix, do_nla, lse, Dsm, scale_sm, dq_sm, dk_sm, dv_sm, dmask, s, st);
    return softmax_bwd_impl<64>(q32, k_sm32, v_sm32, cap, sm_idx, sm_chunk_prefix, do_nla, lse, Dsm, scale_sm, dq_sm, dk_sm, dv_sm, dmask, s, st);
}

template <int D, int G = 1>
static cudaError_t own_block_impl(const float *q32, const float *k32, const float *v32, const float *do_nla,
                                  const float *lse, const float *Dsm, const uint8_t *route, float scale_sm,
                                  float *dq_sm, float *dk_x, float *dv_x, const int32_t *gsc, Shape s,
                                  cudaStream_t st) {
    const size_t smem = sizeof(float) * (4 * kC * (D + 1) + 2 * kC * (kC + 1));
    cudaError_t e = set_smem(softmax_bwd_own_block_simt_kernel<D, G>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(s.L / kC, s.B * s.H * G);
    softmax_bwd_own_block_simt_kernel<D, G><<<grid, kThreads, smem, st>>>(q32, k32, v32, do_nla, lse, Dsm, route,
                                                                      scale_sm, dq_sm, dk_x, dv_x, gsc, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_softmax_bwd_own_block_simt(const float *q32, const float *k32, const float *v32,
                                              const float *do_nla, const float *lse, const float *Dsm,
                                              const uint8_t *route, float scale_sm, float *dq_sm,
                                              float *dk_x, float *dv_x, const int32_t *gsc, Shape s,
                                              cudaStream_t st, int G) {
    if (G > 1) {
#define NATSL_GROUPED(DS, GG)                                                                               \
        if (s.d == DS * GG && G == GG)                                                                      \
            return own_block_impl<DS, GG>(q32, k32, v32, do_nla, lse, Dsm, route, scale_sm, dq_sm, dk_x, dv_x, \
                                          gsc, s, st)
        NATSL_GROUPED(32, 2);
        NATSL_GROUPED(64, 2);
        NATSL_GROUPED(32, 4);
#undef NATSL_GROUPED
        return cudaErrorInvalidValue;
    }
    if (s.d == 128) return own_block_impl<128>(q32, k32, v32, do_nla, lse, Dsm, route, scale_sm, dq_sm, dk_x, dv_x, gsc, s, st);
    return own_block_impl<64>(q32, k32, v32, do_nla, lse, Dsm, route, scale_sm, dq_sm, dk_x, dv_x, gsc, s, st);
}

template <int D>
static cudaError_t rscan_impl(const float *q32, const float *k32, const float *Gcum, const float *W,
                              const float *P, const float *do_la, const float *chunk_states,
                              float scale_la, float *dUt, float *dS_c, float *gS,
                              const float *dstate_out, float *dstate_in, const uint8_t *block_route, Shape s,
                              cudaStream_t st) {
    const size_t smem = sizeof(float) * (D * kDvs + 3 * kC * (D + 1) + kC * (kC + 1) +
                                         2 * kC * (kDvs + 1) + kC + 8);
    cudaError_t e = set_smem(gdn_rscan_kernel<D>, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(D / kDvs, s.B * s.H);
    gdn_rscan_kernel<D><<<grid, kThreads, smem, st>>>(q32, k32, Gcum, W, P, do_la, chunk_states,
                                                      scale_la, dUt, dS_c, gS, dstate_out, dstate_in, block_route,
                                                      s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_rscan(const float *q32, const float *k32, const float *Gcum, const float *W,
                             const float *P, const float *do_la, const float *chunk_states,
                             float scale_la, float *dUt, float *dS_c, float *gS,
                             const float *dstate_out, float *dstate_in, Shape s, cudaStream_t st,
                             const uint8_t *block_route) {
    if (s.d == 128)
        return rscan_impl<128>(q32, k32, Gcum, W, P, do_la, chunk_states, scale_la, dUt, dS_c, gS, dstate_out, dstate_in, block_route, s, st);
    return rscan_impl<64>(q32, k32, Gcum, W, P, do_la, chunk_states, scale_la, dUt, dS_c, gS, dstate_out, dstate_in, block_route, s, st);
}

cudaError_t launch_gdn_tsolve(const float *Abar, const float *beta, const uint8_t *route,
                              const float *dW, const float *dUt, float *dKb, float *dVb, Shape s,
                              cudaStream_t st) {
    dim3 grid(s.L / kC, s.B * s.H);
    if (s.d == 128)
        gdn_tsolve_kernel<128><<<grid, kThreads, 0, st>>>(Abar, beta, route, dW, dUt, dKb, dVb, s.L, s.H);
    else
        gdn_tsolve_kernel<64><<<grid, kThreads, 0, st>>>(Abar, beta, route, dW, dUt, dKb, dVb, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_mask_scale(const float *M, const float *N, const float *Gcum, const float *beta,
                              const uint8_t *route, float scale_la, float *Mg, float *Ms, float *Ns,
                              Shape s, cudaStream_t st) {
    dim3 grid(s.L / kC, s.B * s.H);
    mask_scale_kernel<<<grid, kThreads, 0, st>>>(M, N, Gcum, beta, route, scale_la, Mg, Ms, Ns, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t assemble_impl(const AssembleArgs &a, void *dq, void *dk, void *dv, Shape s,
                                 cudaStream_t st) {
    const size_t rows = (size_t)s.B * s.L * s.H;
    gdn_assemble_kernel<T, D><<<(unsigned)((rows + 7) / 8), kThreads, 0, st>>>(
        a.q32, a.k32, a.v32, a.Gcum, a.beta, a.route, a.dQg, a.dKb, a.dVb, a.dKt, a.X1p, a.X2, a.X3,
        a.X4, a.dq_sm, a.dk_x, a.dv_x, a.scale_la, (T *)dq, (T *)dk, (T *)dv, a.dGrow, a.kappa, a.dbeta, s.B,
        s.L, s.H);
    count_launch();
    const int NC = s.L / kC;
    const size_t nch = (size_t)s.B * s.H * NC;
    dg_kernel<<<(unsigned)((nch + 127) / 128), 128, 0, st>>>(a.dGrow, a.kappa, a.gS, a.Gcum,
                                                            s.d / kDvs, a.dg, s.B, s.L, s.H);
    count_launch();
    if (a.no_scatter) return cudaGetLastError();   // (the retained tokens' gradients came in through dk_x, dv_x)
    constexpr int kRows = kThreads / (D / 4);
    dim3 grid((a.cap + kRows - 1) / kRows, s.B * s.H);
    scatter_sm_kernel<T, D><<<grid, kThreads, 0, st>>>(a.dk_sm, a.dv_sm, a.cap, a.sm_idx, a.sm_prefix,
                                                       (T *)dk, (T *)dv, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t finish_impl(const AssembleArgs &a, void *dk, void *dv, Shape s, cudaStream_t st,
                               bool with_dg) {
    const int NC = s.L / kC;
    const size_t nch = (size_t)s.B * s.H * NC;
    if (with_dg) {
        dg_kernel<<<(unsigned)((nch + 127) / 128), 128, 0, st>>>(a.dGrow, a.kappa, a.gS, a.Gcum,
                                                                s.d / kDvs, a.dg, s.B, s.L, s.H);
        count_launch();
    }
    constexpr int kRows = kThreads / (D / 4);
    dim3 grid((a.cap + kRows - 1) / kRows, s.B * s.H);
    scatter_sm_kernel<T, D><<<grid, kThreads, 0, st>>>(a.dk_sm, a.dv_sm, a.cap, a.sm_idx, a.sm_prefix,
                                                       (T *)dk, (T *)dv, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_tm(const float *Tinv, const float *dW, const float *dUt, const float *W, const float *U,
                          const float *dO, const float *Ut, const float *Gcum, const float *beta,
                          const uint8_t *route, float scale_la, float *dKb, float *dVb, float *Mg, float *Ms,
                          float *Ns, Shape s, cudaStream_t st) {
    const unsigned nch = (unsigned)(s.B * s.H * (s.L / kC));
    auto kernel = s.d == 128 ? gdn_tm_kernel<128> : gdn_tm_kernel<64>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTmSmem);
    if (e != cudaSuccess) return e;
    kernel<<<nch, kThreads, kTmSmem, st>>>(Tinv, dW, dUt, W, U, dO, Ut, Gcum, beta, route, scale_la, dKb, dVb, Mg,
                                          Ms, Ns, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t xassemble_impl(const AssembleArgs &a, const float *Mg, const float *Ms, const float *Ns,
                                  void *dq, void *dk, void *dv, Shape s, cudaStream_t st) {
    const int NC = s.L / kC;
    const size_t nch = (size_t)s.B * s.H * NC;
    cudaError_t e = cudaFuncSetAttribute(gdn_xassemble_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)kXaSmem);
    if (e != cudaSuccess) return e;
    gdn_xassemble_kernel<T, D><<<(unsigned)nch, kThreads, kXaSmem, st>>>(
        a.q32, a.k32, a.v32, a.Gcum, a.beta, a.route, a.dQg, a.dKb, a.dVb, a.dKt, Mg, Ms, Ns, a.dq_sm, a.dk_x,
        a.dv_x, a.scale_la, (T *)dq, (T *)dk, (T *)dv, a.dGrow, a.kappa, a.dbeta, s.L, s.H);
    count_launch();
    dg_kernel<<<(unsigned)((nch + 127) / 128), 128, 0, st>>>(a.dGrow, a.kappa, a.gS, a.Gcum,
                                                            s.d / kDvs, a.dg, s.B, s.L, s.H);
    count_launch();
    if (a.no_scatter) return cudaGetLastError();
    constexpr int kRows = kThreads / (D / 4);
    dim3 grid((a.cap + kRows - 1) / kRows, s.B * s.H);
    scatter_sm_kernel<T, D><<<grid, kThreads, 0, st>>>(a.dk_sm, a.dv_sm, a.cap, a.sm_idx, a.sm_prefix,
                                                       (T *)dk, (T *)dv, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_gdn_xassemble(const AssembleArgs &a, const float *Mg, const float *Ms, const float *Ns,
                                 void *dq, void *dk, void *dv, Shape s, cudaStream_t st) {
    if (s.bf16) {
        if (s.d == 128) return xassemble_impl<__nv_bfloat16, 128>(a, Mg, Ms, Ns, dq, dk, dv, s, st);
        return xassemble_impl<__nv_bfloat16, 64>(a, Mg, Ms, Ns, dq, dk, dv, s, st);
    }
    if (s.d == 128) return xassemble_impl<float, 128>(a, Mg, Ms, Ns, dq, dk, dv, s, st);
    return xassemble_impl<float, 64>(a, Mg, Ms, Ns, dq, dk, dv, s, st);
}

cudaError_t launch_gdn_finish(const AssembleArgs &a, void *dk, void *dv, Shape s, cudaStream_t st,
                              bool with_dg) {
    if (s.bf16) {
        if (s.d == 128) return finish_impl<__nv_bfloat16, 128>(a, dk, dv, s, st, with_dg);
        return finish_impl<__nv_bfloat16, 64>(a, dk, dv, s, st, with_dg);
    }
    if (s.d == 128) return finish_impl<float, 128>(a, dk, dv, s, st, with_dg);
    return finish_impl<float, 64>(a, dk, dv, s, st, with_dg);
}

cudaError_t launch_gdn_assemble(const AssembleArgs &a, void *dq, void *dk, void *dv, Shape s,
                                cudaStream_t st) {
    if (s.bf16) {
        if (s.d == 128) return assemble_impl<__nv_bfloat16, 128>(a, dq, dk, dv, s, st);
        return assemble_impl<__nv_bfloat16, 64>(a, dq, dk, dv, s, st);
    }
    if (s.d == 128) return assemble_impl<float, 128>(a, dq, dk, dv, s, st);
    return assemble_impl<float, 64>(a, dq, dk, dv, s, st);
}

}  // namespace natsl

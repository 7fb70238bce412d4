// Backward of the softmax branch through a query's own block under block-level routing
// (Section 4.1: both operations compute the inner-chunk correlations; Section 4.2: ds = p (dp -
// <do, o>)).  A query in a linear block reads, besides the retained tokens of earlier softmax
// blocks (handled by the kernels over the compacted K/V), the causal part of its own block of 64
// tokens.  This kernel adds that part: one CTA per linear block,
//   p_ij = exp(scale q_i k_j - lse_i),  ds_ij = p_ij (do_i v_j - D_i)        (j <= i, same block)
//   dq_i += scale sum_j ds_ij k_j;  dk_j = scale sum_i ds_ij q_i;  dv_j = sum_i p_ij do_i,
// with lse_i and D_i = <do_i, o_i> of the whole softmax row.  The tokens of a linear block have no
// other softmax-branch gradient, so dk_j, dv_j are written, not accumulated.  fp32 on CUDA cores:
// a 64 x 64 x d problem per block.
#include "common.cuh"
#include "natsl_internal.h"

namespace natsl {

namespace {

constexpr int kOwnThreads = 256;

template <int D>
__global__ void __launch_bounds__(kOwnThreads)
softmax_bwd_own_block_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k,
                             const __nv_bfloat16 *__restrict__ v, const float *__restrict__ do_nla,
                             const float *__restrict__ lse, const float *__restrict__ Dsm,
                             const uint8_t *__restrict__ route, float scale_sm,
                             float *__restrict__ dq_sm, float *__restrict__ dk_x,
                             float *__restrict__ dv_x, int L, int H) {
    constexpr int kLd = D + 1;
    extern __shared__ float sm[];
    float *Qs = sm, *Ks = Qs + kC * kLd, *Vs = Ks + kC * kLd, *Os = Vs + kC * kLd;   // [64][D+1]
    float *Ps = Os + kC * kLd, *Ss = Ps + kC * (kC + 1);                             // [64][65]: p, ds
    const int c = blockIdx.x, bh = blockIdx.y, b = bh / H, h = bh % H;
    const size_t tok0 = ((size_t)b * L + (size_t)c * kC) * H + h;
    if (route[tok0]) return;                       // a softmax block: its tokens are among the retained ones
    const size_t ts = (size_t)H * D;
    const int tid = threadIdx.x;
    for (int idx = tid; idx < kC * D; idx += kOwnThreads) {
        const int r = idx / D, cc = idx % D;
        const size_t off = tok0 * D + (size_t)r * ts + cc;
        Qs[r * kLd + cc] = __bfloat162float(q[off]);
        Ks[r * kLd + cc] = __bfloat162float(k[off]);
        Vs[r * kLd + cc] = __bfloat162float(v[off]);
        Os[r * kLd + cc] = do_nla[off];
    }
    __syncthreads();
    {   // p and ds: thread (i, j mod 4)
        const int i = tid >> 2;
        const float lse_i = lse[(size_t)bh * L + c * kC + i], D_i = Dsm[(size_t)bh * L + c * kC + i];
        for (int j = tid & 3; j < kC; j += 4) {
            float pij = 0.f, ds = 0.f;
            if (j <= i) {
                float s = 0.f, dp = 0.f;
#pragma unroll 8
                for (int x = 0; x < D; ++x) {
                    s = fmaf(Qs[i * kLd + x], Ks[j * kLd + x], s);
                    dp = fmaf(Os[i * kLd + x], Vs[j * kLd + x], dp);
                }
                pij = __expf(scale_sm * s - lse_i);
                ds = scale_sm * pij * (dp - D_i);
            }
            Ps[i * (kC + 1) + j] = pij;
            Ss[i * (kC + 1) + j] = ds;
        }
    }
    __syncthreads();
    // thread (row, 16 columns): dq of query `row`; dk, dv of key `row`
    const int row = tid >> 2, c0 = (tid & 3) * (D / 4);
    constexpr int kPer = D / 4;
    float aq[kPer], ak[kPer], av[kPer];
#pragma unroll
    for (int x = 0; x < kPer; ++x) { aq[x] = 0.f; ak[x] = 0.f; av[x] = 0.f; }
    for (int m = 0; m < kC; ++m) {
        const float ds_rm = Ss[row * (kC + 1) + m];     // query row, key m
        const float ds_mr = Ss[m * (kC + 1) + row];     // query m, key row
        const float p_mr = Ps[m * (kC + 1) + row];
#pragma unroll
        for (int x = 0; x < kPer; ++x) {
            aq[x] = fmaf(ds_rm, Ks[m * kLd + c0 + x], aq[x]);
            ak[x] = fmaf(ds_mr, Qs[m * kLd + c0 + x], ak[x]);
            av[x] = fmaf(p_mr, Os[m * kLd + c0 + x], av[x]);
        }
    }
    const size_t off = tok0 * D + (size_t)row * ts + c0;
#pragma unroll
    for (int x = 0; x < kPer; x += 4) {
        float4 cur = *reinterpret_cast<const float4 *>(dq_sm + off + x);
        cur.x += aq[x]; cur.y += aq[x + 1]; cur.z += aq[x + 2]; cur.w += aq[x + 3];
        *reinterpret_cast<float4 *>(dq_sm + off + x) = cur;
        *reinterpret_cast<float4 *>(dk_x + off + x) = make_float4(ak[x], ak[x + 1], ak[x + 2], ak[x + 3]);
        *reinterpret_cast<float4 *>(dv_x + off + x) = make_float4(av[x], av[x + 1], av[x + 2], av[x + 3]);
    }
}

}  // namespace

cudaError_t launch_softmax_bwd_own_block(const void *q, const void *k, const void *v,
                                         const float *do_nla, const float *lse, const float *Dsm,
                                         const uint8_t *route, float scale_sm, float *dq_sm,
                                         float *dk_x, float *dv_x, Shape s, cudaStream_t st) {
    if (s.d != 64 || !s.bf16) return cudaErrorInvalidValue;
    constexpr int D = 64;
    const size_t smem = sizeof(float) * (4 * kC * (D + 1) + 2 * kC * (kC + 1));
    cudaError_t e = cudaFuncSetAttribute(softmax_bwd_own_block_kernel<D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid(s.L / kC, s.B * s.H);
    softmax_bwd_own_block_kernel<D><<<grid, kOwnThreads, smem, st>>>(
        (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, do_nla, lse, Dsm,
        route, scale_sm, dq_sm, dk_x, dv_x, s.L, s.H);
    count_launch();
    return cudaGetLastError();
}

}  // namespace natsl

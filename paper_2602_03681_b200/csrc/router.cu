// Attention score layer (Section 4.1, the score equation and the arg max that follows it): for
// every chunk of C = 64 tokens the mean of the chunk's input rows, a linear map to one score per
// operation and head, and the operation with the higher score as the chunk's route.
//
// HBM-bound: X [B, L, d_model] is read exactly once; the score weights (2 H rows of d_model) stay
// in L2.  One CTA per pair of chunks, half of its threads per chunk: a thread owns 16 bytes of
// every row of its chunk, so a warp reads 512 contiguous bytes per row, and sixteen rows are in
// flight per thread (the grid is small, so the bytes in flight have to come from the threads).
// The pooled rows are kept in shared memory; one warp per (head, operation) pair reads its weight
// row once and forms the dot products with both pooled rows; the route bytes of the chunks'
// tokens go out as one contiguous run.
#include "common.cuh"
#include "natsl_internal.h"

namespace natsl {

namespace {

constexpr int kScoreChunks = 2;                    // chunks per CTA
constexpr int kHalfThreads = 256;                  // threads per chunk
constexpr int kScoreThreads = kScoreChunks * kHalfThreads;
constexpr int kRowsInFlight = 16;

__device__ __forceinline__ void unpack16(const uint4 u, float (&x)[4], float) {
    x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
    x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
}
__device__ __forceinline__ void unpack16(const uint4 u, float (&x)[8], __nv_bfloat16) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

template <typename T>
__global__ void __launch_bounds__(kScoreThreads)
score_layer_kernel(const T *__restrict__ x, const float *__restrict__ w_score,
                   float *__restrict__ scores, uint8_t *__restrict__ route, int L, int Dm, int H) {
    constexpr int kE = 16 / (int)sizeof(T);          // elements per 16-byte piece
    extern __shared__ __align__(16) float pooled[];  // [kScoreChunks][Dm] pooled rows, then [kScoreChunks][2 H] scores
    float *sc = pooled + kScoreChunks * Dm;
    const int NC = L / kC, b = blockIdx.y, c0 = blockIdx.x * kScoreChunks;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = tid / kHalfThreads, ht = tid % kHalfThreads;       // chunk of the pair, thread within it
    const bool live = c0 + g < NC;                                   // the last pair may be half empty
    const T *xc = x + ((size_t)b * L + (size_t)(c0 + g) * kC) * Dm;

    for (int col = ht * kE; col < Dm; col += kHalfThreads * kE) {
        float acc[kE];
#pragma unroll
        for (int e = 0; e < kE; ++e) acc[e] = 0.f;
        if (live) {
            for (int i = 0; i < kC; i += kRowsInFlight) {
                uint4 u[kRowsInFlight];
#pragma unroll
                for (int j = 0; j < kRowsInFlight; ++j)
                    u[j] = *reinterpret_cast<const uint4 *>(xc + (size_t)(i + j) * Dm + col);
#pragma unroll
                for (int j = 0; j < kRowsInFlight; ++j) {
                    float v[kE];
                    unpack16(u[j], v, T());
#pragma unroll
                    for (int e = 0; e < kE; ++e) acc[e] += v[e];
                }
            }
        }
#pragma unroll
        for (int e = 0; e < kE; ++e) pooled[g * Dm + col + e] = acc[e] * (1.f / kC);
    }
    __syncthreads();
    for (int pair = warp; pair < 2 * H; pair += kScoreThreads / 32) {   // pair = 2 head + operation
        const float *wr = w_score + (size_t)pair * Dm;
        float s[kScoreChunks];
#pragma unroll
        for (int q = 0; q < kScoreChunks; ++q) s[q] = 0.f;
        for (int dd = lane * 4; dd < Dm; dd += 128) {
            const float4 wv = __ldg(reinterpret_cast<const float4 *>(wr + dd));
#pragma unroll
            for (int q = 0; q < kScoreChunks; ++q) {
                const float4 pv = *reinterpret_cast<const float4 *>(pooled + q * Dm + dd);
                s[q] = fmaf(wv.x, pv.x, fmaf(wv.y, pv.y, fmaf(wv.z, pv.z, fmaf(wv.w, pv.w, s[q]))));
            }
        }
#pragma unroll
        for (int q = 0; q < kScoreChunks; ++q) {
            const float t = warp_sum(s[q]);
            if (lane == 0 && c0 + q < NC) {
                sc[q * 2 * H + pair] = t;
                if (scores) scores[((size_t)b * NC + c0 + q) * H * 2 + pair] = t;
            }
        }
    }
    __syncthreads();
    // arg max over (linear, softmax); a tie keeps the first operation (linear)
    const int nch = min(kScoreChunks, NC - c0);
    uint8_t *rt = route + ((size_t)b * L + (size_t)c0 * kC) * H;
    for (int idx = tid; idx < nch * kC * H; idx += kScoreThreads) {
        const int q = idx / (kC * H), h = idx % H;
        rt[idx] = sc[q * 2 * H + 2 * h + 1] > sc[q * 2 * H + 2 * h] ? 1 : 0;
    }
}

template <typename T>
cudaError_t score_layer_impl(const void *x, const float *w_score, float *scores, uint8_t *route,
                             int d_model, Shape s, cudaStream_t st) {
    dim3 grid((s.L / kC + kScoreChunks - 1) / kScoreChunks, s.B);
    const size_t smem = (size_t)kScoreChunks * ((size_t)d_model + 2 * s.H) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(score_layer_kernel<T>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    score_layer_kernel<T><<<grid, kScoreThreads, smem, st>>>((const T *)x, w_score, scores, route, s.L,
                                                             d_model, s.H);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_layer(const void *x, const float *w_score, float *scores, uint8_t *route,
                               int d_model, Shape s, cudaStream_t st) {
    if (s.bf16) return score_layer_impl<__nv_bfloat16>(x, w_score, scores, route, d_model, s, st);
    return score_layer_impl<float>(x, w_score, scores, route, d_model, s, st);
}

}  // namespace natsl

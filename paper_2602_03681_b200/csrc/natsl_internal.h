// Host-side launch functions of the natsl kernels (one per .cu file), called by api.cu.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/natsl.h"

namespace natsl {

constexpr int kC = 64;  // chunk size (NAtS chunk = GDN chunk)

// Every launch_* function calls this once per kernel it enqueues.
void count_launch(int n = 1);

struct Shape {
    int B, H, L, d;
    bool bf16;
};

// compact.cu
cudaError_t launch_route_compact(const uint8_t *route, int32_t *sm_idx, int32_t *sm_chunk_prefix,
                                 int32_t *lin_idx, int32_t *n_lin, int32_t *sm_len, int B, int L,
                                 int H, cudaStream_t st);
cudaError_t launch_gather_kv(const void *k, const void *v, const int32_t *sm_idx,
                             const int32_t *sm_chunk_prefix, void *k_sm, void *v_sm, int32_t cap,
                             int32_t *status, Shape s, cudaStream_t st);

// fwd_simt.cu -- fp32 CUDA-core forward (exact-precision path; bf16 storage allowed)
size_t simt_prepare_smem(int d);
size_t simt_scan_smem(int d);
cudaError_t launch_gdn_prepare_simt(const void *q, const void *k, const void *v, const float *g,
                                    const float *beta, const uint8_t *route, float scale_la,
                                    float *W, float *U, float *P, Shape s, cudaStream_t st);
cudaError_t launch_gdn_scan_simt(const void *q, const void *k, const float *g, const float *W,
                                 const float *U, const float *P, float scale_la,
                                 const float *state_in, float *state_out, float *chunk_states,
                                 float *o_la, Shape s, cudaStream_t st);
cudaError_t launch_softmax_combine_simt(const void *q, const void *k_sm, const void *v_sm,
                                        int32_t cap, const int32_t *sm_idx,
                                        const int32_t *sm_chunk_prefix, const float *o_la,
                                        const float *w, float scale_sm, float eps, void *out,
                                        float *o_nla, float *lse, Shape s, cudaStream_t st);

// decode.cu
cudaError_t launch_decode_step(const void *q, const void *k, const void *v, const float *g,
                               const float *beta, const uint8_t *route, const float *w,
                               float *state, void *k_cache, void *v_cache, int32_t *cache_len,
                               int32_t cache_cap, void *out, float scale_la, float scale_sm,
                               float eps, int32_t *status, Shape s, cudaStream_t st);

}  // namespace natsl

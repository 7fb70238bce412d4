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

// Block-level routing (Section 4.1: one decision per block of C tokens, and both operations see
// the query's own block): the route bytes [B,L,H] and the layer's K and V, from which the softmax
// kernel reads the own block of a query in a linear block.  route == nullptr: token-level routing.
struct BlockRouting {
    const uint8_t *route;
    const void *k, *v;
};

// Grouped softmax heads and per-operation q/k normalisation (Section 4.3): G softmax heads per
// linear head, each a slice of d / G columns of the linear head's q, k, v; norm_eps >= 0: q and k are
// L2-normalised for the linear operation and RMS-normalised (per softmax head) for the softmax one,
// inside the kernels; norm_eps < 0: used as given.
struct HeadGroups {
    int G = 1;
    float norm_eps = -1.f;
};

// router.cu -- attention score layer: scores [B,L/C,H,2] (may be nullptr) and route [B,L,H]
cudaError_t launch_score_layer(const void *x, const float *w_score, float *scores, uint8_t *route,
                               int d_model, Shape s, cudaStream_t st);

// compact.cu  (block_status: where a route that changes inside a chunk is reported, or nullptr;
// base_in [B,H]: retained tokens already in the cache the call appends to, or nullptr for none;
// cap: rows per head of the cache sm_len describes -- the stored length is clamped to it; 0: none)
cudaError_t launch_route_compact(const uint8_t *route, int32_t *sm_idx, int32_t *sm_chunk_prefix,
                                 int32_t *lin_idx, int32_t *n_lin, int32_t *sm_len,
                                 const int32_t *base_in, int32_t *block_status, int cap, int B, int L,
                                 int H, cudaStream_t st);
cudaError_t launch_gather_kv(const void *k, const void *v, const int32_t *sm_idx,
                             const int32_t *sm_chunk_prefix, void *k_sm, void *v_sm, int32_t cap,
                             int32_t *status, Shape s, cudaStream_t st);

// fwd_simt.cu -- fp32 CUDA-core forward (exact-precision path; bf16 storage allowed)
size_t simt_prepare_smem(int d);
size_t simt_scan_smem(int d);
cudaError_t launch_gdn_prepare_simt(const void *q, const void *k, const void *v, const float *g,
                                    const float *beta, const uint8_t *route, float scale_la,
                                    float *W, float *U, float *P, float *Abar, float *Gcum, Shape s,
                                    cudaStream_t st);
cudaError_t launch_gdn_scan_simt(const void *q, const void *k, const float *g, const float *W,
                                 const float *U, const float *P, float scale_la,
                                 const float *state_in, float *state_out, float *chunk_states,
                                 float *Ut, float *o_la, const uint8_t *block_route, Shape s,
                                 cudaStream_t st);
cudaError_t launch_softmax_combine_simt(const void *q, const void *k_sm, const void *v_sm,
                                        int32_t cap, const int32_t *sm_idx,
                                        const int32_t *sm_chunk_prefix, const float *o_la,
                                        const float *w, float scale_sm, float eps, void *out,
                                        float *o_nla, float *lse, BlockRouting br, Shape s,
                                        cudaStream_t st, int G = 1);
// (G > 1: grouped softmax heads, fp32 storage only; see HeadGroups)
// fp32 storage: q, k [rows, d] -> L2-normalised rows (q_la, k_la) and rows with each of the G slices
// RMS-normalised (q_sm, k_sm)
cudaError_t launch_qk_norm_f32(const void *q, const void *k, bool bf16, float *q_la, float *k_la, float *q_sm,
                               float *k_sm, size_t rows, int d, int G, float norm_eps, cudaStream_t st);
// (q, k in fp32 or bf16 storage; q_sm, k_sm may be nullptr)
// Its backward, in place: dq (gradient w.r.t. the L2 copy) and dq_sm (w.r.t. the RMS copy) -> dq;
// dk (w.r.t. the L2 copy for a linear token, the RMS copy for a retained one) -> dk.
cudaError_t launch_qk_norm_bwd_f32(const void *q, const void *k, bool bf16, const uint8_t *route,
                                   const float *dq_la, const float *dq_sm, const float *dk_in,
                                   const float *dv_in, void *dq, void *dk, void *dv, size_t rows, int d, int G,
                                   float norm_eps, cudaStream_t st, const float *dk_sm = nullptr);
// (dk_sm given -- block-level routing, where every token's k reaches both operations: dk_in is the gradient
// w.r.t. the L2 copy and dk_sm the one w.r.t. the RMS copy, for every token, like q)
// (fp32 gradients in: dq_la, dq_sm, dk_in, and dv_in or nullptr; out in the storage type: dq, dk, and dv =
// dv_in converted when given.  In place is fine for fp32 storage: dq_la == dq, dk_in == dk.)

// softmax_tc.cu -- tensor-core softmax branch + combination (bf16 storage)
cudaError_t launch_gather_kv_tc(const void *k, const void *v, const int32_t *sm_idx,
                                const int32_t *sm_chunk_prefix, void *k_sm, void *v_sm, void *v16,
                                void *k16, int32_t cap, int32_t capv, bool appending, int32_t *status,
                                Shape s, cudaStream_t st, HeadGroups hg = HeadGroups{}, bool raw_k_sm = false);
// (hg.norm_eps >= 0: the keys are RMS-normalised per softmax head and stored as fp16 -- in k_sm and k16, or,
// with raw_k_sm, in k16 only while k_sm, a cache handed on to the decode step, keeps them as given)
cudaError_t launch_softmax_combine_tc(const void *q, const void *k_sm, const void *v16, int32_t cap,
                                      int32_t capv, const int32_t *sm_idx,
                                      const int32_t *sm_chunk_prefix, const void *o_la16,
                                      const int32_t *emit_flags, const float *w, float scale_sm,
                                      float eps, void *out, float *o_nla, float *lse, BlockRouting br,
                                      bool appending, int32_t *status, Shape s, cudaStream_t st,
                                      HeadGroups hg = HeadGroups{});
// (o_la16: the linear branch's read-out, o_laT [B,H,L/C,8,d,8] fp16; emit_flags: see ScanOut -- when given, the
// kernel is launched as a programmatic dependent of the kernel before it in the stream, the scan)
int sm_count();   // multiprocessors of the current device (cached per device)
// Bound of the device-side waits in units of 1024 cycles, 0 = the default (about two seconds);
// non-zero only after natsl_debug_set_wait_limit.  Every tensor-core kernel launch passes it on.
int debug_wait_kcycles();

// softmax_bwd_tc.cu -- tensor-core backward of the softmax branch (bf16 storage).  Qh is scratch
// for the fp16 copy of q [B,H,L,d]; dO16 the fp16 branch-output gradient [B,H,L,d]; k16, v16 the
// fp16 retained K/V [B,H,cap,d]; dq_sm is token-major [B,L,H,d], dk_sm / dv_sm compacted.
cudaError_t launch_softmax_bwd_tc(const void *q, void *Qh, const void *dO16, const void *k16,
                                  const void *v16, int cap, const int32_t *sm_idx,
                                  const int32_t *sm_chunk_prefix, const float *lse, const float *Dsm,
                                  float scale_sm, float *dq_sm, float *dk_sm, float *dv_sm,
                                  float *dmask, bool qh_ready, int32_t *status, Shape s, cudaStream_t st,
                                  cudaStream_t st_kv,    // st: query-side kernel, st_kv: key-side kernel
                                  HeadGroups hg = HeadGroups{});
// (hg.G = 2 at d = 128: softmax heads are column slices, lse / Dsm [B,H,G,L]; hg.norm_eps >= 0: Qh is
// written here as the slice-wise RMS-normalised q, k16 must hold the normalised keys already)

// gdn_tc.cu -- tensor-core chunkwise Gated DeltaNet (bf16 storage): intermediates in workspace
struct GdnTcWs {
    void *Qh, *Kh;   // fp16 copies of q, k              [B,H,L,d]
    void *Wt;        // W^T per chunk, fp16              [B,H,L/C,d,64]
    float *Ut;       // U^T per chunk, fp32, in 4-token pieces   [B,H,L/C,16,d,4]
    void *Ph;        // P per chunk, fp16                [B,H,L/C,64,64]
    float *Gd;       // per chunk: gamma_i (64), gamma_C / gamma_i (64), fp32   [B,H,L/C,128]
};
// Optional fp32 copies of the chunkwise quantities the backward needs (all may be null).
struct GdnTcExport {
    float *W, *U;    // token-major [B,L,H,d]
    float *P;        // [B,H,L/C,64,64]
    float *T;        // (I + A)^-1, [B,H,L/C,64,64]
    float *Gcum;     // in-chunk cumulative log decay [B,H,L]
    float *S_c;      // chunk-entry states [B,H,L/C,d,d]
    float *Ut;       // U~ = U - W S, token-major [B,L,H,d]
};
// norm_eps >= 0: q and k rows are L2-normalised as the tiles are converted (Section 4.3, HeadGroups)
cudaError_t launch_gdn_prepare_tc(const void *q, const void *k, const void *v, const float *g,
                                  const float *beta, const uint8_t *route, float scale_la,
                                  const GdnTcWs &ws, const GdnTcExport &ex, int32_t *status, Shape s,
                                  cudaStream_t st, float norm_eps = -1.f);
// Splitting the scan of one (batch, head) over several CTAs when there are few (batch, head)
// pairs.  The state recurrence S <- (gamma_C I - K~^T W) S + K~^T U is affine in S with a factor
// that acts on the key dimension only, so a segment of chunks maps its entry state S0 to
// M_seg S0 + B_seg, and the same scan kernel yields both parts: B_seg as the exit state of a run
// from S0 = 0, M_seg as the exit state of a run from S0 = I with U = 0.
//   mode 0: one CTA per (batch, head) over all chunks (state_in / state_out as given);
//   mode 1: two CTAs per (batch, head, segment), no outputs: B_seg -> incr, M_seg -> trans;
//   mode 2: one CTA per (batch, head, segment) from the entry state in `start`, with outputs;
//           the last segment writes state_out.
// incr, trans, start: [B*H, nseg, d, d] fp32.  Between modes 1 and 2 launch_scan_combine chains the
// segments: start[0] = state_in (or 0), start[s+1] = M_s start[s] + B_s.
struct ScanSegments {
    int mode, nseg, ncs;       // ncs = chunks per segment
    float *incr, *trans, *start;
};
// Where the scan's read-out goes: o_la16 = o_laT [B,H,L/C,8,d,8] fp16 always (one transposed tile per
// chunk: what the softmax kernel's epilogue reads), o_la32 the same in fp32 or nullptr, and emit_flags [B*H, L/C] (or nullptr): one counter
// per chunk, zeroed by the caller, that each of the eight row warps of the scan CTA raises by one
// (release) once its rows of the chunk are written, so that a kernel running beside the scan can
// consume o_la chunk by chunk.
struct ScanOut {
    void *o_la16;
    float *o_la32;
    int32_t *emit_flags;
};
constexpr int kScanRowWarps = 8;
cudaError_t launch_gdn_scan_tc(const GdnTcWs &ws, float scale_la, const float *state_in,
                               float *state_out, const ScanOut &out, const GdnTcExport &ex,
                               const ScanSegments &sg, const uint8_t *block_route, int32_t *status,
                               Shape s, cudaStream_t st);
cudaError_t launch_scan_combine(const float *state_in, const ScanSegments &sg, Shape s, cudaStream_t st);

// bwd_simt.cu -- fp32 CUDA-core backward
// A batched matrix operand: element (r, c) of batch (b, h, chunk) is
// p[b*sb + h*sh + chunk*sc + r*ld + c].
struct BMat {
    const float *p;
    long long sb, sh, sc;
    int ld;
};
// C = alpha * op(A) op(B) (+ C) per (batch, head, chunk); m, n multiples of 64, k of 16.
// mask: 0 none, 1 keep col <= row, 2 keep col < row (64x64 outputs).
cudaError_t launch_bgemm(bool ta, bool tb, int mask, BMat A, BMat B, BMat C, int m, int n, int k,
                         float alpha, bool accumulate, Shape s, cudaStream_t st);
cudaError_t launch_to_f32(const void *a, const void *b, const void *c, float *a32, float *b32,
                          float *c32, size_t n, bool bf16, cudaStream_t st);
// do16: optional fp16 copy of do_nla in [B,H,L,d] layout (tensor-core softmax backward).
// gsc: the status page holding max |dout| (see grad_scale in common.cuh), or nullptr for no scaling.
// With it the fp16 copies and Dsm are written times the scale.
cudaError_t launch_combine_bwd(const float *o_la, const float *o_nla, const void *dout,
                               const float *w, float eps, float *do_la, float *do_nla, float *dw,
                               float *Dsm, void *do16, void *dola16, void *dolag16, const float *Gd,
                               float scale_la, const int32_t *gsc, Shape s, cudaStream_t st, int G = 1);
// (G > 1: the softmax branch's output was normalised per slice of d / G columns; Dsm is [B,H,G,L])
// max |dout| (n elements) into word kGradAmaxWord of the status page (zeroed first)
cudaError_t launch_dout_amax(const void *dout, size_t n, bool bf16, int32_t *status, cudaStream_t st);
cudaError_t launch_softmax_bwd(const float *q32, const float *k_sm32, const float *v_sm32, int cap,
                               const int32_t *sm_idx, const int32_t *sm_chunk_prefix,
                               const float *do_nla, const float *lse, const float *Dsm,
                               float scale_sm, float *dq_sm, float *dk_sm, float *dv_sm, Shape s,
                               cudaStream_t st, float *dmask = nullptr, int G = 1);
// (dmask [B,H,cap] or nullptr: per retained key the sum of the mask gradients of Section 4.2)
// Block-level routing, fp32: the softmax branch's backward through the own block of the queries of a
// linear block (adds to dq_sm, writes the dk_x / dv_x rows of the linear blocks).  gsc: gradient
// scale of the tensor-core kernels that Dsm carries (nullptr: none).
cudaError_t launch_softmax_bwd_own_block_simt(const float *q32, const float *k32, const float *v32,
                                              const float *do_nla, const float *lse, const float *Dsm,
                                              const uint8_t *route, float scale_sm, float *dq_sm,
                                              float *dk_x, float *dv_x, const int32_t *gsc, Shape s,
                                              cudaStream_t st, int G = 1);
// (G > 1: slices of d / G columns, lse / Dsm [B,H,G,L]; q32, k32: the softmax operation's copies of q, k)
// dstate_out [B,H,d,d] (or nullptr: zero): the gradient the scan starts from, at the final state;
// dstate_in (or nullptr): receives what is left after the first chunk, the initial state's gradient.
cudaError_t launch_gdn_rscan(const float *q32, const float *k32, const float *Gcum, const float *W,
                             const float *P, const float *do_la, const float *chunk_states,
                             float scale_la, float *dUt, float *dS_c, float *gS,
                             const float *dstate_out, float *dstate_in, Shape s, cudaStream_t st,
                             const uint8_t *block_route = nullptr);
// Tensor-core reverse scan (gdn_bwd_tc.cu): dO16 / dOg16 are fp16 [B,H,L,d] copies of the read-out
// gradient and of scale_la gamma times it; outputs as launch_gdn_rscan (gS: slot 0 of each row).
cudaError_t launch_gdn_rscan_tc(const void *dO16, const void *dOg16, const GdnTcWs &ws,
                                const float *S_c, float *dUt, float *dS_c, float *gS,
                                const float *dstate_out, float *dstate_in,
                                const uint8_t *block_route, int32_t *status, Shape s, cudaStream_t st);
cudaError_t launch_gdn_tsolve(const float *Abar, const float *beta, const uint8_t *route,
                              const float *dW, const float *dUt, float *dKb, float *dVb, Shape s,
                              cudaStream_t st);
cudaError_t launch_mask_scale(const float *M, const float *N, const float *Gcum, const float *beta,
                              const uint8_t *route, float scale_la, float *Mg, float *Ms, float *Ns,
                              Shape s, cudaStream_t st);
struct AssembleArgs {
    const float *q32, *k32, *v32, *Gcum, *beta;
    const uint8_t *route;
    const float *dQg, *dKb, *dVb, *dKt, *X1p, *X2, *X3, *X4, *dq_sm, *dk_sm, *dv_sm, *gS;
    const int32_t *sm_idx, *sm_prefix;
    int cap;
    float scale_la;
    float *dGrow, *kappa, *dbeta, *dg;
    // block-level routing on the path with separate chunk-level products: route == nullptr (every token
    // takes part in the delta rule) and the softmax-branch dk, dv of every token, fp32 token-major
    const float *dk_x = nullptr, *dv_x = nullptr;
    bool no_scatter = false;     // the retained tokens' dk, dv are part of dk_x, dv_x (or handled by the caller)
};
// dq (all tokens), dk/dv (linear tokens from the GDN branch, retained tokens scattered from the
// compacted softmax-branch gradients), dbeta, dg.  Three kernels.
cudaError_t launch_gdn_assemble(const AssembleArgs &a, void *dq, void *dk, void *dv, Shape s,
                                cudaStream_t st);
// Tensor-core path (tf32 products), one kernel per chunk: dKb = Tinv^T dW, dVb = Tinv^T dU~ (written out),
// M = -strictly_lower(dKb W^T + dVb U^T), N = lower(dO U~^T), then Mg, Ms, Ns as launch_mask_scale forms them.
cudaError_t launch_gdn_tm(const float *Tinv, const float *dW, const float *dUt, const float *W, const float *U,
                          const float *dO, const float *Ut, const float *Gcum, const float *beta,
                          const uint8_t *route, float scale_la, float *dKb, float *dVb, float *Mg, float *Ms,
                          float *Ns, Shape s, cudaStream_t st);
// The same with the four products X1 = Mg K, X2 = Ms^T K, X3 = Ns K, X4 = Ns^T Q formed inside (tf32
// tensor-core products; a.X1p .. a.X4 are not read); s.bf16 says what dq, dk, dv are stored as.
cudaError_t launch_gdn_xassemble(const AssembleArgs &a, const float *Mg, const float *Ms, const float *Ns,
                                 void *dq, void *dk, void *dv, Shape s, cudaStream_t st);
// The last two of those kernels only (dg from the per-token sums, scatter of the retained tokens'
// dk, dv), for callers that formed dq, dk, dv of the linear tokens and the sums themselves.
cudaError_t launch_gdn_finish(const AssembleArgs &a, void *dk, void *dv, Shape s, cudaStream_t st,
                              bool with_dg = true);
// gdn_bwd_tc.cu: everything of the linear branch's backward that follows the reverse scan, fused
// per chunk (d = 64, bf16 storage): dq (with dq_sm added), dk, dv of the linear tokens, dg, dbeta.
cudaError_t launch_gdn_bwd_chunk(const void *q, const void *k, const void *v, const float *dO,
                                 const float *dUt, const float *Ut, const float *S_c, const float *dS_c,
                                 const float *Tinv, const void *Wt, const float *Up, const float *Gcum,
                                 const float *beta, const uint8_t *route, const float *dq_sm,
                                 float scale_la, void *dq, void *dk, void *dv, float *dg,
                                 float *dbeta, bool block, const float *dk_x, const float *dv_x,
                                 float *kap_c, Shape s, cudaStream_t st);
// (kap_c [B,H,L/C]: the chunk sums of kappa, or kappa_tok [B,H,L]: kappa per token, summed here)
cudaError_t launch_dscore(const uint8_t *route, const int32_t *sm_chunk_prefix, const float *dmask,
                          const float *kap_c, const float *kappa_tok, int cap, float *dscore, Shape s,
                          cudaStream_t st, int G = 1);
// (G > 1: dmask is [B,H,G,cap], summed over the group's softmax heads)

// block-level routing: softmax-branch backward through the own block of the queries of a linear
// block (adds to dq_sm, writes the dk_x / dv_x rows of the linear blocks); do16: fp16 [B,H,L,d]
cudaError_t launch_softmax_bwd_own_block(const void *q, const void *k, const void *v,
                                         const void *do16, const float *lse, const float *Dsm,
                                         const uint8_t *route, float scale_sm, float *dq_sm,
                                         float *dk_x, float *dv_x, const int32_t *gsc, Shape s,
                                         cudaStream_t st, int G = 1, const float *qn = nullptr,
                                         const float *kn = nullptr);
// (softmax heads of 64 columns: d = 64, or G = 2 at d = 128 with lse / Dsm [B,H,G,L]; qn, kn: fp32 copies
// holding the softmax operation's normalised q, k [B,L,H,d], read instead of q, k)

// decode.cu
constexpr int kDecodeParts = 4;   // CTAs that share the retained K/V of one (sequence, head)
// Bytes of workspace of a decode step: status word, per-head tickets, partial softmax results and
// linear read-outs.  Zero-filled once by the caller; the kernel leaves the tickets at zero.
size_t decode_workspace_bytes(int B, int H, int d);
cudaError_t launch_decode_step(const void *q, const void *k, const void *v, const float *g,
                               const float *beta, const uint8_t *route, const float *w,
                               float *state, void *k_cache, void *v_cache, int32_t *cache_len,
                               int32_t cache_cap, void *out, float scale_la, float scale_sm,
                               float eps, void *ws, Shape s, cudaStream_t st, HeadGroups hg = HeadGroups{});
cudaError_t launch_decode_block_end(const uint8_t *route_block, const float *g_block, float *state,
                                    float *state_start, int32_t *cache_len, int32_t block_len,
                                    void *ws, Shape s, cudaStream_t st);

}  // namespace natsl

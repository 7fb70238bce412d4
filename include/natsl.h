/*
 * natsl.h -- C ABI of the B200 (sm_100a) hybrid attention layer of NAtS-L.
 *
 * The layer, per (batch, head), for tokens i = 0..L-1 with route r_i in {0,1}
 * (1 = softmax token, K/V retained; 0 = linear token, folded into the state):
 *
 *   linear branch  (Section 4.3, Gated DeltaNet equation; decay on every token, the
 *                   decay-update equation of the same section; update only for linear tokens,
 *                   Section 4.1 case equation for the chunk state):
 *       Sbar = exp(g_i) S ;  S = r_i ? Sbar : Sbar + beta_i k_i^T (v_i - k_i Sbar)
 *       o_la_i = scale_la * q_i S
 *   softmax branch (Section 4.1, O_nla equation with column mask M^nla):
 *       o_nla_i = sum_{j<=i, r_j=1} softmax_j(scale_sm * q_i.k_j) v_j    (0 if no such j)
 *   combination    (Section 4.3, Norm equation):
 *       out_i = w_nla_i RMSnorm(o_nla_i) + w_la_i RMSnorm(o_la_i),
 *       RMSnorm(x) = x / sqrt(mean_d(x^2) + eps)
 *
 * Every pointer below is a DEVICE pointer unless it says "host".  The caller owns all
 * buffers and the stream; the library allocates no device memory and keeps no per-call state.
 * Calls are asynchronous and ordered on `stream` (a cudaStream_t passed as void*; NULL = default
 * stream) like any other work of that stream.  What the library does own, per device and created
 * on the first forward or backward call there that may use it: one non-blocking stream and two
 * events, on which stages that do not depend on each other run beside the caller's stream (forked
 * from it and joined back into it within the call), and one process-wide mutex that covers the
 * enqueue of such a call, because the two events are shared.  NATSL_SINGLE_STREAM and
 * natsl_hybrid_fwd_static use none of this.  The device of `stream` and of all tensors must be
 * the current device of the calling thread.
 * All tensors are dense, row-major, innermost dimension contiguous, in the shapes given (no
 * strides are taken: a caller with another layout makes a contiguous copy).  Base pointers of
 * q,k,v,out,dout,dq,dk,dv, the caches and the workspace must be 16-byte aligned.
 *
 * Precision of the default path for NATSL_BF16 (tcgen05 tensor cores): q, k, v are used as
 * given; every computed tensor-core operand is held in fp16 with fp32 accumulation, and q, k, v
 * are converted to fp16 on the way, so their magnitudes must stay below 65504 (values below
 * 6e-8 in magnitude flush to zero).  NATSL_FORCE_SIMT selects fp32 arithmetic throughout.
 *
 * Return value: NATSL_OK or a negative natsl_status.  Arguments are validated on the host
 * before anything is launched; an invalid call launches nothing.  Conditions only the
 * device can see (decode cache full) are written to a status word that
 * natsl_device_status() reads back; kernels never trap.
 */
#ifndef NATSL_H_
#define NATSL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum natsl_status {
    NATSL_OK = 0,
    NATSL_ERR_NULL = -1,        /* a required pointer is NULL */
    NATSL_ERR_SHAPE = -2,       /* B,H,L <= 0, L % C != 0, d not in {64,128}, C != 64 */
    NATSL_ERR_DTYPE = -3,       /* dtype not NATSL_F32 / NATSL_BF16 */
    NATSL_ERR_ALIGN = -4,       /* a tensor base is not 16-byte aligned */
    NATSL_ERR_WORKSPACE = -5,   /* workspace NULL or smaller than natsl_workspace_size */
    NATSL_ERR_CUDA = -6,        /* a launch or runtime call failed */
    NATSL_ERR_CACHE_FULL = -7,  /* decode: a retained-KV cache has no room (device-detected) */
    NATSL_ERR_UNSUPPORTED = -8, /* valid request this build does not implement */
    NATSL_ERR_TOO_LARGE = -9,   /* natsl_hybrid_fwd_static: problem needs more than the built-in scratch */
    NATSL_ERR_TIMEOUT = -10,    /* a bounded device-side wait expired (device-detected); kernel drained */
    NATSL_ERR_ROUTE = -11       /* block-level routing: route changes inside a block, or a block end
                                   without the block's cache entries (device-detected) */
} natsl_status;

enum { NATSL_F32 = 0, NATSL_BF16 = 1 };
enum { NATSL_OP_FWD = 0, NATSL_OP_BWD = 1, NATSL_OP_DECODE = 2, NATSL_OP_COMPACT = 3 };

/* flags */
enum {
    NATSL_FORCE_SIMT = 1u << 0,  /* use the fp32 CUDA-core kernels even for bf16 tensors (the
                                    default for bf16 is the tcgen05 tensor-core path) */
    NATSL_SINGLE_PASS_SCAN = 1u << 1,  /* forward, tensor-core path: keep the scan over the chunks of a
                                    (batch, head) in one CTA even when B*H is small.  By default
                                    such calls split the chunks into segments that run in
                                    parallel (a second run per segment yields the segment's
                                    state transition, a small kernel chains the segments); the
                                    results agree to rounding */
    NATSL_BLOCK_ROUTING = 1u << 2,     /* forward (both paths), backward: block-level routing, the paper's
                                    default (Section 4.1, paragraph on intra-chunk correlations;
                                    Section 4.3, chunk size = GDN chunk size).  `route` holds one
                                    decision per block of C = 64 tokens, repeated over the block's
                                    tokens.  The decision is known only when the block is complete,
                                    so both operations treat the tokens of the query's own block as
                                    theirs: the softmax branch reads the retained tokens of earlier
                                    blocks plus the causal part of the own block; the linear branch
                                    reads the state committed by earlier linear blocks and runs the
                                    delta rule over the own block, whose update is committed to the
                                    state only if the block is linear (a softmax block leaves the
                                    decay alone).  state_out, k_sm, v_sm, sm_len hold what is kept
                                    after the last block.  A route that changes inside a block is
                                    reported as NATSL_ERR_ROUTE by natsl_device_status.  Backward:
                                    built on every path (bf16 storage with d = 64: fused per
                                    chunk; d = 128 and fp32 storage: the chunk-level products as
                                    separate kernels).  Generation: route 2 in
                                    natsl_decode_step and natsl_decode_block_end (no flag needed) */
    NATSL_APPEND_CACHE = 1u << 3,      /* forward, tensor-core path: prefill in pieces.  p->k_sm, p->v_sm,
                                    p->sm_len (required) are read AND written: the cache already
                                    holds sm_len[b,h] retained tokens of earlier pieces of the same
                                    sequences; the softmax branch of this piece reads them as
                                    earlier tokens, and the piece's own retained tokens are
                                    appended behind them (sm_len grows; NATSL_ERR_CACHE_FULL in the
                                    status word if sm_cap would be exceeded).  Together with
                                    p->state_in = the previous piece's state_out this continues a
                                    sequence exactly where the last call stopped (Section 4.1: the
                                    two hidden states kept during generation are the linear state
                                    and the KV cache).  natsl_workspace_size depends on the flag
                                    and on p->sm_cap.  Backward: NATSL_ERR_UNSUPPORTED */
    NATSL_SINGLE_STREAM = 1u << 4,     /* forward and backward, tensor-core path: launch everything on
                                    the caller's stream.  By default stages that do not depend on
                                    each other (route compaction + gather beside the linear branch's
                                    prepare kernel; in the backward also the reverse scan beside the
                                    softmax branch's backward) run side by side, one of them on a
                                    stream the library creates once per device, forked from and
                                    joined to the caller's stream with events, so the call is still
                                    ordered like any other work on that stream.  Also implied by
                                    p->stage_events.  natsl_hybrid_fwd_static always sets it.  The
                                    forward then also runs its kernels strictly one after the other
                                    (by default the softmax branch starts while the scan of the linear
                                    branch is still running and picks its read-out up chunk by chunk) */
    NATSL_SAVE_FOR_BWD = 1u << 5,      /* forward of a training step: `ws` is a BACKWARD workspace
                                    (natsl_workspace_size(p, NATSL_OP_BWD) bytes).  The forward runs in
                                    it and leaves there what the backward needs (chunk-entry states,
                                    the chunkwise operands, log-sum-exp, the raw branch outputs), so
                                    that natsl_hybrid_bwd with NATSL_SAVED_FWD on the same inputs, the
                                    same p and the same ws starts at the gradients.  Produces `out`
                                    and p->state_out; the other optional outputs, NATSL_APPEND_CACHE
                                    and p->stage_events are NATSL_ERR_UNSUPPORTED with it */
    NATSL_SAVED_FWD = 1u << 6,         /* backward: `ws` holds such a forward (same inputs, same p apart
                                    from this flag).  One backward per saved forward: the backward
                                    reuses some of the saved buffers for its own results */
    NATSL_QK_NORM = 1u << 7            /* forward and backward: q and k are normalised inside the kernels, differently
                                    for the two operations that share them (Section 4.3): L2 over the
                                    d columns of the head for the linear operation,
                                    x / sqrt(sum x^2 + norm_eps), and RMS per softmax head for the
                                    softmax operation, x / sqrt(mean x^2 + norm_eps), no gain.
                                    Without the flag q and k are used as given.  See p->G for what
                                    is built */
};

typedef struct natsl_params {
    int32_t B, H, L, d;     /* d = d_k = d_v in {64, 128}; L % C == 0; decode ignores L */
    int32_t C;              /* chunk size; must be 64 (Section 5: NAtS chunk = GDN chunk = 64) */
    int32_t dtype;          /* storage type of q,k,v,out,dout,dq,dk,dv and the KV caches */
    float scale_la;         /* logit scale of the linear read-out */
    float scale_sm;         /* logit scale of the softmax branch; > 0 on the tensor-core path */
    float eps;              /* RMS-norm epsilon, > 0 */
    uint32_t flags;
    const float *w;         /* [B,L,H,2] (decode: [B,H,2]) = (w_nla, w_la); NULL => (0.5, 0.5) */
    const float *state_in;  /* [B,H,d,d] fp32, row = key dim, col = value dim; NULL => zeros */
    float *state_out;       /* [B,H,d,d] fp32 or NULL */
    float *o_la;            /* optional raw linear-branch output  [B,L,H,d] fp32, or NULL */
    float *o_nla;           /* optional raw softmax-branch output [B,L,H,d] fp32, or NULL */
    float *lse;             /* optional log-sum-exp of the softmax logits [B,H,L] fp32, or NULL */
    void *k_sm, *v_sm;      /* optional compacted K/V of the retained tokens [B,H,sm_cap,d], */
    int32_t *sm_len;        /*   in `dtype`, with their counts [B,H]; all three or none.     */
    int32_t sm_cap;         /*   This is the decode cache layout (prefill -> decode handoff). */
    void *const *stage_events; /* host array of cudaEvent_t owned by the caller, or NULL: the    */
    int32_t n_stage_events;    /*   library records event[i] on `stream` before stage i and one  */
                               /*   after the last stage (see natsl_stage_name); for profiling.  */
    const float *dstate_out; /* backward, optional: gradient w.r.t. state_out [B,H,d,d] fp32; NULL => 0 */
    float *dstate_in;       /* backward, optional: receives the gradient w.r.t. state_in [B,H,d,d]    */
    float *dscore;          /* backward with NATSL_BLOCK_ROUTING, optional: gradients of the score    */
                            /*   layer's two masks per block [B,L/C,H,2] fp32 = (linear, softmax), */
                            /*   Section 4.2: for a softmax block the sum over its keys j and all  */
                            /*   queries i >= j of dM_ij = p_ij (dp_ij - <do_i, o_i>); for a linear */
                            /*   block <dS_next, U> with U the update the block commits to the     */
                            /*   state; zero for the operation the block did not choose.  NULL:    */
                            /*   not computed.  Without the flag: NATSL_ERR_UNSUPPORTED.           */
    int32_t G;              /* softmax heads per linear head (Section 4.3: several softmax heads are   */
                            /*   grouped under one linear head and share its route); 0 or 1: none.     */
                            /*   The paper does not say how one q, k, v serves two head counts; here   */
                            /*   the G softmax heads of head h are the G slices of d / G columns of    */
                            /*   q, k, v [B,L,H,d]: softmax head (h, s) attends with columns           */
                            /*   [s d/G, (s+1) d/G) over the retained tokens of route[:,:,h] and fills */
                            /*   those columns of the softmax output, which is RMS-normalised per      */
                            /*   slice; the linear operation, its state and the two weights stay per   */
                            /*   head h over all d columns.  p->lse becomes [B,H,G,L].                 */
                            /*   Built: natsl_hybrid_fwd with token-level and block-level routing, for */
                            /*   fp32 storage (d / G in {32, 64, 128}) and on the tensor-core path for */
                            /*   d = 128, G = 2 (the appendix's two softmax heads per linear head;     */
                            /*   three would need d = 192); natsl_hybrid_bwd with either routing for   */
                            /*   the same shapes (self-contained or                                    */
                            /*   from a saved forward; p->dscore: the softmax heads of a group share   */
                            /*   the block's mask, their gradients add); natsl_decode_step for d / G in */
                            /*   {32, 64, 128}.  A cache returned or read with NATSL_QK_NORM holds the */
                            /*   keys as given: they are normalised as they are read                   */
                            /*   (NATSL_APPEND_CACHE included).  G > 1 or NATSL_QK_NORM with           */
                            /*   NATSL_FORCE_SIMT on bf16: NATSL_ERR_UNSUPPORTED.                      */
    float norm_eps;         /* NATSL_QK_NORM: epsilon under the square roots, >= 0                     */
} natsl_params;

/* Bytes of workspace `op` needs for these shapes (host call, launches nothing). */
int natsl_workspace_size(const natsl_params *p, int op, size_t *bytes /* host */);

/*
 * Route compaction: the column masks M^nla / M^la of Section 4.1 as index lists, so that the
 * softmax branch loads only retained tokens and the linear branch only linear tokens.
 *   route           [B,L,H] u8
 *   sm_idx          [B,H,L]      ascending positions with route=1 (entries >= n_sm untouched)
 *   sm_chunk_prefix [B,H,L/C+1]  exclusive prefix of per-chunk softmax counts, last = n_sm
 *   lin_idx         [B,H,L/C,C]  ascending in-chunk offsets with route=0, padded with C
 *   n_lin           [B,H,L/C]
 * Integer work; exactly one result is correct.  No workspace needed (ws may be NULL).
 */
int natsl_route_compact(const uint8_t *route, int32_t *sm_idx, int32_t *sm_chunk_prefix,
                        int32_t *lin_idx, int32_t *n_lin, const natsl_params *p,
                        void *ws, size_t ws_bytes, void *stream);

/*
 * Attention score layer (Section 4.1, the score equation and the arg max after it): per chunk of
 * C = 64 tokens, score = W^score Mean(X_chunk), one score per operation and head, and the
 * operation with the higher score becomes the chunk's route.  Its output is a `route` for
 * NATSL_BLOCK_ROUTING.
 *   x       [B,L,d_model] in p->dtype (the layer's input features), d_model a multiple of 8
 *           (bf16) or 4 (fp32), 16-byte aligned;
 *   w_score [H,2,d_model] fp32, 16-byte aligned: row (h, 0) scores linear attention, row (h, 1)
 *           softmax attention (every head has its own mask, Section 4.3);
 *   scores  [B,L/C,H,2] fp32, or NULL;
 *   route   [B,L,H] u8: 1 where the softmax score is strictly higher (a tie keeps linear, the first
 *           operation), repeated over the chunk's tokens.
 * The softmax over the two scores is monotone and is not formed.  fp32 accumulation throughout.
 * Only B, L, H, C, dtype of `p` are used (d must still be valid).  No workspace.
 * Errors: NULL, SHAPE, DTYPE, ALIGN, CUDA.
 */
int natsl_score_layer(const void *x, const float *w_score, float *scores, uint8_t *route,
                      int32_t d_model, const natsl_params *p, void *stream);

/*
 * Forward of the whole layer (header comment; Sections 4.1 and 4.3).
 *   q,k,v [B,L,H,d] in p->dtype; g,beta [B,L,H] fp32 (g = log decay <= 0);
 *   route [B,L,H] u8; out [B,L,H,d] in p->dtype.
 * The linear branch is computed chunkwise (Section 3, chunkwise equations) with C = 64.
 * Optional outputs are taken from `p`.  Errors: NULL, SHAPE, DTYPE, ALIGN, WORKSPACE, CUDA;
 * UNSUPPORTED for NATSL_APPEND_CACHE off the tensor-core path (fp32 storage, NATSL_FORCE_SIMT).
 */
int natsl_hybrid_fwd(const void *q, const void *k, const void *v, const float *g,
                     const float *beta, const uint8_t *route, void *out,
                     const natsl_params *p, void *ws, size_t ws_bytes, void *stream);

/*
 * natsl_hybrid_fwd for callers that cannot allocate device memory (no counterpart in the paper;
 * it computes exactly what natsl_hybrid_fwd computes).  A plug-in inside a server that owns the
 * memory pool, or a latency-critical loop that must not hit the device-wide synchronisation of
 * cudaMalloc, has no workspace to hand over.  Here the scratch is a fixed array of
 * NATSL_STATIC_WS_BYTES inside the library (each GPU that loads the library holds it until the
 * process exits); the caller passes only inputs and outputs, including the optional ones in `p`.
 *   - Problems whose natsl_workspace_size(p, NATSL_OP_FWD) exceeds NATSL_STATIC_WS_BYTES are
 *     rejected with NATSL_ERR_TOO_LARGE before anything is launched.
 *   - The first call on each device looks up the array's device address (a host-side set-up
 *     step); make that first call outside any stream capture.
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the
 *     library re-initialises what it needs.  Two calls that overlap on the GPU (different
 *     streams, no ordering between them) race on it: keep them on one stream or order them.
 *   - The array is the one of the calling thread's current device: `stream` and all tensors must
 *     belong to that device.
 *   - Conditions only the device can see (NATSL_ERR_ROUTE, NATSL_ERR_CACHE_FULL, NATSL_ERR_TIMEOUT)
 *     go to the status word at the head of the array; natsl_static_status reads it.
 * Errors otherwise as natsl_hybrid_fwd.
 */
#define NATSL_STATIC_WS_BYTES (32u << 20)
int natsl_hybrid_fwd_static(const void *q, const void *k, const void *v, const float *g,
                            const float *beta, const uint8_t *route, void *out,
                            const natsl_params *p, void *stream);

/* natsl_device_status for the built-in scratch of the current device (no counterpart in the
 * paper): synchronises `stream`, returns and clears the status word.  Allocates nothing. */
int natsl_static_status(void *stream);

/*
 * Backward of natsl_hybrid_fwd's `out` (Section 4.2 states the properties: the softmax-branch
 * logit gradient is p (dp - <do,o>), and k, v gradients of an operation vanish for tokens
 * inactive for it).  Self-contained: recomputes what it needs from the inputs, unless the forward
 * was run with NATSL_SAVE_FOR_BWD in the same workspace (then pass NATSL_SAVED_FWD).
 *   dout [B,L,H,d] in p->dtype; dq,dk,dv [B,L,H,d] in p->dtype;
 *   dg,dbeta [B,L,H] fp32; dw [B,L,H,2] fp32 or NULL.
 * The linear state is carried across calls (Section 3, chunkwise recurrence): with p->state_in the
 * sequence continues an earlier piece; p->dstate_out is the gradient arriving at this piece's
 * final state from the pieces after it, p->dstate_in receives the gradient for the piece before
 * (both optional).  The retained K/V of earlier pieces are not part of this call: their gradients
 * belong to the calls that produced them.  Errors as forward.
 */
int natsl_hybrid_bwd(const void *q, const void *k, const void *v, const float *g,
                     const float *beta, const uint8_t *route, const void *dout,
                     void *dq, void *dk, void *dv, float *dg, float *dbeta, float *dw,
                     const natsl_params *p, void *ws, size_t ws_bytes, void *stream);

/*
 * One generation step (Section 4.1, per-token generation): decay the state, apply the delta
 * rule (route 0) or append the token's K/V to the retained cache (route 1), then read both
 * branches and combine.  With routes 0 / 1 the new token's route is known (token-level routing)
 * and no roll-back is needed.  route 2 is a token of a block whose decision is still open
 * (block-level routing): it is folded into the state and appended to the cache, so that both
 * operations see it (the paper's pseudo-update of both hidden states); natsl_decode_block_end
 * undoes one of the two when the block is complete.
 *   q,k,v [B,H,d] in p->dtype; g,beta [B,H] fp32; route [B,H] u8; p->w [B,H,2] or NULL;
 *   state [B,H,d,d] fp32, updated in place;
 *   k_cache,v_cache [B,H,cache_cap,d] in p->dtype; cache_len [B,H] i32, updated in place;
 *   out [B,H,d] in p->dtype.
 * A sequence whose cache is full and whose token is to be appended is left untouched,
 * its out row is zero-filled and NATSL_ERR_CACHE_FULL is recorded in the status word at the
 * start of the workspace.  ws must hold natsl_workspace_size(p, NATSL_OP_DECODE) bytes and be
 * zero-filled once before its first use; besides the status word it holds per-head tickets and
 * partial results of the step in flight, so two steps that use the same ws must not overlap on
 * the GPU (successive steps on one stream are fine).
 */
int natsl_decode_step(const void *q, const void *k, const void *v, const float *g,
                      const float *beta, const uint8_t *route, float *state,
                      void *k_cache, void *v_cache, int32_t *cache_len, int32_t cache_cap,
                      void *out, const natsl_params *p, void *ws, size_t ws_bytes, void *stream);

/*
 * End of a block during generation under block-level routing (Section 4.1: after observing the
 * entire chunk, the hidden state of the operation that was not selected is rolled back).
 * block_len tokens were decoded with route 2 since the previous call (or since the prefill).
 *   route_block [B,H] u8: the block's decision.  1 (softmax): the linear state is reset to its
 *       value at the start of the block, state_start, times the block's decay exp(g_block)
 *       (Section 4.3: the decay is applied on softmax blocks too); the block's K/V stay in the
 *       cache.  0 (linear): the state stays; the block's block_len cache entries are dropped
 *       (cache_len -= block_len).
 *   g_block [B,H] fp32: sum of the g values of the block's tokens.
 *   state, state_start [B,H,d,d] fp32, device; state_start is then set to the new state, the
 *       start of the next block.  Before the first block the caller makes it a copy of `state`.
 *   cache_len [B,H] i32, in place.  A linear block with fewer than block_len entries in its cache
 *       records NATSL_ERR_ROUTE in the status word (ws: the decode workspace).
 * Errors: NULL, SHAPE, ALIGN, WORKSPACE, CUDA.
 */
int natsl_decode_block_end(const uint8_t *route_block, const float *g_block, float *state,
                           float *state_start, int32_t *cache_len, int32_t block_len,
                           const natsl_params *p, void *ws, size_t ws_bytes, void *stream);

/* Synchronises `stream`, returns (and clears) the status word kernels wrote at ws[0]. */
int natsl_device_status(void *ws, void *stream);

const char *natsl_strerror(int status);

/* Name of stage i of operation `op` (the interval between stage events i and i+1), or NULL
 * when i is past the last stage.  Host call. */
const char *natsl_stage_name(int op, int i);

/* Number of kernels this library has launched in this process so far (host counter). */
uint64_t natsl_launch_count(void);

/*
 * Test hook for the time-out path (no counterpart in the paper).  Every device-side wait of the
 * tensor-core kernels is bounded (about two seconds by default); when a wait runs out the kernel
 * records NATSL_ERR_TIMEOUT in the status word, waits for its own copies in flight, frees its
 * tensor memory and returns.  This call sets, for all following forward calls of the process,
 *   kcycles              the bound in units of 1024 clock cycles (0: back to the default), and
 *   withhold_scan_flags  non-zero: the scan does not raise the per-chunk counters the softmax
 *                        kernel's epilogue waits for, so that exactly this wait runs out.
 * Nothing faults and nothing hangs: the call returns after the bound and reports the time-out.
 */
void natsl_debug_set_wait_limit(uint32_t kcycles, int withhold_scan_flags);

#ifdef __cplusplus
}
#endif
#endif /* NATSL_H_ */

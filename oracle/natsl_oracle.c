/*
 * fp64 CPU oracle for the token-level hybrid attention layer (NAtS-L).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * layer computes; the parity tests, the smoke check and the benchmark's CPU
 * baseline are its only callers.  It shares no code with the CUDA library and
 * the CUDA library never calls it.
 *
 * Everything here is the token-by-token definition, per (batch, head):
 *
 *   linear branch   : Gated DeltaNet recurrence (Section 4.3, the GDN equation
 *                     S_t = S_{t-1} alpha_t (I - beta_t k_t k_t^T) + beta_t v_t k_t^T),
 *                     with the decay applied on every token, also on tokens routed
 *                     to softmax (Section 4.3, the "always apply the decay" equation),
 *                     and the delta update applied only for linear tokens
 *                     (Section 4.1, the case equation for the chunk state).
 *   softmax branch  : softmax over the retained tokens j <= i only (Section 4.1,
 *                     the O_nla equation with the column mask M^nla).
 *   combination     : RMS-normalise each branch output and add them with the
 *                     per-token, per-head weights (Section 4.3, the Norm equation).
 *
 * Conventions (the paper's S is the transpose of ours):
 *   q,k,v,out   [B, L, H, d]   row vectors, d contiguous
 *   g,beta      [B, L, H]      g = log alpha <= 0
 *   route       [B, L, H]      1 = softmax (K/V retained), 0 = linear (folded into S)
 *   w           [B, L, H, 2]   (w_nla, w_la);  NULL means (0.5, 0.5)
 *   state       [B, H, dk, dv] o_la = scale_la * q S  (read after the token's own update)
 *   lse         [B, H, L]      log-sum-exp of the softmax logits, -inf for an empty row
 *
 * natsl_oracle_hybrid_fwd_block is the same layer with one routing decision per block of
 * tokens, written the way the paper describes generation: both operations run inside a block
 * and the one not chosen is rolled back at its end.
 *
 * Parity pins live in tests/ (closed forms, a library attention routine, brute
 * force on tiny inputs, finite differences); none of them calls back into the
 * formula they check.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define AT3(b, l, h) ((((size_t)(b)) * L + (size_t)(l)) * H + (size_t)(h))

int natsl_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------------------
 * Route compaction (the column masks of Section 4.1 written as index lists).
 *   sm_idx          [B,H,L]       ascending positions with route = 1; entries past n_sm untouched
 *   sm_chunk_prefix [B,H,L/C+1]   exclusive prefix of per-chunk softmax counts; last = n_sm
 *   lin_idx         [B,H,L/C,C]   ascending in-chunk offsets with route = 0, padded with C
 *   n_lin           [B,H,L/C]
 * ------------------------------------------------------------------------- */
int natsl_oracle_route_compact(const uint8_t *route, int B, int L, int H, int C,
                               int32_t *sm_idx, int32_t *sm_chunk_prefix,
                               int32_t *lin_idx, int32_t *n_lin)
{
    if (C <= 0 || L % C != 0) return -1;
    int NC = L / C;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            size_t bh = (size_t)b * H + h;
            int n_sm = 0;
            for (int c = 0; c < NC; ++c) {
                sm_chunk_prefix[bh * (NC + 1) + c] = n_sm;
                int nl = 0;
                for (int t = 0; t < C; ++t) {
                    int l = c * C + t;
                    if (route[AT3(b, l, h)]) {
                        sm_idx[bh * L + n_sm] = l;
                        ++n_sm;
                    } else {
                        lin_idx[(bh * NC + c) * C + nl] = t;
                        ++nl;
                    }
                }
                n_lin[bh * NC + c] = nl;
                for (int t = nl; t < C; ++t) lin_idx[(bh * NC + c) * C + t] = C;
            }
            sm_chunk_prefix[bh * (NC + 1) + NC] = n_sm;
        }
    return 0;
}

/* RMS normalisation of one row: y = o / sqrt(mean(o^2) + eps); returns the factor. */
static double rms_factor(const double *o, int d, double eps)
{
    double ss = 0.0;
    for (int a = 0; a < d; ++a) ss += o[a] * o[a];
    return 1.0 / sqrt(ss / d + eps);
}

/* One token of the hybrid layer for one (batch, head).
 * S      : dk x dv state, updated in place
 * kc, vc : retained keys / values so far, n_c rows of d
 * delta  : apply the delta update of this token to S;  append: add its K/V to kc, vc.
 *          Token-level routing sets exactly one of the two (delta for a linear token, append for
 *          a softmax token); inside an undecided block both are set (see the block-mode forward).
 * Outputs (each may be NULL): o_la, o_nla rows, lse, out row. */
static void hybrid_token(int d, const double *q, const double *k, const double *v,
                         double g, double beta, int delta, int append, double w_nla, double w_la,
                         double scale_la, double scale_sm, double eps,
                         double *S, double *kc, double *vc, int *n_c,
                         double *logit /* scratch, >= n_c+1 */,
                         double *o_la_out, double *o_nla_out, double *lse_out, double *out)
{
    /* decay on every token */
    double alpha = exp(g);
    for (int a = 0; a < d * d; ++a) S[a] *= alpha;
    if (delta) {
        /* delta rule against the decayed state: S += beta k^T (v - k S) */
        for (int c = 0; c < d; ++c) {
            double ks = 0.0;
            for (int a = 0; a < d; ++a) ks += k[a] * S[(size_t)a * d + c];
            double e = v[c] - ks;
            for (int a = 0; a < d; ++a) S[(size_t)a * d + c] += beta * k[a] * e;
        }
    }
    if (append) {
        memcpy(kc + (size_t)(*n_c) * d, k, sizeof(double) * d);
        memcpy(vc + (size_t)(*n_c) * d, v, sizeof(double) * d);
        *n_c += 1;
    }
    /* linear branch reads the state that already contains this token */
    double o_la[512], o_nla[512];
    for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int a = 0; a < d; ++a) acc += q[a] * S[(size_t)a * d + c];
        o_la[c] = scale_la * acc;
    }
    /* softmax branch over the retained tokens (this one included when it was appended) */
    int n = *n_c;
    double lse = -INFINITY;
    for (int c = 0; c < d; ++c) o_nla[c] = 0.0;
    if (n > 0) {
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) {
            double s = 0.0;
            for (int a = 0; a < d; ++a) s += q[a] * kc[(size_t)j * d + a];
            logit[j] = scale_sm * s;
            if (logit[j] > m) m = logit[j];
        }
        double z = 0.0;
        for (int j = 0; j < n; ++j) {
            logit[j] = exp(logit[j] - m);
            z += logit[j];
        }
        for (int j = 0; j < n; ++j) {
            double p = logit[j] / z;
            for (int c = 0; c < d; ++c) o_nla[c] += p * vc[(size_t)j * d + c];
        }
        lse = m + log(z);
    }
    double f_la = rms_factor(o_la, d, eps), f_nla = rms_factor(o_nla, d, eps);
    for (int c = 0; c < d; ++c) {
        if (out) out[c] = w_nla * o_nla[c] * f_nla + w_la * o_la[c] * f_la;
        if (o_la_out) o_la_out[c] = o_la[c];
        if (o_nla_out) o_nla_out[c] = o_nla[c];
    }
    if (lse_out) *lse_out = lse;
}

/* ---------------------------------------------------------------------------
 * Forward over a whole sequence.  Optional outputs may be NULL.
 *   kc_out, vc_out [B,H,L,d]  retained K/V in order of arrival (first n_sm rows valid)
 *   n_sm_out       [B,H]
 * ------------------------------------------------------------------------- */
int natsl_oracle_hybrid_fwd(const double *q, const double *k, const double *v,
                            const double *g, const double *beta, const uint8_t *route,
                            const double *w, int B, int L, int H, int d,
                            double scale_la, double scale_sm, double eps,
                            const double *state_in, double *out, double *o_la, double *o_nla,
                            double *lse, double *state_out, double *kc_out, double *vc_out,
                            int32_t *n_sm_out)
{
    if (d > 512 || d <= 0) return -1;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H;
        double *S = (double *)calloc((size_t)d * d, sizeof(double));
        double *kc = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *vc = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *logit = (double *)malloc(sizeof(double) * (size_t)(L + 1));
        if (!S || !kc || !vc || !logit) {
            err = 1;
        } else {
            if (state_in) memcpy(S, state_in + (size_t)bh * d * d, sizeof(double) * d * d);
            int n_c = 0;
            for (int i = 0; i < L; ++i) {
                size_t t = AT3(b, i, h);
                double wn = w ? w[t * 2 + 0] : 0.5, wl = w ? w[t * 2 + 1] : 0.5;
                hybrid_token(d, q + t * d, k + t * d, v + t * d, g[t], beta[t], route[t] == 0,
                             route[t] != 0,
                             wn, wl, scale_la, scale_sm, eps, S, kc, vc, &n_c, logit,
                             o_la ? o_la + t * d : NULL, o_nla ? o_nla + t * d : NULL,
                             lse ? lse + (size_t)bh * L + i : NULL, out ? out + t * d : NULL);
            }
            if (state_out) memcpy(state_out + (size_t)bh * d * d, S, sizeof(double) * d * d);
            if (kc_out) memcpy(kc_out + (size_t)bh * L * d, kc, sizeof(double) * (size_t)n_c * d);
            if (vc_out) memcpy(vc_out + (size_t)bh * L * d, vc, sizeof(double) * (size_t)n_c * d);
            if (n_sm_out) n_sm_out[bh] = n_c;
        }
        free(S); free(kc); free(vc); free(logit);
    }
    return err ? -2 : 0;
}

/* ---------------------------------------------------------------------------
 * Block-mode forward (Section 4.1, the paragraphs after the chunk-state case equation and on
 * per-token generation): one routing decision per block of R tokens, known only when the block
 * is complete.  Until then both branches treat every token of the block as their own -- the
 * linear state takes the token's delta update and the token's K/V join the retained set -- so
 * that each output contains the intra-block correlations of both operations.  At the end of the
 * block the operation that was not chosen is rolled back: for a linear block the block's K/V are
 * removed again; for a softmax block the linear state is reset to its value at the start of the
 * block, with the block's decay applied (Section 4.3, the decay-always equation).
 *   route [B,L,H] must be constant within each block of R tokens (-4 otherwise); L % R == 0.
 * Outputs as natsl_oracle_hybrid_fwd.
 * ------------------------------------------------------------------------- */
int natsl_oracle_hybrid_fwd_block(const double *q, const double *k, const double *v,
                                  const double *g, const double *beta, const uint8_t *route,
                                  const double *w, int B, int L, int H, int d, int R,
                                  double scale_la, double scale_sm, double eps,
                                  const double *state_in, double *out, double *o_la,
                                  double *o_nla, double *lse, double *state_out, double *kc_out,
                                  double *vc_out, int32_t *n_sm_out)
{
    if (d > 512 || d <= 0 || R <= 0 || L % R != 0) return -1;
    int err = 0, bad_route = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H;
        double *S = (double *)calloc((size_t)d * d, sizeof(double));
        double *S_start = (double *)malloc(sizeof(double) * (size_t)d * d);
        double *kc = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *vc = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *logit = (double *)malloc(sizeof(double) * (size_t)(L + 1));
        if (!S || !S_start || !kc || !vc || !logit) {
            err = 1;
        } else {
            if (state_in) memcpy(S, state_in + (size_t)bh * d * d, sizeof(double) * d * d);
            int n_c = 0;
            for (int i0 = 0; i0 < L; i0 += R) {
                const int r = route[AT3(b, i0, h)] != 0;
                const int n_start = n_c;
                double g_block = 0.0;
                memcpy(S_start, S, sizeof(double) * d * d);
                for (int i = i0; i < i0 + R; ++i) {
                    size_t t = AT3(b, i, h);
                    if ((route[t] != 0) != r) bad_route = 1;
                    double wn = w ? w[t * 2 + 0] : 0.5, wl = w ? w[t * 2 + 1] : 0.5;
                    g_block += g[t];
                    hybrid_token(d, q + t * d, k + t * d, v + t * d, g[t], beta[t], 1, 1,
                                 wn, wl, scale_la, scale_sm, eps, S, kc, vc, &n_c, logit,
                                 o_la ? o_la + t * d : NULL, o_nla ? o_nla + t * d : NULL,
                                 lse ? lse + (size_t)bh * L + i : NULL, out ? out + t * d : NULL);
                }
                if (r) {
                    double decay = exp(g_block);
                    for (int a = 0; a < d * d; ++a) S[a] = decay * S_start[a];
                } else {
                    n_c = n_start;
                }
            }
            if (state_out) memcpy(state_out + (size_t)bh * d * d, S, sizeof(double) * d * d);
            if (kc_out) memcpy(kc_out + (size_t)bh * L * d, kc, sizeof(double) * (size_t)n_c * d);
            if (vc_out) memcpy(vc_out + (size_t)bh * L * d, vc, sizeof(double) * (size_t)n_c * d);
            if (n_sm_out) n_sm_out[bh] = n_c;
        }
        free(S); free(S_start); free(kc); free(vc); free(logit);
    }
    if (err) return -2;
    return bad_route ? -4 : 0;
}

/* ---------------------------------------------------------------------------
 * One decode step (Section 4.1, per-token generation).  route 0 / 1: the route of the new
 * token is known (token-level routing), so nothing has to be rolled back.  route 2: the token
 * belongs to a block whose decision is still open -- it is folded into the state AND appended
 * to the retained K/V (the pseudo-update of both hidden states); natsl_oracle_block_end undoes
 * one of the two when the block is complete.
 *   q,k,v [B,H,d]; g,beta [B,H]; route [B,H]; w [B,H,2] or NULL
 *   state [B,H,d,d] in place; k_cache,v_cache [B,H,cap,d]; cache_len [B,H] in place
 * Returns -3 if a sequence would overflow its cache (nothing is modified for it).
 * ------------------------------------------------------------------------- */
int natsl_oracle_decode_step(const double *q, const double *k, const double *v,
                             const double *g, const double *beta, const uint8_t *route,
                             const double *w, int B, int H, int d,
                             double scale_la, double scale_sm, double eps,
                             double *state, double *k_cache, double *v_cache,
                             int32_t *cache_len, int cache_cap, double *out,
                             double *o_la, double *o_nla)
{
    if (d > 512 || d <= 0) return -1;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        int n_c = cache_len[bh];
        if (route[bh] != 0 && n_c >= cache_cap) { err = 3; continue; }
        double *logit = (double *)malloc(sizeof(double) * (size_t)(n_c + 2));
        double wn = w ? w[(size_t)bh * 2] : 0.5, wl = w ? w[(size_t)bh * 2 + 1] : 0.5;
        hybrid_token(d, q + (size_t)bh * d, k + (size_t)bh * d, v + (size_t)bh * d, g[bh], beta[bh],
                     route[bh] != 1, route[bh] != 0, wn, wl, scale_la, scale_sm, eps,
                     state + (size_t)bh * d * d, k_cache + (size_t)bh * cache_cap * d,
                     v_cache + (size_t)bh * cache_cap * d, &n_c, logit,
                     o_la ? o_la + (size_t)bh * d : NULL, o_nla ? o_nla + (size_t)bh * d : NULL,
                     NULL, out + (size_t)bh * d);
        cache_len[bh] = n_c;
        free(logit);
    }
    return err ? -3 : 0;
}

/* ---------------------------------------------------------------------------
 * End of a block during generation (Section 4.1: "reroll the hidden states of the operations
 * that are not selected"): R tokens were decoded with route 2 since the last call.
 *   route_block [B,H]: the block's decision.  1 (softmax): the linear state is reset to its value
 *       at the start of the block, state_start, times the block's decay exp(g_block) (Section 4.3,
 *       decay-always equation); the appended K/V stay.  0 (linear): the state stays, the block's
 *       R cache entries are removed.
 *   state_start [B,H,d,d] is then set to the new state: the start of the next block.
 * ------------------------------------------------------------------------- */
int natsl_oracle_block_end(const uint8_t *route_block, const double *g_block, int B, int H, int d,
                           int R, double *state, double *state_start, int32_t *cache_len)
{
    for (int bh = 0; bh < B * H; ++bh) {
        double *S = state + (size_t)bh * d * d, *S0 = state_start + (size_t)bh * d * d;
        if (route_block[bh]) {
            double decay = exp(g_block[bh]);
            for (int a = 0; a < d * d; ++a) S[a] = decay * S0[a];
        } else {
            if (cache_len[bh] < R) return -1;
            cache_len[bh] -= R;
        }
        memcpy(S0, S, sizeof(double) * (size_t)d * d);
    }
    return 0;
}

/* ---------------------------------------------------------------------------
 * Analytic backward of natsl_oracle_hybrid_fwd (reverse-mode, token by token).
 * The paper gives no backward for the delta rule itself; this is the chain rule
 * applied to the forward loop above, statement by statement, in reverse order.
 * The softmax part is the usual ds = p (dp - <do, o>) (Section 4.2, the dM^nla
 * equation is that same quantity).
 *
 * Inputs as forward plus dout [B,L,H,d] and optional dstate_out [B,H,d,d].
 * Outputs: dq,dk,dv [B,L,H,d]; dg,dbeta [B,L,H]; dw [B,L,H,2] (may be NULL);
 *          dstate_in [B,H,d,d] (may be NULL).
 * ------------------------------------------------------------------------- */
int natsl_oracle_hybrid_bwd(const double *q, const double *k, const double *v,
                            const double *g, const double *beta, const uint8_t *route,
                            const double *w, const double *dout, int B, int L, int H, int d,
                            double scale_la, double scale_sm, double eps,
                            const double *state_in, const double *dstate_out,
                            double *dq, double *dk, double *dv, double *dg, double *dbeta,
                            double *dw, double *dstate_in)
{
    if (d > 512 || d <= 0) return -1;
    int err = 0;
    size_t dd = (size_t)d * d;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H;
        /* states[i] = S_{i-1} (before token i), states[L] = final */
        double *states = (double *)malloc(sizeof(double) * dd * (size_t)(L + 1));
        double *o_la = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *o_nla = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *do_la = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *do_nla = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *lse = (double *)malloc(sizeof(double) * (size_t)L);
        double *dS = (double *)calloc(dd, sizeof(double));
        double *Sbar = (double *)malloc(sizeof(double) * dd);
        double *p = (double *)malloc(sizeof(double) * (size_t)(L + 1));
        int *ret = (int *)malloc(sizeof(int) * (size_t)(L + 1));
        if (!states || !o_la || !o_nla || !do_la || !do_nla || !lse || !dS || !Sbar || !p || !ret) {
            err = 1;
            goto done;
        }
        /* ---- forward recomputation, keeping every state ---- */
        if (state_in) memcpy(states, state_in + (size_t)bh * dd, sizeof(double) * dd);
        else memset(states, 0, sizeof(double) * dd);
        int n_ret = 0;
        for (int i = 0; i < L; ++i) {
            size_t t = AT3(b, i, h);
            const double *qi = q + t * d, *ki = k + t * d, *vi = v + t * d;
            double *Sp = states + dd * i, *Sn = states + dd * (i + 1);
            double alpha = exp(g[t]);
            for (size_t a = 0; a < dd; ++a) Sn[a] = alpha * Sp[a];
            if (!route[t]) {
                for (int c = 0; c < d; ++c) {
                    double ks = 0.0;
                    for (int a = 0; a < d; ++a) ks += ki[a] * Sn[(size_t)a * d + c];
                    double e = vi[c] - ks;
                    for (int a = 0; a < d; ++a) Sn[(size_t)a * d + c] += beta[t] * ki[a] * e;
                }
            } else {
                ret[n_ret++] = i;
            }
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int a = 0; a < d; ++a) acc += qi[a] * Sn[(size_t)a * d + c];
                o_la[(size_t)i * d + c] = scale_la * acc;
                o_nla[(size_t)i * d + c] = 0.0;
            }
            lse[i] = -INFINITY;
            if (n_ret > 0) {
                double m = -INFINITY;
                for (int j = 0; j < n_ret; ++j) {
                    const double *kj = k + AT3(b, ret[j], h) * d;
                    double s = 0.0;
                    for (int a = 0; a < d; ++a) s += qi[a] * kj[a];
                    p[j] = scale_sm * s;
                    if (p[j] > m) m = p[j];
                }
                double z = 0.0;
                for (int j = 0; j < n_ret; ++j) { p[j] = exp(p[j] - m); z += p[j]; }
                for (int j = 0; j < n_ret; ++j) {
                    const double *vj = v + AT3(b, ret[j], h) * d;
                    for (int c = 0; c < d; ++c) o_nla[(size_t)i * d + c] += p[j] / z * vj[c];
                }
                lse[i] = m + log(z);
            }
        }
        /* ---- combination backward, row by row ---- */
        for (int i = 0; i < L; ++i) {
            size_t t = AT3(b, i, h);
            double wn = w ? w[t * 2] : 0.5, wl = w ? w[t * 2 + 1] : 0.5;
            const double *ol = o_la + (size_t)i * d, *on = o_nla + (size_t)i * d;
            const double *dy = dout + t * d;
            double fl = rms_factor(ol, d, eps), fn = rms_factor(on, d, eps);
            double dwn = 0.0, dwl = 0.0, ml = 0.0, mn = 0.0;
            for (int c = 0; c < d; ++c) {
                dwn += dy[c] * on[c] * fn;
                dwl += dy[c] * ol[c] * fl;
                mn += wn * dy[c] * on[c] * fn;
                ml += wl * dy[c] * ol[c] * fl;
            }
            mn /= d; ml /= d;
            for (int c = 0; c < d; ++c) {
                /* y = o f, f = (mean(o^2)+eps)^(-1/2):  do = f (dy' - y mean(dy' y)),  dy' = w dy */
                do_nla[(size_t)i * d + c] = fn * (wn * dy[c] - on[c] * fn * mn);
                do_la[(size_t)i * d + c] = fl * (wl * dy[c] - ol[c] * fl * ml);
            }
            if (dw) { dw[t * 2] = dwn; dw[t * 2 + 1] = dwl; }
        }
        for (int i = 0; i < L; ++i) {
            size_t t = AT3(b, i, h);
            for (int a = 0; a < d; ++a) { dq[t * d + a] = 0.0; dk[t * d + a] = 0.0; dv[t * d + a] = 0.0; }
        }
        /* ---- softmax branch backward ---- */
        {
            int n_vis = n_ret;
            for (int i = L - 1; i >= 0; --i) {
                while (n_vis > 0 && ret[n_vis - 1] > i) --n_vis;
                if (n_vis == 0) continue;
                size_t t = AT3(b, i, h);
                const double *qi = q + t * d;
                const double *doi = do_nla + (size_t)i * d, *oi = o_nla + (size_t)i * d;
                double D = 0.0;
                for (int c = 0; c < d; ++c) D += doi[c] * oi[c];
                for (int j = 0; j < n_vis; ++j) {
                    size_t tj = AT3(b, ret[j], h);
                    const double *kj = k + tj * d, *vj = v + tj * d;
                    double s = 0.0, dp = 0.0;
                    for (int a = 0; a < d; ++a) s += qi[a] * kj[a];
                    double pij = exp(scale_sm * s - lse[i]);
                    for (int c = 0; c < d; ++c) dp += doi[c] * vj[c];
                    double ds = pij * (dp - D);
                    for (int c = 0; c < d; ++c) dv[tj * d + c] += pij * doi[c];
                    for (int a = 0; a < d; ++a) {
                        dq[t * d + a] += scale_sm * ds * kj[a];
                        dk[tj * d + a] += scale_sm * ds * qi[a];
                    }
                }
            }
        }
        /* ---- linear branch backward: reverse recurrence carrying dS ---- */
        if (dstate_out) memcpy(dS, dstate_out + (size_t)bh * dd, sizeof(double) * dd);
        for (int i = L - 1; i >= 0; --i) {
            size_t t = AT3(b, i, h);
            const double *qi = q + t * d, *ki = k + t * d, *vi = v + t * d;
            const double *Sp = states + dd * i, *Sn = states + dd * (i + 1);
            const double *doi = do_la + (size_t)i * d;
            double alpha = exp(g[t]);
            double bt = route[t] ? 0.0 : beta[t];
            /* o_la = scale_la q S_i */
            for (int a = 0; a < d; ++a) {
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += doi[c] * Sn[(size_t)a * d + c];
                dq[t * d + a] += scale_la * acc;
                for (int c = 0; c < d; ++c) dS[(size_t)a * d + c] += scale_la * qi[a] * doi[c];
            }
            for (size_t a = 0; a < dd; ++a) Sbar[a] = alpha * Sp[a];
            double dbt = 0.0;
            if (!route[t]) {
                /* S_i = Sbar + bt k^T e,  e = v - k Sbar */
                for (int c = 0; c < d; ++c) {
                    double ks = 0.0, kds = 0.0;
                    for (int a = 0; a < d; ++a) {
                        ks += ki[a] * Sbar[(size_t)a * d + c];
                        kds += ki[a] * dS[(size_t)a * d + c];
                    }
                    double e = vi[c] - ks;
                    double de = bt * kds;
                    dbt += kds * e;
                    dv[t * d + c] += de;
                    for (int a = 0; a < d; ++a) {
                        dk[t * d + a] += bt * e * dS[(size_t)a * d + c] - de * Sbar[(size_t)a * d + c];
                    }
                    /* dSbar = dS - k^T de  (column c) */
                    for (int a = 0; a < d; ++a) dS[(size_t)a * d + c] -= ki[a] * de;
                }
            }
            /* Sbar = alpha S_{i-1},  alpha = exp(g) */
            double da = 0.0;
            for (size_t a = 0; a < dd; ++a) da += dS[a] * Sp[a];
            dg[t] = alpha * da;
            dbeta[t] = route[t] ? 0.0 : dbt;
            for (size_t a = 0; a < dd; ++a) dS[a] *= alpha;
        }
        if (dstate_in) memcpy(dstate_in + (size_t)bh * dd, dS, sizeof(double) * dd);
    done:
        free(states); free(o_la); free(o_nla); free(do_la); free(do_nla); free(lse);
        free(dS); free(Sbar); free(p); free(ret);
    }
    return err ? -2 : 0;
}

/* ---------------------------------------------------------------------------
 * Analytic backward of natsl_oracle_hybrid_fwd_block (reverse mode, token by token): the chain
 * rule applied to that forward, statement by statement, in reverse order.
 *   - softmax branch: query i reads key j <= i when j's block is a softmax block or j is in i's
 *     own block; ds = p (dp - <do, o>) as in the token-level backward (Section 4.2).
 *   - linear branch: inside a block the delta rule runs over every token from the block's start
 *     state.  A linear block hands its last state on, so the state gradient flows back through
 *     the block's tokens.  A softmax block hands on exp(sum g) * (start state): the incoming
 *     gradient goes straight to the start state (times the decay) and to every g of the block;
 *     the block's own token chain receives gradient from its outputs only.
 * Arguments as natsl_oracle_hybrid_bwd, plus the block length R and
 *   dscore [B, L/R, H, 2] (may be NULL): gradients of the two operation scores' masks per block
 *   (Section 4.2), index 0 = linear, 1 = softmax, computed for the active operation only and
 *   zero for the other ("set d score = 0 if the mask is 0"):
 *     softmax block t: sum over its keys j and all queries i >= j of dM_ij = p_ij (dp_ij - <do_i, o_i>)
 *                      (the dM^nla and d score^nla equations);
 *     linear block t : <dS_next, U_t>, U_t = the update the block commits to the state, i.e. the
 *                      gradient of a mask m_t in S_next = decay S_start + m_t U_t (the paper's
 *                      d score^la equation names the two factors dS and S without indices).
 * ------------------------------------------------------------------------- */
int natsl_oracle_hybrid_bwd_block(const double *q, const double *k, const double *v,
                                  const double *g, const double *beta, const uint8_t *route,
                                  const double *w, const double *dout, int B, int L, int H, int d,
                                  int R, double scale_la, double scale_sm, double eps,
                                  const double *state_in, const double *dstate_out,
                                  double *dq, double *dk, double *dv, double *dg, double *dbeta,
                                  double *dw, double *dstate_in, double *dscore)
{
    if (d > 512 || d <= 0 || R <= 0 || L % R != 0) return -1;
    int err = 0, bad_route = 0;
    if (dscore) memset(dscore, 0, sizeof(double) * (size_t)B * (L / R) * H * 2);
    size_t dd = (size_t)d * d;
    int NB = L / R;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H;
        double *after = (double *)malloc(sizeof(double) * dd * (size_t)L);        /* state after token i */
        double *start = (double *)malloc(sizeof(double) * dd * (size_t)(NB + 1)); /* state at block starts */
        double *o_la = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *o_nla = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *do_la = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *do_nla = (double *)malloc(sizeof(double) * (size_t)L * d);
        double *lse = (double *)malloc(sizeof(double) * (size_t)L);
        double *dS = (double *)calloc(dd, sizeof(double));
        double *dC = (double *)malloc(sizeof(double) * dd);
        double *Sbar = (double *)malloc(sizeof(double) * dd);
        double *p = (double *)malloc(sizeof(double) * (size_t)(L + 1));
        if (!after || !start || !o_la || !o_nla || !do_la || !do_nla || !lse || !dS || !dC || !Sbar || !p) {
            err = 1;
            goto done;
        }
        /* ---- forward recomputation, keeping every state ---- */
        if (state_in) memcpy(start, state_in + (size_t)bh * dd, sizeof(double) * dd);
        else memset(start, 0, sizeof(double) * dd);
        for (int c = 0; c < NB; ++c) {
            int i0 = c * R, r = route[AT3(b, i0, h)] != 0;
            double g_block = 0.0;
            for (int i = i0; i < i0 + R; ++i) {
                size_t t = AT3(b, i, h);
                if ((route[t] != 0) != r) bad_route = 1;
                const double *qi = q + t * d, *ki = k + t * d, *vi = v + t * d;
                const double *Sp = i == i0 ? start + dd * c : after + dd * (i - 1);
                double *Sn = after + dd * i;
                double alpha = exp(g[t]);
                g_block += g[t];
                for (size_t a = 0; a < dd; ++a) Sn[a] = alpha * Sp[a];
                for (int cc = 0; cc < d; ++cc) {
                    double ks = 0.0;
                    for (int a = 0; a < d; ++a) ks += ki[a] * Sn[(size_t)a * d + cc];
                    double e = vi[cc] - ks;
                    for (int a = 0; a < d; ++a) Sn[(size_t)a * d + cc] += beta[t] * ki[a] * e;
                }
                for (int cc = 0; cc < d; ++cc) {
                    double acc = 0.0;
                    for (int a = 0; a < d; ++a) acc += qi[a] * Sn[(size_t)a * d + cc];
                    o_la[(size_t)i * d + cc] = scale_la * acc;
                    o_nla[(size_t)i * d + cc] = 0.0;
                }
                /* softmax branch: keys of softmax blocks and of the own block, j <= i */
                double m = -INFINITY;
                for (int j = 0; j <= i; ++j) {
                    size_t tj = AT3(b, j, h);
                    p[j] = -INFINITY;
                    if (!(route[tj] || j >= i0)) continue;
                    const double *kj = k + tj * d;
                    double sc = 0.0;
                    for (int a = 0; a < d; ++a) sc += qi[a] * kj[a];
                    p[j] = scale_sm * sc;
                    if (p[j] > m) m = p[j];
                }
                double z = 0.0;
                for (int j = 0; j <= i; ++j) if (p[j] > -INFINITY) { p[j] = exp(p[j] - m); z += p[j]; } else p[j] = 0.0;
                for (int j = 0; j <= i; ++j) {
                    if (p[j] == 0.0) continue;
                    const double *vj = v + AT3(b, j, h) * d;
                    for (int cc = 0; cc < d; ++cc) o_nla[(size_t)i * d + cc] += p[j] / z * vj[cc];
                }
                lse[i] = m + log(z);               /* the own token is always visible: z > 0 */
            }
            double *Snext = start + dd * (c + 1);
            if (r) {
                double decay = exp(g_block);
                for (size_t a = 0; a < dd; ++a) Snext[a] = decay * start[dd * c + a];
            } else {
                memcpy(Snext, after + dd * (i0 + R - 1), sizeof(double) * dd);
            }
        }
        /* ---- combination backward, row by row (as in the token-level backward) ---- */
        for (int i = 0; i < L; ++i) {
            size_t t = AT3(b, i, h);
            double wn = w ? w[t * 2] : 0.5, wl = w ? w[t * 2 + 1] : 0.5;
            const double *ol = o_la + (size_t)i * d, *on = o_nla + (size_t)i * d;
            const double *dy = dout + t * d;
            double fl = rms_factor(ol, d, eps), fn = rms_factor(on, d, eps);
            double dwn = 0.0, dwl = 0.0, ml = 0.0, mn = 0.0;
            for (int c = 0; c < d; ++c) {
                dwn += dy[c] * on[c] * fn;
                dwl += dy[c] * ol[c] * fl;
                mn += wn * dy[c] * on[c] * fn;
                ml += wl * dy[c] * ol[c] * fl;
            }
            mn /= d; ml /= d;
            for (int c = 0; c < d; ++c) {
                do_nla[(size_t)i * d + c] = fn * (wn * dy[c] - on[c] * fn * mn);
                do_la[(size_t)i * d + c] = fl * (wl * dy[c] - ol[c] * fl * ml);
            }
            if (dw) { dw[t * 2] = dwn; dw[t * 2 + 1] = dwl; }
        }
        for (int i = 0; i < L; ++i) {
            size_t t = AT3(b, i, h);
            for (int a = 0; a < d; ++a) { dq[t * d + a] = 0.0; dk[t * d + a] = 0.0; dv[t * d + a] = 0.0; }
            dg[t] = 0.0;
        }
        /* ---- softmax branch backward ---- */
        for (int i = 0; i < L; ++i) {
            size_t t = AT3(b, i, h);
            int i0 = i / R * R;
            const double *qi = q + t * d;
            const double *doi = do_nla + (size_t)i * d, *oi = o_nla + (size_t)i * d;
            double D = 0.0;
            for (int c = 0; c < d; ++c) D += doi[c] * oi[c];
            for (int j = 0; j <= i; ++j) {
                size_t tj = AT3(b, j, h);
                if (!(route[tj] || j >= i0)) continue;
                const double *kj = k + tj * d, *vj = v + tj * d;
                double sc = 0.0, dp = 0.0;
                for (int a = 0; a < d; ++a) sc += qi[a] * kj[a];
                double pij = exp(scale_sm * sc - lse[i]);
                for (int c = 0; c < d; ++c) dp += doi[c] * vj[c];
                double ds = pij * (dp - D);
                if (dscore && route[tj]) dscore[(((size_t)b * NB + j / R) * H + h) * 2 + 1] += ds;
                for (int c = 0; c < d; ++c) dv[tj * d + c] += pij * doi[c];
                for (int a = 0; a < d; ++a) {
                    dq[t * d + a] += scale_sm * ds * kj[a];
                    dk[tj * d + a] += scale_sm * ds * qi[a];
                }
            }
        }
        /* ---- linear branch backward: blocks in reverse order ---- */
        if (dstate_out) memcpy(dS, dstate_out + (size_t)bh * dd, sizeof(double) * dd);
        for (int c = NB - 1; c >= 0; --c) {
            int i0 = c * R, r = route[AT3(b, i0, h)] != 0;
            double dg_block = 0.0;
            if (r) {
                /* next start = exp(sum g) * start_c: straight to the start state and to every g */
                double g_block = 0.0, acc = 0.0;
                for (int i = i0; i < i0 + R; ++i) g_block += g[AT3(b, i, h)];
                double decay = exp(g_block);
                for (size_t a = 0; a < dd; ++a) {
                    acc += dS[a] * start[dd * c + a];
                    dC[a] = decay * dS[a];
                    dS[a] = 0.0;                   /* the block's own chain feeds nothing later */
                }
                dg_block = decay * acc;
            } else {
                memset(dC, 0, sizeof(double) * dd);
                if (dscore) {   /* <dS_next, committed update>, update = last state - decayed start */
                    double g_block = 0.0, acc = 0.0;
                    for (int i = i0; i < i0 + R; ++i) g_block += g[AT3(b, i, h)];
                    double decay = exp(g_block);
                    const double *Se = after + dd * (i0 + R - 1);
                    for (size_t a = 0; a < dd; ++a) acc += dS[a] * (Se[a] - decay * start[dd * c + a]);
                    dscore[(((size_t)b * NB + c) * H + h) * 2] = acc;
                }
            }
            for (int i = i0 + R - 1; i >= i0; --i) {
                size_t t = AT3(b, i, h);
                const double *qi = q + t * d, *ki = k + t * d, *vi = v + t * d;
                const double *Sp = i == i0 ? start + dd * c : after + dd * (i - 1);
                const double *Sn = after + dd * i;
                const double *doi = do_la + (size_t)i * d;
                double alpha = exp(g[t]), bt = beta[t];
                for (int a = 0; a < d; ++a) {
                    double acc = 0.0;
                    for (int cc = 0; cc < d; ++cc) acc += doi[cc] * Sn[(size_t)a * d + cc];
                    dq[t * d + a] += scale_la * acc;
                    for (int cc = 0; cc < d; ++cc) dS[(size_t)a * d + cc] += scale_la * qi[a] * doi[cc];
                }
                for (size_t a = 0; a < dd; ++a) Sbar[a] = alpha * Sp[a];
                double dbt = 0.0;
                for (int cc = 0; cc < d; ++cc) {
                    double ks = 0.0, kds = 0.0;
                    for (int a = 0; a < d; ++a) {
                        ks += ki[a] * Sbar[(size_t)a * d + cc];
                        kds += ki[a] * dS[(size_t)a * d + cc];
                    }
                    double e = vi[cc] - ks;
                    double de = bt * kds;
                    dbt += kds * e;
                    dv[t * d + cc] += de;
                    for (int a = 0; a < d; ++a)
                        dk[t * d + a] += bt * e * dS[(size_t)a * d + cc] - de * Sbar[(size_t)a * d + cc];
                    for (int a = 0; a < d; ++a) dS[(size_t)a * d + cc] -= ki[a] * de;
                }
                double da = 0.0;
                for (size_t a = 0; a < dd; ++a) da += dS[a] * Sp[a];
                dg[t] = alpha * da + dg_block;
                dbeta[t] = dbt;
                for (size_t a = 0; a < dd; ++a) dS[a] *= alpha;
            }
            for (size_t a = 0; a < dd; ++a) dS[a] += dC[a];
        }
        if (dstate_in) memcpy(dstate_in + (size_t)bh * dd, dS, sizeof(double) * dd);
    done:
        free(after); free(start); free(o_la); free(o_nla); free(do_la); free(do_nla); free(lse);
        free(dS); free(dC); free(Sbar); free(p);
    }
    if (err) return -2;
    return bad_route ? -4 : 0;
}

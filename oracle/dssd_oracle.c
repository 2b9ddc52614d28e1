/*
 * CPU oracle for one round of split speculative verification (DSSD, Algorithm 2).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision
 * statement of what the verification round computes.  It exists to check the
 * CUDA library and to be timed as a CPU baseline; the product never calls it
 * and it shares no code, tables or helpers with the CUDA sources.
 *
 * Everything is sequential and in float64; sums run in index order; there is no
 * blocking, fusion or reordering.  A batch is B independent sequences, each a
 * separate run of the paper's single-sequence algorithm.
 *
 * Reading of the acceptance rule: Algorithm 2 prints the ratio as q/p while the
 * residual it pairs with is norm(max(0, P - Q)) (Section 2.1, "Resample").  Only
 * u < min(1, p(x)/q(x)) together with that residual reproduces the target
 * distribution, so that direction is used here.
 *
 * Indices are 0-based: accept_len n = j - 1 where j is the paper's 1-based
 * position of the first rejected token (j = gamma + 1 when all are accepted).
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1

#define FLAG_BAD_TOKEN 1u      /* edge: a drafted token id outside [0, V)          */
#define FLAG_NONFINITE 2u      /* edge: a target row without a finite log-sum-exp  */

#define RS_FLAG_BONUS 1u       /* device: n == gamma, sampled from P_{gamma+1}     */
#define RS_FLAG_FALLBACK 2u    /* device: residual mass <= 0, sampled from P_j     */
#define RS_FLAG_INVALID 4u     /* device: no positive mass, or n outside [0,gamma] */

static double load_logit(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORACLE_BF16) {
        union { uint32_t u; float f; } cvt;
        cvt.u = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        return (double)cvt.f;
    }
    return (double)((const float *)base)[idx];
}

/*
 * Target distribution of one row: P(v) = softmax(l_v / T)  (the "P_j(x)" that
 * Algorithm 2 obtains from M_p; temperature as in Section 4).
 *   z_v = l_v / T;  m = max z;  S = sum_v exp(z_v - m);  lse = m + ln S.
 * Returns lse; *ok = 0 when lse is not finite (NaN, +inf, or an all -inf row).
 */
static double row_lse(const void *row, int dtype, int V, double T, int *ok)
{
    double m = -INFINITY, S = 0.0, lse;
    int has_nan = 0;
    for (int v = 0; v < V; ++v) {
        double z = load_logit(row, dtype, v) / T;
        if (z != z) has_nan = 1;
        if (z > m) m = z;
    }
    if (has_nan || !(m > -INFINITY) || !(m < INFINITY)) { *ok = 0; return NAN; }
    for (int v = 0; v < V; ++v)
        S += exp(load_logit(row, dtype, v) / T - m);
    lse = m + log(S);
    *ok = (lse == lse) && (lse > -INFINITY) && (lse < INFINITY);
    return lse;
}

/*
 * Edge half of Algorithm 2 ("Verification Process" + "Downlink Transmission").
 *
 * target_logits [B, gamma+1, V] with row_stride elements between rows
 * draft_tokens  [B, gamma]   x_i
 * draft_q_tok   [B, gamma]   q_i(x_i) as uploaded by the device
 * uniforms      [B, gamma]   r_i
 * outputs:
 *   accept_len [B]           n = number of accepted draft tokens
 *   p_row      [B, V]        P_{n+1}(.) rounded to float32 (the downlink payload,
 *                            b_prob = 32 bits); row of the bonus position when n == gamma
 *   p_row64    [B, V]        the same row before rounding (may be NULL)
 *   p_tok      [B, gamma]    p_i(x_i)   (may be NULL)
 *   lse        [B, gamma+1]  (may be NULL)
 *   flags      [B]           (may be NULL)
 *   margin_acc [B]           min over tested positions of |u_i - min(1, ratio_i)| (may be NULL)
 */
int dssd_oracle_edge_verify(const void *target_logits, int dtype, int64_t row_stride,
                            const int32_t *draft_tokens, const float *draft_q_tok,
                            const float *uniforms, float temperature,
                            int B, int gamma, int V,
                            int32_t *accept_len, float *p_row, double *p_row64,
                            double *p_tok, double *lse, uint32_t *flags, double *margin_acc)
{
    const double T = (double)temperature;
    const size_t esz = (dtype == ORACLE_BF16) ? 2 : 4;
    if (B < 1 || gamma < 0 || V < 1 || !(T > 0.0) || row_stride < V) return 1;
    for (int b = 0; b < B; ++b) {
        uint32_t fl = 0;
        int n = gamma;          /* j - 1; stays gamma when Flag remains 1 */
        int flag_open = 1;      /* the paper's Flag */
        double margin = INFINITY;
        for (int i = 0; i <= gamma; ++i) {
            const char *row = (const char *)target_logits +
                              ((size_t)b * (size_t)(gamma + 1) + (size_t)i) * (size_t)row_stride * esz;
            int ok;
            double l = row_lse(row, dtype, V, T, &ok);
            if (!ok) fl |= FLAG_NONFINITE;
            if (lse) lse[(size_t)b * (gamma + 1) + i] = l;
            if (i == gamma) break;
            /* p_i(x_i) and the acceptance test  r_i < min{1, p_i(x_i)/q_i(x_i)} */
            int32_t x = draft_tokens[(size_t)b * gamma + i];
            double u = (double)uniforms[(size_t)b * gamma + i];
            double q = (double)draft_q_tok[(size_t)b * gamma + i];
            double p, ratio;
            int accept;
            if (x < 0 || x >= V) {
                fl |= FLAG_BAD_TOKEN;
                p = NAN;
                accept = 0;
                ratio = NAN;
            } else {
                p = exp(load_logit(row, dtype, x) / T - l);
                if (q != q) ratio = NAN;
                else if (q <= 0.0) ratio = (p > 0.0) ? INFINITY : 0.0;
                else ratio = p / q;
                accept = (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
            }
            if (p_tok) p_tok[(size_t)b * gamma + i] = p;
            if (flag_open) {
                if (ratio == ratio) {
                    double d = fabs(u - (ratio < 1.0 ? ratio : 1.0));
                    if (d < margin) margin = d;
                }
                if (!accept) { n = i; flag_open = 0; }
            }
        }
        accept_len[b] = n;
        if (flags) flags[b] = fl;
        if (margin_acc) margin_acc[b] = margin;
        /* downlink payload: the single row P_{n+1}(.) */
        {
            const char *row = (const char *)target_logits +
                              ((size_t)b * (size_t)(gamma + 1) + (size_t)n) * (size_t)row_stride * esz;
            int ok;
            double l = row_lse(row, dtype, V, T, &ok);
            for (int v = 0; v < V; ++v) {
                double pv = exp(load_logit(row, dtype, v) / T - l);
                if (p_row64) p_row64[(size_t)b * V + v] = pv;
                p_row[(size_t)b * V + v] = (float)pv;
            }
        }
    }
    return 0;
}

/*
 * Inverse-CDF draw in index order from unnormalised non-negative weights r_v:
 * token = min{k : sum_{v<=k} r_v > u * Z},  Z = sum_v r_v;
 * when rounding leaves no such k, the last index with r_v > 0.
 * mode 0: r = max(0, p - q); mode 1: r = p.  Returns -1 if Z is not > 0 and finite.
 */
static int32_t inverse_cdf(const float *p, const float *q, int mode, int V, double u,
                           double *Z_out, double *margin)
{
    double Z = 0.0;
    for (int v = 0; v < V; ++v) {
        double r = mode ? (double)p[v] : fmax(0.0, (double)p[v] - (double)q[v]);
        Z += r;
    }
    *Z_out = Z;
    if (!(Z > 0.0) || !(Z < INFINITY)) return -1;
    double t = u * Z, C = 0.0, Cprev = 0.0;
    int32_t last_pos = -1;
    for (int v = 0; v < V; ++v) {
        double r = mode ? (double)p[v] : fmax(0.0, (double)p[v] - (double)q[v]);
        Cprev = C;
        C += r;
        if (r > 0.0) last_pos = v;
        if (C > t) {
            if (margin) {
                double lo = t - Cprev, hi = C - t;
                *margin = (lo < hi ? lo : hi) / Z;
            }
            return v;
        }
    }
    if (margin) *margin = 0.0;
    return last_pos;
}

/*
 * Device half of Algorithm 2 ("Resample"), plus the bonus draw x_{gamma+1} ~ P_{gamma+1}
 * for sequences whose drafts were all accepted.
 *
 * p_row      [B, V]         float32 row received over the downlink
 * draft_q    [B, gamma, V]  float32 Q_i(.) kept on the device; only row n is read
 * accept_len [B]            n
 * uniforms   [B]            u'
 * outputs: token [B]; flags [B] (may be NULL); margin_cdf [B] = distance of u'Z to the
 * nearest CDF step, relative to Z (may be NULL); Z [B] (may be NULL).
 */
int dssd_oracle_device_resample(const float *p_row, const float *draft_q,
                                const int32_t *accept_len, const float *uniforms,
                                int B, int gamma, int V,
                                int32_t *token, uint32_t *flags, double *margin_cdf, double *Z_out)
{
    if (B < 1 || gamma < 0 || V < 1) return 1;
    for (int b = 0; b < B; ++b) {
        const float *p = p_row + (size_t)b * V;
        int n = accept_len[b];
        double u = (double)uniforms[b];
        double Z = 0.0, mg = 0.0;
        uint32_t fl = 0;
        int32_t tok;
        if (n < 0 || n > gamma) {
            fl = RS_FLAG_INVALID;
            tok = -1;
        } else {
            if (n == gamma) {
                fl |= RS_FLAG_BONUS;
                tok = inverse_cdf(p, NULL, 1, V, u, &Z, &mg);
            } else {
                const float *q = draft_q + ((size_t)b * gamma + n) * (size_t)V;
                tok = inverse_cdf(p, q, 0, V, u, &Z, &mg);
                if (tok < 0) {
                    fl |= RS_FLAG_FALLBACK;
                    tok = inverse_cdf(p, NULL, 1, V, u, &Z, &mg);
                }
            }
            if (tok < 0) { fl |= RS_FLAG_INVALID; mg = 0.0; }
        }
        token[b] = tok;
        if (flags) flags[b] = fl;
        if (margin_cdf) margin_cdf[b] = mg;
        if (Z_out) Z_out[b] = Z;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Truncated-support variant (Section 4: the experiments sample with top-k, k = 10, T = 1).
 *
 * Reading: "top-k sampling" restricts a model's distribution to its k most likely tokens and
 * renormalises over them.  The support of a row is its k largest logits; equal logits are
 * ordered by vocabulary index, lower index first, so the support is unique.  Inside the
 * support P(v) = exp(l_v/T - m) / sum_{w in support} exp(l_w/T - m), outside it P(v) = 0.
 * The draft side truncates its own distributions the same way before it samples, so the
 * scalars q_i(x_i) it uploads and the rows Q_i it keeps are truncated ones; Algorithm 2 then
 * runs unchanged on the truncated P and Q, and the downlink carries k (index, value) pairs
 * instead of |V| values.
 * ------------------------------------------------------------------------------------------ */

#define TOPK_MAX 32

/*
 * Support and probabilities of one row.  Selection by k successive maxima: pick r is the
 * largest element that comes strictly after pick r-1 in the order (logit descending, index
 * ascending).  idx/prob are in that order.  *ok = 0 (idx = -1, prob = NaN) when the row
 * holds a NaN or +inf, or has no entry above -inf.
 */
static void row_topk(const void *row, int dtype, int V, int k, double T,
                     int32_t *idx, double *prob, int *ok)
{
    double val[TOPK_MAX];
    int bad = 0;
    double top = -INFINITY;
    for (int v = 0; v < V; ++v) {
        double l = load_logit(row, dtype, v);
        if (l != l || l == INFINITY) bad = 1;
        if (l > top) top = l;
    }
    if (bad || !(top > -INFINITY)) {
        for (int r = 0; r < k; ++r) { idx[r] = -1; prob[r] = NAN; }
        *ok = 0;
        return;
    }
    double prev_val = INFINITY;
    int32_t prev_idx = -1;
    for (int r = 0; r < k; ++r) {
        double best = 0.0;
        int32_t best_idx = -1;
        for (int v = 0; v < V; ++v) {
            double l = load_logit(row, dtype, v);
            int after_prev = (l < prev_val) || (l == prev_val && v > prev_idx);
            if (!after_prev) continue;
            if (best_idx < 0 || l > best) { best = l; best_idx = v; }
        }
        idx[r] = best_idx;
        val[r] = best;
        prev_val = best;
        prev_idx = best_idx;
    }
    {
        double m = val[0] / T, S = 0.0;
        for (int r = 0; r < k; ++r) S += exp(val[r] / T - m);
        for (int r = 0; r < k; ++r) prob[r] = exp(val[r] / T - m) / S;
    }
    *ok = 1;
}

/*
 * Edge half of Algorithm 2 on truncated distributions.
 *
 * inputs as dssd_oracle_edge_verify, plus k (1 <= k <= min(V, 32)); draft_q_tok holds the
 * draft's truncated q_i(x_i).
 * outputs:
 *   accept_len [B]
 *   p_idx  [B, k]   support of row n in (logit descending, index ascending) order; -1 for a
 *                   row without a finite distribution
 *   p_val  [B, k]   its probabilities rounded to float32 (the downlink payload)
 *   p_val64 [B, k]  before rounding (may be NULL)
 *   p_tok  [B, gamma]  P_i(x_i): 0 outside the support (may be NULL)
 *   flags  [B], margin_acc [B]  as in dssd_oracle_edge_verify (may be NULL)
 */
int dssd_oracle_edge_verify_topk(const void *target_logits, int dtype, int64_t row_stride,
                                 const int32_t *draft_tokens, const float *draft_q_tok,
                                 const float *uniforms, float temperature,
                                 int B, int gamma, int V, int k,
                                 int32_t *accept_len, int32_t *p_idx, float *p_val, double *p_val64,
                                 double *p_tok, uint32_t *flags, double *margin_acc)
{
    const double T = (double)temperature;
    const size_t esz = (dtype == ORACLE_BF16) ? 2 : 4;
    if (B < 1 || gamma < 0 || V < 1 || !(T > 0.0) || row_stride < V) return 1;
    if (k < 1 || k > V || k > TOPK_MAX) return 1;
    for (int b = 0; b < B; ++b) {
        uint32_t fl = 0;
        int n = gamma;
        int flag_open = 1;
        double margin = INFINITY;
        int32_t idx[TOPK_MAX];
        double prob[TOPK_MAX];
        for (int i = 0; i <= gamma; ++i) {
            const char *row = (const char *)target_logits +
                              ((size_t)b * (size_t)(gamma + 1) + (size_t)i) * (size_t)row_stride * esz;
            int ok;
            row_topk(row, dtype, V, k, T, idx, prob, &ok);
            if (!ok) fl |= FLAG_NONFINITE;
            if (i == gamma) break;
            int32_t x = draft_tokens[(size_t)b * gamma + i];
            double u = (double)uniforms[(size_t)b * gamma + i];
            double q = (double)draft_q_tok[(size_t)b * gamma + i];
            double p, ratio;
            int accept;
            if (x < 0 || x >= V) {
                fl |= FLAG_BAD_TOKEN;
                p = NAN;
                accept = 0;
                ratio = NAN;
            } else {
                if (!ok) p = NAN;
                else {
                    p = 0.0;
                    for (int r = 0; r < k; ++r) if (idx[r] == x) p = prob[r];
                }
                if (q != q || p != p) ratio = NAN;
                else if (q <= 0.0) ratio = (p > 0.0) ? INFINITY : 0.0;
                else ratio = p / q;
                accept = (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
            }
            if (p_tok) p_tok[(size_t)b * gamma + i] = p;
            if (flag_open) {
                if (ratio == ratio) {
                    double d = fabs(u - (ratio < 1.0 ? ratio : 1.0));
                    if (d < margin) margin = d;
                }
                if (!accept) { n = i; flag_open = 0; }
            }
        }
        accept_len[b] = n;
        if (flags) flags[b] = fl;
        if (margin_acc) margin_acc[b] = margin;
        {
            const char *row = (const char *)target_logits +
                              ((size_t)b * (size_t)(gamma + 1) + (size_t)n) * (size_t)row_stride * esz;
            int ok;
            row_topk(row, dtype, V, k, T, idx, prob, &ok);
            for (int r = 0; r < k; ++r) {
                p_idx[(size_t)b * k + r] = idx[r];
                p_val[(size_t)b * k + r] = (float)prob[r];
                if (p_val64) p_val64[(size_t)b * k + r] = prob[r];
            }
        }
    }
    return 0;
}

/*
 * Device half on truncated distributions: the residual max(0, P - Q_n) lives on P's support,
 * so the draw walks P's k entries in increasing vocabulary index (the order the dense draw
 * walks the vocabulary in) with Q_n looked up by index (0 where Q_n has no such entry; the
 * first match if an index is listed twice).
 *
 * p_idx, p_val [B, k]; q_idx, q_val [B, gamma, k] (only row n is read); accept_len, uniforms [B].
 * A negative p_idx marks a sequence without a row: token = -1, RS_FLAG_INVALID.
 */
int dssd_oracle_device_resample_topk(const int32_t *p_idx, const float *p_val,
                                     const int32_t *q_idx, const float *q_val,
                                     const int32_t *accept_len, const float *uniforms,
                                     int B, int gamma, int k,
                                     int32_t *token, uint32_t *flags, double *margin_cdf, double *Z_out)
{
    if (B < 1 || gamma < 0 || k < 1 || k > TOPK_MAX) return 1;
    for (int b = 0; b < B; ++b) {
        int n = accept_len[b];
        double u = (double)uniforms[b];
        double Z = 0.0, mg = 0.0;
        uint32_t fl = 0;
        int32_t tok = -1;
        int32_t sid[TOPK_MAX];
        float sp[TOPK_MAX], sq[TOPK_MAX];
        int has_row = 1;
        for (int e = 0; e < k; ++e) if (p_idx[(size_t)b * k + e] < 0) has_row = 0;
        if (n < 0 || n > gamma || !has_row) {
            fl = RS_FLAG_INVALID;
        } else {
            /* P's entries in increasing index (insertion sort) */
            for (int e = 0; e < k; ++e) {
                int32_t id = p_idx[(size_t)b * k + e];
                float pv = p_val[(size_t)b * k + e];
                int pos = e;
                while (pos > 0 && sid[pos - 1] > id) {
                    sid[pos] = sid[pos - 1];
                    sp[pos] = sp[pos - 1];
                    --pos;
                }
                sid[pos] = id;
                sp[pos] = pv;
            }
            int pos_tok;
            if (n == gamma) {
                fl |= RS_FLAG_BONUS;
                pos_tok = inverse_cdf(sp, NULL, 1, k, u, &Z, &mg);
            } else {
                const int32_t *qi = q_idx + ((size_t)b * gamma + n) * (size_t)k;
                const float *qv = q_val + ((size_t)b * gamma + n) * (size_t)k;
                for (int e = 0; e < k; ++e) {
                    sq[e] = 0.0f;
                    for (int f = k - 1; f >= 0; --f) if (qi[f] == sid[e]) sq[e] = qv[f];
                }
                pos_tok = inverse_cdf(sp, sq, 0, k, u, &Z, &mg);
                if (pos_tok < 0) {
                    fl |= RS_FLAG_FALLBACK;
                    pos_tok = inverse_cdf(sp, NULL, 1, k, u, &Z, &mg);
                }
            }
            if (pos_tok < 0) { fl |= RS_FLAG_INVALID; mg = 0.0; }
            else tok = sid[pos_tok];
        }
        token[b] = tok;
        if (flags) flags[b] = fl;
        if (margin_cdf) margin_cdf[b] = mg;
        if (Z_out) Z_out[b] = Z;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Algorithm 1 (DSD): the verification that the paper's split scheme is compared with.  The
 * edge holds the full draft rows Q_i(.) (they were uploaded), so it tests every position with
 * q_i(x_i) read from the row, and on the first rejection resamples from
 * norm(max(0, P_n - Q_n)) itself; when all drafts pass it samples the bonus token from
 * P_{gamma+1}.  No row is transmitted, so nothing is rounded to a payload format: the residual
 * is formed from the float64 target probabilities.
 *
 * target_logits [B, gamma+1, V] (row_stride elements between rows), draft_q [B, gamma, V] float32,
 * draft_tokens [B, gamma], uniforms [B, gamma] (acceptance), uniforms_rs [B] (the draw).
 * outputs: accept_len [B], token [B], flags [B] (edge flags, may be NULL), rs_flags [B] (may be
 * NULL), margin_acc [B], margin_cdf [B] (may be NULL) as in the split functions, Z_out [B] (may be
 * NULL): the mass sum_v r_v that the returned token was drawn from (0 when there was none).
 * ------------------------------------------------------------------------------------------ */
int dssd_oracle_dsd_verify(const void *target_logits, int dtype, int64_t row_stride,
                           const float *draft_q, const int32_t *draft_tokens,
                           const float *uniforms, const float *uniforms_rs, float temperature,
                           int B, int gamma, int V,
                           int32_t *accept_len, int32_t *token, uint32_t *flags, uint32_t *rs_flags,
                           double *margin_acc, double *margin_cdf, double *Z_out)
{
    const double T = (double)temperature;
    const size_t esz = (dtype == ORACLE_BF16) ? 2 : 4;
    if (B < 1 || gamma < 0 || V < 1 || !(T > 0.0) || row_stride < V) return 1;
    for (int b = 0; b < B; ++b) {
        uint32_t fl = 0, rfl = 0;
        int n = gamma, flag_open = 1;
        double margin = INFINITY;
        for (int i = 0; i <= gamma; ++i) {
            const char *row = (const char *)target_logits +
                              ((size_t)b * (size_t)(gamma + 1) + (size_t)i) * (size_t)row_stride * esz;
            int ok;
            double l = row_lse(row, dtype, V, T, &ok);
            if (!ok) fl |= FLAG_NONFINITE;
            if (i == gamma) break;
            int32_t x = draft_tokens[(size_t)b * gamma + i];
            double u = (double)uniforms[(size_t)b * gamma + i];
            double ratio;
            int accept;
            if (x < 0 || x >= V) {
                fl |= FLAG_BAD_TOKEN;
                accept = 0;
                ratio = NAN;
            } else {
                double q = (double)draft_q[((size_t)b * gamma + i) * (size_t)V + x];
                double p = exp(load_logit(row, dtype, x) / T - l);
                if (q != q) ratio = NAN;
                else if (q <= 0.0) ratio = (p > 0.0) ? INFINITY : 0.0;
                else ratio = p / q;
                accept = (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
            }
            if (flag_open) {
                if (ratio == ratio) {
                    double d = fabs(u - (ratio < 1.0 ? ratio : 1.0));
                    if (d < margin) margin = d;
                }
                if (!accept) { n = i; flag_open = 0; }
            }
        }
        accept_len[b] = n;
        /* the draw at position n: residual against Q_n, or the bonus row itself */
        {
            const char *row = (const char *)target_logits +
                              ((size_t)b * (size_t)(gamma + 1) + (size_t)n) * (size_t)row_stride * esz;
            const float *q = n < gamma ? draft_q + ((size_t)b * gamma + n) * (size_t)V : NULL;
            int ok;
            double l = row_lse(row, dtype, V, T, &ok);
            double u = (double)uniforms_rs[b];
            int32_t tok = -1;
            double mg = 0.0, Z_used = 0.0;
            if (n == gamma) rfl |= RS_FLAG_BONUS;
            for (int pass = 0; pass < 2 && tok < 0; ++pass) {
                /* pass 0: the residual (or the bonus row); pass 1: fall back to P_n when it has no mass */
                const float *qq = pass == 0 ? q : NULL;
                double Z = 0.0;
                if (pass == 1) {
                    if (!q) break;
                    rfl |= RS_FLAG_FALLBACK;
                }
                for (int v = 0; v < V; ++v) {
                    double p = exp(load_logit(row, dtype, v) / T - l);
                    Z += qq ? fmax(0.0, p - (double)qq[v]) : p;
                }
                if (!(Z > 0.0) || !(Z < INFINITY)) continue;
                Z_used = Z;
                double t = u * Z, C = 0.0, Cprev;
                int32_t last_pos = -1;
                for (int v = 0; v < V; ++v) {
                    double p = exp(load_logit(row, dtype, v) / T - l);
                    double r = qq ? fmax(0.0, p - (double)qq[v]) : p;
                    Cprev = C;
                    C += r;
                    if (r > 0.0) last_pos = v;
                    if (C > t) {
                        double lo = t - Cprev, hi = C - t;
                        mg = (lo < hi ? lo : hi) / Z;
                        tok = v;
                        break;
                    }
                }
                if (tok < 0) { tok = last_pos; mg = 0.0; }
            }
            if (tok < 0) { rfl |= RS_FLAG_INVALID; mg = 0.0; }
            token[b] = tok;
            if (margin_cdf) margin_cdf[b] = mg;
            if (Z_out) Z_out[b] = tok < 0 ? 0.0 : Z_used;
        }
        if (flags) flags[b] = fl;
        if (rs_flags) rs_flags[b] = rfl;
        if (margin_acc) margin_acc[b] = margin;
    }
    return 0;
}

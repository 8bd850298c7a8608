/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow, fp64 CPU statement of the two draft-verification procedures of
 * "Block Verification Accelerates Speculative Decoding" (arXiv 2403.10444):
 *
 *   - Token Verification  (Algorithm 1, residual distribution Eq. "pres-token")
 *   - Block Verification  (Algorithm 2, prefix recursion Eq. "def_as",
 *                          residual distribution Eq. "pres-block",
 *                          acceptance weights Eq. "pacc_block")
 *   - Greedy Block Verification (Algorithm 4, residual Eq. "pres_greedy"): one
 *                          iteration only; the distribution modification that must
 *                          follow it (Algorithm 5) needs the models and is not here
 *
 * The first two also on given probabilities instead of logits (oracle_verify_probs, pinned in
 * tests/test_oracle_probs.py).
 *
 * It follows the algorithms step by step in the paper's order and notation,
 * with no blocking, fusion or reordering.  It shares no code with the CUDA
 * library, and only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.
 *
 * Pins (see tests/test_oracle_*.py): the paper's two-token worked example
 * (expected accepted lengths 10/9 and 11/9), brute-force enumeration of every
 * drafted block showing the output law equals the target model's (Theorem 1 /
 * Eq. "output_block_distribution"), Lemma 3 (Pr(tau >= i | X^i) = p_i), the
 * expected-length ordering of Theorem 2, the gamma = 1 coincidence of the two
 * procedures, scipy's logsumexp for the normalisers, and explicit cumulative
 * sums for the sampler.  Algorithm 4 (tests/test_oracle_greedy.py): the paper's
 * account of the same example (12/9 accepted tokens, the 1/3 counter-example),
 * Lemma "block-accept", Theorem "greedy_one_iter" and Lemma
 * "greedy_block_identical" by enumeration in exact rationals.
 *
 * Notation (0-based storage rows, 1-based tokens):
 *   P_r = softmax(target_logits[b, r, :] / T),  r = 0..gamma    (M_b(. | c, X^r))
 *   Q_r = softmax(draft_logits [b, r, :] / T),  r = 0..gamma-1  (M_s(. | c, X^r))
 *   X_i = draft_tokens[b, i-1],  eta_i = uniforms[b, i-1],  i = 1..gamma
 *   uniforms[b, gamma]   drives the residual sample (tau < gamma)
 *   uniforms[b, gamma+1] drives the target sample   (tau == gamma)
 *
 * Readings taken where the paper is silent:
 *   - temperature divides both models' logits before the softmax;
 *   - a position is selectable only if its acceptance weight is > 0, and
 *     h_i := 0 when S_i = 0 (the 0/0 case of Eq. "pacc_block");
 *   - sampling is inverse-CDF in vocabulary-index order with a strict
 *     comparison: Y = min{k : C_k > u * W}; if rounding leaves none, the last
 *     k with positive weight;
 *   - a residual whose total mass is exactly 0 at the position that was selected is a domain
 *     error of the sequence: Eq. "pres-token" / "pres-block" divide by that mass, and the
 *     algorithms cannot arrive there (P_tau == Q_tau makes the ratio of the next test 1, so
 *     Algorithm 1 does not stop at tau and tau + 1 passes its test in Algorithms 2 and 4);
 *   - Algorithm 4: its last test is taken as eta_gamma <= pt_gamma like every other test
 *     (it is printed with "<"; the two differ on a set of measure zero); a test whose
 *     denominator sum is 0 passes; a position whose numerator sum is 0 is not selectable;
 *   - NaN / +inf logits in a row that is used, an all -inf row, a drafted token
 *     outside [0, V) or one whose draft logit is -inf are per-sequence domain
 *     errors: out_len = -1 and out_tokens = -1.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F64 = 2 };
enum { ORACLE_TOKEN_VERIFY = 0, ORACLE_BLOCK_VERIFY = 1, ORACLE_GREEDY_BLOCK_VERIFY = 2 };

/* One logit, widened exactly to double. */
static double logit_at(const void *base, int dtype, size_t idx)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)base)[idx];
    if (dtype == ORACLE_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return ((const double *)base)[idx];
}

/* log sum_x exp(z_x / T) over one row; returns 0, or 1 on a domain error. */
static int row_lse(const void *base, int dtype, size_t off, int V, double T,
                   double *lse_out)
{
    double m = -INFINITY;
    for (int x = 0; x < V; ++x) {
        double z = logit_at(base, dtype, off + (size_t)x) / T;
        if (isnan(z) || z == INFINITY)
            return 1;
        if (z > m)
            m = z;
    }
    if (!isfinite(m))
        return 1; /* every logit is -inf */
    double s = 0.0;
    for (int x = 0; x < V; ++x)
        s += exp(logit_at(base, dtype, off + (size_t)x) / T - m);
    *lse_out = m + log(s);
    return 0;
}

/* softmax probability of token x in a row whose log-normaliser is lse */
static double prob_at(const void *base, int dtype, size_t off, int x, double T,
                      double lse)
{
    return exp(logit_at(base, dtype, off + (size_t)x) / T - lse);
}

/*
 * Unnormalised sampling weight of token x at one position:
 *   max(p * P(x) - Q(x), 0)   (Eq. "pres-block"; p = 1 gives Eq. "pres-token"),
 * or P(x) itself when there is no draft row (the target sample at tau = gamma).
 */
static double weight_at(const void *tgt, size_t toff, double lse_t,
                        const void *drf, size_t doff, double lse_d, int have_draft,
                        int dtype, int x, double T, double p)
{
    double P = prob_at(tgt, dtype, toff, x, T, lse_t);
    if (!have_draft)
        return P;
    double Q = prob_at(drf, dtype, doff, x, T, lse_d);
    double w = p * P - Q;
    return w > 0.0 ? w : 0.0;
}

/*
 * Inverse-CDF sample in vocabulary-index order.  W = sum of weights and the
 * running sums C_k are plain sequential fp64 sums.  Returns the token, or -1
 * when the weights sum to nothing;
 * *margin receives min(u - C_{k-1}/W, C_k/W - u), the distance (in probability)
 * of u from the nearest edge of the chosen token's CDF cell.
 */
static int sample_index_order(const void *tgt, size_t toff, double lse_t,
                              const void *drf, size_t doff, double lse_d,
                              int have_draft, int dtype, int V, double T, double p,
                              double u, double *W_out, double *margin)
{
    double W = 0.0;
    for (int x = 0; x < V; ++x)
        W += weight_at(tgt, toff, lse_t, drf, doff, lse_d, have_draft, dtype, x, T, p);
    *W_out = W;
    if (!(W > 0.0)) {
        /* nothing to sample from: a domain error (see header) */
        *margin = 0.0;
        return -1;
    }
    double t = u * W, C = 0.0;
    int last_pos = -1;
    for (int x = 0; x < V; ++x) {
        double w = weight_at(tgt, toff, lse_t, drf, doff, lse_d, have_draft, dtype, x, T, p);
        double Cprev = C;
        C += w;
        if (w > 0.0)
            last_pos = x;
        if (C > t) {
            double lo = u - Cprev / W, hi = C / W - u;
            *margin = lo < hi ? lo : hi;
            return x;
        }
    }
    *margin = 0.0; /* u*W fell beyond the last running sum by rounding */
    return last_pos;
}

/* Everything one sequence needs; rows are addressed by element offsets. */
typedef struct {
    const void *tgt, *drf;
    const int32_t *X;   /* gamma drafted tokens */
    const float *u;     /* gamma + 2 uniforms   */
    int gamma, V, dtype;
    double T;
    size_t toff, doff;  /* offset of row 0 of this sequence in tgt / drf */
    const float *given_lse_d; /* gamma supplied draft log-normalisers, or NULL: compute them */
} seq_t;

typedef struct {
    double *p, *S, *h, *lse_t, *lse_d; /* per-sequence slices, may be NULL */
    double *margin_eta, *margin_smp;   /* one value each, may be NULL      */
} diag_t;

/*
 * Log-normaliser of draft row r: computed from the row, or, when the caller supplies the
 * normalisers (the drafting step has them already), the supplied value: M_s(x | c, X^r) is then
 * exp(z_x / T - supplied).  Returns 1 on a domain error (a supplied value that is not finite).
 */
static int draft_lse(const seq_t *s, int r, double *out)
{
    if (s->given_lse_d) {
        double v = (double)s->given_lse_d[r];
        if (!isfinite(v))
            return 1;
        *out = v;
        return 0;
    }
    return row_lse(s->drf, s->dtype, s->doff + (size_t)r * (size_t)s->V, s->V, s->T, out);
}

static void diag_fill_nan(const diag_t *d, int gamma)
{
    for (int i = 0; i <= gamma; ++i) {
        if (d->p) d->p[i] = NAN;
        if (d->h) d->h[i] = NAN;
        if (d->lse_t) d->lse_t[i] = NAN;
        if (i < gamma && d->S) d->S[i] = NAN;
        if (i < gamma && d->lse_d) d->lse_d[i] = NAN;
    }
    if (d->margin_eta) *d->margin_eta = NAN;
    if (d->margin_smp) *d->margin_smp = NAN;
}

static void emit(const seq_t *s, int tau, int Y, int32_t *out_tokens, int32_t *out_len)
{
    for (int i = 0; i <= s->gamma; ++i)
        out_tokens[i] = -1;
    if (tau < 0) { /* domain error */
        *out_len = -1;
        return;
    }
    for (int i = 0; i < tau; ++i)
        out_tokens[i] = s->X[i];
    out_tokens[tau] = Y;
    *out_len = tau + 1; /* the accepted prefix X_1..X_tau and the one sampled token Y */
}

/*
 * ln of the ratio M_b(X_i | c, X^{i-1}) / M_s(X_i | c, X^{i-1})  (Algorithm 1
 * "Set h_i", Algorithm 2 "Set p_i"): both distributions are the ones
 * conditioned on X^{i-1}, i.e. storage row i-1.  Returns 1 on a domain error.
 */
static int log_ratio(const seq_t *s, int i, double lse_t, double lse_d, double *lr)
{
    int x = s->X[i - 1];
    if (x < 0 || x >= s->V)
        return 1;
    size_t V = (size_t)s->V;
    double zq = logit_at(s->drf, s->dtype, s->doff + (size_t)(i - 1) * V + (size_t)x);
    double zp = logit_at(s->tgt, s->dtype, s->toff + (size_t)(i - 1) * V + (size_t)x);
    if (zq == -INFINITY)
        return 1; /* a token the draft model cannot have produced */
    *lr = (zp / s->T - lse_t) - (zq / s->T - lse_d);
    return 0;
}

/* ---------------- Algorithm 1: Token Verification ---------------- */
static void token_verify_one(const seq_t *s, const diag_t *d,
                             int32_t *out_tokens, int32_t *out_len)
{
    const int g = s->gamma;
    const size_t V = (size_t)s->V;
    double lse_t = 0.0, lse_d = 0.0, m_eta = INFINITY;
    diag_fill_nan(d, g);

    int tau = 0;
    for (int i = 1; i <= g; ++i) {
        /* the distributions conditioned on X^{i-1} */
        if (row_lse(s->tgt, s->dtype, s->toff + (size_t)(i - 1) * V, s->V, s->T, &lse_t) ||
            draft_lse(s, i - 1, &lse_d)) {
            emit(s, -1, -1, out_tokens, out_len);
            return;
        }
        if (d->lse_t) d->lse_t[i - 1] = lse_t;
        if (d->lse_d) d->lse_d[i - 1] = lse_d;
        double lr;
        if (log_ratio(s, i, lse_t, lse_d, &lr)) {
            emit(s, -1, -1, out_tokens, out_len);
            return;
        }
        double ratio = exp(lr);
        double h = ratio < 1.0 ? ratio : 1.0;       /* h_i^token = min(ratio, 1) */
        if (d->h) d->h[i] = h;
        double eta = (double)s->u[i - 1];
        double gap = fabs(eta - h);
        if (gap < m_eta) m_eta = gap;
        if (h > 0.0 && eta <= h)
            tau = i;
        else
            break;
    }
    if (d->h) d->h[0] = 1.0;

    /* the distributions conditioned on X^tau */
    if (row_lse(s->tgt, s->dtype, s->toff + (size_t)tau * V, s->V, s->T, &lse_t)) {
        emit(s, -1, -1, out_tokens, out_len);
        return;
    }
    if (d->lse_t) d->lse_t[tau] = lse_t;
    int have_draft = tau < g;
    if (have_draft) {
        if (draft_lse(s, tau, &lse_d)) {
            emit(s, -1, -1, out_tokens, out_len);
            return;
        }
        if (d->lse_d) d->lse_d[tau] = lse_d;
    }
    double u = (double)s->u[have_draft ? g : g + 1];
    double W, m_smp;
    int Y = sample_index_order(s->tgt, s->toff + (size_t)tau * V, lse_t,
                               s->drf, s->doff + (size_t)tau * V, lse_d,
                               have_draft, s->dtype, s->V, s->T, 1.0, u, &W, &m_smp);
    if (have_draft && d->S) d->S[tau] = W; /* residual mass sum_x max(P - Q, 0) */
    if (d->margin_eta) *d->margin_eta = m_eta;
    if (d->margin_smp) *d->margin_smp = m_smp;
    emit(s, Y < 0 ? -1 : tau, Y, out_tokens, out_len);
}

/* ---------------- Algorithm 2: Block Verification ---------------- */
static void block_verify_one(const seq_t *s, const diag_t *d,
                             int32_t *out_tokens, int32_t *out_len)
{
    const int g = s->gamma;
    const size_t V = (size_t)s->V;
    diag_fill_nan(d, g);

    double *lse_t = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *lse_d = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *p = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *S = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *h = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    int bad = 0;

    /* the conditional distributions along the sample path */
    for (int r = 0; r <= g && !bad; ++r) {
        bad |= row_lse(s->tgt, s->dtype, s->toff + (size_t)r * V, s->V, s->T, &lse_t[r]);
        if (r < g)
            bad |= draft_lse(s, r, &lse_d[r]);
    }

    /* p_0 = 1;  p_i = min{ p_{i-1} * M_b(X_i|c,X^{i-1}) / M_s(X_i|c,X^{i-1}), 1 } */
    p[0] = 1.0;
    for (int i = 1; i <= g && !bad; ++i) {
        double lr;
        if (log_ratio(s, i, lse_t[i - 1], lse_d[i - 1], &lr)) {
            bad = 1;
            break;
        }
        double v = p[i - 1] * exp(lr);
        p[i] = v < 1.0 ? v : 1.0;
    }
    if (bad) {
        emit(s, -1, -1, out_tokens, out_len);
        goto done;
    }

    /* S_i = sum_x max{ p_i * M_b(x|c,X^i) - M_s(x|c,X^i), 0 },  i = 0..gamma-1 */
    for (int i = 0; i < g; ++i) {
        double acc = 0.0;
        for (int x = 0; x < s->V; ++x)
            acc += weight_at(s->tgt, s->toff + (size_t)i * V, lse_t[i],
                             s->drf, s->doff + (size_t)i * V, lse_d[i], 1,
                             s->dtype, x, s->T, p[i]);
        S[i] = acc;
    }

    /* h_gamma = p_gamma;  h_i = S_i / (S_i + 1 - p_i) for i < gamma */
    h[0] = 1.0; /* tau = 0 is what remains when nothing is selected */
    for (int i = 1; i < g; ++i)
        h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0 - p[i]) : 0.0;
    h[g] = p[g];

    /* tau = the largest i with eta_i <= h_i (every i is tried: "continue") */
    int tau = 0;
    double m_eta = INFINITY;
    for (int i = 1; i <= g; ++i) {
        double eta = (double)s->u[i - 1];
        if (h[i] > 0.0 && eta <= h[i])
            tau = i;
    }
    /* comparisons at i >= tau decide the outcome; those below tau do not */
    for (int i = (tau > 0 ? tau : 1); i <= g; ++i) {
        double gap = fabs((double)s->u[i - 1] - h[i]);
        if (gap < m_eta) m_eta = gap;
    }

    {
        int have_draft = tau < g;
        double u = (double)s->u[have_draft ? g : g + 1];
        double W, m_smp;
        int Y = sample_index_order(s->tgt, s->toff + (size_t)tau * V, lse_t[tau],
                                   s->drf, s->doff + (size_t)tau * V, lse_d[tau],
                                   have_draft, s->dtype, s->V, s->T, p[tau], u, &W, &m_smp);
        if (d->margin_eta) *d->margin_eta = m_eta;
        if (d->margin_smp) *d->margin_smp = m_smp;
        emit(s, Y < 0 ? -1 : tau, Y, out_tokens, out_len);
    }
    for (int i = 0; i <= g; ++i) {
        if (d->p) d->p[i] = p[i];
        if (d->h) d->h[i] = h[i];
        if (d->lse_t) d->lse_t[i] = lse_t[i];
        if (i < g && d->S) d->S[i] = S[i];
        if (i < g && d->lse_d) d->lse_d[i] = lse_d[i];
    }
done:
    free(lse_t); free(lse_d); free(p); free(S); free(h);
}

/* ---------------- Algorithm 4: Greedy Block Verification ---------------- */
/*
 * Diagnostics: p receives the unclipped products pt_0..pt_gamma, S the numerator sums
 * sum_x max(pt_i P_i - Q_i, 0) (i = 0..gamma-1), h the ratios h_i as printed (they may
 * exceed 1, and are +inf when the denominator sum is 0), with h_0 := 1 and h_gamma := pt_gamma.
 */
static void greedy_block_verify_one(const seq_t *s, const diag_t *d,
                                    int32_t *out_tokens, int32_t *out_len)
{
    const int g = s->gamma;
    const size_t V = (size_t)s->V;
    diag_fill_nan(d, g);

    double *lse_t = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *lse_d = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *pt = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *num = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *h = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    int bad = 0;

    for (int r = 0; r <= g && !bad; ++r) {
        bad |= row_lse(s->tgt, s->dtype, s->toff + (size_t)r * V, s->V, s->T, &lse_t[r]);
        if (r < g)
            bad |= draft_lse(s, r, &lse_d[r]);
    }
    if (bad) {
        emit(s, -1, -1, out_tokens, out_len);
        goto done;
    }

    int tau = 0;
    pt[0] = 1.0;
    h[0] = 1.0;
    /* position 0 has no test; its numerator sum is the mass of the residual at tau = 0 */
    {
        double acc = 0.0;
        for (int x = 0; x < s->V; ++x)
            acc += weight_at(s->tgt, s->toff, lse_t[0], s->drf, s->doff, lse_d[0], 1,
                             s->dtype, x, s->T, 1.0);
        num[0] = acc;
    }
    for (int i = 1; i <= g - 1; ++i) {
        /* pt_i = pt_{i-1} * M_b(X_i | c, X^{i-1}) / M_s(X_i | c, X^{i-1}): no minimum */
        double lr;
        if (log_ratio(s, i, lse_t[i - 1], lse_d[i - 1], &lr)) {
            bad = 1;
            break;
        }
        pt[i] = pt[i - 1] * exp(lr);
        /* h_i = sum_x max{pt_i M_b(x) - M_s(x), 0} / sum_x max{M_s(x) - pt_i M_b(x), 0} */
        double a = 0.0, c = 0.0;
        for (int x = 0; x < s->V; ++x) {
            double P = prob_at(s->tgt, s->dtype, s->toff + (size_t)i * V, x, s->T, lse_t[i]);
            double Q = prob_at(s->drf, s->dtype, s->doff + (size_t)i * V, x, s->T, lse_d[i]);
            double w = pt[i] * P - Q;
            if (w > 0.0)
                a += w;
            else
                c += -w;
        }
        num[i] = a;
        h[i] = c > 0.0 ? a / c : (a > 0.0 ? INFINITY : 0.0);
        if (a > 0.0 && (double)s->u[i - 1] <= h[i])
            tau = i;
    }
    if (!bad) {
        double lr;
        if (log_ratio(s, g, lse_t[g - 1], lse_d[g - 1], &lr))
            bad = 1;
        else
            pt[g] = pt[g - 1] * exp(lr);
    }
    if (bad) {
        emit(s, -1, -1, out_tokens, out_len);
        goto done;
    }
    h[g] = pt[g];
    if ((double)s->u[g - 1] <= pt[g])
        tau = g;

    {
        /* tests at i >= tau decide the outcome; a test passes with probability min(h_i, 1) */
        double m_eta = INFINITY;
        for (int i = (tau > 0 ? tau : 1); i <= g; ++i) {
            double gap = fabs((double)s->u[i - 1] - (h[i] < 1.0 ? h[i] : 1.0));
            if (gap < m_eta) m_eta = gap;
        }
        int have_draft = tau < g;
        double u = (double)s->u[have_draft ? g : g + 1];
        double W, m_smp;
        int Y = sample_index_order(s->tgt, s->toff + (size_t)tau * V, lse_t[tau],
                                   s->drf, s->doff + (size_t)tau * V, lse_d[tau],
                                   have_draft, s->dtype, s->V, s->T, pt[tau], u, &W, &m_smp);
        if (d->margin_eta) *d->margin_eta = m_eta;
        if (d->margin_smp) *d->margin_smp = m_smp;
        emit(s, Y < 0 ? -1 : tau, Y, out_tokens, out_len);
    }
    for (int i = 0; i <= g; ++i) {
        if (d->p) d->p[i] = pt[i];
        if (d->h) d->h[i] = h[i];
        if (d->lse_t) d->lse_t[i] = lse_t[i];
        if (i < g && d->S) d->S[i] = num[i];
        if (i < g && d->lse_d) d->lse_d[i] = lse_d[i];
    }
done:
    free(lse_t); free(lse_d); free(pt); free(num); free(h);
}

/*
 * Batch entry.  All pointers are host pointers.
 *   algo: 0 = Token Verification, 1 = Block Verification, 2 = Greedy Block Verification
 *   target [B, gamma+1, V], draft [B, gamma, V] in dtype (0 f32, 1 bf16 bits, 2 f64)
 *   tokens [B, gamma] int32, uniforms [B, gamma+2] f32
 *   out_tokens [B, gamma+1], out_len [B]
 *   diagnostics (each may be NULL): p [B,gamma+1], S [B,gamma], h [B,gamma+1],
 *   lse_t [B,gamma+1], lse_d [B,gamma], margin_eta [B], margin_smp [B].
 *   Values an algorithm never forms are NaN (Token Verification forms h_i up to
 *   the first rejection, S only at tau, and no p).
 * Sequences are independent; the loop over b may run on several threads.
 * Returns 0, or 1 for an invalid argument.
 */
static int verify_impl(int algo, const void *target, const void *draft,
                  const int32_t *tokens, const float *uniforms, const float *given_lse_d,
                  int B, int gamma, int V, int dtype, double temperature,
                  int32_t *out_tokens, int32_t *out_len,
                  double *p, double *S, double *h, double *lse_t, double *lse_d,
                  double *margin_eta, double *margin_smp)
{
    if (!target || !draft || !tokens || !uniforms || !out_tokens || !out_len)
        return 1;
    if (B < 0 || gamma < 1 || V < 1 || !(temperature > 0.0) || !isfinite(temperature))
        return 1;
    if (dtype < 0 || dtype > 2 || algo < 0 || algo > 2)
        return 1;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int b = 0; b < B; ++b) {
        seq_t s;
        s.tgt = target; s.drf = draft;
        s.X = tokens + (size_t)b * (size_t)gamma;
        s.u = uniforms + (size_t)b * (size_t)(gamma + 2);
        s.gamma = gamma; s.V = V; s.dtype = dtype; s.T = temperature;
        s.toff = (size_t)b * (size_t)(gamma + 1) * (size_t)V;
        s.doff = (size_t)b * (size_t)gamma * (size_t)V;
        s.given_lse_d = given_lse_d ? given_lse_d + (size_t)b * (size_t)gamma : NULL;
        diag_t d;
        d.p = p ? p + (size_t)b * (size_t)(gamma + 1) : NULL;
        d.S = S ? S + (size_t)b * (size_t)gamma : NULL;
        d.h = h ? h + (size_t)b * (size_t)(gamma + 1) : NULL;
        d.lse_t = lse_t ? lse_t + (size_t)b * (size_t)(gamma + 1) : NULL;
        d.lse_d = lse_d ? lse_d + (size_t)b * (size_t)gamma : NULL;
        d.margin_eta = margin_eta ? margin_eta + b : NULL;
        d.margin_smp = margin_smp ? margin_smp + b : NULL;
        int32_t *ot = out_tokens + (size_t)b * (size_t)(gamma + 1);
        if (algo == ORACLE_BLOCK_VERIFY)
            block_verify_one(&s, &d, ot, out_len + b);
        else if (algo == ORACLE_GREEDY_BLOCK_VERIFY)
            greedy_block_verify_one(&s, &d, ot, out_len + b);
        else
            token_verify_one(&s, &d, ot, out_len + b);
    }
    return 0;
}

int oracle_verify(int algo, const void *target, const void *draft,
                  const int32_t *tokens, const float *uniforms,
                  int B, int gamma, int V, int dtype, double temperature,
                  int32_t *out_tokens, int32_t *out_len,
                  double *p, double *S, double *h, double *lse_t, double *lse_d,
                  double *margin_eta, double *margin_smp)
{
    return verify_impl(algo, target, draft, tokens, uniforms, NULL, B, gamma, V, dtype, temperature,
                       out_tokens, out_len, p, S, h, lse_t, lse_d, margin_eta, margin_smp);
}

/*
 * The same with the draft rows' log-normalisers supplied, given_lse_d [B, gamma] float
 * (ln sum_x exp(draft[b, r, x] / T), as the drafting step leaves them): the draft distributions
 * are exp(z / T - given).  Everything else as oracle_verify.
 */
int oracle_verify_lse(int algo, const void *target, const void *draft,
                      const int32_t *tokens, const float *uniforms, const float *given_lse_d,
                      int B, int gamma, int V, int dtype, double temperature,
                      int32_t *out_tokens, int32_t *out_len,
                      double *p, double *S, double *h, double *lse_t, double *lse_d,
                      double *margin_eta, double *margin_smp)
{
    if (!given_lse_d)
        return 1;
    return verify_impl(algo, target, draft, tokens, uniforms, given_lse_d, B, gamma, V, dtype,
                       temperature, out_tokens, out_len, p, S, h, lse_t, lse_d, margin_eta, margin_smp);
}

/*
 * The drafting step of Algorithm 3 (the small model draws X_1..X_gamma one after the other and
 * its conditional distribution at each step is kept) for rows of logits: for every row r,
 *   M_s(x) = softmax(logits[r, :] / T)(x),
 *   tokens[r] = inverse-CDF sample in vocabulary-index order with uniforms[r]
 *               (the same convention as the verification samples),
 *   lse[r]    = ln sum_x exp(logits[r, x] / T)   (what the verification needs of the row).
 * A row with a NaN or +inf logit, or with no finite logit, gives tokens[r] = -1, lse[r] = NaN.
 * margin[r] (may be NULL): distance in probability of the uniform from its CDF cell's edges.
 * Returns 0, or 1 for an invalid argument.
 */
int oracle_sample_rows(const void *logits, const float *uniforms, int rows, int V, int dtype,
                       double temperature, int32_t *tokens, double *lse, double *margin)
{
    if (!logits || !uniforms || !tokens || rows < 0 || V < 1)
        return 1;
    if (!(temperature > 0.0) || !isfinite(temperature) || dtype < 0 || dtype > 2)
        return 1;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int r = 0; r < rows; ++r) {
        size_t off = (size_t)r * (size_t)V;
        double l, W, m = NAN;
        if (row_lse(logits, dtype, off, V, temperature, &l)) {
            tokens[r] = -1;
            l = NAN;
        } else {
            tokens[r] = sample_index_order(logits, off, l, NULL, 0, 0.0, 0, dtype, V, temperature,
                                           1.0, (double)uniforms[r], &W, &m);
        }
        if (lse) lse[r] = l;
        if (margin) margin[r] = m;
    }
    return 0;
}

/* ================= the same procedures on given probabilities =================
 *
 * The paper states Algorithms 1 and 2 on the conditional distributions themselves
 * (M_b(. | c, X^i), M_s(. | c, X^i)); here they are the inputs, as stored numbers:
 *   P_r(x) = target_probs[b, r, x], r = 0..gamma;  Q_r(x) = draft_probs[b, r, x], r = 0..gamma-1.
 * Nothing is renormalised: Eq. "def_as", "pacc_block", "pres-token" and "pres-block" are
 * evaluated on the numbers as given (a row that does not sum to one exactly, as after rounding to
 * a narrow type, is used as it is; the samples divide by the sum of their own weights).
 * Domain errors of a sequence: a drafted token outside [0, V); Q_{i-1}(X_i) that is not a
 * positive finite number or P_{i-1}(X_i) that is not a non-negative finite number in a test the
 * algorithm makes; an empty or non-finite weight sum at the position to sample from.
 */
static double stored_prob(const seq_t *s, int target_row, int r, int x)
{
    size_t V = (size_t)s->V;
    return target_row ? logit_at(s->tgt, s->dtype, s->toff + (size_t)r * V + (size_t)x)
                      : logit_at(s->drf, s->dtype, s->doff + (size_t)r * V + (size_t)x);
}

/* weight of token x at position i: max(p P_i(x) - Q_i(x), 0), or P_gamma(x) at i = gamma */
static double weight_probs(const seq_t *s, int i, int x, double p)
{
    double P = stored_prob(s, 1, i, x);
    if (i == s->gamma)
        return P;
    double w = p * P - stored_prob(s, 0, i, x);
    return w > 0.0 ? w : 0.0;
}

/* inverse-CDF sample in index order from the weights of position i (see sample_index_order) */
static int sample_probs(const seq_t *s, int i, double p, double u, double *W_out, double *margin)
{
    double W = 0.0;
    for (int x = 0; x < s->V; ++x)
        W += weight_probs(s, i, x, p);
    *W_out = W;
    *margin = 0.0;
    if (!(W > 0.0) || !isfinite(W))
        return -1;
    double t = u * W, C = 0.0;
    int last_pos = -1;
    for (int x = 0; x < s->V; ++x) {
        double w = weight_probs(s, i, x, p);
        double Cprev = C;
        C += w;
        if (w > 0.0)
            last_pos = x;
        if (C > t) {
            double lo = u - Cprev / W, hi = C / W - u;
            *margin = lo < hi ? lo : hi;
            return x;
        }
    }
    return last_pos;
}

/* M_b(X_i | c, X^{i-1}) / M_s(X_i | c, X^{i-1}) from the stored numbers; 1 on a domain error */
static int ratio_probs(const seq_t *s, int i, double *ratio)
{
    int x = s->X[i - 1];
    if (x < 0 || x >= s->V)
        return 1;
    double P = stored_prob(s, 1, i - 1, x), Q = stored_prob(s, 0, i - 1, x);
    if (!(Q > 0.0) || !isfinite(Q) || !(P >= 0.0) || !isfinite(P))
        return 1;
    *ratio = P / Q;
    return 0;
}

/* Algorithm 1 */
static void token_verify_probs_one(const seq_t *s, const diag_t *d, int32_t *out_tokens, int32_t *out_len)
{
    const int g = s->gamma;
    double m_eta = INFINITY;
    diag_fill_nan(d, g);
    int tau = 0;
    for (int i = 1; i <= g; ++i) {
        double ratio;
        if (ratio_probs(s, i, &ratio)) {
            emit(s, -1, -1, out_tokens, out_len);
            return;
        }
        double h = ratio < 1.0 ? ratio : 1.0;
        if (d->h) d->h[i] = h;
        double eta = (double)s->u[i - 1];
        double gap = fabs(eta - h);
        if (gap < m_eta) m_eta = gap;
        if (h > 0.0 && eta <= h)
            tau = i;
        else
            break;
    }
    if (d->h) d->h[0] = 1.0;
    double W, m_smp;
    int Y = sample_probs(s, tau, 1.0, (double)s->u[tau < g ? g : g + 1], &W, &m_smp);
    if (tau < g && d->S) d->S[tau] = W;
    if (d->margin_eta) *d->margin_eta = m_eta;
    if (d->margin_smp) *d->margin_smp = m_smp;
    emit(s, Y < 0 ? -1 : tau, Y, out_tokens, out_len);
}

/* Algorithm 2 */
static void block_verify_probs_one(const seq_t *s, const diag_t *d, int32_t *out_tokens, int32_t *out_len)
{
    const int g = s->gamma;
    diag_fill_nan(d, g);
    double *p = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *S = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    double *h = (double *)malloc(sizeof(double) * (size_t)(g + 1));
    p[0] = 1.0;
    for (int i = 1; i <= g; ++i) {
        double ratio;
        if (ratio_probs(s, i, &ratio)) {
            emit(s, -1, -1, out_tokens, out_len);
            goto done;
        }
        double v = p[i - 1] * ratio;
        p[i] = v < 1.0 ? v : 1.0;
    }
    for (int i = 0; i < g; ++i) {
        double acc = 0.0;
        for (int x = 0; x < s->V; ++x)
            acc += weight_probs(s, i, x, p[i]);
        S[i] = acc;
    }
    h[0] = 1.0;
    for (int i = 1; i < g; ++i)
        h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0 - p[i]) : 0.0;
    h[g] = p[g];
    int tau = 0;
    double m_eta = INFINITY;
    for (int i = 1; i <= g; ++i)
        if (h[i] > 0.0 && (double)s->u[i - 1] <= h[i])
            tau = i;
    for (int i = (tau > 0 ? tau : 1); i <= g; ++i) {
        double gap = fabs((double)s->u[i - 1] - h[i]);
        if (gap < m_eta) m_eta = gap;
    }
    {
        double W, m_smp;
        int Y = sample_probs(s, tau, p[tau], (double)s->u[tau < g ? g : g + 1], &W, &m_smp);
        if (d->margin_eta) *d->margin_eta = m_eta;
        if (d->margin_smp) *d->margin_smp = m_smp;
        emit(s, Y < 0 ? -1 : tau, Y, out_tokens, out_len);
    }
    for (int i = 0; i <= g; ++i) {
        if (d->p) d->p[i] = p[i];
        if (d->h) d->h[i] = h[i];
        if (i < g && d->S) d->S[i] = S[i];
    }
done:
    free(p); free(S); free(h);
}

/*
 * algo: ORACLE_TOKEN_VERIFY or ORACLE_BLOCK_VERIFY.  target_probs [B, gamma+1, V], draft_probs
 * [B, gamma, V] in dtype (f32, bf16 bits, f64); the other arguments as oracle_verify, without
 * the normalisers.  Returns 0, or 1 for an invalid argument.
 */
int oracle_verify_probs(int algo, const void *target_probs, const void *draft_probs,
                        const int32_t *tokens, const float *uniforms,
                        int B, int gamma, int V, int dtype,
                        int32_t *out_tokens, int32_t *out_len,
                        double *p, double *S, double *h, double *margin_eta, double *margin_smp)
{
    if (!target_probs || !draft_probs || !tokens || !uniforms || !out_tokens || !out_len)
        return 1;
    if (B < 0 || gamma < 1 || V < 1 || dtype < 0 || dtype > 2)
        return 1;
    if (algo != ORACLE_TOKEN_VERIFY && algo != ORACLE_BLOCK_VERIFY)
        return 1;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int b = 0; b < B; ++b) {
        seq_t s;
        s.tgt = target_probs; s.drf = draft_probs;
        s.X = tokens + (size_t)b * (size_t)gamma;
        s.u = uniforms + (size_t)b * (size_t)(gamma + 2);
        s.gamma = gamma; s.V = V; s.dtype = dtype; s.T = 1.0;
        s.toff = (size_t)b * (size_t)(gamma + 1) * (size_t)V;
        s.doff = (size_t)b * (size_t)gamma * (size_t)V;
        s.given_lse_d = NULL;
        diag_t d;
        d.p = p ? p + (size_t)b * (size_t)(gamma + 1) : NULL;
        d.S = S ? S + (size_t)b * (size_t)gamma : NULL;
        d.h = h ? h + (size_t)b * (size_t)(gamma + 1) : NULL;
        d.lse_t = NULL; d.lse_d = NULL;
        d.margin_eta = margin_eta ? margin_eta + b : NULL;
        d.margin_smp = margin_smp ? margin_smp + b : NULL;
        int32_t *ot = out_tokens + (size_t)b * (size_t)(gamma + 1);
        if (algo == ORACLE_BLOCK_VERIFY)
            block_verify_probs_one(&s, &d, ot, out_len + b);
        else
            token_verify_probs_one(&s, &d, ot, out_len + b);
    }
    return 0;
}

/* Number of threads the batch loop uses (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
#else
int oracle_threads(void) { return 1; }
#endif

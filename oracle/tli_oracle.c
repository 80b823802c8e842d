/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow, fp64 CPU oracle for batched Token-Level Intersection (TLI)
 * verification.  It exists so that tests can check the CUDA library and so that
 * the benchmark can time a CPU baseline.  Nothing in the product may call it,
 * and it shares no code, table or helper with the CUDA sources.
 *
 * What it computes, in the paper's notation (T target vocabulary, D drafter
 * vocabulary, p target distribution, q drafter distribution):
 *
 *   - Algorithm 4 (TLI): q'(x) = q(x) / sum_{t in T cap D} q(t) on the
 *     intersection and 0 elsewhere.  The algorithm box writes the sum over T;
 *     q only lives on D, and the expected-acceptance table writes the same
 *     denominator as a sum over T cap D, which is the reading used here (it
 *     also reproduces the worked example q = 1/3,1/3,1/3 -> q' = 1/2,1/2,0).
 *   - Algorithm 5 (standard speculative decoding) run with (p, q'): a draft
 *     d_j is rejected with probability 1 - p(d_j)/q'(d_j) when p <= q', i.e.
 *     accepted iff u < min(1, p/q') for a uniform u in [0,1); the number of
 *     accepted drafts n is the index of the first rejection; the extra token
 *     is drawn from r(t) = (p(t) - min{p(t), q'(t)}) / (1 - sum min{p, q'})
 *     if a draft was rejected and from p otherwise.
 *
 * Readings where the paper is silent (each one is a documented choice):
 *   - logits become distributions by softmax(z / tau), one tau per sequence,
 *     the same for target and drafter; tau == 0 is the arg-max limit with the
 *     lowest index winning ties, and then drafter logits and uniforms are not
 *     read: a draft is accepted iff map[d_j] equals the arg-max of its row;
 *   - draft ids are drafter-vocabulary ids; the id map sends a drafter id to
 *     its target id or to -1;
 *   - a draft id outside [0, V_d) or outside the intersection has q' = 0 and
 *     is rejected with certainty (threshold 0);
 *   - the extra token is found by inverse CDF in increasing target-id order
 *     using one more uniform v = u[b, K]: the smallest t whose cumulative
 *     weight exceeds v * (total weight);
 *   - if the residual has zero total weight (only reachable through a draft
 *     outside the intersection) it falls back to p of that position.
 *
 * Every sum runs in index order in double precision; there is no blocking,
 * fusion or reordering.
 *
 * The file also holds the drafting side of the same algorithms
 * (oracle_tli_draft): drawing the draft ids from q', and the verification step
 * of Algorithm 2, exact matching against sampled target tokens
 * (oracle_slem_verify), and the expected acceptance rates of the paper's table
 * (oracle_tli_rates); all at the end.
 *
 * Parity status: every function here is pinned by tests that do not use this
 * file's own formulas (worked example, brute-force losslessness on tiny
 * vocabularies, chi-square losslessness, closed-form acceptance rate,
 * reduction to single-vocabulary rejection sampling, q == p, disjoint and
 * subset vocabularies).  At benchmark-scale vocabularies nothing beyond those
 * pins is available: the same code is trusted there because it passed them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1

/* row flag bits, same meaning as the library's row_status */
#define FLAG_DRAFT_RANGE 1
#define FLAG_DRAFT_UNMAPPED 2
#define FLAG_NONFINITE 4
#define FLAG_FALLBACK 8
#define FLAG_BAD_TEMPERATURE 32
/* oracle-only: the two ways of forming q' disagree by more than 1e-12 */
#define FLAG_SELFCHECK 64

typedef struct {
    int32_t B, K, V_t, V_d, dtype;
    const void *target_logits;  /* [B, K+1, V_t], strides in elements */
    int64_t t_stride_b, t_stride_k;
    const void *drafter_logits; /* [B, K, V_d] */
    int64_t d_stride_b, d_stride_k;
    const int32_t *id_map;      /* [V_d] drafter id -> target id or -1 */
    const int32_t *draft_ids;   /* [B, K] drafter ids */
    const float *temperature;   /* [B] */
    const float *uniforms;      /* [B, K+1] */
    const int8_t *force_accept; /* [B, K] or NULL: -1 natural, 0 reject, 1 accept */
    const int32_t *probe_token; /* [B] or NULL: report this token's CDF interval */
    /* outputs */
    int32_t *accepted;          /* [B] */
    int32_t *next_token;        /* [B] */
    int32_t *flags;             /* [B] */
    double *thr;                /* [B, K] min(1, p/q') (0 for drafts outside the intersection) */
    double *p_draft;            /* [B, K] p(map[d_j]) */
    double *q_draft;            /* [B, K] q'(d_j) */
    double *cdf_lo;             /* [B] normalised CDF just below next_token */
    double *cdf_hi;             /* [B] normalised CDF at next_token */
    double *total;              /* [B] total weight R of the sampled distribution */
    double *probe_lo;           /* [B] (only if probe_token) */
    double *probe_hi;           /* [B] */
    double *probe_w;            /* [B] normalised weight of the probed token */
    /* optional input, last so that older callers' layouts stay valid */
    const int32_t *draft_lengths; /* [B] or NULL: drafts of sequence b that count, 0..K; the extra token
                                   * then comes from target row draft_lengths[b] when all of them are accepted */
} oracle_args;

static double load_logit(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORACLE_F32) {
        return (double)((const float *)base)[idx];
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* softmax(z / tau) of one row of V logits into out[V]; returns 0 if a logit is not finite */
static int softmax_row(const void *base, int dtype, int64_t off, int V, double tau, double *out)
{
    double m = -INFINITY;
    for (int i = 0; i < V; ++i) {
        double z = load_logit(base, dtype, off + i);
        if (!isfinite(z)) return 0;
        if (z > m) m = z;
    }
    double Z = 0.0;
    for (int i = 0; i < V; ++i) {
        out[i] = exp((load_logit(base, dtype, off + i) - m) / tau);
        Z += out[i];
    }
    for (int i = 0; i < V; ++i) out[i] /= Z;
    return 1;
}

/* lowest index attaining the maximum of one row */
static int argmax_row(const void *base, int dtype, int64_t off, int V)
{
    int best = 0;
    double m = load_logit(base, dtype, off);
    for (int i = 1; i < V; ++i) {
        double z = load_logit(base, dtype, off + i);
        if (z > m) { m = z; best = i; }
    }
    return best;
}

/*
 * Algorithm 4's q' for one drafter row: softmax over all of D, then divide by
 * the mass on the intersection.  qp[x] = 0 for x outside the intersection.
 * Also forms q' by a softmax restricted to the intersection and reports
 * whether the two agree to 1e-12.  Returns 0 on a non-finite logit.
 */
static int qprime_row(const oracle_args *a, int64_t off, double tau, double *q, double *qp,
                      int *selfcheck_ok, int *empty)
{
    const int V_d = a->V_d;
    *selfcheck_ok = 1;
    *empty = 0;
    if (!softmax_row(a->drafter_logits, a->dtype, off, V_d, tau, q)) return 0;
    double M = 0.0;
    int n_in = 0;
    for (int x = 0; x < V_d; ++x)
        if (a->id_map[x] >= 0) { M += q[x]; ++n_in; }
    if (n_in == 0 || !(M > 0.0)) {
        /* empty intersection, or all its mass underflowed */
        *empty = 1;
        for (int x = 0; x < V_d; ++x) qp[x] = 0.0;
        if (n_in == 0) return 1;
    } else {
        for (int x = 0; x < V_d; ++x) qp[x] = (a->id_map[x] >= 0) ? q[x] / M : 0.0;
    }
    /* second route: softmax over the intersection only */
    double m = -INFINITY;
    for (int x = 0; x < V_d; ++x)
        if (a->id_map[x] >= 0) {
            double z = load_logit(a->drafter_logits, a->dtype, off + x);
            if (z > m) m = z;
        }
    double Z = 0.0;
    for (int x = 0; x < V_d; ++x)
        if (a->id_map[x] >= 0) Z += exp((load_logit(a->drafter_logits, a->dtype, off + x) - m) / tau);
    for (int x = 0; x < V_d; ++x)
        if (a->id_map[x] >= 0) {
            double alt = exp((load_logit(a->drafter_logits, a->dtype, off + x) - m) / tau) / Z;
            if (*empty) { qp[x] = alt; }
            else if (fabs(alt - qp[x]) > 1e-12) *selfcheck_ok = 0;
        }
    if (*empty) *empty = 2; /* rescued by the restricted softmax */
    return 1;
}

/*
 * Verify rows [row_begin, row_end).  Returns 0, or -1 on bad arguments, -2 if
 * the id map is not injective / out of range, -3 on allocation failure.
 */
int oracle_tli_verify(const oracle_args *a, int32_t row_begin, int32_t row_end)
{
    if (!a || a->B < 0 || a->K < 1 || a->V_t < 1 || a->V_d < 1) return -1;
    if (a->dtype != ORACLE_F32 && a->dtype != ORACLE_BF16) return -1;
    if (row_begin < 0 || row_end > a->B || row_begin > row_end) return -1;
    const int K = a->K, V_t = a->V_t, V_d = a->V_d;

    int32_t *inv = (int32_t *)malloc(sizeof(int32_t) * (size_t)V_t);
    double *p = (double *)malloc(sizeof(double) * (size_t)V_t);
    double *q = (double *)malloc(sizeof(double) * (size_t)V_d);
    double *qp = (double *)malloc(sizeof(double) * (size_t)V_d);
    double *w = (double *)malloc(sizeof(double) * (size_t)V_t);
    int *acc = (int *)malloc(sizeof(int) * (size_t)K);
    int rc = 0;
    if (!inv || !p || !q || !qp || !w || !acc) { rc = -3; goto done; }

    /* inverse of the id map: target id -> the one drafter id that maps to it */
    for (int t = 0; t < V_t; ++t) inv[t] = -1;
    for (int x = 0; x < V_d; ++x) {
        int32_t t = a->id_map[x];
        if (t == -1) continue;
        if (t < 0 || t >= V_t || inv[t] != -1) { rc = -2; goto done; }
        inv[t] = x;
    }

    for (int b = row_begin; b < row_end; ++b) {
        const double tau = (double)a->temperature[b];
        const int64_t t_off = (int64_t)b * a->t_stride_b;
        const int64_t d_off = (int64_t)b * a->d_stride_b;
        int flags = 0;
        int Kb = a->draft_lengths ? a->draft_lengths[b] : K;   /* drafts of this sequence */
        if (Kb < 0) Kb = 0;
        if (Kb > K) Kb = K;
        int n = Kb;
        int next = 0;
        double lo = 0.0, hi = 0.0, R = 0.0;
        for (int j = 0; j < K; ++j) {
            if (a->thr) a->thr[(int64_t)b * K + j] = 0.0;
            if (a->p_draft) a->p_draft[(int64_t)b * K + j] = 0.0;
            if (a->q_draft) a->q_draft[(int64_t)b * K + j] = 0.0;
        }

        if (!(tau >= 0.0) || !isfinite(tau)) {
            flags |= FLAG_BAD_TEMPERATURE;
            n = 0; next = 0;
            goto row_done;
        }

        if (tau == 0.0) {
            /* arg-max limit: exact match of map[d_j] with the row's arg-max */
            for (int j = 0; j < Kb; ++j) {
                int aj = argmax_row(a->target_logits, a->dtype, t_off + (int64_t)j * a->t_stride_k, V_t);
                int32_t x = a->draft_ids[(int64_t)b * K + j];
                int ok;
                if (x < 0 || x >= V_d) { flags |= FLAG_DRAFT_RANGE; ok = 0; }
                else if (a->id_map[x] < 0) { flags |= FLAG_DRAFT_UNMAPPED; ok = 0; }
                else ok = (a->id_map[x] == aj);
                if (a->force_accept && a->force_accept[(int64_t)b * K + j] >= 0)
                    ok = a->force_accept[(int64_t)b * K + j];
                acc[j] = ok;
                if (a->thr) a->thr[(int64_t)b * K + j] = ok ? 1.0 : 0.0;
            }
            n = Kb;
            for (int j = 0; j < Kb; ++j) if (!acc[j]) { n = j; break; }
            next = argmax_row(a->target_logits, a->dtype, t_off + (int64_t)n * a->t_stride_k, V_t);
            lo = 0.0; hi = 1.0; R = 1.0;
            goto row_done;
        }

        /* acceptance tests, Algorithm 5 with (p, q') */
        for (int j = 0; j < Kb; ++j) {
            int ok_sc, empty;
            if (!softmax_row(a->target_logits, a->dtype, t_off + (int64_t)j * a->t_stride_k, V_t, tau, p) ||
                !qprime_row(a, d_off + (int64_t)j * a->d_stride_k, tau, q, qp, &ok_sc, &empty)) {
                flags |= FLAG_NONFINITE;
                break;
            }
            if (!ok_sc) flags |= FLAG_SELFCHECK;
            if (empty == 1) flags |= FLAG_FALLBACK;
            int32_t x = a->draft_ids[(int64_t)b * K + j];
            double thr, pv = 0.0, qv = 0.0;
            if (x < 0 || x >= V_d) { flags |= FLAG_DRAFT_RANGE; thr = 0.0; }
            else if (a->id_map[x] < 0) { flags |= FLAG_DRAFT_UNMAPPED; thr = 0.0; }
            else {
                pv = p[a->id_map[x]];
                qv = qp[x];
                if (qv > 0.0) { thr = pv / qv; if (thr > 1.0) thr = 1.0; }
                else thr = (pv > 0.0) ? 1.0 : 0.0;
            }
            int ok = ((double)a->uniforms[(int64_t)b * (K + 1) + j] < thr);
            if (a->force_accept && a->force_accept[(int64_t)b * K + j] >= 0)
                ok = a->force_accept[(int64_t)b * K + j];
            acc[j] = ok;
            if (a->thr) a->thr[(int64_t)b * K + j] = thr;
            if (a->p_draft) a->p_draft[(int64_t)b * K + j] = pv;
            if (a->q_draft) a->q_draft[(int64_t)b * K + j] = qv;
        }
        if (flags & FLAG_NONFINITE) { n = 0; next = 0; goto row_done; }

        /* number of accepted drafts */
        n = Kb;
        for (int j = 0; j < Kb; ++j) if (!acc[j]) { n = j; break; }

        /* distribution of the extra token */
        if (!softmax_row(a->target_logits, a->dtype, t_off + (int64_t)n * a->t_stride_k, V_t, tau, p)) {
            flags |= FLAG_NONFINITE; n = 0; next = 0; goto row_done;
        }
        if (n < Kb) {
            int ok_sc, empty;
            if (!qprime_row(a, d_off + (int64_t)n * a->d_stride_k, tau, q, qp, &ok_sc, &empty)) {
                flags |= FLAG_NONFINITE; n = 0; next = 0; goto row_done;
            }
            R = 0.0;
            for (int t = 0; t < V_t; ++t) {
                double qt = (inv[t] >= 0) ? qp[inv[t]] : 0.0;
                double mn = (p[t] < qt) ? p[t] : qt;   /* min{p, q'} */
                w[t] = p[t] - mn;                      /* numerator of r(t) */
                R += w[t];
            }
            if (!(R > 0.0)) {
                flags |= FLAG_FALLBACK;
                R = 0.0;
                for (int t = 0; t < V_t; ++t) { w[t] = p[t]; R += w[t]; }
            }
        } else {
            R = 0.0;
            for (int t = 0; t < V_t; ++t) { w[t] = p[t]; R += w[t]; }
        }
        {
            const double target = (double)a->uniforms[(int64_t)b * (K + 1) + K] * R;
            double C = 0.0;
            int found = -1, last_pos = 0;
            double C_before = 0.0;
            for (int t = 0; t < V_t; ++t) {
                double Cn = C + w[t];
                if (w[t] > 0.0) last_pos = t;
                if (found < 0 && Cn > target) { found = t; C_before = C; hi = Cn / R; }
                C = Cn;
            }
            if (found < 0) { found = last_pos; C_before = C - w[last_pos]; hi = 1.0; }
            next = found;
            lo = C_before / R;
            if (a->probe_token) {
                int g = a->probe_token[b];
                double plo = 0.0, phi = 0.0, pw = 0.0;
                if (g >= 0 && g < V_t) {
                    double Cc = 0.0;
                    for (int t = 0; t < g; ++t) Cc += w[t];
                    plo = Cc / R; phi = (Cc + w[g]) / R; pw = w[g] / R;
                }
                if (a->probe_lo) a->probe_lo[b] = plo;
                if (a->probe_hi) a->probe_hi[b] = phi;
                if (a->probe_w) a->probe_w[b] = pw;
            }
        }
row_done:
        a->accepted[b] = n;
        a->next_token[b] = next;
        if (a->flags) a->flags[b] = flags;
        if (a->cdf_lo) a->cdf_lo[b] = lo;
        if (a->cdf_hi) a->cdf_hi[b] = hi;
        if (a->total) a->total[b] = R;
    }
done:
    free(inv); free(p); free(q); free(qp); free(w); free(acc);
    return rc;
}

/*
 * The two distributions of one (row, position) pair, for inspection by tests:
 * p_out[V_t] = target softmax, qT_out[V_t] = q' carried to target ids
 * (0 where no drafter id maps).  Returns 0 on success.
 */
int oracle_tli_distributions(const oracle_args *a, int32_t b, int32_t j, double *p_out, double *qT_out)
{
    if (!a || b < 0 || b >= a->B || j < 0 || j > a->K) return -1;
    const double tau = (double)a->temperature[b];
    if (!(tau > 0.0)) return -1;
    if (!softmax_row(a->target_logits, a->dtype, (int64_t)b * a->t_stride_b + (int64_t)j * a->t_stride_k,
                     a->V_t, tau, p_out)) return -4;
    for (int t = 0; t < a->V_t; ++t) qT_out[t] = 0.0;
    if (j == a->K) return 0;
    double *q = (double *)malloc(sizeof(double) * (size_t)a->V_d);
    double *qp = (double *)malloc(sizeof(double) * (size_t)a->V_d);
    if (!q || !qp) { free(q); free(qp); return -3; }
    int ok_sc, empty;
    int ok = qprime_row(a, (int64_t)b * a->d_stride_b + (int64_t)j * a->d_stride_k, tau, q, qp, &ok_sc, &empty);
    if (ok)
        for (int x = 0; x < a->V_d; ++x)
            if (a->id_map[x] >= 0 && a->id_map[x] < a->V_t) qT_out[a->id_map[x]] = qp[x];
    free(q); free(qp);
    return ok ? 0 : -4;
}

/*
 * Drafting with Algorithm 4's q' (the sampling step of Algorithm 5 run with
 * q'): for every sequence b and row r of drafter logits, draw a drafter id
 * from q'(x) = q(x) / sum_{T cap D} q on the intersection.  One uniform per
 * row; inverse CDF in increasing drafter-id order: the smallest x whose
 * cumulative q' exceeds v * (sum of q'), so ids outside the intersection
 * (weight 0) are never drawn.  tau == 0: the lowest id among those attaining
 * the largest logit inside the intersection.  No id can be drawn (-1) when the
 * intersection is empty, when a logit is not finite or the temperature is
 * invalid; the row is flagged.  Parity status: pinned by the worked example of
 * q', by a chi-square test of the drawn ids against q' formed independently,
 * by the boundaries of the CDF on tiny vocabularies, and by the reduction to
 * a plain softmax sampler when every id is in the intersection.
 */
typedef struct {
    int32_t B, R, V_d, dtype;
    const void *drafter_logits; /* [B, R, V_d], strides in elements */
    int64_t d_stride_b, d_stride_r;
    const int32_t *id_map;      /* [V_d] */
    const float *temperature;   /* [B] */
    const float *uniforms;      /* [B, R] */
    const int32_t *probe_id;    /* [B, R] or NULL: report this id's CDF interval */
    /* outputs */
    int32_t *draft_ids;         /* [B, R] drafter ids, -1 if none can be drawn */
    int32_t *flags;             /* [B] */
    double *q_draft;            /* [B, R] q'(drawn id) */
    double *cdf_lo, *cdf_hi;    /* [B, R] normalised CDF around the drawn id */
    double *probe_lo, *probe_hi, *probe_w; /* [B, R] (only if probe_id) */
} oracle_draft_args;

int oracle_tli_draft(const oracle_draft_args *a, int32_t row_begin, int32_t row_end)
{
    if (!a || a->B < 1 || a->R < 1 || a->V_d < 1) return -1;
    if (a->dtype != ORACLE_F32 && a->dtype != ORACLE_BF16) return -1;
    if (row_begin < 0 || row_end > a->B || row_begin > row_end) return -1;
    const int V_d = a->V_d, R = a->R;
    double *q = (double *)malloc(sizeof(double) * (size_t)V_d);
    double *qp = (double *)malloc(sizeof(double) * (size_t)V_d);
    if (!q || !qp) { free(q); free(qp); return -3; }
    /* qprime_row() reads the drafter side of the verification arguments */
    oracle_args va;
    memset(&va, 0, sizeof va);
    va.V_d = V_d; va.dtype = a->dtype; va.drafter_logits = a->drafter_logits; va.id_map = a->id_map;

    for (int b = row_begin; b < row_end; ++b) {
        const double tau = (double)a->temperature[b];
        int flags = 0;
        for (int r = 0; r < R; ++r) {
            const int64_t o = (int64_t)b * R + r;
            const int64_t off = (int64_t)b * a->d_stride_b + (int64_t)r * a->d_stride_r;
            int d = -1;
            double qd = 0.0, lo = 0.0, hi = 0.0;
            if (!(tau >= 0.0) || isinf(tau)) {
                flags |= FLAG_BAD_TEMPERATURE;
            } else if (tau == 0.0) {
                /* lowest id attaining the maximum inside the intersection */
                double m = 0.0;
                int finite = 1;
                for (int x = 0; x < V_d; ++x) {
                    double z = load_logit(a->drafter_logits, a->dtype, off + x);
                    if (!isfinite(z)) finite = 0;
                    if (a->id_map[x] >= 0 && (d < 0 || z > m)) { m = z; d = x; }
                }
                if (!finite) { flags |= FLAG_NONFINITE; d = -1; }
                else if (d < 0) flags |= FLAG_FALLBACK;
                else { qd = 1.0; lo = 0.0; hi = 1.0; }
            } else {
                int ok_sc, empty;
                if (!qprime_row(&va, off, tau, q, qp, &ok_sc, &empty)) {
                    flags |= FLAG_NONFINITE;
                } else {
                    if (!ok_sc) flags |= FLAG_SELFCHECK;
                    double total = 0.0;
                    for (int x = 0; x < V_d; ++x) total += qp[x];
                    if (!(total > 0.0)) {
                        flags |= FLAG_FALLBACK;           /* empty intersection */
                    } else {
                        const double target = (double)a->uniforms[o] * total;
                        double C = 0.0, C_before = 0.0;
                        int last_pos = 0;
                        for (int x = 0; x < V_d; ++x) {
                            double Cn = C + qp[x];
                            if (qp[x] > 0.0) last_pos = x;
                            if (d < 0 && Cn > target) { d = x; C_before = C; hi = Cn / total; }
                            C = Cn;
                        }
                        if (d < 0) { d = last_pos; C_before = C - qp[last_pos]; hi = 1.0; }
                        lo = C_before / total;
                        qd = qp[d];
                        if (a->probe_id) {
                            int g = a->probe_id[o];
                            double plo = 0.0, phi = 0.0, pw = 0.0;
                            if (g >= 0 && g < V_d) {
                                double Cc = 0.0;
                                for (int x = 0; x < g; ++x) Cc += qp[x];
                                plo = Cc / total; phi = (Cc + qp[g]) / total; pw = qp[g] / total;
                            }
                            if (a->probe_lo) a->probe_lo[o] = plo;
                            if (a->probe_hi) a->probe_hi[o] = phi;
                            if (a->probe_w) a->probe_w[o] = pw;
                        }
                    }
                }
            }
            a->draft_ids[o] = d;
            if (a->q_draft) a->q_draft[o] = qd;
            if (a->cdf_lo) a->cdf_lo[o] = lo;
            if (a->cdf_hi) a->cdf_hi[o] = hi;
        }
        if (a->flags) a->flags[b] = flags;
    }
    free(q); free(qp);
    return 0;
}

/*
 * Algorithm 2 (string-level exact matching), the part after the drafts have
 * been re-tokenised into target ids t_1..t_m: sample t'_j from each of the
 * m+1 target rows (p_j = softmax(row j / tau); inverse CDF in increasing
 * target-id order with the uniform u[b, j]; tau == 0: the lowest id attaining
 * the maximum), find the first j with t'_j != t_j (j = m+1 if none), accept
 * t_1..t_{j-1} and emit t'_j.  accepted = j-1 in [0, m], next_token = t'_j.
 * Sequences may have different m (lengths[b] <= M); rows beyond m are not
 * sampled (-1).  A non-finite logit in a row that is sampled, or an invalid
 * temperature, flags the sequence (accepted = 0, next_token = 0).  Parity
 * status: pinned by a chi-square of the sampled ids against the softmax, by
 * the closed-form match probability p_j(t_j), by numpy's cumulative-sum
 * search, by brute force over all candidate strings on a tiny vocabulary, and
 * at tau == 0 by agreement with the verification oracle under an identity map.
 */
typedef struct {
    int32_t B, M, V_t, dtype;
    const void *target_logits;  /* [B, M+1, V_t], strides in elements */
    int64_t t_stride_b, t_stride_k;
    const int32_t *candidates;  /* [B, M] target ids of the re-tokenised drafts */
    const int32_t *lengths;     /* [B] m_b in [0, M], or NULL for m_b = M */
    const float *temperature;   /* [B] */
    const float *uniforms;      /* [B, M+1] */
    const int32_t *probe_token; /* [B, M+1] or NULL */
    /* outputs */
    int32_t *sampled;           /* [B, M+1] t'_j; -1 for rows that are not sampled */
    int32_t *accepted;          /* [B] */
    int32_t *next_token;        /* [B] */
    int32_t *flags;             /* [B] */
    double *cdf_lo, *cdf_hi;    /* [B, M+1] normalised CDF around t'_j */
    double *probe_lo, *probe_hi, *probe_w; /* [B, M+1] (only if probe_token) */
} oracle_slem_args;

int oracle_slem_verify(const oracle_slem_args *a, int32_t row_begin, int32_t row_end)
{
    if (!a || a->B < 1 || a->M < 0 || a->V_t < 1) return -1;
    if (a->dtype != ORACLE_F32 && a->dtype != ORACLE_BF16) return -1;
    if (row_begin < 0 || row_end > a->B || row_begin > row_end) return -1;
    const int V = a->V_t, M = a->M;
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    if (!p) return -3;
    for (int b = row_begin; b < row_end; ++b) {
        const double tau = (double)a->temperature[b];
        int m = a->lengths ? a->lengths[b] : M;
        int flags = 0;
        if (m < 0) m = 0;
        if (m > M) m = M;
        for (int j = 0; j <= M; ++j) {
            const int64_t o = (int64_t)b * (M + 1) + j;
            a->sampled[o] = -1;
            if (a->cdf_lo) a->cdf_lo[o] = 0.0;
            if (a->cdf_hi) a->cdf_hi[o] = 0.0;
        }
        if (!(tau >= 0.0) || isinf(tau)) flags |= FLAG_BAD_TEMPERATURE;
        for (int j = 0; j <= m && !flags; ++j) {
            const int64_t o = (int64_t)b * (M + 1) + j;
            const int64_t off = (int64_t)b * a->t_stride_b + (int64_t)j * a->t_stride_k;
            if (tau == 0.0) {
                int finite = 1;
                for (int t = 0; t < V; ++t)
                    if (!isfinite(load_logit(a->target_logits, a->dtype, off + t))) finite = 0;
                if (!finite) { flags |= FLAG_NONFINITE; break; }
                a->sampled[o] = argmax_row(a->target_logits, a->dtype, off, V);
                if (a->cdf_hi) a->cdf_hi[o] = 1.0;
                continue;
            }
            if (!softmax_row(a->target_logits, a->dtype, off, V, tau, p)) { flags |= FLAG_NONFINITE; break; }
            double total = 0.0;
            for (int t = 0; t < V; ++t) total += p[t];
            const double target = (double)a->uniforms[o] * total;
            double C = 0.0, C_before = 0.0, hi = 1.0;
            int found = -1, last_pos = 0;
            for (int t = 0; t < V; ++t) {
                double Cn = C + p[t];
                if (p[t] > 0.0) last_pos = t;
                if (found < 0 && Cn > target) { found = t; C_before = C; hi = Cn / total; }
                C = Cn;
            }
            if (found < 0) { found = last_pos; C_before = C - p[last_pos]; hi = 1.0; }
            a->sampled[o] = found;
            if (a->cdf_lo) a->cdf_lo[o] = C_before / total;
            if (a->cdf_hi) a->cdf_hi[o] = hi;
            if (a->probe_token) {
                int g = a->probe_token[o];
                double plo = 0.0, phi = 0.0, pw = 0.0;
                if (g >= 0 && g < V) {
                    double Cc = 0.0;
                    for (int t = 0; t < g; ++t) Cc += p[t];
                    plo = Cc / total; phi = (Cc + p[g]) / total; pw = p[g] / total;
                }
                if (a->probe_lo) a->probe_lo[o] = plo;
                if (a->probe_hi) a->probe_hi[o] = phi;
                if (a->probe_w) a->probe_w[o] = pw;
            }
        }
        int n = 0, next = 0;
        if (!flags) {
            n = m;
            for (int j = 0; j < m; ++j)
                if (a->sampled[(int64_t)b * (M + 1) + j] != a->candidates[(int64_t)b * M + j]) { n = j; break; }
            next = a->sampled[(int64_t)b * (M + 1) + n];
        } else {
            for (int j = 0; j <= M; ++j) a->sampled[(int64_t)b * (M + 1) + j] = -1;
        }
        a->accepted[b] = n;
        a->next_token[b] = next;
        if (a->flags) a->flags[b] = flags;
    }
    free(p);
    return 0;
}

/*
 * Expected acceptance rates of one draft position, the paper's table of
 * expected acceptance rates: for target p and drafter q of position (b, j),
 *   mass        M       = sum_{x in T cap D} q(x)
 *   alpha_union         = sum_{x in T cap D} min{p(x), q(x)}          (drafting from q)
 *   alpha_tli           = sum_{x in T cap D} min{p(x), q(x) / M}      (drafting from q', Algorithm 4)
 * with p = softmax(target row / tau), q = softmax(drafter row / tau) over all
 * of D and p(x) read at the target id of x.  tau == 0 is the limit of one-hot
 * distributions: q sits on the arg-max over D, q' on the arg-max over the
 * intersection, p on the arg-max over T (lowest id on ties), so each rate is
 * 0 or 1.  An empty intersection gives 0, 0, 0.  Parity status: pinned by the
 * worked example, by Theorem 4.1 (alpha_union <= alpha_tli), by numpy's direct
 * evaluation, by the closed forms for identity and disjoint maps, and by a
 * Monte-Carlo run of the drafting and verification oracles whose empirical
 * acceptance frequency must match alpha_tli.
 */
typedef struct {
    int32_t B, K, V_t, V_d, dtype;
    const void *target_logits;  /* [B, >=K, V_t], strides in elements; rows 0..K-1 are read */
    int64_t t_stride_b, t_stride_k;
    const void *drafter_logits; /* [B, K, V_d] */
    int64_t d_stride_b, d_stride_k;
    const int32_t *id_map;      /* [V_d] */
    const float *temperature;   /* [B] */
    /* outputs, [B, K] */
    double *mass, *alpha_union, *alpha_tli;
    int32_t *flags;             /* [B] */
} oracle_rates_args;

int oracle_tli_rates(const oracle_rates_args *a, int32_t row_begin, int32_t row_end)
{
    if (!a || a->B < 1 || a->K < 1 || a->V_t < 1 || a->V_d < 1) return -1;
    if (a->dtype != ORACLE_F32 && a->dtype != ORACLE_BF16) return -1;
    if (row_begin < 0 || row_end > a->B || row_begin > row_end) return -1;
    const int K = a->K, V_t = a->V_t, V_d = a->V_d;
    double *p = (double *)malloc(sizeof(double) * (size_t)V_t);
    double *q = (double *)malloc(sizeof(double) * (size_t)V_d);
    if (!p || !q) { free(p); free(q); return -3; }
    for (int b = row_begin; b < row_end; ++b) {
        const double tau = (double)a->temperature[b];
        int flags = 0;
        for (int j = 0; j < K; ++j) {
            const int64_t o = (int64_t)b * K + j;
            const int64_t t_off = (int64_t)b * a->t_stride_b + (int64_t)j * a->t_stride_k;
            const int64_t d_off = (int64_t)b * a->d_stride_b + (int64_t)j * a->d_stride_k;
            double M = 0.0, au = 0.0, at = 0.0;
            if (!(tau >= 0.0) || isinf(tau)) {
                flags |= FLAG_BAD_TEMPERATURE;
            } else if (tau == 0.0) {
                int finite = 1;
                for (int t = 0; t < V_t; ++t) if (!isfinite(load_logit(a->target_logits, a->dtype, t_off + t))) finite = 0;
                for (int x = 0; x < V_d; ++x) if (!isfinite(load_logit(a->drafter_logits, a->dtype, d_off + x))) finite = 0;
                if (!finite) { flags |= FLAG_NONFINITE; }
                else {
                    const int at_id = argmax_row(a->target_logits, a->dtype, t_off, V_t);
                    const int ad_all = argmax_row(a->drafter_logits, a->dtype, d_off, V_d);
                    int ad_in = -1; double m = 0.0;
                    for (int x = 0; x < V_d; ++x) {
                        double z = load_logit(a->drafter_logits, a->dtype, d_off + x);
                        if (a->id_map[x] >= 0 && (ad_in < 0 || z > m)) { m = z; ad_in = x; }
                    }
                    M = (a->id_map[ad_all] >= 0) ? 1.0 : 0.0;
                    au = (a->id_map[ad_all] == at_id) ? 1.0 : 0.0;
                    at = (ad_in >= 0 && a->id_map[ad_in] == at_id) ? 1.0 : 0.0;
                    if (ad_in < 0) flags |= FLAG_FALLBACK;
                }
            } else if (!softmax_row(a->target_logits, a->dtype, t_off, V_t, tau, p) ||
                       !softmax_row(a->drafter_logits, a->dtype, d_off, V_d, tau, q)) {
                flags |= FLAG_NONFINITE;
            } else {
                int n_in = 0;
                for (int x = 0; x < V_d; ++x) if (a->id_map[x] >= 0) { M += q[x]; ++n_in; }
                if (n_in == 0) flags |= FLAG_FALLBACK;
                for (int x = 0; x < V_d; ++x) {
                    const int t = a->id_map[x];
                    if (t < 0) continue;
                    const double pt = p[t];
                    au += (pt < q[x]) ? pt : q[x];
                    if (M > 0.0) { const double qp = q[x] / M; at += (pt < qp) ? pt : qp; }
                }
            }
            a->mass[o] = M; a->alpha_union[o] = au; a->alpha_tli[o] = at;
        }
        if (a->flags) a->flags[b] = flags;
    }
    free(p); free(q);
    return 0;
}

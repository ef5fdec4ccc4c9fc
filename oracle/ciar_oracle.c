/*
 * CIAR oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision CPU statement of what the CIAR hot path
 * computes for every image token: the row softmax over the visual codebook,
 * the InterFuse probability interval, the Omega*Sigma uncertainty score, the
 * threshold test that sends a token to the cloud, the speculative-decoding
 * accept/reject test, the residual-distribution resample and the accepted
 * prefix length per draft window, and the per-request position advance.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call this file.  It shares no code, header, table or constant with the CUDA
 * library; the product never routes through it.
 *
 * Every loop runs in code-index order, in double, with no blocking, fusion or
 * reordering beyond what the cited passage states.  bf16 and fp32 inputs are
 * widened to double exactly.
 *
 * Parity status of each function (what pins it is in tests/test_oracle_*.py):
 *   orc_quantify   pinned: closed forms (entropy 0 / ln V, r = 0, V = 2
 *                  logistic form, one-hot row), a hand-worked rational example,
 *                  the validity invariants of the interval appendix, Claims 1-4
 *                  of the uncertainty appendix, a library log-sum-exp.
 *   orc_verify     pinned: acceptance probability 1 - TV(p,q), the chi-square
 *                  test that accept+resample reproduces the target
 *                  distribution, residual mass = TV(p,q), inverse-CDF end
 *                  points, brute force on tiny windows.
 *   orc_decode_step pinned: replay against orc_verify window by window and the
 *                  conservation law (every request emits exactly seq_len tokens).
 *   orc_topk       (discrete top-k quantifier) pinned: brute-force rank counting on
 *                  V <= 64, k = V reproducing orc_quantify, k = 1, closed forms on constant
 *                  and geometric rows.  That it is the discrete method the paper timed:
 *                  parity unpinned (the paper prints no formula for it).
 *   orc_score_variant pinned: the appendix's scaling claim, the reductions to the product.
 *   orc_ensemble / orc_vote pinned: one head and identical heads reproducing
 *                  orc_quantify, a two-head example with a uniform average, head order.
 *   orc_interdro   pinned: library log-softmax / relative entropy, CE = H + KL, V = 2
 *                  closed forms, constant radius, alpha = 0 and large alpha.
 *   The operating point tau = 0.30 and the paper's end-to-end ratios depend on
 *   trained weights and data: parity unpinned (context only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* dtype codes of a logit tensor */
#define ORC_F32 0
#define ORC_BF16 1
/* radius modes (Inter-Head equation: r = Softplus(Linear_radius(h))) */
#define ORC_RADIUS_SCALAR 0
#define ORC_RADIUS_PER_ROW 1
#define ORC_RADIUS_PER_CODE 2
/* flag policies: the paper's interval score, and the baselines it compares with */
#define ORC_POLICY_INTERVAL 0
#define ORC_POLICY_ENTROPY 1
#define ORC_POLICY_MAXPROB 2
#define ORC_POLICY_RANDOM 3
#define ORC_POLICY_ALL 4
/* which rows of a draft window are tested by the cloud */
#define ORC_VERIFY_ANCHORED 0 /* Algorithm 1: buffer starts at the first flagged token */
#define ORC_VERIFY_PER_TOKEN 1 /* only flagged tokens are tested */
#define ORC_VERIFY_ALL 2 /* every token is tested */
/* row status bits */
#define ORC_ROW_NAN 1
#define ORC_ROW_NO_FINITE 2
#define ORC_ROW_BAD_TOKEN 4

typedef struct {
    const void *base;
    int dtype;
    int64_t rows;
    int32_t vocab;
    int64_t row_stride; /* elements between consecutive rows */
    int32_t valid_begin; /* first code of the valid slice */
    int32_t valid_count; /* n = |V| of the row (masked codes are not part of V) */
} orc_tensor;

/* exact widening of one stored logit to double */
static double load_elem(const void *base, int dtype, int64_t idx)
{
    if (dtype == ORC_F32) {
        return (double)((const float *)base)[idx];
    } else {
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* copy the valid slice of one row into a double array; returns status bits */
static int load_row(const orc_tensor *t, int64_t row, double *c)
{
    int status = 0;
    int any_finite = 0;
    for (int32_t i = 0; i < t->valid_count; ++i) {
        double v = load_elem(t->base, t->dtype, row * t->row_stride + t->valid_begin + i);
        c[i] = v;
        if (isnan(v) || (isinf(v) && v > 0)) status |= ORC_ROW_NAN; /* +inf makes exp(c-m) NaN */
        if (isfinite(v)) any_finite = 1;
    }
    if (!any_finite) status |= ORC_ROW_NO_FINITE;
    return status;
}

/*
 * Softmax with the max-trick (interval appendix, closing remark): m = max c,
 * e_i = exp(c_i - m), Z' = sum e_i, p_i = e_i / Z'.  Returns the lowest index
 * attaining the maximum.
 */
static int32_t softmax_row(const double *c, int32_t n, double *e, double *m_out, double *z_out)
{
    double m = -INFINITY;
    int32_t arg = 0;
    for (int32_t i = 0; i < n; ++i)
        if (c[i] > m) { m = c[i]; arg = i; }
    double z = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        e[i] = exp(c[i] - m);
        z += e[i];
    }
    *m_out = m;
    *z_out = z;
    return arg;
}

/* Softplus with beta = 1, written so that large arguments do not overflow */
static double softplus(double x)
{
    if (x > 0) return x + log1p(exp(-x));
    return log1p(exp(x));
}

typedef struct {
    double row_max, sum_exp, lse, p_max, entropy;
    double S_lo, S_up, scale_lo, scale_up;
    double omega, sigma, score;
    int32_t argmax;
    int status;
} orc_row_result;

/*
 * One token row of the device-side quantifier:
 *   softmax of the centre logits           (Inter-DRO section: p = softmax(o))
 *   radius r = min(softplus(rho), r_max)    (Inter-Head equation; clamp: interval appendix)
 *   InterFuse lower / upper bounds          (interval appendix, the two bound equations)
 *   rescale by min(1, lo_cap/S_l), max(1, hi_cap/S_u)   (interval appendix, normalisation step)
 *   delta = p^u - p^l, Omega = sum delta, Sigma = population std of delta, U = Omega * Sigma
 *                                            (uncertainty-score equation)
 * c: valid slice of the row (n values); rad: n radii (already expanded per code).
 * p, p_lo, p_up (each n doubles, nullable) receive the dense vectors.
 */
static void quantify_row(const double *c, const double *rad, int32_t n, int radius_is_raw,
                         double r_max, double lo_cap, double hi_cap,
                         double *e, double *lo, double *up,
                         double *p_out, double *plo_out, double *pup_out, orc_row_result *res)
{
    double m, z;
    res->argmax = softmax_row(c, n, e, &m, &z);
    res->row_max = m;
    res->sum_exp = z;
    res->lse = m + log(z);
    res->p_max = 1.0 / z; /* e = 1 at the maximum */

    /* Shannon entropy of softmax(c), in nats (the entropy-threshold baseline) */
    double h = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        double p = e[i] / z;
        if (p > 0.0) h -= p * log(p);
        if (p_out) p_out[i] = p;
    }
    res->entropy = h;

    /* InterFuse raw bounds.  Z' - e_i is the sum of the OTHER codes' terms; for the
       maximum code it is summed directly so that a dominant code does not cancel. */
    double others_of_max = 0.0;
    for (int32_t j = 0; j < n; ++j)
        if (j != res->argmax) others_of_max += e[j];
    double s_lo = 0.0, s_up = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        double r = radius_is_raw ? softplus(rad[i]) : rad[i];
        if (r > r_max) r = r_max;
        double rest = (i == res->argmax) ? others_of_max : (z - e[i]);
        double el = e[i] * exp(-r); /* exp(c_i - r_i - m) */
        double eu = e[i] * exp(r); /* exp(c_i + r_i - m) */
        lo[i] = (el > 0.0) ? el / (rest + el) : 0.0;
        up[i] = (eu > 0.0) ? eu / (rest + eu) : 0.0;
        s_lo += lo[i];
        s_up += up[i];
    }
    res->S_lo = s_lo;
    res->S_up = s_up;

    /* normalisation step: sum p^l <= lo_cap, sum p^u >= hi_cap */
    double k_lo = 1.0, k_up = 1.0;
    if (s_lo > 0.0 && lo_cap / s_lo < 1.0) k_lo = lo_cap / s_lo;
    if (s_up > 0.0 && hi_cap / s_up > 1.0) k_up = hi_cap / s_up;
    res->scale_lo = k_lo;
    res->scale_up = k_up;
    for (int32_t i = 0; i < n; ++i) {
        lo[i] *= k_lo;
        up[i] *= k_up;
        if (plo_out) plo_out[i] = lo[i];
        if (pup_out) pup_out[i] = up[i];
    }

    /* widths, total ambiguity, confidence disparity (two-pass population std) */
    double omega = 0.0;
    for (int32_t i = 0; i < n; ++i) omega += up[i] - lo[i];
    double mean = omega / (double)n;
    double ss = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        double d = (up[i] - lo[i]) - mean;
        ss += d * d;
    }
    res->omega = omega;
    res->sigma = sqrt(ss / (double)n);
    res->score = res->omega * res->sigma;
}

static double rel_margin(double a, double b)
{
    double d = fabs(a - b);
    double s = fmax(fabs(a), fabs(b));
    return (s > 0.0) ? d / s : 0.0;
}

/*
 * Quantify every row.  All outputs are nullable.  dense_* are [rows, valid_count].
 * radius: SCALAR -> ignored (r_scalar used); PER_ROW -> float32[rows];
 *         PER_CODE -> same dtype and layout as the logits.
 * flag policy: INTERVAL U > tau (Algorithm 1: accept on device iff U <= tau);
 *   ENTROPY H > tau; MAXPROB p_max < tau; RANDOM u_flag < tau; ALL always.
 * margin: relative distance of the decision quantity from tau.
 * A row with a NaN / +inf, or without any finite code, gets NaN scores, flag 1.
 */
int orc_quantify(const void *logits, int dtype, int64_t rows, int32_t vocab, int64_t row_stride,
                 int32_t valid_begin, int32_t valid_count,
                 int radius_mode, const void *radius, int radius_is_raw, double r_scalar,
                 double r_max, double lo_cap, double hi_cap,
                 int policy, double tau, const float *u_flag,
                 double *row_max, double *sum_exp, double *lse, double *p_max, double *entropy,
                 double *S_lo, double *S_up, double *scale_lo, double *scale_up,
                 double *omega, double *sigma, double *score,
                 int32_t *argmax, uint8_t *flag, uint8_t *row_status, double *margin,
                 double *dense_p, double *dense_lo, double *dense_up, int threads)
{
    if (rows < 0 || valid_count < 1 || valid_begin < 0 || valid_begin + (int64_t)valid_count > vocab)
        return 1;
    orc_tensor t = { logits, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    orc_tensor tr = { radius, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    const int32_t n = valid_count;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
    int fail = 0;
#pragma omp parallel
    {
        double *buf = (double *)malloc(sizeof(double) * (size_t)n * 5);
        if (!buf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t row = 0; row < rows; ++row) {
            if (!buf) continue;
            double *c = buf, *rad = buf + n, *e = buf + 2 * (size_t)n, *lo = buf + 3 * (size_t)n,
                   *up = buf + 4 * (size_t)n;
            int status = load_row(&t, row, c);
            if (radius_mode == ORC_RADIUS_PER_CODE) {
                for (int32_t i = 0; i < n; ++i) {
                    rad[i] = load_elem(tr.base, tr.dtype, row * tr.row_stride + valid_begin + i);
                    if (isnan(rad[i])) status |= ORC_ROW_NAN;
                }
            } else {
                double r = (radius_mode == ORC_RADIUS_PER_ROW) ? (double)((const float *)radius)[row] : r_scalar;
                if (isnan(r)) status |= ORC_ROW_NAN;
                for (int32_t i = 0; i < n; ++i) rad[i] = r;
            }
            orc_row_result res;
            memset(&res, 0, sizeof res);
            double *dp = dense_p ? dense_p + row * (int64_t)n : NULL;
            double *dl = dense_lo ? dense_lo + row * (int64_t)n : NULL;
            double *du = dense_up ? dense_up + row * (int64_t)n : NULL;
            uint8_t fl;
            double mg;
            if (status) {
                res.row_max = res.sum_exp = res.lse = res.p_max = res.entropy = NAN;
                res.S_lo = res.S_up = res.scale_lo = res.scale_up = NAN;
                res.omega = res.sigma = res.score = NAN;
                res.argmax = -1;
                for (int32_t i = 0; i < n; ++i) {
                    if (dp) dp[i] = NAN;
                    if (dl) dl[i] = NAN;
                    if (du) du[i] = NAN;
                }
                fl = 1;
                mg = INFINITY;
            } else {
                quantify_row(c, rad, n, radius_is_raw, r_max, lo_cap, hi_cap, e, lo, up, dp, dl, du, &res);
                res.argmax += valid_begin; /* global code index */
                switch (policy) {
                case ORC_POLICY_INTERVAL: fl = res.score > tau; mg = rel_margin(res.score, tau); break;
                case ORC_POLICY_ENTROPY: fl = res.entropy > tau; mg = rel_margin(res.entropy, tau); break;
                case ORC_POLICY_MAXPROB: fl = res.p_max < tau; mg = rel_margin(res.p_max, tau); break;
                case ORC_POLICY_RANDOM: fl = (double)u_flag[row] < tau; mg = rel_margin((double)u_flag[row], tau); break;
                default: fl = 1; mg = INFINITY; break;
                }
            }
            if (row_max) row_max[row] = res.row_max;
            if (sum_exp) sum_exp[row] = res.sum_exp;
            if (lse) lse[row] = res.lse;
            if (p_max) p_max[row] = res.p_max;
            if (entropy) entropy[row] = res.entropy;
            if (S_lo) S_lo[row] = res.S_lo;
            if (S_up) S_up[row] = res.S_up;
            if (scale_lo) scale_lo[row] = res.scale_lo;
            if (scale_up) scale_up[row] = res.scale_up;
            if (omega) omega[row] = res.omega;
            if (sigma) sigma[row] = res.sigma;
            if (score) score[row] = res.score;
            if (argmax) argmax[row] = res.argmax;
            if (flag) flag[row] = fl;
            if (row_status) row_status[row] = (uint8_t)status;
            if (margin) margin[row] = mg;
        }
        free(buf);
    }
    return fail ? 2 : 0;
}

/*
 * One draft window of W consecutive rows starting at row0 (Algorithm 1, the
 * else-branch: buffer, cloud verification, resampling).
 *   f  = first flagged row of the window, else W (the buffer starts there)
 *   tested rows: ANCHORED j >= f; PER_TOKEN flagged rows; ALL every row
 *   accept_j  = (u_acc_j * p_x < q_x), p = softmax(draft row), q = softmax(target row),
 *               x the draft token: the speculative-decoding test u < min(1, q_x / p_x)
 *   a  = first tested row that is rejected, else W;  accepted_len = a
 *   if a < W: token drawn from norm(max(0, q - p)) on row a by inverse CDF with
 *             u_res_a: smallest k with cum_k > u_res * Rs (cum in index order)
 * wlen <= W rows exist (a window cut short by the end of the sequence).
 */
typedef struct {
    int32_t first_flag, accepted_len, resampled;
    uint8_t cloud_call;
    double residual_mass, resample_margin;
} orc_window_result;

/* tokens, flag, u_acc, u_res, accept, p_tok, q_tok, acc_margin, row_status point at the
   window's first row (index j = 0 .. wlen-1); the output ones are nullable. */
static void verify_window(const orc_tensor *draft, const orc_tensor *target, const int32_t *tokens,
                          const uint8_t *flag, const float *u_acc, const float *u_res,
                          int64_t row0, int32_t wlen, int mode, double *work,
                          uint8_t *accept, double *p_tok, double *q_tok, double *acc_margin,
                          uint8_t *row_status, orc_window_result *out)
{
    const int32_t n = draft->valid_count;
    double *c = work, *t = work + n, *ep = work + 2 * (size_t)n, *eq = work + 3 * (size_t)n;
    int32_t f = wlen;
    if (mode == ORC_VERIFY_ALL) {
        f = 0;
    } else {
        for (int32_t j = 0; j < wlen; ++j)
            if (flag[j]) { f = j; break; }
    }
    out->first_flag = f;
    out->cloud_call = (f < wlen);
    int32_t a = wlen;
    for (int32_t j = 0; j < wlen; ++j) {
        int64_t row = row0 + j;
        int tested = (mode == ORC_VERIFY_ALL) || (mode == ORC_VERIFY_ANCHORED && j >= f) ||
                     (mode == ORC_VERIFY_PER_TOKEN && flag[j]);
        uint8_t acc = 1;
        double px = 0.0, qx = 0.0, mg = INFINITY;
        int status = 0;
        if (tested) {
            status |= load_row(draft, row, c);
            status |= load_row(target, row, t);
            int32_t x = tokens[j];
            if (x < 0 || x >= draft->vocab) status |= ORC_ROW_BAD_TOKEN;
            if (status) {
                acc = 0;
                px = qx = NAN;
            } else {
                double mp, zp, mq, zq;
                softmax_row(c, n, ep, &mp, &zp);
                softmax_row(t, n, eq, &mq, &zq);
                int32_t xi = x - draft->valid_begin;
                if (xi >= 0 && xi < n) { /* a code outside the valid slice has probability 0 */
                    px = ep[xi] / zp;
                    qx = eq[xi] / zq;
                }
                double lhs = (double)u_acc[j] * px;
                acc = lhs < qx;
                mg = rel_margin(lhs, qx);
            }
        }
        if (accept) accept[j] = acc;
        if (p_tok) p_tok[j] = px;
        if (q_tok) q_tok[j] = qx;
        if (acc_margin) acc_margin[j] = mg;
        if (row_status) row_status[j] = (uint8_t)status;
        if (tested && !acc && a == wlen) a = j;
    }
    out->accepted_len = a;
    out->resampled = -1;
    out->residual_mass = 0.0;
    out->resample_margin = INFINITY;
    if (a < wlen) {
        int64_t row = row0 + a;
        int status = load_row(draft, row, c) | load_row(target, row, t);
        if (!status) {
            double mp, zp, mq, zq;
            softmax_row(c, n, ep, &mp, &zp);
            int32_t argq = softmax_row(t, n, eq, &mq, &zq);
            double rs = 0.0;
            for (int32_t i = 0; i < n; ++i) {
                double r = eq[i] / zq - ep[i] / zp;
                ep[i] = (r > 0.0) ? r : 0.0; /* residual max(0, q_i - p_i) */
                rs += ep[i];
            }
            out->residual_mass = rs;
            if (rs > 0.0) {
                double thr = (double)u_res[a] * rs;
                double cum = 0.0;
                int32_t pick = -1, last_pos = -1;
                double lo_edge = 0.0, hi_edge = 0.0;
                for (int32_t i = 0; i < n; ++i) {
                    if (ep[i] > 0.0) last_pos = i;
                    double prev = cum;
                    cum += ep[i];
                    if (cum > thr) { pick = i; lo_edge = prev; hi_edge = cum; break; }
                }
                if (pick < 0) { pick = last_pos; lo_edge = hi_edge = cum; }
                out->resampled = pick + draft->valid_begin;
                out->resample_margin = fmin(fabs(thr - lo_edge), fabs(hi_edge - thr)) / rs;
            } else {
                out->resampled = argq + draft->valid_begin; /* p == q on the support: fall back to the mode of q */
                out->resample_margin = INFINITY;
            }
        }
    }
}

int orc_verify(const void *draft_logits, const void *target_logits, int dtype, int64_t rows, int32_t vocab,
               int64_t row_stride, int32_t valid_begin, int32_t valid_count,
               const int32_t *draft_tokens, const uint8_t *flag, const float *u_accept, const float *u_resample,
               int32_t window, int mode,
               uint8_t *accept, double *p_draft_tok, double *p_target_tok, double *accept_margin,
               uint8_t *row_status,
               int32_t *first_flag, int32_t *accepted_len, int32_t *resampled_token, uint8_t *cloud_call,
               double *residual_mass, double *resample_margin, int threads)
{
    if (rows < 0 || window < 1 || rows % window != 0 || valid_count < 1 || valid_begin < 0 ||
        valid_begin + (int64_t)valid_count > vocab)
        return 1;
    if (mode != ORC_VERIFY_ALL && !flag) return 1;
    orc_tensor d = { draft_logits, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    orc_tensor t = { target_logits, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    const int64_t nw = rows / window;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
    int fail = 0;
#pragma omp parallel
    {
        double *work = (double *)malloc(sizeof(double) * (size_t)valid_count * 4);
        if (!work) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t w = 0; w < nw; ++w) {
            if (!work) continue;
            orc_window_result r;
            const int64_t r0 = w * window;
            verify_window(&d, &t, draft_tokens + r0, flag ? flag + r0 : NULL, u_accept + r0, u_resample + r0,
                          r0, window, mode, work,
                          accept ? accept + r0 : NULL, p_draft_tok ? p_draft_tok + r0 : NULL,
                          p_target_tok ? p_target_tok + r0 : NULL, accept_margin ? accept_margin + r0 : NULL,
                          row_status ? row_status + r0 : NULL, &r);
            if (first_flag) first_flag[w] = r.first_flag;
            if (accepted_len) accepted_len[w] = r.accepted_len;
            if (resampled_token) resampled_token[w] = r.resampled;
            if (cloud_call) cloud_call[w] = r.cloud_call;
            if (residual_mass) residual_mass[w] = r.residual_mass;
            if (resample_margin) resample_margin[w] = r.resample_margin;
        }
        free(work);
    }
    return fail ? 2 : 0;
}

/*
 * One decoding step for every request (Algorithm 1, one trip of the device
 * loop in draft windows of `window` tokens; position advance of its last line).
 * Pools hold, for request q and position s, row q*seq_len + s: the logits the
 * device / cloud model would produce there, the drafted token and the uniforms.
 * For a request at position pos < seq_len the window is rows pos .. pos+wlen-1,
 * wlen = min(window, seq_len - pos) (the buffer stops at the sequence end).
 *   quantify each row -> flag;  verify the window -> a, resampled
 *   tokens_out[pos .. pos+a-1] = drafted tokens; if a < wlen: tokens_out[pos+a] = resampled
 *   pos += a + (a < wlen)
 * counters (int64[8], accumulated): 0 windows processed, 1 windows with a cloud
 * call, 2 rows sent to the cloud, 3 rows flagged, 4 drafted tokens kept,
 * 5 tokens resampled, 6 rows quantified, 7 requests finished in this step.
 * min_margin (nullable, double[3], min-accumulated): flag, accept, resample margins.
 */
int orc_decode_step(const void *draft_pool, const void *target_pool, int dtype, int32_t requests, int32_t seq_len,
                    int32_t vocab, int64_t row_stride, int32_t valid_begin, int32_t valid_count,
                    const int32_t *draft_token_pool, const float *u_accept_pool, const float *u_resample_pool,
                    int radius_mode, const void *radius, int radius_is_raw, double r_scalar,
                    double r_max, double lo_cap, double hi_cap, int policy, double tau, const float *u_flag,
                    int32_t window, int mode,
                    int32_t *pos, int32_t *tokens_out, int64_t *counters, double *min_margin, int threads)
{
    if (requests < 0 || seq_len < 1 || window < 1 || window > 64) return 1;
    const int64_t rows = (int64_t)requests * seq_len;
    orc_tensor d = { draft_pool, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    orc_tensor t = { target_pool, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    const int32_t n = valid_count;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
    int64_t cnt[8] = { 0, 0, 0, 0, 0, 0, 0, 0 };
    double mm[3] = { INFINITY, INFINITY, INFINITY };
    int fail = 0;
#pragma omp parallel
    {
        double *buf = (double *)malloc(sizeof(double) * (size_t)n * 5);
        int64_t lc[8] = { 0, 0, 0, 0, 0, 0, 0, 0 };
        double lm[3] = { INFINITY, INFINITY, INFINITY };
        if (!buf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int32_t q = 0; q < requests; ++q) {
            if (!buf) continue;
            int32_t p0 = pos[q];
            if (p0 >= seq_len) continue;
            int32_t wlen = seq_len - p0 < window ? seq_len - p0 : window;
            int64_t row0 = (int64_t)q * seq_len + p0;
            double *c = buf, *rad = buf + n, *e = buf + 2 * (size_t)n, *lo = buf + 3 * (size_t)n,
                   *up = buf + 4 * (size_t)n;
            uint8_t wflag[64];
            for (int32_t j = 0; j < wlen; ++j) {
                int64_t row = row0 + j;
                int status = load_row(&d, row, c);
                double r = r_scalar;
                if (radius_mode == ORC_RADIUS_PER_CODE) {
                    for (int32_t i = 0; i < n; ++i)
                        rad[i] = load_elem(radius, dtype, row * row_stride + valid_begin + i);
                } else {
                    if (radius_mode == ORC_RADIUS_PER_ROW) r = (double)((const float *)radius)[row];
                    for (int32_t i = 0; i < n; ++i) rad[i] = r;
                }
                uint8_t fl = 1;
                if (!status) {
                    orc_row_result res;
                    quantify_row(c, rad, n, radius_is_raw, r_max, lo_cap, hi_cap, e, lo, up, NULL, NULL, NULL, &res);
                    double mg = INFINITY;
                    switch (policy) {
                    case ORC_POLICY_INTERVAL: fl = res.score > tau; mg = rel_margin(res.score, tau); break;
                    case ORC_POLICY_ENTROPY: fl = res.entropy > tau; mg = rel_margin(res.entropy, tau); break;
                    case ORC_POLICY_MAXPROB: fl = res.p_max < tau; mg = rel_margin(res.p_max, tau); break;
                    case ORC_POLICY_RANDOM: fl = (double)u_flag[row] < tau; mg = rel_margin((double)u_flag[row], tau); break;
                    default: fl = 1; break;
                    }
                    if (mg < lm[0]) lm[0] = mg;
                }
                wflag[j] = fl;
                lc[3] += fl;
                lc[6] += 1;
            }
            orc_window_result r;
            uint8_t acc[64];
            double amg[64];
            verify_window(&d, &t, draft_token_pool + row0, wflag, u_accept_pool + row0, u_resample_pool + row0,
                          row0, wlen, mode, buf, acc, NULL, NULL, amg, NULL, &r);
            for (int32_t j = 0; j < wlen; ++j)
                if (amg[j] < lm[1]) lm[1] = amg[j];
            if (r.resample_margin < lm[2]) lm[2] = r.resample_margin;
            int32_t a = r.accepted_len;
            for (int32_t j = 0; j < a; ++j) tokens_out[(int64_t)q * seq_len + p0 + j] = draft_token_pool[row0 + j];
            int32_t adv = a;
            if (a < wlen) {
                tokens_out[(int64_t)q * seq_len + p0 + a] = r.resampled;
                adv = a + 1;
                lc[5] += 1;
            }
            pos[q] = p0 + adv;
            lc[0] += 1;
            lc[1] += r.cloud_call;
            if (mode == ORC_VERIFY_PER_TOKEN) {
                for (int32_t j = 0; j < wlen; ++j) lc[2] += wflag[j];
            } else {
                lc[2] += wlen - r.first_flag;
            }
            lc[4] += a;
            if (pos[q] >= seq_len) lc[7] += 1;
        }
#pragma omp critical
        {
            for (int k = 0; k < 8; ++k) cnt[k] += lc[k];
            for (int k = 0; k < 3; ++k)
                if (lm[k] < mm[k]) mm[k] = lm[k];
        }
        free(buf);
    }
    if (counters)
        for (int k = 0; k < 8; ++k) counters[k] += cnt[k];
    if (min_margin)
        for (int k = 0; k < 3; ++k)
            if (mm[k] < min_margin[k]) min_margin[k] = mm[k];
    return fail ? 2 : 0;
}

int orc_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------
 * Discrete top-k quantifier (the "Discrete" rows of the paper's discrete-vs-continuous
 * comparison, k = 100 .. 400).  The paper gives no formula for it; the reading taken here:
 * the solution set of a row is T_k = its k most probable codes (largest logits, equal
 * logits by lowest index), found by a FULL SORT of the row; the row's discrete uncertainty
 * is the interval score of the quantifier above applied to the k kept codes alone
 * (softmax renormalised over T_k, n = k).  Also reported: the k-th largest logit, how many
 * codes lie strictly above it, the mass of T_k under the full-row softmax, and the
 * Shannon entropy of the renormalised distribution.
 *
 * Parity status: pinned by brute-force rank counting on V <= 64, k = V (must reproduce
 * orc_quantify), k = 1 (mass = p_max, Omega = 0.02, U = 0), closed forms for constant and
 * geometric rows.  That this is the discrete method the paper timed: parity unpinned.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    double v;
    int32_t i;
} orc_kv;

static int cmp_value_desc_index_asc(const void *a, const void *b)
{
    const orc_kv *x = (const orc_kv *)a, *y = (const orc_kv *)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->i > y->i) - (x->i < y->i);
}

static int cmp_int32_asc(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int orc_topk(const void *logits, int dtype, int64_t rows, int32_t vocab, int64_t row_stride,
             int32_t valid_begin, int32_t valid_count, int32_t k,
             int radius_mode, const void *radius, int radius_is_raw, double r_scalar,
             double r_max, double lo_cap, double hi_cap, double tau,
             double *kth_logit, int32_t *n_above, double *mass, double *entropy,
             double *S_lo, double *S_up, double *omega, double *sigma, double *score,
             uint8_t *flag, uint8_t *row_status, double *margin,
             int32_t *indices /* [rows, k] ascending global code ids, nullable */, int threads)
{
    if (rows < 0 || valid_count < 1 || valid_begin < 0 || valid_begin + (int64_t)valid_count > vocab)
        return 1;
    if (k < 1 || k > valid_count) return 1;
    orc_tensor t = { logits, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    const int32_t n = valid_count;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
    int fail = 0;
#pragma omp parallel
    {
        double *buf = (double *)malloc(sizeof(double) * ((size_t)n * 2 + (size_t)k * 5));
        orc_kv *kv = (orc_kv *)malloc(sizeof(orc_kv) * (size_t)n);
        int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
        if (!buf || !kv || !idx) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t row = 0; row < rows; ++row) {
            if (!buf || !kv || !idx) continue;
            double *c = buf, *e = buf + n, *ck = buf + 2 * (size_t)n, *rk = ck + k, *ek = rk + k,
                   *lo = ek + k, *up = lo + k;
            int status = load_row(&t, row, c);
            double r_row = r_scalar;
            if (radius_mode == ORC_RADIUS_PER_ROW) r_row = (double)((const float *)radius)[row];
            if (radius_mode != ORC_RADIUS_PER_CODE && isnan(r_row)) status |= ORC_ROW_NAN;
            if (!status) {
                /* full sort, most probable first */
                for (int32_t i = 0; i < n; ++i) { kv[i].v = c[i]; kv[i].i = i; }
                qsort(kv, (size_t)n, sizeof(orc_kv), cmp_value_desc_index_asc);
                for (int32_t j = 0; j < k; ++j) idx[j] = kv[j].i;
                qsort(idx, (size_t)k, sizeof(int32_t), cmp_int32_asc);
                double kth = kv[k - 1].v;
                int32_t above = 0;
                for (int32_t i = 0; i < n; ++i) above += (c[i] > kth);
                /* mass of the set under the full-row softmax */
                double m, z;
                softmax_row(c, n, e, &m, &z);
                double ms = 0.0;
                for (int32_t j = 0; j < k; ++j) ms += e[idx[j]];
                ms /= z;
                /* the quantifier on the kept codes alone */
                for (int32_t j = 0; j < k; ++j) {
                    ck[j] = c[idx[j]];
                    if (radius_mode == ORC_RADIUS_PER_CODE) {
                        rk[j] = load_elem(radius, dtype, row * row_stride + valid_begin + idx[j]);
                        if (isnan(rk[j])) status |= ORC_ROW_NAN;
                    } else {
                        rk[j] = r_row;
                    }
                }
                if (!status) {
                    orc_row_result res;
                    memset(&res, 0, sizeof res);
                    quantify_row(ck, rk, k, radius_is_raw, r_max, lo_cap, hi_cap, ek, lo, up, NULL, NULL, NULL, &res);
                    if (kth_logit) kth_logit[row] = kth;
                    if (n_above) n_above[row] = above;
                    if (mass) mass[row] = ms;
                    if (entropy) entropy[row] = res.entropy;
                    if (S_lo) S_lo[row] = res.S_lo;
                    if (S_up) S_up[row] = res.S_up;
                    if (omega) omega[row] = res.omega;
                    if (sigma) sigma[row] = res.sigma;
                    if (score) score[row] = res.score;
                    if (flag) flag[row] = res.score > tau;
                    if (margin) margin[row] = rel_margin(res.score, tau);
                    if (indices)
                        for (int32_t j = 0; j < k; ++j) indices[row * (int64_t)k + j] = idx[j] + valid_begin;
                }
            }
            if (status) {
                if (kth_logit) kth_logit[row] = NAN;
                if (n_above) n_above[row] = -1;
                if (mass) mass[row] = NAN;
                if (entropy) entropy[row] = NAN;
                if (S_lo) S_lo[row] = NAN;
                if (S_up) S_up[row] = NAN;
                if (omega) omega[row] = NAN;
                if (sigma) sigma[row] = NAN;
                if (score) score[row] = NAN;
                if (flag) flag[row] = 1;
                if (margin) margin[row] = INFINITY;
                if (indices)
                    for (int32_t j = 0; j < k; ++j) indices[row * (int64_t)k + j] = -1;
            }
            if (row_status) row_status[row] = (uint8_t)status;
        }
        free(buf);
        free(kv);
        free(idx);
    }
    return fail ? 2 : 0;
}

/* ------------------------------------------------------------------------------------------
 * Score variants (uncertainty appendix, "Practical Remarks for Thresholding and
 * Normalization"): from a row's Omega, Sigma and n,
 *   PRODUCT     U = Omega * Sigma                       (the uncertainty-score equation)
 *   PER_N       U / n                                    (remark 1: normalise by n)
 *   PER_OMEGA2  U / Omega^2 = Sigma / Omega              (remark 1: normalise by Omega^2)
 *   SMOOTHED    Omega * sqrt(Sigma^2 + eps)              (remark 2)
 *   ADDITIVE    lambda1 * Omega + lambda2 * Omega * Sigma (remark 2)
 * flag = variant > tau; a NaN input (unusable row) gives NaN and flag 1.
 * Parity status: pinned by the scaling claim U(alpha delta) = alpha^2 U(delta) (PER_OMEGA2 is
 * invariant, ADDITIVE with lambda2 = 0 is linear), eps = 0 and (lambda1, lambda2) = (0, 1)
 * reducing to PRODUCT, and uniform widths giving Omega * sqrt(eps).
 * ---------------------------------------------------------------------------------------- */
#define ORC_SCORE_PRODUCT 0
#define ORC_SCORE_PER_N 1
#define ORC_SCORE_PER_OMEGA2 2
#define ORC_SCORE_SMOOTHED 3
#define ORC_SCORE_ADDITIVE 4

int orc_score_variant(int64_t rows, int32_t n, const double *omega, const double *sigma, int variant,
                      double eps, double lambda1, double lambda2, double tau,
                      double *out, uint8_t *flag, double *margin)
{
    if (rows < 0 || n < 1 || variant < 0 || variant > ORC_SCORE_ADDITIVE) return 1;
    for (int64_t row = 0; row < rows; ++row) {
        double om = omega[row], sg = sigma[row], v;
        switch (variant) {
        case ORC_SCORE_PRODUCT: v = om * sg; break;
        case ORC_SCORE_PER_N: v = om * sg / (double)n; break;
        case ORC_SCORE_PER_OMEGA2: v = sg / om; break;
        case ORC_SCORE_SMOOTHED: v = om * sqrt(sg * sg + eps); break;
        default: v = lambda1 * om + lambda2 * om * sg; break;
        }
        if (out) out[row] = v;
        if (flag) flag[row] = isnan(v) ? 1 : (v > tau);
        if (margin) margin[row] = isnan(v) ? INFINITY : rel_margin(v, tau);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Several Inter-Heads (appendix "Impact of Inter-Head Capacity").
 * Ensemble (soft voting): the heads' probability distributions are averaged code by code,
 *   pbar_i = (1/H) sum_h softmax(c^h)_i, and the interval is formed around the averaged
 *   distribution (InterFuse on the logits ln pbar_i) with the mean of the heads' clamped
 *   radii.  Reading: the paper says only that the distributions are averaged "to obtain a
 *   calibrated score"; one radius per head and row (or one scalar) is supported.
 * Voting (hard voting): the row is flagged when more than half of the heads flag it.
 * heads: [H, rows, row_stride] stacked; radius: float32[H, rows] (PER_ROW) or r_scalar.
 * Parity status: pinned by H = 1 (must reproduce orc_quantify), identical heads, a
 * permutation of the heads, and a two-head example whose averaged distribution is uniform.
 * ---------------------------------------------------------------------------------------- */
int orc_ensemble(const void *heads, int dtype, int32_t n_heads, int64_t head_stride, int64_t rows,
                 int32_t vocab, int64_t row_stride, int32_t valid_begin, int32_t valid_count,
                 int radius_mode, const float *radius, int radius_is_raw, double r_scalar,
                 double r_max, double lo_cap, double hi_cap, double tau,
                 double *p_max, double *entropy, double *S_lo, double *S_up,
                 double *omega, double *sigma, double *score, uint8_t *flag, uint8_t *row_status,
                 double *margin, double *dense_pbar, int threads)
{
    if (rows < 0 || n_heads < 1 || valid_count < 1 || valid_begin < 0 || valid_begin + (int64_t)valid_count > vocab)
        return 1;
    if (radius_mode == ORC_RADIUS_PER_CODE) return 1;
    const int32_t n = valid_count;
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
    int fail = 0;
#pragma omp parallel
    {
        double *buf = (double *)malloc(sizeof(double) * (size_t)n * 7);
        if (!buf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t row = 0; row < rows; ++row) {
            if (!buf) continue;
            double *c = buf, *e = buf + n, *pbar = buf + 2 * (size_t)n, *cb = buf + 3 * (size_t)n,
                   *rad = buf + 4 * (size_t)n, *lo = buf + 5 * (size_t)n, *up = buf + 6 * (size_t)n;
            int status = 0;
            double rsum = 0.0;
            for (int32_t i = 0; i < n; ++i) pbar[i] = 0.0;
            for (int32_t h = 0; h < n_heads; ++h) {
                orc_tensor t = { (const char *)heads + (size_t)h * (size_t)head_stride * (dtype == ORC_F32 ? 4 : 2),
                                 dtype, rows, vocab, row_stride, valid_begin, valid_count };
                status |= load_row(&t, row, c);
                double r = (radius_mode == ORC_RADIUS_PER_ROW) ? (double)radius[(int64_t)h * rows + row] : r_scalar;
                if (isnan(r)) status |= ORC_ROW_NAN;
                if (status) continue;
                if (radius_is_raw) r = softplus(r);
                if (r > r_max) r = r_max;
                rsum += r;
                double m, z;
                softmax_row(c, n, e, &m, &z);
                for (int32_t i = 0; i < n; ++i) pbar[i] += e[i] / z;
            }
            if (!status) {
                for (int32_t i = 0; i < n; ++i) {
                    pbar[i] /= (double)n_heads;
                    cb[i] = (pbar[i] > 0.0) ? log(pbar[i]) : -INFINITY;
                    rad[i] = rsum / (double)n_heads;
                    if (dense_pbar) dense_pbar[row * (int64_t)n + i] = pbar[i];
                }
                orc_row_result res;
                memset(&res, 0, sizeof res);
                quantify_row(cb, rad, n, 0, r_max, lo_cap, hi_cap, e, lo, up, NULL, NULL, NULL, &res);
                if (p_max) p_max[row] = res.p_max;
                if (entropy) entropy[row] = res.entropy;
                if (S_lo) S_lo[row] = res.S_lo;
                if (S_up) S_up[row] = res.S_up;
                if (omega) omega[row] = res.omega;
                if (sigma) sigma[row] = res.sigma;
                if (score) score[row] = res.score;
                if (flag) flag[row] = res.score > tau;
                if (margin) margin[row] = rel_margin(res.score, tau);
            } else {
                if (p_max) p_max[row] = NAN;
                if (entropy) entropy[row] = NAN;
                if (S_lo) S_lo[row] = NAN;
                if (S_up) S_up[row] = NAN;
                if (omega) omega[row] = NAN;
                if (sigma) sigma[row] = NAN;
                if (score) score[row] = NAN;
                if (flag) flag[row] = 1;
                if (margin) margin[row] = INFINITY;
                if (dense_pbar)
                    for (int32_t i = 0; i < n; ++i) dense_pbar[row * (int64_t)n + i] = NAN;
            }
            if (row_status) row_status[row] = (uint8_t)status;
        }
        free(buf);
    }
    return fail ? 2 : 0;
}

int orc_vote(int32_t n_heads, int64_t rows, const uint8_t *flags /* [H, rows] */, uint8_t *out, int32_t *votes)
{
    if (n_heads < 1 || rows < 0) return 1;
    for (int64_t row = 0; row < rows; ++row) {
        int32_t cnt = 0;
        for (int32_t h = 0; h < n_heads; ++h) cnt += flags[(int64_t)h * rows + row] != 0;
        if (votes) votes[row] = cnt;
        if (out) out[row] = (uint8_t)(2 * cnt > n_heads);
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Inter-DRO loss, forward value (method section, paragraph "Inter-DRO Loss").
 * Per sample (row) n, with centre logits c, radius r = min(Softplus(rho), r_max) per code,
 * cloud logits t:   o_mid = c, o_up = c + r, o_lo = c - r   (Inter-Head: the logit interval),
 *   p_x = softmax(o_x) for x in {mid, up, lo},  p_cloud = softmax(t),
 *   L1_x  = sum_i |p_x,i - p_cloud,i|,
 *   CE_x  = - sum_i p_cloud,i ln p_x,i          (terms with p_cloud,i = 0 are 0),
 *   KL    = sum_i p_cloud,i (ln p_cloud,i - ln p_mid,i).
 * Over the batch of N rows (reading: the paper writes the per-sample losses without a
 * reduction; the mean is taken, and the DRO term is the softmax-weighted sum it prints):
 *   anchor(x) = lambda_v mean_n L1_x + lambda_p mean_n CE_x        (anchor-loss equation)
 *   align     = lambda_beta mean_n KL                               (alignment equation)
 *   w_n = exp(alpha CE_lo^(n)) / sum_k exp(alpha CE_lo^(k)),  dro = sum_n w_n CE_lo^(n)
 *   total = [anchor(mid) + align] + anchor(up) + [anchor(lo) + dro]  (complete-loss equation)
 * l1, ce: [3, rows] in the order mid, up, lo.  loss[6] = total, centre, upper, lower, dro, align.
 * Parity status: pinned by c = t with r = 0 (L1 = 0, KL = 0, CE = entropy of p_cloud), a
 * constant radius (all three distributions coincide), V = 2 closed forms, CE - H = KL,
 * alpha = 0 (dro = mean CE_lo) and large alpha (dro -> max CE_lo), library log-softmax.
 * ---------------------------------------------------------------------------------------- */
static double log_sum_exp(const double *o, int32_t n, double *m_out)
{
    double m = -INFINITY;
    for (int32_t i = 0; i < n; ++i)
        if (o[i] > m) m = o[i];
    double z = 0.0;
    for (int32_t i = 0; i < n; ++i) z += exp(o[i] - m);
    *m_out = m;
    return m + log(z);
}

int orc_interdro(const void *center, const void *radius, const void *cloud, int dtype, int64_t rows,
                 int32_t vocab, int64_t row_stride, int32_t valid_begin, int32_t valid_count,
                 int radius_is_raw, double r_max,
                 double lambda_v, double lambda_p, double lambda_beta, double alpha,
                 double *l1, double *ce, double *kl, double *weights, double *loss, int threads)
{
    if (rows < 1 || valid_count < 1 || valid_begin < 0 || valid_begin + (int64_t)valid_count > vocab)
        return 1;
    const int32_t n = valid_count;
    orc_tensor tc = { center, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    orc_tensor tt = { cloud, dtype, rows, vocab, row_stride, valid_begin, valid_count };
    double *rl1 = (double *)malloc(sizeof(double) * (size_t)rows * 3);
    double *rce = (double *)malloc(sizeof(double) * (size_t)rows * 3);
    double *rkl = (double *)malloc(sizeof(double) * (size_t)rows);
    if (!rl1 || !rce || !rkl) { free(rl1); free(rce); free(rkl); return 2; }
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
    int fail = 0;
#pragma omp parallel
    {
        double *buf = (double *)malloc(sizeof(double) * (size_t)n * 4);
        if (!buf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t row = 0; row < rows; ++row) {
            if (!buf) continue;
            double *c = buf, *t = buf + n, *r = buf + 2 * (size_t)n, *o = buf + 3 * (size_t)n;
            load_row(&tc, row, c);
            load_row(&tt, row, t);
            for (int32_t i = 0; i < n; ++i) {
                double rho = load_elem(radius, dtype, row * row_stride + valid_begin + i);
                double rr = radius_is_raw ? softplus(rho) : rho;
                r[i] = rr > r_max ? r_max : rr;
            }
            double mt;
            double lse_t = log_sum_exp(t, n, &mt);
            for (int x = 0; x < 3; ++x) {
                for (int32_t i = 0; i < n; ++i) o[i] = (x == 0) ? c[i] : (x == 1) ? c[i] + r[i] : c[i] - r[i];
                double mo;
                double lse_o = log_sum_exp(o, n, &mo);
                double s1 = 0.0, sce = 0.0, skl = 0.0;
                for (int32_t i = 0; i < n; ++i) {
                    double lp = o[i] - lse_o, lq = t[i] - lse_t; /* ln p_x,i and ln p_cloud,i */
                    double p = exp(lp), q = exp(lq);
                    s1 += fabs(p - q);
                    if (q > 0.0) {
                        sce -= q * lp;
                        skl += q * (lq - lp);
                    }
                }
                rl1[(size_t)x * rows + row] = s1;
                rce[(size_t)x * rows + row] = sce;
                if (x == 0) rkl[row] = skl;
            }
        }
        free(buf);
    }
    if (!fail) {
        double ml1[3] = { 0, 0, 0 }, mce[3] = { 0, 0, 0 }, mkl = 0.0;
        for (int x = 0; x < 3; ++x) {
            for (int64_t row = 0; row < rows; ++row) {
                ml1[x] += rl1[(size_t)x * rows + row];
                mce[x] += rce[(size_t)x * rows + row];
            }
            ml1[x] /= (double)rows;
            mce[x] /= (double)rows;
        }
        for (int64_t row = 0; row < rows; ++row) mkl += rkl[row];
        mkl /= (double)rows;
        /* adversarial re-weighting of the batch by the lower bound's cross-entropy */
        const double *cel = rce + (size_t)2 * rows;
        double mx = -INFINITY;
        for (int64_t row = 0; row < rows; ++row)
            if (alpha * cel[row] > mx) mx = alpha * cel[row];
        double zs = 0.0;
        for (int64_t row = 0; row < rows; ++row) zs += exp(alpha * cel[row] - mx);
        double dro = 0.0;
        for (int64_t row = 0; row < rows; ++row) {
            double w = exp(alpha * cel[row] - mx) / zs;
            if (weights) weights[row] = w;
            dro += w * cel[row];
        }
        double anchor_mid = lambda_v * ml1[0] + lambda_p * mce[0];
        double anchor_up = lambda_v * ml1[1] + lambda_p * mce[1];
        double anchor_lo = lambda_v * ml1[2] + lambda_p * mce[2];
        double align = lambda_beta * mkl;
        if (loss) {
            loss[1] = anchor_mid + align;
            loss[2] = anchor_up;
            loss[3] = anchor_lo + dro;
            loss[4] = dro;
            loss[5] = align;
            loss[0] = loss[1] + loss[2] + loss[3];
        }
        if (l1) memcpy(l1, rl1, sizeof(double) * (size_t)rows * 3);
        if (ce) memcpy(ce, rce, sizeof(double) * (size_t)rows * 3);
        if (kl) memcpy(kl, rkl, sizeof(double) * (size_t)rows);
    }
    free(rl1);
    free(rce);
    free(rkl);
    return fail ? 2 : 0;
}

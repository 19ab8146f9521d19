/*
 * CPU oracle for the Arbitrage hot path: paged grouped-query attention, the router head and
 * step rollback.  TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline leg of
 * the benchmark call it; the product (the CUDA library) never does and shares no code with it.
 *
 * Everything is the plain definition written out in fp64, one key at a time in logical order:
 * no tiling, no online softmax, no splits.  Inputs are the very bits the GPU reads (fp32 or
 * bf16), widened exactly.  OpenMP only spreads independent output rows over cores.
 *
 * What each function follows:
 *  - oracle_attn: the forward passes inside Algorithm 1 ("Sample draft step", "Sample target step",
 *    and the router's forward over (x, z_d)) reduce, per layer, to causal scaled-dot-product
 *    attention of the new tokens against the cached context x (Section 3.1: a step z is generated
 *    token by token given x and z_<i).  The paper does not print the attention formula; this is the
 *    textbook one, softmax(scale * q.k) v, with grouped-query head sharing and a paged cache.
 *  - oracle_route: Section 4.2 (the router outputs y_hat, the likelihood that the target beats
 *    the draft; reject iff y_hat > tau), Figure 1 caption and Algorithm 1 (accept iff
 *    y_hat <= tau), with the classification head applied to the final-token embedding
 *    (Section 4.2, "Training").  A two-class softmax head equals the sigmoid of the logit
 *    difference, which is the single (w, b) used here.
 *  - oracle_rollback: Algorithm 1, escalation branch: the target regenerates the step from the same
 *    prefix x, so every cache that absorbed the rejected draft step forgets it.
 *  - oracle_policy: the escalation rules the paper compares on PRM scores: the RSD baseline of
 *    Section 3.1 (accept iff s_d > tau), the oracle threshold rule a = 1{Delta > tau} with
 *    Delta = s_t - s_d and the arg-max rule of Section 4.1, the budgeted rule of Appendix B
 *    (Theorem: the min(B, #{Delta > 0}) largest positive advantages), with the wasted-call count of
 *    Section 3.2 (escalated although s_t <= s_d) and the realised score S(a) = s_d + a Delta.
 *  - oracle_route_classes: the C-way heads of the ablation (Section 6.1, Label Granularity and
 *    Classification vs. Regression): a softmax head over C ordered advantage classes, or an ordinal
 *    head (one logit, C - 1 ordered cut points).
 *  - oracle_kv_append: the write of a step's new keys and values into the paged cache that every
 *    "Sample ... step" line of Algorithm 1 implies before the next token attends to them.
 *  - oracle_spearman: the rank correlation the paper reports between the router's predictions and the
 *    oracle advantage (Section 4.2, "Evaluation"; Tables 1-3): Pearson correlation of the two rank
 *    variables, ties sharing the mean of the ranks they span.
 *  - oracle_e4m3_decode / oracle_e4m3_encode: the 8-bit floating-point format E4M3 (1 sign, 4 exponent bits
 *    with bias 7, 3 mantissa bits, no infinities, S.1111.111 = NaN, largest finite value 448) used for
 *    the reduced-precision KV cache of a quantised draft model (Section 5.1 names 4-bit / 3-bit drafts; the
 *    cache format is this library's choice).  Encoding rounds to nearest, ties to the even code, and
 *    saturates at +-448.
 *  - oracle_phase_lens: which sequences take part in a phase of Algorithm 1 (accepted steps are
 *    absorbed by the target's cache, escalated ones are regenerated token by token by the target).
 *
 * Pins (tests/test_oracle_*.py): rows of softmax sum to one; uniform keys give the mean of V;
 * a single key returns its V; a dominant key returns its V; score-shift invariance; brute-force
 * dense numpy attention; a library SDPA routine in fp64; page-permutation invariance; a chunk equals
 * a sequence of decodes; GQA head sharing; hand-built router scores and the tie rule.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

/* status bits reported for inputs that have no defined result */
enum {
    ORACLE_BAD_SEQ_LEN = 1u,   /* seq_len < q_len, or seq_len > max_pages_per_seq * page_size */
    ORACLE_BAD_PAGE = 2u,      /* block_table entry outside [0, num_pages) */
    ORACLE_ROLLBACK_UNDERFLOW = 4u
};

static double widen(const void *base, int dtype, size_t idx)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* element offset of K/V[page][kv_head][slot][0] in the head-major page layout
 * [num_pages, num_kv_heads, page_size, head_dim] */
static size_t kv_offset(long page, int kvh, int slot, int Hkv, int P, int D)
{
    return (((size_t)page * Hkv + kvh) * P + slot) * (size_t)D;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * One output row: query token `i` of sequence `b`, query head `h`.
 *   pos = L_b - n_b + i;  keys j = 0..pos inclusive (a token sees itself)
 *   s_j = scale * q . k_j ; p_j = exp(s_j - max) / sum ; out = sum_j p_j v_j
 * If probs != NULL it receives p_0..p_pos.  Returns status bits (0 = fine).
 */
static unsigned attn_row(int dtype, int Hq, int Hkv, int D, int P, long num_pages, int max_pages,
                         const void *q, const void *k_pages, const void *v_pages,
                         const int32_t *block_row, long q_row, int h, long pos, double scale,
                         double *out_row, double *probs)
{
    int g = Hq / Hkv;
    int kvh = h / g;
    long nkeys = pos + 1;
    double *s = (double *)malloc(sizeof(double) * (size_t)nkeys);
    size_t qoff = ((size_t)q_row * Hq + h) * (size_t)D;
    unsigned status = 0;
    (void)max_pages;

    for (long j = 0; j < nkeys; ++j) {
        long page = block_row[j / P];
        if (page < 0 || page >= num_pages) { status |= ORACLE_BAD_PAGE; break; }
        size_t koff = kv_offset(page, kvh, (int)(j % P), Hkv, P, D);
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += widen(q, dtype, qoff + d) * widen(k_pages, dtype, koff + d);
        s[j] = scale * acc;
    }
    if (status) {
        for (int d = 0; d < D; ++d) out_row[d] = 0.0;
        free(s);
        return status;
    }
    double mx = s[0];
    for (long j = 1; j < nkeys; ++j) if (s[j] > mx) mx = s[j];
    double Z = 0.0;
    for (long j = 0; j < nkeys; ++j) { s[j] = exp(s[j] - mx); Z += s[j]; }
    for (int d = 0; d < D; ++d) out_row[d] = 0.0;
    for (long j = 0; j < nkeys; ++j) {
        double p = s[j] / Z;
        if (probs) probs[j] = p;
        long page = block_row[j / P];
        size_t voff = kv_offset(page, kvh, (int)(j % P), Hkv, P, D);
        for (int d = 0; d < D; ++d)
            out_row[d] += p * widen(v_pages, dtype, voff + d);
    }
    free(s);
    return status;
}

/*
 * Paged grouped-query attention.
 *   q           [total_q, Hq, D]   rows packed by sequence (sequence b owns q_lens[b] rows)
 *   k_pages,
 *   v_pages     [num_pages, Hkv, P, D]
 *   block_table int32 [B, max_pages]
 *   seq_lens    int32 [B]  tokens in the cache INCLUDING the q_lens[b] new ones
 *   q_lens      int32 [B]
 *   out         fp64 [total_q, Hq, D]
 * scale <= 0 means 1/sqrt(D).  Returns the OR of the status bits; a sequence with a bad length
 * gets zero rows, a row that meets a bad page id gets zeros.
 */
unsigned oracle_attn(int dtype, int B, int Hq, int Hkv, int D, int P, long num_pages, int max_pages,
                     const void *q, const void *k_pages, const void *v_pages,
                     const int32_t *block_table, const int32_t *seq_lens, const int32_t *q_lens,
                     double scale, double *out)
{
    if (scale <= 0.0) scale = 1.0 / sqrt((double)D);
    long *row0 = (long *)malloc(sizeof(long) * (size_t)(B + 1));
    row0[0] = 0;
    for (int b = 0; b < B; ++b) row0[b + 1] = row0[b] + (q_lens[b] > 0 ? q_lens[b] : 0);
    unsigned status = 0;

    for (int b = 0; b < B; ++b) {
        long n = q_lens[b], L = seq_lens[b];
        if (n <= 0) continue;
        if (L < n || L > (long)max_pages * P) {
            status |= ORACLE_BAD_SEQ_LEN;
            memset(out + (size_t)row0[b] * Hq * D, 0, sizeof(double) * (size_t)n * Hq * D);
            continue;
        }
        unsigned st_b = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1) reduction(| : st_b)
        for (long i = 0; i < n; ++i)
            for (int h = 0; h < Hq; ++h) {
                long row = row0[b] + i;
                st_b |= attn_row(dtype, Hq, Hkv, D, P, num_pages, max_pages, q, k_pages, v_pages,
                                 block_table + (size_t)b * max_pages, row, h, L - n + i, scale,
                                 out + ((size_t)row * Hq + h) * D, NULL);
            }
        status |= st_b;
    }
    free(row0);
    return status;
}

/* Same as one row of oracle_attn, also returning the softmax probabilities (length pos+1). */
unsigned oracle_attn_row_probs(int dtype, int Hq, int Hkv, int D, int P, long num_pages,
                               int max_pages, const void *q, const void *k_pages,
                               const void *v_pages, const int32_t *block_row, long q_row, int h,
                               long pos, double scale, double *out_row, double *probs)
{
    if (scale <= 0.0) scale = 1.0 / sqrt((double)D);
    return attn_row(dtype, Hq, Hkv, D, P, num_pages, max_pages, q, k_pages, v_pages, block_row,
                    q_row, h, pos, scale, out_row, probs);
}

/*
 * Router head: z = hidden_i . w + b ; score = 1 / (1 + exp(-z)) ; decision = (score > tau).
 * decision 1 = escalate to the target, 0 = accept the draft step (a tie accepts).
 * The comparison is taken on the score rounded to fp32 against tau as fp32, the precision in which
 * the score is stored and the threshold is given.
 */
void oracle_route(int dtype, int n_steps, int hidden_dim, const void *hidden, const void *w,
                  double b, float tau, double *scores, uint8_t *decisions)
{
    for (int i = 0; i < n_steps; ++i) {
        double z = b;
        for (int k = 0; k < hidden_dim; ++k)
            z += widen(hidden, dtype, (size_t)i * hidden_dim + k) * widen(w, dtype, (size_t)k);
        double sc = 1.0 / (1.0 + exp(-z));
        scores[i] = sc;
        decisions[i] = ((float)sc > tau) ? 1 : 0;
    }
}

/*
 * Step rollback: seq_lens[i] -= step_lens[i] * (decisions ? decisions[i] != 0 : 1).
 * No KV bytes move.  A step longer than the sequence clamps to 0 and raises a status bit.
 */
unsigned oracle_rollback(int B, int32_t *seq_lens, const int32_t *step_lens,
                         const uint8_t *decisions)
{
    unsigned status = 0;
    for (int i = 0; i < B; ++i) {
        if (decisions && !decisions[i]) continue;
        long r = (long)seq_lens[i] - (long)step_lens[i];
        if (r < 0 || step_lens[i] < 0) { status |= ORACLE_ROLLBACK_UNDERFLOW; r = r < 0 ? 0 : seq_lens[i]; }
        seq_lens[i] = (int32_t)r;
    }
    return status;
}


/*
 * Escalation policies on PRM scores.  s_d, s_t: fp32 scores of the draft step and of the target's
 * counterpart; decisions[i] = 1 escalates step i to the target, 0 keeps the draft step.
 *   kind 0, RSD (Section 3.1):  accept iff s_d > tau, so escalate iff s_d <= tau; s_t is not read for the
 *           decision (it may be NULL when stats is NULL).
 *   kind 1, oracle threshold (Section 4.1):  escalate iff Delta = s_t - s_d > tau.
 *   kind 2, oracle arg max (Section 4.1):  keep whichever step scores higher; escalate iff s_t > s_d
 *           (a tie keeps the draft: no target call buys nothing).
 *   kind 3, budgeted oracle (Appendix B, Theorem):  escalate the k = min(budget, #{Delta > 0}) steps with
 *           the largest positive Delta; equal advantages go to the lower index.
 * Delta and the comparisons are taken in fp32, the precision the scores are given in.
 * stats (may be NULL): [0] escalations, [1] wasted escalations (a = 1 and s_t <= s_d, Section 3.2),
 * [2] realised score sum_i (a_i ? s_t,i : s_d,i), [3] gain sum_i a_i (s_t,i - s_d,i) in fp64.
 */
typedef struct { float delta; int idx; } oracle_adv;

static int adv_desc(const void *x, const void *y)
{
    const oracle_adv *a = (const oracle_adv *)x, *b = (const oracle_adv *)y;
    if (a->delta > b->delta) return -1;
    if (a->delta < b->delta) return 1;
    return a->idx - b->idx;
}

int oracle_policy(int kind, int n, const float *s_d, const float *s_t, float tau, int budget,
                  uint8_t *decisions, double *stats)
{
    if (kind < 0 || kind > 3 || n < 0) return 1;
    if (kind != 0 && s_t == NULL) return 1;
    if (kind == 3) {
        oracle_adv *adv = (oracle_adv *)malloc(sizeof(oracle_adv) * (size_t)(n > 0 ? n : 1));
        if (!adv) return 2;
        for (int i = 0; i < n; ++i) {
            adv[i].delta = s_t[i] - s_d[i];
            adv[i].idx = i;
            decisions[i] = 0;
        }
        qsort(adv, (size_t)n, sizeof(oracle_adv), adv_desc);
        for (int r = 0; r < n && r < budget; ++r) {
            if (!(adv[r].delta > 0.0f)) break;   /* only positive advantages are worth a call */
            decisions[adv[r].idx] = 1;
        }
        free(adv);
    } else {
        for (int i = 0; i < n; ++i) {
            int a;
            if (kind == 0) a = !(s_d[i] > tau);
            else if (kind == 1) { float delta = s_t[i] - s_d[i]; a = delta > tau; }
            else a = s_t[i] > s_d[i];
            decisions[i] = (uint8_t)a;
        }
    }
    if (stats) {
        double esc = 0, wasted = 0, realised = 0, gain = 0;
        for (int i = 0; i < n; ++i) {
            const double sd = (double)s_d[i], st = s_t ? (double)s_t[i] : sd;
            if (decisions[i]) {
                esc += 1;
                if (!(st > sd)) wasted += 1;
                realised += st;
                gain += st - sd;
            } else {
                realised += sd;
            }
        }
        stats[0] = esc; stats[1] = wasted; stats[2] = realised; stats[3] = gain;
    }
    return 0;
}

/*
 * C-way router heads (Section 6.1 ablation).  The paper says the classes are quantile bins of the
 * advantage, ordered, and that class 0 / 1 of the default head mean accept / escalate; it does not say
 * how a C-way head is turned into one routing score.  Reading taken: the score is the expected class
 * level scaled to [0, 1], score = sum_c p_c * c / (C - 1), and the step escalates iff score > tau (a tie
 * accepts), which for C = 2 is exactly the default head, softmax([l0, l1])_1 = sigmoid(l1 - l0).
 *   mode 0, softmax head:  l_c = hidden . W[c] + b[c],  p = softmax(l).        W: [C, H], b: fp64 [C]
 *   mode 1, ordinal head (cumulative link):  z = hidden . W[0] + b[0];  P(y >= k) = sigmoid(z - cut[k-1]),
 *           k = 1 .. C-1, cut ascending (b[1 .. C-1]);  p_k = P(y >= k) - P(y >= k + 1).  W: [1, H]
 * probs: fp64 [S, C]; scores fp64 [S]; decisions uint8 [S] from the score rounded to fp32.
 */
int oracle_route_classes(int dtype, int mode, int n_steps, int hidden_dim, int n_classes,
                         const void *hidden, const void *w, const double *b, float tau,
                         double *probs, double *scores, uint8_t *decisions)
{
    if (n_classes < 2 || n_classes > 64 || (mode != 0 && mode != 1)) return 1;
    const int C = n_classes;
    for (int i = 0; i < n_steps; ++i) {
        double *p = probs + (size_t)i * C;
        if (mode == 0) {
            double l[64], mx = -INFINITY, z = 0;
            for (int c = 0; c < C; ++c) {
                double acc = b[c];
                for (int k = 0; k < hidden_dim; ++k)
                    acc += widen(hidden, dtype, (size_t)i * hidden_dim + k) * widen(w, dtype, (size_t)c * hidden_dim + k);
                l[c] = acc;
                if (acc > mx) mx = acc;
            }
            for (int c = 0; c < C; ++c) { p[c] = exp(l[c] - mx); z += p[c]; }
            for (int c = 0; c < C; ++c) p[c] /= z;
        } else {
            double acc = b[0], ge[65];
            for (int k = 0; k < hidden_dim; ++k)
                acc += widen(hidden, dtype, (size_t)i * hidden_dim + k) * widen(w, dtype, (size_t)k);
            ge[0] = 1.0;
            for (int k = 1; k < C; ++k) ge[k] = 1.0 / (1.0 + exp(-(acc - b[k])));
            ge[C] = 0.0;
            for (int c = 0; c < C; ++c) p[c] = ge[c] - ge[c + 1];
        }
        double sc = 0;
        for (int c = 0; c < C; ++c) sc += p[c] * (double)c / (double)(C - 1);
        scores[i] = sc;
        decisions[i] = ((float)sc > tau) ? 1 : 0;
    }
    return 0;
}

/*
 * KV append: the new tokens of every sequence go to the slots right behind its cached tokens.
 * k_new, v_new: [total_new, Hkv, D] packed by sequence (new_lens[b] consecutive rows each);
 * token j of sequence b lands at position pos = seq_lens[b] + j, i.e. page block_table[b][pos / P],
 * slot pos % P, of the head-major pools [num_pages, Hkv, P, D].  Values are copied bit for bit (esz
 * bytes per element).  seq_lens is updated to seq_lens + new_lens when update_lens is non-zero.
 * A sequence whose new tokens do not fit (pos >= max_pages * P), with a negative length, or with a
 * block-table entry outside the pool, is left untouched and reported in the status bits.
 */
unsigned oracle_kv_append(int esz, int B, int Hkv, int D, int P, long num_pages, int max_pages,
                          const void *k_new, const void *v_new, const int32_t *block_table,
                          int32_t *seq_lens, const int32_t *new_lens, int update_lens,
                          void *k_pages, void *v_pages)
{
    unsigned status = 0;
    size_t row = 0;
    const size_t tok_bytes = (size_t)D * (size_t)esz;
    for (int b = 0; b < B; ++b) {
        const int n = new_lens[b], L = seq_lens[b];
        if (n <= 0) { if (n < 0) status |= ORACLE_BAD_SEQ_LEN; continue; }
        int ok = L >= 0 && (long)L + n <= (long)max_pages * P;
        if (ok) {
            for (int pos = L; pos < L + n; ++pos) {
                long page = block_table[(size_t)b * max_pages + pos / P];
                if (page < 0 || page >= num_pages) ok = 0;
            }
            if (!ok) status |= ORACLE_BAD_PAGE;
        } else {
            status |= ORACLE_BAD_SEQ_LEN;
        }
        if (ok) {
            for (int j = 0; j < n; ++j) {
                const int pos = L + j;
                const long page = block_table[(size_t)b * max_pages + pos / P];
                for (int h = 0; h < Hkv; ++h) {
                    const size_t dst = kv_offset(page, h, pos % P, Hkv, P, D) * (size_t)esz;
                    const size_t src = ((row + (size_t)j) * Hkv + h) * tok_bytes;
                    memcpy((char *)k_pages + dst, (const char *)k_new + src, tok_bytes);
                    memcpy((char *)v_pages + dst, (const char *)v_new + src, tok_bytes);
                }
            }
            if (update_lens) seq_lens[b] = L + n;
        }
        row += (size_t)n;
    }
    return status;
}


/*
 * Lengths of the next call of a phase of Algorithm 1, from the step lengths and the routing decisions.
 * A sequence takes part in the phase iff decisions is NULL or (decisions[b] != 0) == (want != 0):
 *   token t of a step generated token by token:  out[b] = 1 if it takes part and t < step_lens[b], else 0
 *   a whole step absorbed at once (t < 0):        out[b] = step_lens[b] if it takes part, else 0
 * Negative step lengths count as 0.
 */
void oracle_phase_lens(int B, const int32_t *step_lens, const uint8_t *decisions, int want, int t,
                       int32_t *out)
{
    for (int b = 0; b < B; ++b) {
        const int n = step_lens[b] > 0 ? step_lens[b] : 0;
        const int in = decisions == NULL || ((decisions[b] != 0) == (want != 0));
        out[b] = !in ? 0 : (t < 0 ? n : (t < n ? 1 : 0));
    }
}


/*
 * Spearman's rho of two samples: each value is replaced by its rank among its own sample (1 = smallest;
 * equal values share the average of the ranks they occupy), and rho is the Pearson correlation of the two
 * rank variables, rho = sum (rx - m)(ry - m) / sqrt(sum (rx - m)^2 * sum (ry - m)^2) with m = (n + 1) / 2.
 * Returns NaN when n < 2 or a sample is constant (the correlation is undefined).  ranks_x / ranks_y
 * (nullable) receive the ranks.
 */
double oracle_spearman(int n, const float *x, const float *y, double *ranks_x, double *ranks_y)
{
    if (n < 2) return NAN;
    double *rx = (double *)malloc(sizeof(double) * (size_t)n * 2), *ry = rx + n;
    if (!rx) return NAN;
    for (int i = 0; i < n; ++i) {
        long lx = 0, ex = 0, ly = 0, ey = 0;
        for (int j = 0; j < n; ++j) {
            lx += x[j] < x[i]; ex += x[j] == x[i];
            ly += y[j] < y[i]; ey += y[j] == y[i];
        }
        rx[i] = (double)lx + ((double)ex + 1.0) / 2.0;   /* ranks lx + 1 .. lx + ex, averaged */
        ry[i] = (double)ly + ((double)ey + 1.0) / 2.0;
    }
    const double m = ((double)n + 1.0) / 2.0;
    double sxy = 0, sxx = 0, syy = 0;
    for (int i = 0; i < n; ++i) {
        sxy += (rx[i] - m) * (ry[i] - m);
        sxx += (rx[i] - m) * (rx[i] - m);
        syy += (ry[i] - m) * (ry[i] - m);
    }
    if (ranks_x) memcpy(ranks_x, rx, sizeof(double) * (size_t)n);
    if (ranks_y) memcpy(ranks_y, ry, sizeof(double) * (size_t)n);
    free(rx);
    if (!(sxx > 0) || !(syy > 0)) return NAN;
    return sxy / sqrt(sxx * syy);
}


/* E4M3 code -> value.  e = 0: subnormal m * 2^-9; otherwise (1 + m / 8) * 2^(e - 7); 0x7f / 0xff: NaN. */
double oracle_e4m3_decode(uint8_t code)
{
    const int e = (code >> 3) & 15, m = code & 7;
    const double sign = (code & 0x80) ? -1.0 : 1.0;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) return sign * (double)m * ldexp(1.0, -9);
    return sign * (1.0 + (double)m / 8.0) * ldexp(1.0, e - 7);
}

/* value -> nearest E4M3 code, by search over the 127 finite magnitudes: ties go to the even code, anything
 * beyond the largest finite value saturates to it, NaN gives the NaN code. */
uint8_t oracle_e4m3_encode(float x)
{
    if (x != x) return 0x7f;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const double a = fabs((double)x);
    int best = 0;
    double best_err = a;   /* code 0 = 0.0 */
    for (int c = 1; c <= 0x7e; ++c) {
        const double err = fabs(oracle_e4m3_decode((uint8_t)c) - a);
        if (err < best_err || (err == best_err && (c & 1) == 0)) { best = c; best_err = err; }
    }
    return (uint8_t)(sign | best);
}

/* codes[i] = encode(x[i] * inv_scale), the product taken in fp32 */
void oracle_e4m3_encode_array(long n, const float *x, float inv_scale, uint8_t *codes)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) {   /* independent elements */
        volatile float y = x[i] * inv_scale;
        codes[i] = oracle_e4m3_encode(y);
    }
}

void oracle_e4m3_decode_array(long n, const uint8_t *codes, float *x)
{
    for (long i = 0; i < n; ++i) x[i] = (float)oracle_e4m3_decode(codes[i]);
}

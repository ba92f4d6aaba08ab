/*
 * CPU oracle for arithmetic sampling -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, fp64 restatement of decoding a code point against a
 * next-token distribution, written from the paper (Vilnis et al.,
 * "Arithmetic Sampling", arXiv 2210.15458).  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may call it.  It shares no code with
 * the CUDA library.
 *
 * What each function follows:
 *   orc_lattice_codes     Definition "Arithmetic sampling" (Sec. 4.2) and Eq. 2:
 *                         a regular lattice with one shared uniform shift,
 *                         taken modulo 1; spacing 1/N so that every gap on the
 *                         circle (including the wrap) is exactly 1/N.
 *   orc_step              one pass of the loop body of Algorithm 1 ("Sampling
 *                         from a Code Point"): CDF w over the ordered
 *                         vocabulary, the token whose interval holds the code,
 *                         and the rescaled code c <- (c - m)/(M - m); with the
 *                         logit modifiers the paper names as compatible
 *                         (temperature, top-k: Sec. 2 and "Top-k sampling" in
 *                         Sec. 5.1; nucleus: Sec. 2).
 *   orc_decode_bigram*    Algorithm 1's REPEAT ... UNTIL X = EOS loop over a
 *                         bigram model (row = next-token logits given the
 *                         previous token), stopping at EOS and padding
 *                         (Sec. 3.3, last paragraph).
 *   orc_encode_bigram     the other direction of the codebook (Sec. 4.1): the
 *                         interval [w, w + P(sequence)) of a sequence in
 *                         dictionary order.
 *   orc_ngram_diversity   the n-gram diversity score of Sec. 5.1 ("Diverse beam
 *                         generation"): d = sum_{n=1..4} d_n, d_n = unique
 *                         n-grams / all n-grams in the N sequences of a group.
 *   orc_reward_mean       the sample-mean estimator (1/N) sum_i s(x_i) of Sec. 4.2
 *                         (Proposition on its unbiasedness) for an additive
 *                         reward s(x) = sum_t r[x_t].
 *   orc_xp_*              Algorithm 1 with the code carried to unlimited precision:
 *                         c <- (c - m)/(M - m) is real arithmetic in the paper, and a
 *                         lattice code (j + u)/N is a rational whose binary digits never
 *                         run out.  The step is that of an arithmetic decoder: the CDF of
 *                         each step is quantised to 2^32 cells, the interval (m, M) of the
 *                         chosen token becomes an integer sub-range, and further digits of
 *                         the code are shifted in as the range narrows.
 *
 * Readings taken where the paper is silent (all also stated in the design
 * notes): intervals are half-open [F_{i-1}, F_i); order of modifiers is
 * temperature -> top-k -> softmax -> nucleus on that renormalised distribution
 * -> renormalise; ties in top-k / nucleus order go to the lower token index;
 * nucleus keeps the smallest probability-sorted prefix with mass >= top_p;
 * -inf logits are masked; NaN / +inf logits, an all-masked row or a code
 * outside [0,1] give status ORC_ERR_NUMERIC, token -1, code unchanged; pad
 * id is -1; the typical cut takes the nucleus's place; the extended-precision
 * step quantises each step's CDF to 2^32 cells.  Parity unpinned by the paper
 * for: modifier order (typical decoding's place included), pad id, the
 * non-finite policy, the choice of 2^32 cells (they are pinned only by these
 * stated readings; the arithmetic that follows from them is pinned exactly).
 *
 * All sums are Neumaier-compensated so the oracle's own rounding (~1e-16) is
 * far below every tolerance used against it.
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1
#define ORC_OK 0
#define ORC_ERR_INVALID_ARG (-1)
#define ORC_ERR_NUMERIC (-5)

static const double ORC_ONE_BELOW = 1.0 - 0x1p-53; /* largest double below 1 */

/* ---- exact widening of a stored logit to fp64 ---- */
static double load_logit(const void *base, int dtype, long idx)
{
    if (dtype == ORC_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[idx];
}

/* ---- Neumaier compensated sum ---- */
typedef struct { double s, c; } nsum;
static void nsum_add(nsum *a, double x)
{
    double t = a->s + x;
    if (fabs(a->s) >= fabs(x)) a->c += (a->s - t) + x;
    else                       a->c += (x - t) + a->s;
    a->s = t;
}
static double nsum_val(const nsum *a) { return a->s + a->c; }

typedef struct { double key; long idx; } ranked;
static int cmp_key_desc_idx_asc(const void *pa, const void *pb)
{
    const ranked *a = (const ranked *)pa, *b = (const ranked *)pb;
    if (a->key > b->key) return -1;
    if (a->key < b->key) return 1;
    if (a->idx < b->idx) return -1;
    if (a->idx > b->idx) return 1;
    return 0;
}

typedef struct {
    int32_t token;
    double code_out, p_tok, cdf_lo, d_tok, d_topp;
    int32_t n_kept, tie_topk, status;
} step_result;

/*
 * The modified next-token distribution of one row (steps 1-6 of the loop body of
 * Algorithm 1 with the logit modifiers): on return keep[j] marks the kept tokens,
 * e[j] holds their unnormalised masses exp(l_j/temp - max) (0 for the others) and
 * *Z_out their sum in index order.  Work arrays l, e (V doubles), keep (V bytes),
 * rk (V ranked) are supplied by the caller.  Returns ORC_OK or ORC_ERR_NUMERIC
 * (NaN / +inf logit, no finite logit); fills n_kept, d_topp, tie_topk of `out`.
 */
static int kept_masses(const void *row, int dtype, long V, double temp, long top_k, double top_p,
                       double typical_p, double *l, double *e, char *keep, ranked *rk, double *Z_out,
                       step_result *out)
{
    long j, nK = 0;
    out->d_topp = INFINITY; out->n_kept = 0; out->tie_topk = 0;

    /* 1-2: widen exactly; masked = -inf; NaN / +inf are errors */
    for (j = 0; j < V; ++j) {
        l[j] = load_logit(row, dtype, j);
        if (isnan(l[j]) || l[j] == INFINITY) return ORC_ERR_NUMERIC;
        keep[j] = (l[j] > -INFINITY);
        nK += keep[j];
    }
    if (nK == 0) return ORC_ERR_NUMERIC;

    /* 3: top-k on the logits, order (value desc, index asc) */
    if (top_k > 0 && top_k < nK) {
        long n = 0, r;
        for (j = 0; j < V; ++j) if (keep[j]) { rk[n].key = l[j]; rk[n].idx = j; ++n; }
        qsort(rk, (size_t)n, sizeof(ranked), cmp_key_desc_idx_asc);
        for (r = top_k; r < n; ++r) keep[rk[r].idx] = 0;
        for (r = 0; r < n; ++r) if (rk[r].key == rk[top_k - 1].key) out->tie_topk++;
        nK = top_k;
    }

    /* 4: temperature and stable softmax numerators over the survivors */
    double m = -INFINITY;
    for (j = 0; j < V; ++j) if (keep[j]) { double x = l[j] / temp; if (x > m) m = x; }
    nsum z1 = {0.0, 0.0};
    for (j = 0; j < V; ++j) {
        if (keep[j]) { e[j] = exp(l[j] / temp - m); nsum_add(&z1, e[j]); }
        else e[j] = 0.0;
    }
    double Z1 = nsum_val(&z1);

    /* 4b: locally typical set (Sec. 2 names typical decoding among the compatible logit modifiers;
     * rule of Meister et al.): with H the entropy of the distribution over the survivors, order
     * them by |-ln p_j - H| ascending (index ascending among equals) and keep the smallest prefix
     * with mass >= typical_p.  It takes the nucleus's place: a step has one or the other.
     * d_topp reports how far the cut is from being ambiguous: the normalised distance of the two
     * straddling prefix masses from the target, or 0 when the last kept and the first dropped
     * token are nearer than 1e-9 in |-ln p - H| (their order then hangs on rounding). */
    if (typical_p > 0.0 && typical_p < 1.0) {
        long n = 0, r, cut;
        double lnZ = log(Z1);
        nsum h = {0.0, 0.0};
        for (j = 0; j < V; ++j)
            if (keep[j] && e[j] > 0.0) nsum_add(&h, -(e[j] / Z1) * ((l[j] / temp - m) - lnZ));
        double H = nsum_val(&h);
        for (j = 0; j < V; ++j)
            if (keep[j]) { rk[n].key = -fabs(-((l[j] / temp - m) - lnZ) - H); rk[n].idx = j; ++n; }
        qsort(rk, (size_t)n, sizeof(ranked), cmp_key_desc_idx_asc);     /* -distance descending */
        double target = typical_p * Z1, before = 0.0, after = 0.0;
        nsum run = {0.0, 0.0};
        cut = n;
        for (r = 0; r < n; ++r) {
            before = nsum_val(&run);
            nsum_add(&run, e[rk[r].idx]);
            after = nsum_val(&run);
            if (after >= target) { cut = r + 1; break; }
        }
        for (r = cut; r < n; ++r) { keep[rk[r].idx] = 0; e[rk[r].idx] = 0.0; }
        if (cut < n || after >= target) {
            double a = fabs(target - before), b = fabs(after - target);
            out->d_topp = (a < b ? a : b) / Z1;
        }
        if (cut < n && rk[cut - 1].key - rk[cut].key < 1e-9 &&
            l[rk[cut - 1].idx] != l[rk[cut].idx])
            out->d_topp = 0.0;
        nK = cut;
        /* renormalised total for whatever follows */
        nsum z2 = {0.0, 0.0};
        for (j = 0; j < V; ++j) if (keep[j]) nsum_add(&z2, e[j]);
        Z1 = nsum_val(&z2);
    }

    /* 5: nucleus: smallest (prob desc, index asc) prefix with mass >= top_p */
    if (top_p > 0.0 && top_p < 1.0) {
        long n = 0, r, cut;
        for (j = 0; j < V; ++j) if (keep[j]) { rk[n].key = e[j]; rk[n].idx = j; ++n; }
        qsort(rk, (size_t)n, sizeof(ranked), cmp_key_desc_idx_asc);
        double target = top_p * Z1, before = 0.0, after = 0.0;
        nsum run = {0.0, 0.0};
        cut = n;                                   /* keep everything if never reached */
        for (r = 0; r < n; ++r) {
            before = nsum_val(&run);
            nsum_add(&run, rk[r].key);
            after = nsum_val(&run);
            if (after >= target) { cut = r + 1; break; }
        }
        for (r = cut; r < n; ++r) { keep[rk[r].idx] = 0; e[rk[r].idx] = 0.0; }
        if (cut < n || after >= target) {
            double a = fabs(target - before), b = fabs(after - target);
            out->d_topp = (a < b ? a : b) / Z1;
        }
        nK = cut;
    }

    /* 6: renormalise over the final kept set, summed in index order */
    nsum z = {0.0, 0.0};
    for (j = 0; j < V; ++j) if (keep[j]) nsum_add(&z, e[j]);
    *Z_out = nsum_val(&z);
    out->n_kept = (int32_t)nK;
    return ORC_OK;
}

/*
 * One step for one lane (Algorithm 1, loop body).  row points at V stored
 * logits.  Work arrays as for kept_masses.
 */
static void step_lane_t(const void *row, int dtype, long V, double c, double temp,
                        long top_k, double top_p, double typical_p, double *l, double *e, char *keep,
                        ranked *rk, step_result *out)
{
    long j;
    double Z;
    out->token = -1; out->code_out = c; out->p_tok = 0.0; out->cdf_lo = 0.0;
    out->d_tok = 0.0; out->d_topp = INFINITY; out->n_kept = 0; out->tie_topk = 0;
    out->status = ORC_ERR_NUMERIC;

    if (!(c >= 0.0 && c <= 1.0)) return;          /* also rejects NaN */
    if (c == 1.0) c = ORC_ONE_BELOW;              /* code domain is [0,1) */

    if (kept_masses(row, dtype, V, temp, top_k, top_p, typical_p, l, e, keep, rk, &Z, out) != ORC_OK) {
        out->n_kept = 0; out->d_topp = INFINITY; out->tie_topk = 0;
        return;
    }

    /* 7: first kept j (ascending index) with c*Z < S_j (inclusive prefix) */
    double t = c * Z, S_excl = 0.0;
    long chosen = -1, last = -1;
    double S_last = 0.0;
    nsum run = {0.0, 0.0};
    for (j = 0; j < V; ++j) {
        if (!keep[j]) continue;
        double before = nsum_val(&run);
        nsum_add(&run, e[j]);
        last = j; S_last = before;
        if (t < nsum_val(&run)) { chosen = j; S_excl = before; break; }
    }
    if (chosen < 0) { chosen = last; S_excl = S_last; }  /* rounding at the top end */

    /* 8: rescale the code into the chosen interval */
    double cn = (t - S_excl) / e[chosen];
    if (!(cn >= 0.0)) cn = 0.0;
    if (cn > ORC_ONE_BELOW) cn = ORC_ONE_BELOW;

    /* 9: diagnostics */
    double lo = S_excl / Z, hi = (S_excl + e[chosen]) / Z;
    double da = c - lo, db = hi - c;
    out->token = (int32_t)chosen;
    out->code_out = cn;
    out->p_tok = e[chosen] / Z;
    out->cdf_lo = lo;
    out->d_tok = da < db ? da : db;
    out->status = ORC_OK;
}

static void step_lane(const void *row, int dtype, long V, double c, double temp,
                      long top_k, double top_p, double *l, double *e, char *keep,
                      ranked *rk, step_result *out)
{
    step_lane_t(row, dtype, V, c, temp, top_k, top_p, 1.0, l, e, keep, rk, out);
}

typedef struct { double *l, *e; char *keep; ranked *rk; } workspace;
static int ws_alloc(workspace *w, long V)
{
    w->l = (double *)malloc(sizeof(double) * (size_t)V);
    w->e = (double *)malloc(sizeof(double) * (size_t)V);
    w->keep = (char *)malloc((size_t)V);
    w->rk = (ranked *)malloc(sizeof(ranked) * (size_t)V);
    return w->l && w->e && w->keep && w->rk;
}
static void ws_free(workspace *w) { free(w->l); free(w->e); free(w->keep); free(w->rk); }

static int check_params(long V, double temp, long top_k, double top_p)
{
    if (V < 1) return 0;
    if (!(temp > 0.0) || isinf(temp)) return 0;
    if (top_k < 0) return 0;
    if (isnan(top_p)) return 0;
    return 1;
}

/*
 * Lattice of N codes with one shared shift u in [0,1):  c_j = (j + u)/N, j = 0..N-1.
 */
int orc_lattice_codes(long N, double u, double *codes)
{
    long j;
    if (N < 1 || !(u >= 0.0 && u < 1.0) || !codes) return ORC_ERR_INVALID_ARG;
    for (j = 0; j < N; ++j) {
        double c = ((double)j + u) / (double)N;
        if (c >= 1.0) c -= 1.0;
        codes[j] = c;
    }
    return ORC_OK;
}

/*
 * One decode step for lanes [lane_begin, lane_end) of logits[lanes, ld].
 * Any output pointer may be NULL.  Outputs are indexed by absolute lane.
 */
/*
 * The code sets the paper itself writes down, as variants of the lattice above:
 *   variant 1  Definition "Arithmetic sampling" (Sec. 4.2) as printed:
 *              c_i = (i/(N+1) + b) mod 1, i = 1..N, one shared b in [0,1);
 *   variant 2  the naive codebook of the proposition "Naive arithmetic
 *              sampling" (Sec. 4.2): c_i = i/(N+1), i = 1..N, no shift (the
 *              example after it: N = 1 gives the single code 0.5).
 * codes[i-1] receives c_i.  Variant 0 is orc_lattice_codes.
 */
int orc_lattice_codes_variant(long N, double b, long variant, double *codes)
{
    long i;
    if (variant == 0) return orc_lattice_codes(N, b, codes);
    if (N < 1 || !codes || (variant != 1 && variant != 2)) return ORC_ERR_INVALID_ARG;
    if (variant == 1 && !(b >= 0.0 && b < 1.0)) return ORC_ERR_INVALID_ARG;
    for (i = 1; i <= N; ++i) {
        double c = (double)i / (double)(N + 1);
        if (variant == 1) {
            c += b;
            if (c >= 1.0) c -= 1.0;
        }
        codes[i - 1] = c;
    }
    return ORC_OK;
}

static int step_all(const void *logits, int dtype, long lanes, long V, long ld,
             const double *codes, double temp, long top_k, double top_p, double typical_p,
             int32_t *tokens, double *codes_out, double *p_tok, double *cdf_lo,
             int32_t *n_kept, double *d_tok, double *d_topp, int32_t *tie_topk,
             int32_t *status, long lane_begin, long lane_end)
{
    workspace w;
    long i;
    size_t esz = dtype == ORC_BF16 ? 2 : 4;
    if (!logits || !codes || lanes < 0 || ld < V || !check_params(V, temp, top_k, top_p))
        return ORC_ERR_INVALID_ARG;
    if (dtype != ORC_F32 && dtype != ORC_BF16) return ORC_ERR_INVALID_ARG;
    if (lane_begin < 0 || lane_end > lanes) return ORC_ERR_INVALID_ARG;
    if (!ws_alloc(&w, V)) { ws_free(&w); return ORC_ERR_INVALID_ARG; }
    for (i = lane_begin; i < lane_end; ++i) {
        step_result r;
        const char *row = (const char *)logits + (size_t)i * (size_t)ld * esz;
        step_lane_t(row, dtype, V, codes[i], temp, top_k, top_p, typical_p, w.l, w.e, w.keep, w.rk, &r);
        if (tokens) tokens[i] = r.token;
        if (codes_out) codes_out[i] = r.code_out;
        if (p_tok) p_tok[i] = r.p_tok;
        if (cdf_lo) cdf_lo[i] = r.cdf_lo;
        if (n_kept) n_kept[i] = r.n_kept;
        if (d_tok) d_tok[i] = r.d_tok;
        if (d_topp) d_topp[i] = r.d_topp;
        if (tie_topk) tie_topk[i] = r.tie_topk;
        if (status) status[i] = r.status;
    }
    ws_free(&w);
    return ORC_OK;
}

int orc_step(const void *logits, int dtype, long lanes, long V, long ld,
             const double *codes, double temp, long top_k, double top_p,
             int32_t *tokens, double *codes_out, double *p_tok, double *cdf_lo,
             int32_t *n_kept, double *d_tok, double *d_topp, int32_t *tie_topk,
             int32_t *status, long lane_begin, long lane_end)
{
    return step_all(logits, dtype, lanes, V, ld, codes, temp, top_k, top_p, 1.0, tokens, codes_out, p_tok,
                    cdf_lo, n_kept, d_tok, d_topp, tie_topk, status, lane_begin, lane_end);
}

/* orc_step with the locally typical cut of mass typical_p in place of the nucleus */
int orc_step_typical(const void *logits, int dtype, long lanes, long V, long ld,
                     const double *codes, double temp, long top_k, double typical_p,
                     int32_t *tokens, double *codes_out, double *p_tok, double *cdf_lo,
                     int32_t *n_kept, double *d_tok, double *d_topp, int32_t *tie_topk,
                     int32_t *status, long lane_begin, long lane_end)
{
    if (isnan(typical_p)) return ORC_ERR_INVALID_ARG;
    return step_all(logits, dtype, lanes, V, ld, codes, temp, top_k, 1.0, typical_p, tokens, codes_out, p_tok,
                    cdf_lo, n_kept, d_tok, d_topp, tie_topk, status, lane_begin, lane_end);
}

/*
 * Algorithm 1's loop over a bigram model for lanes [lane_begin, lane_end):
 * lane i starts from previous token prev[i] and code codes_in[i]; at each of
 * at most T steps the row table[prev] gives the next-token logits.  A lane
 * stops after emitting eos (pass eos < 0 for "no EOS"); the rest of its row of
 * seq[lanes, T] is padded with -1 and len[i] = number of tokens emitted.
 * Optional per-step traces (each [lanes, T], may be NULL): the code the step
 * started from, its rescaled code, p_tok and d_tok.
 */
int orc_decode_bigram_codes(const void *table, int dtype, long V, long ld,
                            const int32_t *prev, const double *codes_in, long lanes,
                            long T, long eos, double temp, long top_k, double top_p,
                            int32_t *seq, int32_t *len, double *codes_final,
                            int32_t *status, double *trace_code_in,
                            double *trace_code_out, double *trace_p_tok,
                            double *trace_d_tok, long lane_begin, long lane_end)
{
    workspace w;
    long i, t;
    size_t esz = dtype == ORC_BF16 ? 2 : 4;
    if (!table || !prev || !codes_in || !seq || lanes < 0 || T < 0 || ld < V ||
        !check_params(V, temp, top_k, top_p))
        return ORC_ERR_INVALID_ARG;
    if (dtype != ORC_F32 && dtype != ORC_BF16) return ORC_ERR_INVALID_ARG;
    if (lane_begin < 0 || lane_end > lanes) return ORC_ERR_INVALID_ARG;
    for (i = lane_begin; i < lane_end; ++i)
        if (prev[i] < 0 || prev[i] >= V) return ORC_ERR_INVALID_ARG;
    if (!ws_alloc(&w, V)) { ws_free(&w); return ORC_ERR_INVALID_ARG; }
    for (i = lane_begin; i < lane_end; ++i) {
        long p = prev[i], n = 0;
        double c = codes_in[i];
        int32_t st = ORC_OK;
        for (t = 0; t < T; ++t) {
            seq[i * T + t] = -1;
            if (trace_code_in) trace_code_in[i * T + t] = NAN;
            if (trace_code_out) trace_code_out[i * T + t] = NAN;
            if (trace_p_tok) trace_p_tok[i * T + t] = NAN;
            if (trace_d_tok) trace_d_tok[i * T + t] = NAN;
        }
        for (t = 0; t < T; ++t) {
            step_result r;
            const char *row = (const char *)table + (size_t)p * (size_t)ld * esz;
            step_lane(row, dtype, V, c, temp, top_k, top_p, w.l, w.e, w.keep, w.rk, &r);
            if (r.status != ORC_OK) { st = r.status; break; }
            if (trace_code_in) trace_code_in[i * T + t] = c;
            if (trace_code_out) trace_code_out[i * T + t] = r.code_out;
            if (trace_p_tok) trace_p_tok[i * T + t] = r.p_tok;
            if (trace_d_tok) trace_d_tok[i * T + t] = r.d_tok;
            seq[i * T + t] = r.token;
            n = t + 1;
            c = r.code_out;
            p = r.token;
            if (r.token == eos) break;
        }
        if (len) len[i] = (int32_t)n;
        if (codes_final) codes_final[i] = c;
        if (status) status[i] = st;
    }
    ws_free(&w);
    return ORC_OK;
}

/*
 * Same loop with the code set of the Definition in Sec. 4.2: S start tokens,
 * N lattice codes each sharing one shift u; lane = s*N + j decodes code c_j
 * from previous token start[s].
 */
int orc_decode_bigram(const void *table, int dtype, long V, long ld,
                      const int32_t *start, long S, long N, double u, long T, long eos,
                      double temp, long top_k, double top_p,
                      int32_t *seq, int32_t *len, double *codes_final, int32_t *status)
{
    long s, j, lanes = S * N;
    int rc;
    if (S < 0 || N < 1 || !start) return ORC_ERR_INVALID_ARG;
    double *lat = (double *)malloc(sizeof(double) * (size_t)N);
    double *codes = (double *)malloc(sizeof(double) * (size_t)(lanes > 0 ? lanes : 1));
    int32_t *prev = (int32_t *)malloc(sizeof(int32_t) * (size_t)(lanes > 0 ? lanes : 1));
    if (!lat || !codes || !prev) { free(lat); free(codes); free(prev); return ORC_ERR_INVALID_ARG; }
    rc = orc_lattice_codes(N, u, lat);
    if (rc == ORC_OK) {
        for (s = 0; s < S; ++s)
            for (j = 0; j < N; ++j) { codes[s * N + j] = lat[j]; prev[s * N + j] = start[s]; }
        rc = orc_decode_bigram_codes(table, dtype, V, ld, prev, codes, lanes, T, eos, temp,
                                     top_k, top_p, seq, len, codes_final, status,
                                     NULL, NULL, NULL, NULL, 0, lanes);
    }
    free(lat); free(codes); free(prev);
    return rc;
}

/*
 * Codebook, sequence -> interval (Sec. 4.1): for each lane, the interval
 * [lo, lo + width) in dictionary order of the token sequence seq[i, 0..len-1]
 * continued from prev[i]: lo accumulates width * F_{i-1}, width multiplies by
 * p_i, with the same modified conditional distributions as orc_step.  A token
 * of probability zero gives status ORC_ERR_NUMERIC.
 */
int orc_encode_bigram(const void *table, int dtype, long V, long ld,
                      const int32_t *prev, const int32_t *seq, const int32_t *len,
                      long lanes, long T, double temp, long top_k, double top_p,
                      double *lo_out, double *width_out, int32_t *status)
{
    workspace w;
    long i, t, j;
    size_t esz = dtype == ORC_BF16 ? 2 : 4;
    if (!table || !prev || !seq || !len || lanes < 0 || T < 0 || ld < V ||
        !check_params(V, temp, top_k, top_p))
        return ORC_ERR_INVALID_ARG;
    if (!ws_alloc(&w, V)) { ws_free(&w); return ORC_ERR_INVALID_ARG; }
    for (i = 0; i < lanes; ++i) {
        nsum lo = {0.0, 0.0};
        double width = 1.0;
        long p = prev[i];
        int32_t st = ORC_OK;
        for (t = 0; t < len[i] && t < T; ++t) {
            long tok = seq[i * T + t];
            if (p < 0 || p >= V || tok < 0 || tok >= V) { st = ORC_ERR_INVALID_ARG; break; }
            /* the distribution of this step: run the step with a code that
               cannot fail, then rebuild the kept set's masses from keep/e */
            step_result r;
            const char *row = (const char *)table + (size_t)p * (size_t)ld * esz;
            step_lane(row, dtype, V, 0.0, temp, top_k, top_p, w.l, w.e, w.keep, w.rk, &r);
            if (r.status != ORC_OK) { st = r.status; break; }
            if (!w.keep[tok]) { st = ORC_ERR_NUMERIC; break; }
            nsum z = {0.0, 0.0}, below = {0.0, 0.0};
            for (j = 0; j < V; ++j) if (w.keep[j]) {
                nsum_add(&z, w.e[j]);
                if (j < tok) nsum_add(&below, w.e[j]);
            }
            double Z = nsum_val(&z);
            nsum_add(&lo, width * (nsum_val(&below) / Z));
            width *= w.e[tok] / Z;
            p = tok;
        }
        if (lo_out) lo_out[i] = nsum_val(&lo);
        if (width_out) width_out[i] = width;
        if (status) status[i] = st;
    }
    ws_free(&w);
    return ORC_OK;
}

/*
 * n-gram diversity (Sec. 5.1, "Diverse beam generation"): for every group g
 * of N consecutive lanes and n = 1..4,
 *   total[g][n-1]  = number of n-grams in the group's sequences
 *                  = sum_i max(len_i - n + 1, 0)
 *   unique[g][n-1] = number of distinct ones among them (an n-gram is the
 *                    tuple of n consecutive emitted tokens; padding is not
 *                    part of any n-gram)
 *   d[g] = sum_n unique/total, a term with total = 0 contributing 0
 * (reading: the paper does not say what an empty denominator gives).
 * By the definition: write out all n-grams, sort them, count the distinct.
 */
static long g_ng_n;
static int cmp_ngram(const void *pa, const void *pb)
{
    const int32_t *a = (const int32_t *)pa, *b = (const int32_t *)pb;
    long k;
    for (k = 0; k < g_ng_n; ++k) {
        if (a[k] < b[k]) return -1;
        if (a[k] > b[k]) return 1;
    }
    return 0;
}

int orc_ngram_diversity(const int32_t *seq, const int32_t *len, long S, long N, long T,
                        int64_t *unique, int64_t *total, double *d)
{
    long g, n, i, t, k;
    if (!seq || !len || !unique || !total || !d || S < 0 || N < 1 || T < 0) return ORC_ERR_INVALID_ARG;
    int32_t *buf = (int32_t *)malloc(sizeof(int32_t) * 4 * (size_t)(N * T + 1));
    if (!buf) return ORC_ERR_INVALID_ARG;
    for (g = 0; g < S; ++g) {
        double dsum = 0.0;
        for (n = 1; n <= 4; ++n) {
            long m = 0;
            for (i = 0; i < N; ++i) {
                long lane = g * N + i;
                long L = len[lane] < T ? len[lane] : T;
                for (t = 0; t + n <= L; ++t, ++m)
                    for (k = 0; k < n; ++k) buf[m * n + k] = seq[lane * T + t + k];
            }
            g_ng_n = n;
            qsort(buf, (size_t)m, sizeof(int32_t) * (size_t)n, cmp_ngram);
            long u = 0;
            for (i = 0; i < m; ++i)
                if (i == 0 || cmp_ngram(buf + (i - 1) * n, buf + i * n) != 0) ++u;
            unique[g * 4 + n - 1] = u;
            total[g * 4 + n - 1] = m;
            if (m > 0) dsum += (double)u / (double)m;
        }
        d[g] = dsum;
    }
    free(buf);
    return ORC_OK;
}

/*
 * Sample-mean estimator (Sec. 4.2, Proposition "estimator unbiased and
 * consistent"; used in Sec. 5.2): with the additive reward
 * s(x) = sum_{t < len} r[x_t], per lane s, per group of N consecutive lanes
 * mean[g] = (1/N) sum_i s(x_i).
 */
int orc_reward_mean(const int32_t *seq, const int32_t *len, long S, long N, long T,
                    const double *r, long V, double *lane_reward, double *mean)
{
    long g, i, t;
    if (!seq || !len || !r || !mean || S < 0 || N < 1 || T < 0 || V < 1) return ORC_ERR_INVALID_ARG;
    for (g = 0; g < S; ++g) {
        nsum acc = {0.0, 0.0};
        for (i = 0; i < N; ++i) {
            long lane = g * N + i;
            long L = len[lane] < T ? len[lane] : T;
            nsum s = {0.0, 0.0};
            for (t = 0; t < L; ++t) {
                long tok = seq[lane * T + t];
                if (tok < 0 || tok >= V) return ORC_ERR_INVALID_ARG;
                nsum_add(&s, r[tok]);
            }
            if (lane_reward) lane_reward[lane] = nsum_val(&s);
            nsum_add(&acc, nsum_val(&s));
        }
        mean[g] = nsum_val(&acc) / (double)N;
    }
    return ORC_OK;
}


/* ------------------------------------------------------------------------------------------
 * Extended-precision codes (Algorithm 1 in exact arithmetic).
 *
 * The code of lane j is the rational c = (j + u')/N with u' = floor(u 2^53)/2^53 (the shift
 * read to 53 fractional bits).  With A = j 2^53 + floor(u 2^53), q0 = A div N, rem = A mod N:
 *   c = q0 / 2^53 + (rem / N) / 2^53,
 * so its binary digits are the 53 bits of q0 followed by the digits of rem/N, which long
 * division produces one at a time for ever.
 *
 * Lane state, four 64-bit words:
 *   [0] range   the current interval has `range` units; (2^62, 2^63] after every step
 *   [1] code    the code's offset inside it, in the same units, < range
 *   [2] q       the bits of q0 not yet shifted in (right-aligned)
 *   [3] (nq << 32) | rem    how many those are, and the long-division remainder
 * One step: r = range >> 32 is the size of one of 2^32 cells; the code lies in cell
 * t = min(code div r, 2^32 - 1).  With P_0 = 0 <= P_1 <= ... the prefix sums of the kept masses
 * in index order and F(P) = floor(P * (2^32 / Z)) (F of the last one := 2^32), token j owns
 * the cells [F(P_j), F(P_{j+1})): the token is the first kept j with F(P_{j+1}) > t; then
 * code -= r F(P_j), range = r (F(P_{j+1}) - F(P_j)) -- the last kept token also takes the
 * range mod 2^32 units left over -- and digits of c are shifted in until range > 2^62 again.
 * All of this is integer arithmetic: the decoded sequence is exactly the one whose interval
 * in this nested subdivision holds c.
 * ------------------------------------------------------------------------------------------ */
#define XP_CELLS 4294967296.0          /* 2^32 */
#define XP_RANGE_TOP (1ull << 63)
#define XP_RANGE_LOW (1ull << 62)

static uint64_t xp_next_bit(uint64_t *st, uint64_t N)
{
    uint64_t nq = st[3] >> 32, rem = st[3] & 0xFFFFFFFFull, bit;
    if (nq > 0) {
        --nq;
        bit = (st[2] >> nq) & 1ull;
        st[2] &= (nq ? ((1ull << nq) - 1ull) : 0ull);
    } else {
        rem <<= 1;
        bit = rem >= N;
        if (bit) rem -= N;
    }
    st[3] = (nq << 32) | rem;
    return bit;
}

/* state of the lattice codes (j + u)/N for j = j0 .. j0 + count - 1, written S times over
 * (one copy per start token: lane = s*count + (j - j0)) */
int orc_xp_lattice_state(long N, double u, long j0, long count, long S, uint64_t *state)
{
    long i, s, k;
    if (N < 1 || N > 0x7FFFFFFFL || S < 0 || j0 < 0 || count < 0 || j0 + count > N || !state ||
        !(u >= 0.0 && u < 1.0))
        return ORC_ERR_INVALID_ARG;
    uint64_t U = (uint64_t)floor(u * 9007199254740992.0);            /* floor(u 2^53), exact */
    for (i = 0; i < count; ++i) {
        unsigned __int128 A = ((unsigned __int128)(uint64_t)(j0 + i) << 53) + U;
        uint64_t st[4];
        st[0] = XP_RANGE_TOP;
        st[1] = 0;
        st[2] = (uint64_t)(A / (uint64_t)N);
        st[3] = ((uint64_t)53 << 32) | (uint64_t)(A % (uint64_t)N);
        for (k = 0; k < 63; ++k) st[1] = (st[1] << 1) | xp_next_bit(st, (uint64_t)N);
        for (s = 0; s < S; ++s) memcpy(state + ((size_t)s * (size_t)count + (size_t)i) * 4, st, sizeof st);
    }
    return ORC_OK;
}

/* cell boundaries of one row: cells[j] = F(P_j) for j = 0..V, cells[V] = 2^32; a token that is
 * not kept owns no cell (cells[j+1] == cells[j]).  Returns the status of the row. */
static int xp_row_cells(const void *row, int dtype, long V, double temp, long top_k, double top_p,
                        workspace *w, uint64_t *cells, step_result *info)
{
    long j, last = -1;
    double Z;
    int rc = kept_masses(row, dtype, V, temp, top_k, top_p, 1.0, w->l, w->e, w->keep, w->rk, &Z, info);
    if (rc != ORC_OK) return rc;
    const double K = XP_CELLS / Z;
    nsum run = {0.0, 0.0};
    cells[0] = 0;
    for (j = 0; j < V; ++j) {
        if (w->keep[j]) {
            nsum_add(&run, w->e[j]);
            double f = nsum_val(&run) * K;
            uint64_t F = f >= XP_CELLS ? 0x100000000ull : (uint64_t)f;
            if (F < cells[j]) F = cells[j];            /* (the sums are non-decreasing; kept for safety) */
            cells[j + 1] = F;
            last = j;
        } else {
            cells[j + 1] = cells[j];
        }
    }
    for (j = last; j < V; ++j) cells[j + 1] = 0x100000000ull;   /* the last kept token ends at 2^32 */
    return ORC_OK;
}

int orc_xp_row_cells(const void *row, int dtype, long V, double temp, long top_k, double top_p,
                     uint64_t *cells)
{
    workspace w;
    step_result info;
    if (!row || !cells || !check_params(V, temp, top_k, top_p)) return ORC_ERR_INVALID_ARG;
    if (!ws_alloc(&w, V)) { ws_free(&w); return ORC_ERR_INVALID_ARG; }
    int rc = xp_row_cells(row, dtype, V, temp, top_k, top_p, &w, cells, &info);
    ws_free(&w);
    return rc;
}

/*
 * Algorithm 1's loop with extended-precision codes over a bigram model, lanes
 * [lane_begin, lane_end): lane i starts from previous token prev[i] and state[4 i .. 4 i + 3]
 * (updated in place, so a decode can be split and resumed).  seq, len, status as for
 * orc_decode_bigram_codes.  Optional traces, each [lanes, T]: the position of the code inside
 * the step's distribution, (code / r) / 2^32, and its distance to the nearest end of the
 * chosen token's cell range, both before the step.
 */
int orc_xp_decode_bigram(const void *table, int dtype, long V, long ld, const int32_t *prev,
                         uint64_t *state, long lanes, long N, long T, long eos, double temp,
                         long top_k, double top_p, int32_t *seq, int32_t *len, int32_t *status,
                         double *trace_pos, double *trace_d_tok, long lane_begin, long lane_end)
{
    workspace w;
    long i, t, j;
    size_t esz = dtype == ORC_BF16 ? 2 : 4;
    if (!table || !prev || !state || !seq || lanes < 0 || T < 0 || ld < V || N < 1 || N > 0x7FFFFFFFL ||
        !check_params(V, temp, top_k, top_p))
        return ORC_ERR_INVALID_ARG;
    if (dtype != ORC_F32 && dtype != ORC_BF16) return ORC_ERR_INVALID_ARG;
    if (lane_begin < 0 || lane_end > lanes) return ORC_ERR_INVALID_ARG;
    if (!ws_alloc(&w, V)) { ws_free(&w); return ORC_ERR_INVALID_ARG; }
    uint64_t *cells = (uint64_t *)malloc(sizeof(uint64_t) * (size_t)(V + 1));
    if (!cells) { ws_free(&w); return ORC_ERR_INVALID_ARG; }
    for (i = lane_begin; i < lane_end; ++i) {
        uint64_t *st = state + (size_t)i * 4;
        long p = prev[i], n = 0;
        int32_t rc = ORC_OK;
        for (t = 0; t < T; ++t) {
            seq[i * T + t] = -1;
            if (trace_pos) trace_pos[i * T + t] = NAN;
            if (trace_d_tok) trace_d_tok[i * T + t] = NAN;
        }
        for (t = 0; t < T; ++t) {
            step_result info;
            if (p < 0 || p >= V || st[0] <= XP_RANGE_LOW || st[0] > XP_RANGE_TOP || st[1] >= st[0]) {
                rc = ORC_ERR_NUMERIC;
                break;
            }
            const char *row = (const char *)table + (size_t)p * (size_t)ld * esz;
            rc = xp_row_cells(row, dtype, V, temp, top_k, top_p, &w, cells, &info);
            if (rc != ORC_OK) break;
            const uint64_t r = st[0] >> 32;
            uint64_t tcell = st[1] / r;
            if (tcell > 0xFFFFFFFFull) tcell = 0xFFFFFFFFull;
            long tok = -1;
            for (j = 0; j < V; ++j) if (cells[j + 1] > tcell) { tok = j; break; }
            /* (cells[V] = 2^32 > tcell: a token is always found) */
            const uint64_t lo = cells[tok], hi = cells[tok + 1];
            if (trace_pos || trace_d_tok) {
                double pos = ((double)st[1] / (double)r) / XP_CELLS;
                double a = pos - (double)lo / XP_CELLS, b = (double)hi / XP_CELLS - pos;
                if (trace_pos) trace_pos[i * T + t] = pos;
                if (trace_d_tok) trace_d_tok[i * T + t] = a < b ? a : b;
            }
            st[1] -= r * lo;
            st[0] = hi == 0x100000000ull ? st[0] - r * lo : r * (hi - lo);
            while (st[0] <= XP_RANGE_LOW) {
                st[0] <<= 1;
                st[1] = (st[1] << 1) | xp_next_bit(st, (uint64_t)N);
            }
            seq[i * T + t] = (int32_t)tok;
            n = t + 1;
            p = tok;
            if (tok == eos) break;
        }
        if (len) len[i] = (int32_t)n;
        if (status) status[i] = rc;
    }
    free(cells);
    ws_free(&w);
    return ORC_OK;
}

int orc_version(void) { return 2; }

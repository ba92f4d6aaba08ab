/*
 * arith_sampling.h -- C ABI of the B200 (sm_100a) arithmetic-sampling decode library.
 *
 * Arithmetic sampling (Vilnis et al., arXiv 2210.15458) decodes a set of code
 * points in [0,1) against a sequence model: every code lane repeatedly takes
 * the model's next-token distribution, finds the token whose CDF interval
 * (vocabulary-index order) holds the code, and rescales the code into that
 * interval (Algorithm 1, "Sampling from a Code Point").  The code set is a
 * regular lattice with one shared uniform shift (Definition "Arithmetic
 * sampling", Sec. 4.2; Eq. 2).  Lanes never communicate (Remark after
 * Proposition 1).
 *
 * Conventions common to every call
 *   - All functions are extern "C", return an int status (AS_OK = 0, errors < 0)
 *     and never throw.  as_last_error() gives a text for the calling thread's
 *     last failure.
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller
 *     owns every buffer; unless a function's comment says otherwise, nothing is
 *     allocated and no buffer is kept after the call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Device-buffer calls only enqueue work on it and return; results are ready
 *     once the stream has reached that point.  Host-detectable errors return at
 *     once with nothing enqueued.
 *   - There is no CPU implementation behind these calls: without a usable CUDA
 *     device they return AS_ERR_CUDA.
 *   - Logits are row-major [rows, ld] with ld >= V elements between rows, dtype
 *     AS_F32 (IEEE binary32) or AS_BF16 (bfloat16 bit patterns).  The base
 *     pointer and the pitch need only be element-aligned: rows that start off a
 *     16-byte boundary are bulk-copied from the boundary below their start (the
 *     bytes in front lie in the same 16-byte granule and are masked), at nearly
 *     the speed of aligned rows.
 *   - Codes are fp64 in [0,1).  An input code of exactly 1.0 is read as the
 *     largest double below 1.  Rescaled codes are clamped to [0, 1 - 2^-53].
 *
 * Per-lane conditions found on the device never trap; they are reported through
 * the optional lane-status array: AS_OK, or AS_ERR_NUMERIC for a NaN or +inf
 * logit, a row with every logit -inf, or a code outside [0,1] / NaN.  Such a
 * lane gets token -1 and its code is returned unchanged.
 *
 * Readings of the paper fixed by this library (the paper is silent on them):
 * half-open intervals [F_{i-1}, F_i); modifiers applied as temperature, then
 * top-k, then softmax over the survivors, then nucleus on that renormalised
 * distribution, then renormalisation; ties in top-k / nucleus order go to the
 * lower token index; the nucleus is the smallest probability-sorted prefix with
 * mass >= top_p; -inf logits are masked out.
 */
#ifndef ARITH_SAMPLING_H_
#define ARITH_SAMPLING_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AS_F32 0
#define AS_BF16 1

#define AS_OK 0
#define AS_ERR_INVALID_ARG (-1)  /* NULL pointer, size or parameter out of range */
#define AS_ERR_UNSUPPORTED (-2)  /* valid request this build cannot serve (e.g. V too large) */
#define AS_ERR_CUDA (-3)         /* a CUDA runtime call failed (no device, launch error) */
#define AS_ERR_TIMEOUT (-4)      /* a bounded on-device wait ran out (reported per lane) */
#define AS_ERR_NUMERIC (-5)      /* per-lane: non-finite logits / empty row / bad code */

/* Largest vocabulary size accepted by as_step / as_decode_bigram* / as_encode_bigram. */
#define AS_MAX_V (1 << 20)

/*
 * Optional per-lane diagnostics of as_step; any member may be NULL.
 *   d_p_tok       [lanes] f64  probability of the chosen token under the modified distribution
 *   d_cdf_lo      [lanes] f64  F_{i-1}, the lower end of the chosen token's interval
 *   d_n_kept      [lanes] i32  number of tokens with non-zero probability after the cuts
 *   d_lane_status [lanes] i32  AS_OK or AS_ERR_NUMERIC / AS_ERR_TIMEOUT
 *   d_path        [lanes] i32  which routine decided the lane: AS_PATH_COMPACT (candidate
 *                              compaction from shared memory) or AS_PATH_GENERAL (full-row
 *                              fp64 routine; slower, serves every input)
 */
#define AS_PATH_COMPACT 0
#define AS_PATH_GENERAL 1
typedef struct as_step_diag {
    double *d_p_tok;
    double *d_cdf_lo;
    int32_t *d_n_kept;
    int32_t *d_lane_status;
    int32_t *d_path;
} as_step_diag;

/*
 * Shifted lattice of codes (Definition "Arithmetic sampling", Sec. 4.2; Eq. 2):
 *   d_codes[j] = (j + u) / N  (mod 1),  j = 0..N-1,
 * a lattice of spacing 1/N -- every gap on the circle, the wrap included, is
 * exactly 1/N -- moved by one shared shift; u is the caller's uniform draw.
 *   N        number of codes, >= 1
 *   u        shift in [0,1)
 *   d_codes  [N] f64 device, written
 * Errors: AS_ERR_INVALID_ARG for N < 1, u outside [0,1) or NaN, NULL d_codes.
 */
int as_lattice_codes(int N, double u, double *d_codes, void *stream);

/*
 * The code sets in the forms the paper itself prints (Sec. 4.2), next to the
 * evenly spaced one above:
 *   AS_LATTICE_SHIFTED           (j + b)/N mod 1, j = 0..N-1: as_lattice_codes
 *   AS_LATTICE_PAPER_DEFINITION  (i/(N+1) + b) mod 1, i = 1..N: Definition
 *                                "Arithmetic sampling" as printed (on the circle
 *                                its wrap gap is 2/(N+1), the others 1/(N+1))
 *   AS_LATTICE_NAIVE             i/(N+1), i = 1..N, no shift (b ignored): the
 *                                codebook of the proposition "Naive arithmetic
 *                                sampling" -- consistent but biased
 * d_codes[i-1] = c_i, [N] f64 device.  Feed the codes to as_step or
 * as_decode_bigram_codes.  Errors: AS_ERR_INVALID_ARG for an unknown variant,
 * N < 1, b outside [0,1) where it is used, NULL d_codes.
 */
#define AS_LATTICE_SHIFTED 0
#define AS_LATTICE_PAPER_DEFINITION 1
#define AS_LATTICE_NAIVE 2
int as_lattice_codes_variant(int N, double b, int variant, double *d_codes, void *stream);

/*
 * One decode step for every lane (the loop body of Algorithm 1, with the logit
 * modifiers named in Sec. 2 and "Top-k sampling", Sec. 5.1):
 *   x_j = logits[lane, j] / temp; optional top-k and nucleus cuts; p = softmax
 *   over the kept tokens; F = CDF of p in vocabulary-index order;
 *   token = the i with F_{i-1} <= c < F_i;  c' = (c - F_{i-1}) / p_i.
 *   d_logits     [lanes, ld] device, dtype AS_F32 or AS_BF16, read once
 *   lanes        >= 0 (0 is a no-op);  V in [1, AS_MAX_V];  ld >= V (elements)
 *   d_codes      [lanes] f64 device, the lanes' current codes
 *   temp         softmax temperature, > 0 and finite
 *   top_k        keep the k largest logits; <= 0 or >= V disables
 *   top_p        nucleus mass; <= 0 or >= 1 disables
 *   d_tokens     [lanes] i32 device, written
 *   d_codes_out  [lanes] f64 device, written; may be the same pointer as d_codes
 *   diag         NULL or a struct of optional device arrays (see as_step_diag)
 * Errors: AS_ERR_INVALID_ARG (NULL pointers, lanes < 0, V < 1, ld < V, temp not
 * positive/finite, NaN top_p, unknown dtype, misaligned element pointer),
 * AS_ERR_UNSUPPORTED (V > AS_MAX_V), AS_ERR_CUDA.
 */
int as_step(const void *d_logits, int dtype, int lanes, int V, long long ld,
            const double *d_codes, double temp, int top_k, double top_p,
            int32_t *d_tokens, double *d_codes_out, const as_step_diag *diag,
            void *stream);

/*
 * as_step with the locally typical cut in place of the nucleus (Sec. 2 names typical decoding
 * among the logit modifiers the method composes with; the rule is that of locally typical
 * sampling): after temperature and the optional top-k, with p the softmax over the survivors and
 * H its entropy, the tokens are ordered by |-ln p_j - H| ascending (lower index first among
 * equals) and the smallest prefix with mass >= typical_p is kept, then renormalised.
 *   typical_p  mass of the typical set; <= 0 or >= 1 disables (the call is then as_step
 *              without a nucleus).  Everything else as as_step.
 * Served by the general full-row routine (d_path reports AS_PATH_GENERAL).
 * Errors: as as_step, plus AS_ERR_INVALID_ARG for a NaN typical_p.
 */
int as_step_typical(const void *d_logits, int dtype, int lanes, int V, long long ld,
                    const double *d_codes, double temp, int top_k, double typical_p,
                    int32_t *d_tokens, double *d_codes_out, const as_step_diag *diag,
                    void *stream);

/*
 * The first step of a decode (Algorithm 1 entered with the codes of the
 * Definition "Arithmetic sampling", Sec. 4.2): as_step with lane i taking the
 * lattice code c = (j0 + i + u)/N mod 1 formed in the kernel -- bit-identical to
 * the value as_lattice_codes writes for index j0 + i -- so that the codes need
 * not be written out and read back.  j0 lets a caller that shards the N lanes
 * of one lattice over several devices give each its slice.
 *   N >= 1, u in [0,1), j0 >= 0, j0 + lanes <= N; everything else as as_step.
 * Errors: as as_step, plus AS_ERR_INVALID_ARG for N, u, j0 out of range.
 */
int as_step_lattice(const void *d_logits, int dtype, int lanes, int V, long long ld,
                    int N, double u, int j0, double temp, int top_k, double top_p,
                    int32_t *d_tokens, double *d_codes_out,
                    const as_step_diag *diag, void *stream);

/*
 * Same step with HOST buffers: copies logits and codes to the device, runs
 * as_step, copies tokens and codes back, and returns after the results are in
 * the host buffers (it synchronises `stream`).  Pinned host memory makes the
 * copies fast but is not required.
 *   h_logits [lanes, ld] host;  h_codes [lanes] host;  h_tokens, h_codes_out
 *   [lanes] host, written;  h_lane_status NULL or [lanes] host, written.
 *   d_work   device scratch of at least as_step_host_work_bytes(...) bytes,
 *            256-byte aligned, owned by the caller; contents undefined after.
 *            The rows are staged there at a pitch that is a multiple of 16
 *            bytes whatever ld is, so every row takes the fast kernel path.
 * Errors: as as_step, plus AS_ERR_INVALID_ARG if work_bytes is too small.
 */
int as_step_host(const void *h_logits, int dtype, int lanes, int V, long long ld,
                 const double *h_codes, double temp, int top_k, double top_p,
                 int32_t *h_tokens, double *h_codes_out, int32_t *h_lane_status,
                 void *d_work, size_t work_bytes, void *stream);
size_t as_step_host_work_bytes(int dtype, int lanes, long long ld);

/*
 * as_step_host without any allocation, for callers that cannot provide device memory.
 * (The paper has no counterpart to this call: it is a packaging of as_step_host.)
 *
 * Who needs it: code that is handed a stream but owns no device memory and may not ask for any --
 * a plug-in running inside a serving runtime that keeps the whole GPU in its own fixed pool, or a
 * call site where cudaMalloc's implicit device-wide synchronisation would stall other streams.
 * as_step_host needs a device work buffer (d_work) for the copied logits, codes and results; this
 * variant uses a buffer built into the library instead: AS_STATIC_WORK_BYTES of device memory that
 * every GPU which loads the library holds until the process exits.
 *
 * Arguments and results are those of as_step_host, minus d_work / work_bytes.  It calls no
 * cudaMalloc, cudaFree or other allocating routine.
 *   - A request whose as_step_host_work_bytes(dtype, lanes, ld) exceeds AS_STATIC_WORK_BYTES is
 *     refused with AS_ERR_UNSUPPORTED (as_last_error() names both sizes); nothing is enqueued.
 *   - The first call on each device looks up the buffer's device address (one-time set-up with
 *     that device current); make that first call before any stream capture.
 *   - All calls on a device share the one buffer.  Nothing in it has to start at zero: every byte
 *     the step reads is written by this call's own copies first, and every result the host
 *     receives is written by this call's kernel.  Two calls that overlap on the GPU (different
 *     streams, or two host threads) race on the buffer: serialise them.  The call returns after
 *     its results have reached the host buffers (it synchronises `stream`), so back-to-back calls
 *     from one thread are safe.
 */
#define AS_STATIC_WORK_BYTES (24u << 20)
int as_step_host_static(const void *h_logits, int dtype, int lanes, int V, long long ld,
                        const double *h_codes, double temp, int top_k, double top_p,
                        int32_t *h_tokens, double *h_codes_out, int32_t *h_lane_status,
                        void *stream);

/*
 * Full decode loop of Algorithm 1 (REPEAT ... UNTIL X = EOS) over a bigram
 * model: row table[prev] holds the next-token logits given the previous token.
 * The code set is the shifted lattice of as_lattice_codes, one copy per start
 * token: lane = s*N + j decodes code (j+u)/N starting from d_start[s] (the
 * start token is not part of the output).  Each lane runs up to T steps, stops
 * after emitting `eos` and pads the rest of its row with -1 (Sec. 3.3: EOS
 * terminates a sequence, padding makes lengths uniform).
 *   d_table   [V, ld] device (row index = previous token), read only
 *   d_start   [S] i32 device, each in [0, V);  S >= 0, N >= 1, u in [0,1)
 *   T         maximum number of steps, >= 0;  eos: token id, or < 0 for none
 *   temp, top_k, top_p   as in as_step, the same for every step
 *   d_seq         [S*N, T] i32 device, written (tokens, then -1 padding)
 *   d_len         [S*N] i32 device, written: tokens emitted (EOS included)
 *   d_codes_final NULL or [S*N] f64 device: each lane's code after its last step.
 *                 It doubles as the loop's state: with a top-k / nucleus cut and this
 *                 buffer given, the loop runs as one launch of the step kernel per
 *                 step, rows gathered from the table by the previous tokens (several
 *                 times faster than the single general kernel that runs otherwise)
 *   d_lane_status NULL or [S*N] i32 device: AS_OK, or the status that stopped the
 *                 lane early (a start/previous token outside [0,V) counts as
 *                 AS_ERR_NUMERIC)
 * Errors: AS_ERR_INVALID_ARG, AS_ERR_UNSUPPORTED, AS_ERR_CUDA as for as_step.
 */
int as_decode_bigram(const void *d_table, int dtype, int V, long long ld,
                     const int32_t *d_start, int S, int N, double u, int T, int eos,
                     double temp, int top_k, double top_p,
                     int32_t *d_seq, int32_t *d_len, double *d_codes_final,
                     int32_t *d_lane_status, void *stream);

/*
 * The same loop from caller-supplied per-lane state (Algorithm 1's inputs: a
 * code point and a prefix): lane i starts from previous token d_prev[i] and
 * code d_codes_in[i].  With iid uniform codes this is ordinary ancestral
 * sampling by inverse CDF (Sec. 3.1, last paragraph; Proposition 1); it also
 * serves to split a decode and resume it (T steps = T1 steps, then T - T1 from
 * the returned state).
 */
int as_decode_bigram_codes(const void *d_table, int dtype, int V, long long ld,
                           const int32_t *d_prev, const double *d_codes_in, int lanes,
                           int T, int eos, double temp, int top_k, double top_p,
                           int32_t *d_seq, int32_t *d_len, double *d_codes_final,
                           int32_t *d_lane_status, void *stream);

/*
 * Decoding with extended-precision codes.  Algorithm 1's update c <- (c - m)/(M - m) is real
 * arithmetic; in fp64 every step spends -log2 p_i of the code's 53 bits, so after a few dozen
 * tokens a lane is no longer steered by its lattice code and the properties of Sec. 4.3 / 4.4
 * hold for a prefix only.  A lattice code (j + u)/N is a rational number, though, whose binary
 * digits never run out: these two calls carry it as the state of an arithmetic decoder.
 *
 * Lane state: four 64-bit words [range, code, q, packed] -- the current interval has `range`
 * units, in (2^62, 2^63]; `code` < range is the code's offset inside it; q and packed hold the
 * source of the code's further digits (the unread part of its first 53 bits, their number in
 * the upper half of packed, and in the lower half the remainder of the long division by N that
 * yields every later digit).  Each step cuts the interval into 2^32 cells of range >> 32 units;
 * with P_j the prefix sums (vocabulary-index order) of the kept tokens' masses under the same
 * temperature / top-k / nucleus treatment as as_step and F(P) = floor(P * 2^32 / Z), token j owns
 * the cells [F(P_j), F(P_{j+1})), the last token with mass ending at 2^32; the token whose cells
 * hold the code is emitted, the interval becomes that token's, and digits are shifted in until
 * range > 2^62 again.  All of it is integer arithmetic on cell boundaries that depend on the row
 * alone: the sequences of a lattice are exactly those whose intervals in this subdivision hold
 * the codes, at any length.  A token of probability below 2^-32 may own no cell.
 *
 * as_xp_lattice_state writes the state of the codes (j + u')/N, j = j0 .. j0+count-1, with
 * u' = floor(u 2^53) / 2^53 (the shift read to 53 fractional bits), S times over:
 *   d_state [S*count, 4] u64 device, lane = s*count + (j - j0)
 * Errors: AS_ERR_INVALID_ARG (N < 1, u outside [0,1), j0 / count outside [0, N], S < 0, NULL).
 *
 * as_decode_bigram_xp runs Algorithm 1's loop (as as_decode_bigram_codes) from d_prev[lanes] and
 * d_state[lanes, 4], which it updates in place, so that a decode can be split and resumed.
 *   N   the lattice size the states were made for (it drives the digit source)
 *   d_lane_status NULL or [lanes]: AS_OK, or AS_ERR_NUMERIC (unusable row, previous token
 *       outside [0, V), state outside its domain); the lane stops there
 * Errors: as as_decode_bigram_codes.
 */
int as_xp_lattice_state(int N, double u, int j0, int count, int S, uint64_t *d_state, void *stream);
int as_decode_bigram_xp(const void *d_table, int dtype, int V, long long ld, const int32_t *d_prev,
                        uint64_t *d_state, int lanes, int N, int T, int eos, double temp, int top_k,
                        double top_p, int32_t *d_seq, int32_t *d_len, int32_t *d_lane_status,
                        void *stream);

/*
 * Sequence -> interval, the codebook of Sec. 4.1 read in the other direction:
 * in dictionary order every sequence owns the interval [lo, lo + P(sequence)),
 * and a code decodes to that sequence exactly when it falls inside.  For lane i
 * with tokens d_seq[i, 0..len-1] continued from d_prev[i] under the bigram
 * table of as_decode_bigram:
 *   lo    = sum_t ( prod_{s<t} p_s ) * F_t   (F_t: mass below token t in
 *           vocabulary-index order under that step's modified distribution)
 *   width = prod_t p_t
 * with the same temperature / top-k / nucleus treatment as as_step.
 *   d_prev  [lanes] i32 device   previous token of each lane, in [0, V)
 *   d_seq   [lanes, T] i32 device, read only;  d_len [lanes] i32 device: tokens
 *           to take from each row (values above T are read as T; padding is ignored)
 *   d_lo, d_width  [lanes] f64 device, written
 *   d_lane_status  NULL or [lanes] i32 device: AS_OK; AS_ERR_NUMERIC if a token
 *           has probability zero under its step's distribution (cut by top-k /
 *           nucleus, or masked) or the row is not usable; AS_ERR_INVALID_ARG if a
 *           token id lies outside [0, V).  lo and width then hold the interval of
 *           the prefix before the failing token.
 * Errors: AS_ERR_INVALID_ARG, AS_ERR_UNSUPPORTED, AS_ERR_CUDA as for as_step.
 */
int as_encode_bigram(const void *d_table, int dtype, int V, long long ld,
                     const int32_t *d_prev, const int32_t *d_seq, const int32_t *d_len,
                     int lanes, int T, double temp, int top_k, double top_p,
                     double *d_lo, double *d_width, int32_t *d_lane_status, void *stream);

/*
 * n-gram diversity score of a set of sequences (Sec. 5.1, "Diverse beam
 * generation"): d = sum_{n=1..4} d_n with
 *   d_n = (number of distinct n-grams) / (number of n-grams) in the N sequences
 * of a group.  Lanes g*N .. g*N+N-1 of d_seq form group g (the layout that
 * as_decode_bigram writes for start token g).  An n-gram is n consecutive
 * emitted tokens of one sequence; padding belongs to none.  A d_n whose
 * denominator is zero contributes 0.
 *   d_seq  [S*N, T] i32 device, read only;  d_len [S*N] i32 device (clamped to [0, T])
 *   d_unique, d_total  [S, 4] i64 device, written: the counts for n = 1..4
 *   d_div  [S] f64 device, written: d
 * One group must fit shared memory: N * T <= AS_NGRAM_MAX_ITEMS, else
 * AS_ERR_UNSUPPORTED.  Other errors: AS_ERR_INVALID_ARG (NULL pointer, S < 0,
 * N < 1, T < 0), AS_ERR_CUDA.
 */
#define AS_NGRAM_MAX_ITEMS 16384
int as_ngram_diversity(const int32_t *d_seq, const int32_t *d_len, int S, int N, int T,
                       int64_t *d_unique, int64_t *d_total, double *d_div, void *stream);

/*
 * Sample-mean estimator of Sec. 4.2 (the proposition that (1/N) sum_i s(x_i)
 * over the sequences of one shifted lattice is unbiased and consistent; used
 * for the variance comparison of Sec. 5.2) for an additive reward
 *   s(x) = sum_{t < len} d_r[x_t]:
 *   d_lane_reward[lane] = s(x_lane)            (NULL to skip)
 *   d_mean[g] = (1/N) sum of s over lanes g*N .. g*N+N-1
 *   d_r  [V] f64 device;  d_seq, d_len as for as_ngram_diversity
 *   d_group_status  NULL or [S] i32 device: AS_OK, or AS_ERR_INVALID_ARG if a
 *                   token of the group lies outside [0, V) (it then adds nothing)
 * Errors: AS_ERR_INVALID_ARG (NULL pointer, S < 0, N outside [1, AS_REWARD_MAX_N],
 * T < 0, V < 1), AS_ERR_CUDA.
 */
#define AS_REWARD_MAX_N 4096
int as_reward_mean(const int32_t *d_seq, const int32_t *d_len, int S, int N, int T,
                   const double *d_r, int V, double *d_lane_reward, double *d_mean,
                   int32_t *d_group_status, void *stream);

/*
 * Launch-shape overrides for measurement sweeps and tests (0 restores the built-in
 * choice).  Keys:
 *   AS_TUNE_STEP_PATH     0 = streaming kernel (one CTA per lane), 1 = general kernel only,
 *                         2 = cluster kernel (row split over the CTAs of a cluster)
 *   AS_TUNE_CLUSTER       CTAs per lane for the cluster kernel (1, 2, 4, 8)
 *   AS_TUNE_CTAS_PER_SM   resident CTAs per SM the grid is sized for
 *   AS_TUNE_STAGES        16 KB ring stages of the streaming kernel (2..12); rows longer than
 *                         the ring stream through it, so a small value also makes rows stream
 *                         that would otherwise stay resident
 *   AS_TUNE_MIN_CTAS      streaming kernel build for bf16 rows that do not fit the ring:
 *                         3 = three CTAs per SM (1024-entry hit list, <= 72 registers; default),
 *                         2 = two CTAs per SM (2048-entry hit list)
 *   AS_TUNE_SERIAL_LAUNCH 1 = launch the streaming kernel as an ordinary stream-ordered kernel.
 *                         By default it is launched so that its CTAs may be set up while the
 *                         kernel before it on the stream drains (programmatic dependent launch;
 *                         it still waits for that kernel's completion before it reads or
 *                         writes global memory, so results do not depend on this key)
 *   AS_TUNE_WAIT_KCYCLES  bound on every on-device wait for a copy, in units of 1000 clock
 *                         cycles (default: 2,000,000 = about one second).  A wait that runs out
 *                         ends the lane with status AS_ERR_TIMEOUT (token -1, code unchanged);
 *                         the kernel returns normally and later calls are not affected
 *   AS_TUNE_DEBUG_NO_COPY 1 = the copy-issuing thread of the step kernels issues nothing, so
 *                         every wait runs out: exists only so that a test can exercise the
 *                         AS_ERR_TIMEOUT path without any copy in flight; use it with a small
 *                         AS_TUNE_WAIT_KCYCLES
 *   AS_TUNE_RADIX_NUCLEUS 1 = the general routine of the step calls finds every nucleus by its
 *                         radix select on mass-weighted keys.  By default a nucleus without a
 *                         top-k is first looked for through bins of the logit value (two passes
 *                         over the row for a nucleus of any width), and the radix select takes
 *                         the rows that the bins cannot settle; the results are the same
 * Returns AS_ERR_INVALID_ARG for an unknown key or value.  The keys are process-wide; a launch
 * reads each once (concurrent calls see the old or the new value).
 */
#define AS_TUNE_STEP_PATH 1
#define AS_TUNE_CLUSTER 2
#define AS_TUNE_CTAS_PER_SM 3
#define AS_TUNE_STAGES 4
#define AS_TUNE_MIN_CTAS 5
#define AS_TUNE_SERIAL_LAUNCH 6
#define AS_TUNE_WAIT_KCYCLES 7
#define AS_TUNE_DEBUG_NO_COPY 8
#define AS_TUNE_RADIX_NUCLEUS 9
int as_tune(int key, int value);

/* Text of the calling thread's most recent error ("" if none). Never NULL. */
const char *as_last_error(void);

/* Library version: major * 1000 + minor. */
int as_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ARITH_SAMPLING_H_ */

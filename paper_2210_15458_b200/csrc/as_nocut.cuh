// Lanes without a top-k / nucleus cut (temperature only: Algorithm 1 as the paper states it,
// and the setting of its main experiments, Sec. 5.1): every token is kept, so the whole row
// contributes to Z and to the prefix sums, and all of it has to be summed to fp64 accuracy --
// c' = (c Z - S_{i-1}) / e_i magnifies an error of the prefix by up to 1e5 on lanes that are
// compared at 1e-6.
//
// One CTA holds up to three independent groups of 256 threads.  A group owns one lane at a
// time and a row buffer in shared memory that thread 0 of the group fills with bulk async
// copies (16 KB pieces, one mbarrier each); while one group waits for its row the others
// compute, which is what keeps HBM busy in the decode loop, where a lane's next row is known
// only after its current step.  Per row:
//   sum pass   chunks of 32 consecutive 16-byte vectors, one warp per chunk: per-chunk mass
//              sums in vocabulary-index order (the CDF w of Algorithm 1 at chunk granularity);
//   locate     warp 0 scans the chunk sums (Z = the total), finds the chunk whose interval
//              holds c Z, re-evaluates that chunk element by element, picks the token and
//              rescales the code (Algorithm 1: (m, M), c <- (c - m)/(M - m)).
// Masses.  bf16 logits take only 65536 values, and e_j = exp(l_j / temp) depends on nothing
// else: a shared-memory table over the magnitudes [2^-8, 2^6) of both signs (4096 slots,
// 3584 in use, filled once per CTA with the fp64 exponential) turns every mass into one 8-byte load and
// one fp64 add instead of a 13-operation fp64 exponential.  The masses are not divided by
// exp(max / temp): token choice and rescaled code do not depend on a common factor, and with
// temp >= 0.1 the table's range stays far inside fp64.  Elements outside the table: tiny
// magnitudes (and zeros) are evaluated directly, -inf counts as masked, NaN / +inf fail the
// lane, and a finite magnitude >= 64 sends the row once more through the direct evaluation
// relative to the row maximum (`robust`: the same passes with the fp64 exponential), which
// is also what fp32 rows and temperatures below 0.1 always take.
#pragma once
#include "as_staged.cuh"

namespace asx {

constexpr int NC_GT = 256;                        // threads per group
constexpr int NC_GW = NC_GT / 32;
constexpr int NC_MAXG = 3;                        // groups per CTA
constexpr int NC_PIECE_BYTES = 16384;
constexpr int NC_MAXPIECE = 6;
constexpr int NC_MAXROW = NC_MAXPIECE * NC_PIECE_BYTES;        // rows up to 96 KB
constexpr int NC_R = 4;                           // chunks a warp takes together in the sum pass
constexpr int NC_MAXCH = NC_MAXROW / 16 / 32;                  // 192 chunks of 32 vectors
constexpr int NC_EXP_LO = 119;                    // biased exponent of 2^-8
constexpr int NC_BINADES = 14;                    // [2^-8, 2^6)
constexpr int NC_ENT = NC_BINADES * 128;          // table entries per sign
constexpr uint32_t NC_MAG_LO = (uint32_t)NC_EXP_LO << 7;
constexpr int NC_TBL_DOUBLES = 4096;              // sign (1) | low four exponent bits | mantissa (7)
constexpr double NC_MIN_TEMP = 0.1;               // below: exp(64 / temp) leaves fp64's comfortable range

constexpr int NC_STEP = 0, NC_DECODE = 1, NC_ENCODE = 2, NC_DECODE_XP = 3;
constexpr int NCF_BAD = 1, NCF_BIG = 2;

struct NocutArgs {
    const void* data;          // logits [lanes, ld] (step) or table [V, ld] (decode / encode)
    long long ld;
    int V;
    int lanes;
    double inv_tau;
    int use_table;             // bf16 and temp >= NC_MIN_TEMP
    // step
    const double* codes;
    int lat_N, lat_j0;
    double lat_u;
    int* tokens;
    double* codes_out;
    DiagOut diag;
    // decode: lane state from (tok_in[ln / N], N, u) when codes_in is null, else (tok_in[ln], codes_in[ln])
    const int* tok_in;
    const double* codes_in;
    int N;
    double u;
    int T, eos;
    int* seq;
    int* len;
    double* codes_final;
    int* lane_status;
    // encode
    const int* seq_in;
    const int* len_in;
    double* lo_out;
    double* width_out;
    // decode with extended-precision codes: lane state [lanes, 4], read and written back
    unsigned long long* xp_state;
    long long wait_cycles;
    int debug_no_copy;
};

struct NcGroupSmem {
    unsigned long long full[NC_MAXPIECE];
    double chunk_sum[NC_MAXCH + 1];
    unsigned red_u[NC_GW];
    unsigned red_u2[NC_GW];
    int flags;
    int masked;          // table mode: -inf elements (padding included); robust mode: finite elements
    int poisoned;
    unsigned has[6];             // bit c: chunk c holds mass (not to be read off the scanned sums, whose
                                 // lane totals are added in another order than the sums inside a lane)
    LaneResult res;
    unsigned long long xp_lo, xp_hi;     // extended-precision steps: the chosen token's cells [xp_lo, xp_hi)
};

// shared memory in front of the row buffers: mass table, 2^(j/64) table, the groups' control blocks
__host__ __device__ constexpr size_t nc_fixed_bytes() {
    return ((NC_TBL_DOUBLES + 64) * sizeof(double) + NC_MAXG * sizeof(NcGroupSmem) + 127) & ~(size_t)127;
}

template <int G>
__device__ __forceinline__ void nc_bar(int gi) {
    asm volatile("bar.sync %0, %1;" ::"r"(gi + 1), "n"(G) : "memory");
}

// One row for one group.  `rowv` is the group's buffer; the ragged end of a row (< 16 bytes)
// is not part of the bulk copies: the thread that owns the last vector reads it from `grow`.
template <int DT>
struct NcRow {
    using Tr = Traits<DT>;
    using P = Pass<DT>;
    static constexpr int E = Tr::E;

    NcGroupSmem& g;
    const double* tbl;         // mass table (bf16) or nullptr
    const double* exp_tbl;     // 2^(j/64)
    const uint4* rowv;
    const char* grow;          // the row in global memory
    int V, nvec, bulk_vec, nch, npiece;
    int gi, gtid, lane, warp;
    double inv_tau;
    double s64, c64;           // robust mode: t = x * s64 + c64 in units of 1/64 of a bit
    uint32_t parity;
    long long wait_cycles;

    __device__ __forceinline__ void wait_piece(int p) {
        if (*(volatile int*)&g.poisoned) return;
        if (!mbar_wait_bounded(smem_u32(&g.full[p]), parity, wait_cycles)) *(volatile int*)&g.poisoned = 1;
    }

    __device__ __forceinline__ static uint4 ninf_vec() {
        const uint32_t w = DT == DT_BF16 ? 0xFF80FF80u : 0xFF800000u;
        return make_uint4(w, w, w, w);
    }
    __device__ __forceinline__ static uint4 ones_vec() {           // the value 1.0 in every element
        const uint32_t w = DT == DT_BF16 ? 0x3F803F80u : 0x3F800000u;
        return make_uint4(w, w, w, w);
    }
    // vector v of the row; elements at or past V read as -inf
    __device__ __forceinline__ uint4 load_vec(int v) const {
        if (v < bulk_vec) return rowv[ASX_AT(v, NC_MAXROW / 16, 70)];
        uint32_t w[4];
        const int base = v * E;
        if (DT == DT_BF16) {
            const unsigned short* src = reinterpret_cast<const unsigned short*>(grow);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t lo = base + 2 * i < V ? src[base + 2 * i] : 0xFF80u;
                const uint32_t hi = base + 2 * i + 1 < V ? src[base + 2 * i + 1] : 0xFF80u;
                w[i] = lo | (hi << 16);
            }
        } else {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(grow);
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = base + i < V ? src[base + i] : 0xFF800000u;
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }

    // ---- masses of one vector, table mode (bf16).  Table entry of a bf16 pattern h = s|eeeeeeee|mmmmmmm
    //      with exponent field in [119, 133): index s<<11 | (e & 15)<<7 | m -- the low four exponent
    //      bits are distinct over those 14 binades, so the byte offset is two shifts and two masks
    //      of the pattern itself.  A vector with any element outside the table goes, element by
    //      element, through `slow1` (rare on real rows; kept out of line).
    __device__ __forceinline__ static uint32_t tbl_off(uint32_t w, bool high) {
        return high ? (((w >> 13) & 0x3FF8u) | ((w >> 17) & 0x4000u)) : (((w << 3) & 0x3FF8u) | ((w >> 1) & 0x4000u));
    }
    // one element outside the fast path (free of `this`, so that the row's state stays in registers):
    // its mass, or -1 for -inf (a masked token), -2 for NaN / +inf, -3 for a finite magnitude >= 64
    __device__ __noinline__ static double slow1(uint32_t b, const double* tbl_, const double* exp_tbl_, double inv_tau_) {
        const uint32_t mag = b & 0x7FFFu;
        if (mag >= 0x7F80u) return b == 0xFF80u ? -1.0 : -2.0;
        if (mag >= NC_MAG_LO + NC_ENT) return -3.0;
        if (mag >= NC_MAG_LO) return *reinterpret_cast<const double*>(reinterpret_cast<const char*>(tbl_) + tbl_off(b, false));
        return exp_core((double)__uint_as_float(b << 16) * inv_tau_, exp_tbl_);   // |x| < 2^-8 (zeros, subnormals)
    }
    __device__ __forceinline__ void masses_tbl(const uint4& q, double (&e)[8], int& flags, int& masked) const {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        // every magnitude in [NC_MAG_LO, NC_MAG_LO + NC_ENT)?  Packed per 16-bit half: t = |h| - NC_MAG_LO
        // must stay below NC_ENT = 0x700, i.e. neither t nor t + 0x100 may reach bit 11.  (A borrow out
        // of the low half only occurs when that half is already out of range.)
        uint32_t bad = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t t = (w[i] & 0x7FFF7FFFu) - (NC_MAG_LO | (NC_MAG_LO << 16));
            bad |= t | (t + 0x01000100u);
        }
        if (bad & 0xF800F800u) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                double v = slow1((k & 1) ? (w[k >> 1] >> 16) : (w[k >> 1] & 0xFFFFu), tbl, exp_tbl, inv_tau);
                if (v < 0.0) {
                    masked += (v == -1.0);
                    flags |= v == -2.0 ? NCF_BAD : v == -3.0 ? NCF_BIG : 0;
                    v = 0.0;
                }
                e[k] = v;
            }
            return;
        }
        const char* tb = reinterpret_cast<const char*>(tbl);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            e[2 * i] = *reinterpret_cast<const double*>(tb + ASX_AT(tbl_off(w[i], false), NC_TBL_DOUBLES * 8, 71));
            e[2 * i + 1] = *reinterpret_cast<const double*>(tb + ASX_AT(tbl_off(w[i], true), NC_TBL_DOUBLES * 8, 71));
        }
    }
    // ---- robust mode: fp64 exponential relative to the row maximum; counts the finite elements
    __device__ __forceinline__ void masses_dir(const uint4& q, double (&e)[E], int& nfin) const {
        float x[E];
        P::floats(q, x);
#pragma unroll
        for (int k = 0; k < E; ++k) {
            e[k] = exp2_64th(fma((double)x[k], s64, c64), exp_tbl);
            nfin += (x[k] > __uint_as_float(0xFF800000u));
        }
    }
    template <bool TBL>
    __device__ __forceinline__ void masses(const uint4& q, double (&e)[E], int& flags, int& count) const {
        if constexpr (TBL && DT == DT_BF16) masses_tbl(q, e, flags, count);
        else masses_dir(q, e, count);
    }

    __device__ __forceinline__ bool chunk_has(int c) const { return (g.has[c >> 5] >> (c & 31)) & 1u; }

    // ---- per-chunk sums in index order (a chunk = 32 consecutive vectors, one per lane).
    //      g.flags / g.masked / g.has must be zero on entry (group-wide).  A warp takes NC_R
    //      consecutive chunks at once: their table loads are in flight together and their
    //      reductions interleave (a lone reduction is a chain of five dependent shuffle-add rounds).
    template <bool TBL>
    __device__ void sum_pass() {
        int flags = 0, count = 0, cur = -1;
        const int nsuper = (nch + NC_R - 1) / NC_R;
        for (int sc = warp; sc < nsuper; sc += NC_GW) {
            const int piece = (sc * NC_R * 512) / NC_PIECE_BYTES;
            if (piece != cur && piece < npiece) { wait_piece(piece); cur = piece; }
            // (no branches in here: the four vectors' index arithmetic and table loads interleave.  A
            //  vector past the row is replaced by a harmless in-table pattern and its sum dropped;
            //  inside the row's last chunk it counts as masked padding)
            uint4 q[NC_R];
            bool valid[NC_R];
#pragma unroll
            for (int r = 0; r < NC_R; ++r) {
                const int v = (sc * NC_R + r) * 32 + lane;
                valid[r] = v < nvec;
                q[r] = valid[r] ? load_vec(v) : ((TBL && DT == DT_BF16) ? ones_vec() : ninf_vec());
                count += (!valid[r] && sc * NC_R + r < nch) ? (TBL && DT == DT_BF16 ? E : 0) : 0;
            }
            double s[NC_R];
#pragma unroll
            for (int r = 0; r < NC_R; ++r) {
                double e[E];
                masses<TBL>(q[r], e, flags, count);
                double t;
                if constexpr (E == 8) t = ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
                else t = (e[0] + e[1]) + (e[2] + e[3]);
                s[r] = valid[r] ? t : 0.0;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
                for (int r = 0; r < NC_R; ++r) s[r] += __shfl_xor_sync(FULL, s[r], o);
            }
            if (lane < NC_R) {
                double mine = s[0];
#pragma unroll
                for (int r = 1; r < NC_R; ++r) mine = lane == r ? s[r] : mine;
                const int c = sc * NC_R + lane;
                if (c < nch) {
                    g.chunk_sum[ASX_AT(c, NC_MAXCH + 1, 72)] = mine;
                    if (mine > 0.0) atomicOr(&g.has[c >> 5], 1u << (c & 31));
                }
            }
        }
        flags = __reduce_or_sync(FULL, flags);
        count = __reduce_add_sync(FULL, count);
        if (lane == 0) {
            if (flags) atomicOr(&g.flags, flags);
            if (count) atomicAdd(&g.masked, count);
        }
    }

    // ---- row maximum for the robust mode (NaN and +inf propagate into it).  Ends with a barrier.
    __device__ uint32_t max_pass() {
        for (int p = 0; p < npiece; ++p) wait_piece(p);
        typename P::Acc acc = P::init();
        for (int v = gtid; v < nvec; v += NC_GT) P::merge(acc, P::reduce(load_vec(v)));
        uint32_t k0, k1;
        P::keys(acc, k0, k1);
        const uint32_t km = warp_max_u(max(k0, k1));
        if (lane == 0) g.red_u[warp] = km;
        nc_bar<NC_GT>(gi);
        uint32_t kmax = 0;
#pragma unroll
        for (int w = 0; w < NC_GW; ++w) kmax = max(kmax, g.red_u[w]);
        nc_bar<NC_GT>(gi);
        return kmax;
    }

    // ---- warp 0: scan of the chunk sums in place (exclusive; [nch] = Z, continuing the same
    //      running sum so that sum[c+1] > sum[c] exactly when chunk c added something)
    __device__ void scan_chunks() {
        const int per = (nch + 31) / 32;
        const int b = min(lane * per, nch), en = min(b + per, nch);
        double s = 0.0;
        for (int i = b; i < en; ++i) s += g.chunk_sum[i];
        const double incl = warp_incl_scan_d(s, lane);
        double run = __shfl_up_sync(FULL, incl, 1);
        if (lane == 0) run = 0.0;
        for (int i = b; i < en; ++i) {
            const double v = g.chunk_sum[i];
            g.chunk_sum[i] = run;
            run += v;
        }
        if (en == nch && b < nch) g.chunk_sum[nch] = run;
        __syncwarp();
    }

    // masses of this lane's vector of chunk c (zeros past the row); returns its first token index
    template <bool TBL>
    __device__ __forceinline__ int chunk_masses(int c, double (&ev)[E]) const {
        const int v = c * 32 + lane;
        int f = 0, cnt = 0;
        masses<TBL>(v < nvec ? load_vec(v) : ninf_vec(), ev, f, cnt);
        return v * E;
    }
    // three quotients on three lanes (an fp64 division is a long dependent chain): lane 0 returns
    // n0 / d0, and q1 = n1 / d1, q2 = n2 / d1 come back to it through shuffles
    __device__ __forceinline__ double div3(double n0, double d0, double n1, double n2, double d1, double& q1, double& q2) const {
        const double num = lane == 0 ? n0 : lane == 1 ? n1 : n2;
        const double den = lane == 0 ? d0 : d1;
        const double quo = num / den;
        q1 = __shfl_sync(FULL, quo, 1);
        q2 = __shfl_sync(FULL, quo, 2);
        return quo;
    }

    // ---- warp 0: the token whose interval holds c * Z, and the rescaled code
    template <bool TBL>
    __device__ void locate(double c, double c_in, int n_kept) {
        scan_chunks();
        const double Z = g.chunk_sum[nch];
        const double t = c * Z;
        int first = INT_MAX, last_c = -1;
        for (int ci = lane; ci < nch; ci += 32) {
            if (chunk_has(ci)) {
                last_c = ci;
                if (t < g.chunk_sum[ci + 1]) first = min(first, ci);
            }
        }
        first = (int)warp_min_u((unsigned)first);
        last_c = (int)warp_max_u((unsigned)(last_c + 1)) - 1;
        const bool force_last = first == INT_MAX;
        const int cstar = force_last ? last_c : first;
        int tok = -1;
        double tok_S = 0.0, tok_e = 1.0;
        if (cstar >= 0) {
            const double run = g.chunk_sum[ASX_AT(cstar, NC_MAXCH + 1, 73)];
            double ev[E];
            const int base = chunk_masses<TBL>(cstar, ev);
            double local = 0.0;
#pragma unroll
            for (int k = 0; k < E; ++k) local += ev[k];
            const double incl = warp_incl_scan_d(local, lane);
            double excl = __shfl_up_sync(FULL, incl, 1);
            if (lane == 0) excl = 0.0;
            int pick = -1, last_idx = -1;
            double pick_S = 0.0, pick_e = 1.0, last_S = 0.0, last_e = 1.0;
            double S = run + excl;
#pragma unroll
            for (int k = 0; k < E; ++k) {
                if (ev[k] > 0.0) {
                    if (pick < 0 && t < S + ev[k]) { pick = base + k; pick_S = S; pick_e = ev[k]; }
                    last_idx = base + k; last_S = S; last_e = ev[k];
                    S += ev[k];
                }
            }
            const bool cross = !force_last && local > 0.0 && (t < run + incl);
            const unsigned bal = __ballot_sync(FULL, cross);
            if (bal) {
                const int L = __ffs(bal) - 1;
                if (pick < 0) { pick = last_idx; pick_S = last_S; pick_e = last_e; }
                tok = __shfl_sync(FULL, pick, L);
                tok_S = __shfl_sync(FULL, pick_S, L);
                tok_e = __shfl_sync(FULL, pick_e, L);
            } else {   // rounding at the top end: the last token with mass in the chunk
                const unsigned best = warp_max_u((unsigned)(last_idx + 1));
                const unsigned bal2 = __ballot_sync(FULL, (unsigned)(last_idx + 1) == best);
                const int L = __ffs(bal2) - 1;
                tok = __shfl_sync(FULL, last_idx, L);
                tok_S = __shfl_sync(FULL, last_S, L);
                tok_e = __shfl_sync(FULL, last_e, L);
            }
        }
        double p_tok, cdf_lo;
        double cn = div3(t - tok_S, tok_e, tok_e, tok_S, Z, p_tok, cdf_lo);
        if (lane == 0) {
            if (!(cn >= 0.0)) cn = 0.0;
            if (cn > ASX_ONE_BELOW) cn = ASX_ONE_BELOW;
            LaneResult r;
            r.token = tok; r.status = tok < 0 ? ST_NUMERIC : ST_OK; r.n_kept = n_kept;
            r.code_out = tok < 0 ? c_in : cn;
            r.p_tok = p_tok;
            r.cdf_lo = cdf_lo;
            g.res = r;
        }
    }

    // ---- warp 0: the token that owns the cell `tcell` of the 2^32 cells of this step's CDF
    //      (extended-precision codes); the token's cells go to g.xp_lo / g.xp_hi
    template <bool TBL>
    __device__ void locate_xp(unsigned long long tcell, int n_kept) {
        scan_chunks();
        const double Z = g.chunk_sum[nch];
        const double K = 4294967296.0 / Z;
        int last_c = -1;
        for (int ci = lane; ci < nch; ci += 32)
            if (chunk_has(ci)) last_c = ci;
        last_c = (int)warp_max_u((unsigned)(last_c + 1)) - 1;
        int tok = -1;
        unsigned long long plo = 0, phi = 0;
        double pe = 1.0;
        if (last_c >= 0) {
            // the first chunk with mass whose end cell lies beyond the code's cell, and the chunk
            // with mass before it: a chunk starts in the cell where that one ended
            int first = INT_MAX;
            for (int ci = lane; ci <= last_c; ci += 32) {
                const unsigned long long fe = ci == last_c ? XP_TOP : xp_cell(g.chunk_sum[ci + 1], K);
                if (fe > tcell && chunk_has(ci)) first = min(first, ci);
            }
            const int cstar = (int)warp_min_u((unsigned)first);
            int prev_c = -1;
            for (int ci = lane; ci < cstar; ci += 32)
                if (chunk_has(ci)) prev_c = ci;
            prev_c = (int)warp_max_u((unsigned)(prev_c + 1)) - 1;
            const unsigned long long Fend = cstar == last_c ? XP_TOP : xp_cell(g.chunk_sum[cstar + 1], K);
            double run = g.chunk_sum[cstar];
            unsigned long long carry = prev_c < 0 ? 0ull : xp_cell(g.chunk_sum[prev_c + 1], K);
            double ev[E];
            const int base = chunk_masses<TBL>(cstar, ev);
            int pk = 0;
            const int L = xp_subrow<E>(ev, lane, K, tcell, true, Fend, run, carry, pk, plo, phi, pe);
            if (L >= 0) tok = __shfl_sync(FULL, base, L) + pk;
        }
        if (lane == 0) {
            LaneResult r;
            r.token = tok; r.status = tok < 0 ? ST_NUMERIC : ST_OK; r.n_kept = n_kept;
            r.code_out = 0.0;
            r.p_tok = pe / Z;
            r.cdf_lo = (double)plo * (1.0 / 4294967296.0);
            g.xp_lo = plo; g.xp_hi = phi;
            g.res = r;
        }
    }

    // ---- warp 0: interval of a given token (the other direction, Sec. 4.1)
    template <bool TBL>
    __device__ void interval(int tok, int n_kept) {
        scan_chunks();
        const double Z = g.chunk_sum[nch];
        const int cstar = (tok / E) >> 5;
        double ev[E];
        const int base = chunk_masses<TBL>(cstar, ev);
        double below = 0.0, e_tok = 0.0;
#pragma unroll
        for (int k = 0; k < E; ++k) {
            if (base + k < tok) below += ev[k];
            if (base + k == tok) e_tok = ev[k];
        }
        below = warp_sum_d(below);
        e_tok = warp_sum_d(e_tok);                 // one lane holds it, the others add zero
        double p_tok, unused;
        const double cdf_lo = div3(g.chunk_sum[ASX_AT(cstar, NC_MAXCH + 1, 74)] + below, Z, e_tok, 0.0, Z, p_tok, unused);
        if (lane == 0) {
            // kept = not masked (a finite logit whose mass underflows still has its empty interval)
            bool kept;
            if (DT == DT_BF16) kept = reinterpret_cast<const unsigned short*>(grow)[tok] != 0xFF80u;
            else kept = reinterpret_cast<const uint32_t*>(grow)[tok] != 0xFF800000u;
            LaneResult r;
            r.token = kept ? tok : -1; r.status = kept ? ST_OK : ST_NUMERIC; r.n_kept = n_kept;
            r.code_out = 0.0;
            r.p_tok = p_tok;
            r.cdf_lo = cdf_lo;
            g.res = r;
        }
    }

    // One decode step (tok_given < 0) or one interval (tok_given >= 0) on the row in the buffer.
    // All threads of the group call it; the result is returned to all of them.
    // xp: the code's cell comes from an extended-precision state instead of c_in.
    __device__ LaneResult run(double c_in, int tok_given, bool use_table, bool xp = false, unsigned long long tcell = 0) {
        double c = c_in;
        if (c == 1.0) c = ASX_ONE_BELOW;
        bool robust = !(use_table && DT == DT_BF16);
        bool failed = false;
        if (!robust) {
            sum_pass<true>();
            nc_bar<NC_GT>(gi);
            const int flags = g.flags;
            if (flags & NCF_BAD) failed = true;
            else if (flags & NCF_BIG) robust = true;
            if (!failed && !robust && warp == 0 && !g.poisoned) {
                const int n_kept = nch * 32 * E - g.masked;       // (padding counts as masked)
                if (n_kept <= 0) { if (lane == 0) g.res = failed_lane(c_in, ST_NUMERIC); }
                else if (xp) locate_xp<true>(tcell, n_kept);
                else if (tok_given < 0) locate<true>(c, c_in, n_kept);
                else interval<true>(tok_given, n_kept);
            }
            if (robust) {                                        // (the counters start again)
                nc_bar<NC_GT>(gi);
                if (gtid == 0) { g.flags = 0; g.masked = 0; g.has[0] = g.has[1] = g.has[2] = g.has[3] = g.has[4] = g.has[5] = 0u; }
                nc_bar<NC_GT>(gi);
            }
        }
        if (robust && !failed) {
            const uint32_t kmax = max_pass();
            if (kmax >= Tr::KEY_PINF || kmax <= Tr::KEY_NINF) {
                failed = true;
            } else {
                s64 = inv_tau * 0x1.71547652b82fep+6;            // 64 log2(e) / temp
                c64 = -(double)Tr::value_f(kmax) * s64;
                sum_pass<false>();
                nc_bar<NC_GT>(gi);
                if (warp == 0 && !g.poisoned) {
                    if (xp) locate_xp<false>(tcell, g.masked);
                    else if (tok_given < 0) locate<false>(c, c_in, g.masked);
                    else interval<false>(tok_given, g.masked);
                }
            }
        }
        if (gtid == 0) {
            if (*(volatile int*)&g.poisoned) g.res = failed_lane(c_in, ST_TIMEOUT);
            else if (failed) g.res = failed_lane(c_in, ST_NUMERIC);
        }
        nc_bar<NC_GT>(gi);
        const LaneResult out = g.res;
        if (gtid == 0) { g.flags = 0; g.masked = 0; g.has[0] = g.has[1] = g.has[2] = g.has[3] = g.has[4] = g.has[5] = 0u; }
        nc_bar<NC_GT>(gi);          // the buffer and the result slot are free again
        return out;
    }
};

template <int DT, int MODE>
__global__ void __launch_bounds__(NC_MAXG * NC_GT, 1) nocut_kernel(const NocutArgs a, const int groups, const int row_stride) {
    using Tr = Traits<DT>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    double* tbl = reinterpret_cast<double*>(smem_raw);
    double* exp_tbl = tbl + NC_TBL_DOUBLES;
    NcGroupSmem* gs = reinterpret_cast<NcGroupSmem*>(exp_tbl + 64);
    unsigned char* bufs = smem_raw + nc_fixed_bytes();

    const int tid = threadIdx.x;
    const int gi = tid / NC_GT, gtid = tid % NC_GT;
    NcGroupSmem& g = gs[gi];
    fill_exp_table(exp_tbl, tid);
    if (gtid == 0) {
        for (int p = 0; p < NC_MAXPIECE; ++p) mbar_init(smem_u32(&g.full[p]), 1);
        g.flags = 0; g.masked = 0; g.poisoned = 0; g.has[0] = g.has[1] = g.has[2] = g.has[3] = g.has[4] = g.has[5] = 0u;
    }
    if (tid == 0) fence_mbar_init();
    __syncthreads();
    if (a.use_table && DT == DT_BF16) {
        for (int i = tid; i < NC_TBL_DOUBLES; i += blockDim.x) {
            const uint32_t e4 = (i >> 7) & 15u;
            const uint32_t ex = e4 >= (NC_EXP_LO & 15u) ? (NC_EXP_LO & ~15u) + e4 : (NC_EXP_LO & ~15u) + 16u + e4;
            const uint32_t bits = ((uint32_t)(i >> 11) << 15) | (ex << 7) | (uint32_t)(i & 127);
            const bool used = ex >= (uint32_t)NC_EXP_LO && ex < (uint32_t)(NC_EXP_LO + NC_BINADES);
            tbl[i] = used ? exp_core((double)__uint_as_float(bits << 16) * a.inv_tau, exp_tbl) : 0.0;
        }
    }
    __syncthreads();

    const int V = a.V;
    NcRow<DT> R{g};
    R.tbl = tbl; R.exp_tbl = exp_tbl;
    R.rowv = reinterpret_cast<const uint4*>(bufs + (size_t)gi * row_stride);
    R.V = V;
    R.nvec = (V + Tr::E - 1) / Tr::E;
    const int bulk_bytes = (V * Tr::BYTES) & ~15;
    R.bulk_vec = bulk_bytes >> 4;
    R.nch = (R.nvec + 31) / 32;
    R.npiece = (bulk_bytes + NC_PIECE_BYTES - 1) / NC_PIECE_BYTES;
    R.gi = gi; R.gtid = gtid; R.lane = gtid & 31; R.warp = gtid >> 5;
    R.inv_tau = a.inv_tau; R.s64 = 0.0; R.c64 = 0.0;
    R.parity = 0;
    R.wait_cycles = a.wait_cycles;
    bool armed = false;              // copies issued under the current parity (uniform in the group)

    // bring a row into the group's buffer (every reader of the previous row has passed the group
    // barrier that precedes this call)
    auto fetch = [&](const char* src) {
        R.grow = src;
        if (!a.debug_no_copy && !*(volatile int*)&g.poisoned) {
            if (gtid < R.npiece) {                 // one piece per thread: the issues do not queue behind one another
                fence_proxy_async();
                const int p = gtid;
                const uint32_t bytes = (uint32_t)min(NC_PIECE_BYTES, bulk_bytes - p * NC_PIECE_BYTES);
                const uint32_t bar = smem_u32(&g.full[p]);
                mbar_expect_tx(bar, bytes);
                bulk_g2s(smem_u32(R.rowv) + p * NC_PIECE_BYTES, src + (size_t)p * NC_PIECE_BYTES, bytes, bar);
            }
            armed = true;
        }
    };
    // (after a time-out nothing more is issued: parity and `armed` keep describing the last copies)
    auto row_done = [&]() { if (!*(volatile int*)&g.poisoned) { R.parity ^= 1u; armed = false; } };
    auto row_ptr = [&](long long r) -> const char* {
        return reinterpret_cast<const char*>(a.data) + (size_t)r * (size_t)a.ld * Tr::BYTES;
    };

    const int ngroups = gridDim.x * groups;
    if (gi < groups) {
        for (int ln = blockIdx.x * groups + gi; ln < a.lanes; ln += ngroups) {
            if (MODE == NC_STEP) {
                double c;
                if (a.lat_N > 0) {
                    c = ((double)(a.lat_j0 + ln) + a.lat_u) / (double)a.lat_N;
                    if (c >= 1.0) c -= 1.0;
                } else {
                    c = a.codes[ln];
                }
                LaneResult r;
                if (!(c >= 0.0 && c <= 1.0)) {
                    r = failed_lane(c, ST_NUMERIC);
                } else {
                    fetch(row_ptr(ln));
                    r = R.run(c, -1, a.use_table != 0);
                    row_done();
                }
                if (gtid == 0) {
                    a.tokens[ln] = r.token;
                    a.codes_out[ln] = r.code_out;
                    if (a.diag.p_tok) a.diag.p_tok[ln] = r.p_tok;
                    if (a.diag.cdf_lo) a.diag.cdf_lo[ln] = r.cdf_lo;
                    if (a.diag.n_kept) a.diag.n_kept[ln] = r.n_kept;
                    if (a.diag.lane_status) a.diag.lane_status[ln] = r.status;
                    if (a.diag.path) a.diag.path[ln] = PATH_GENERAL;
                }
            } else if (MODE == NC_DECODE) {
                // Algorithm 1's REPEAT ... UNTIL X = EOS for one lane
                int prev;
                double c;
                if (a.codes_in) {
                    prev = a.tok_in[ln];
                    c = a.codes_in[ln];
                } else {
                    prev = a.tok_in[ln / a.N];
                    c = ((double)(ln % a.N) + a.u) / (double)a.N;
                    if (c >= 1.0) c -= 1.0;
                }
                int n = 0, status = ST_OK;
                for (int t = 0; t < a.T; ++t) {
                    if (prev < 0 || prev >= V || !(c >= 0.0 && c <= 1.0)) { status = ST_NUMERIC; break; }
                    fetch(row_ptr(prev));
                    const LaneResult r = R.run(c, -1, a.use_table != 0);
                    row_done();
                    if (r.status != ST_OK) { status = r.status; break; }
                    if (gtid == 0) a.seq[(size_t)ln * a.T + t] = r.token;
                    n = t + 1;
                    c = r.code_out;
                    prev = r.token;
                    if (r.token == a.eos) break;
                }
                for (int t = n + gtid; t < a.T; t += NC_GT) a.seq[(size_t)ln * a.T + t] = -1;
                if (gtid == 0) {
                    a.len[ln] = n;
                    if (a.codes_final) a.codes_final[ln] = c;
                    if (a.lane_status) a.lane_status[ln] = status;
                }
            } else if (MODE == NC_DECODE_XP) {
                // the same loop with the code carried in exact arithmetic: every thread keeps the
                // lane's state and advances it by the chosen token's cells
                XpState xs;
                xs.range = a.xp_state[(size_t)ln * 4]; xs.code = a.xp_state[(size_t)ln * 4 + 1];
                xs.q = a.xp_state[(size_t)ln * 4 + 2]; xs.packed = a.xp_state[(size_t)ln * 4 + 3];
                int prev = a.tok_in[ln];
                int n = 0, status = ST_OK;
                for (int t = 0; t < a.T; ++t) {
                    if (prev < 0 || prev >= V || !xp_state_ok(xs)) { status = ST_NUMERIC; break; }
                    fetch(row_ptr(prev));
                    const LaneResult r = R.run(0.0, -1, a.use_table != 0, true, xp_target(xs));
                    row_done();
                    if (r.status != ST_OK) { status = r.status; break; }
                    xp_advance(xs, g.xp_lo, g.xp_hi, (unsigned)a.N);
                    if (gtid == 0) a.seq[(size_t)ln * a.T + t] = r.token;
                    n = t + 1;
                    prev = r.token;
                    if (r.token == a.eos) break;
                }
                for (int t = n + gtid; t < a.T; t += NC_GT) a.seq[(size_t)ln * a.T + t] = -1;
                if (gtid == 0) {
                    a.len[ln] = n;
                    a.xp_state[(size_t)ln * 4] = xs.range; a.xp_state[(size_t)ln * 4 + 1] = xs.code;
                    a.xp_state[(size_t)ln * 4 + 2] = xs.q; a.xp_state[(size_t)ln * 4 + 3] = xs.packed;
                    if (a.lane_status) a.lane_status[ln] = status;
                }
            } else {
                // sequence -> interval: lo gathers width * F_{i-1}, width multiplies by p_i
                int prev = a.tok_in[ln];
                const int n = min(a.len_in[ln], a.T);
                double lo = 0.0, comp = 0.0, width = 1.0;
                int status = ST_OK;
                for (int t = 0; t < n; ++t) {
                    const int tok = a.seq_in[(size_t)ln * a.T + t];
                    if (prev < 0 || prev >= V || tok < 0 || tok >= V) { status = -1; break; }   // invalid argument
                    fetch(row_ptr(prev));
                    const LaneResult r = R.run(0.0, tok, a.use_table != 0);
                    row_done();
                    if (r.status != ST_OK) { status = r.status; break; }
                    const double term = width * r.cdf_lo;          // compensated: the terms shrink with t
                    const double s = lo + term;
                    comp += (fabs(lo) >= fabs(term)) ? (lo - s) + term : (term - s) + lo;
                    lo = s;
                    width *= r.p_tok;
                    prev = tok;
                }
                if (gtid == 0) {
                    a.lo_out[ln] = lo + comp;
                    a.width_out[ln] = width;
                    if (a.lane_status) a.lane_status[ln] = status;
                }
            }
        }
        // a wait ran out: copies armed before that may still be in flight into this buffer
        if (gtid == 0 && armed && *(volatile int*)&g.poisoned)
            for (int p = 0; p < R.npiece; ++p)
                if (!mbar_wait_bounded(smem_u32(&g.full[p]), R.parity, a.wait_cycles)) break;
    }
}

}  // namespace asx

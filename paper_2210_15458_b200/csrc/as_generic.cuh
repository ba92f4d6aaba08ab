// General decode step for one lane, run by one CTA on a row it can address
// (global or shared memory).  Correct for every input: any V, any top_k /
// top_p, ties, masked tokens.  All masses are fp64.
//
// Steps (Algorithm 1's loop body with the logit modifiers):
//   1. max key, non-finite detection
//   2. top-k: exact radix select on the ordered keys -> threshold key T and the
//      number of elements equal to T that are kept (lowest indices first)
//   3. Z1 = sum of exp((l - l_max)/temp) over the kept set
//   4. nucleus: radix select on the keys weighted by mass -> new threshold
//   5. per-chunk masses in index order, exclusive scan, Z
//   6. the chunk, then the element, whose interval holds c*Z; rescale
//
// The row is cut into chunks of 32*E*R consecutive elements, one warp per chunk
// at a time, lane l of the warp owning E consecutive elements of each of the R
// sub-rows, so that (chunk, sub-row, lane, element) order is index order.
#pragma once
#include "as_common.cuh"
#include <limits.h>

namespace asx {

constexpr int MAXCH = 512;  // chunks per row (R grows so that this suffices)
constexpr int HIST_REP = 4; // replicas of every histogram bin

// kept(key) = key > T, or key == T and: eq_mode 1 -> always; eq_mode 2 -> only the
// first `need` such elements in index order; eq_mode 0 -> never.
struct Pred {
    uint32_t T;
    int need;
    int eq_mode;
};

// Locally typical cut: kept(j) also needs tkey(j) > T, or tkey(j) == T and: eq_mode 1 -> always;
// eq_mode 2 -> only the first `need` such kept elements in index order.  tkey orders the tokens
// by |y_j - mu| ascending (y the scaled logit, mu its mean under the distribution = ln Z - H).
struct TypPred {
    int on;
    double mu;
    unsigned long long T;
    int need;
    int eq_mode;
};

template <int NT>
struct GenericSmem {
    double chunk_sum[MAXCH + 1];
    int chunk_eq[MAXCH + 1];
    int chunk_eq2[MAXCH + 1];             // typical cut: ties at its threshold, per chunk
    unsigned chunk_has[MAXCH / 32];       // bit ci: chunk ci holds mass (set with chunk_sum, before its scan)
    double hist_mass[256 * HIST_REP];     // bin d, replica r at [d * HIST_REP + r]: lanes spread over
    int hist_cnt[256 * HIST_REP];         // the replicas, so that a crowded bin is hit by fewer threads
    double red_d[NT / 32];
    unsigned red_u[NT / 32];
    unsigned red_u2[NT / 32];
    int red_i[NT / 32];
    double exp_tbl[64];
    double b_d[4];
    int b_i[4];
    unsigned b_u[2];
    LaneResult res;
    unsigned long long xp_lo, xp_hi;      // extended-precision steps: the chosen token's cells
};

// Barrier over the NT threads that run a lane: the whole CTA, or (in kernels with a
// separate copy-issuing warp) the consumer warps only, through named barrier 1.
struct SyncAll {
    __device__ __forceinline__ static void sync() { __syncthreads(); }
};
template <int NTHREADS>
struct SyncNamed {
    __device__ __forceinline__ static void sync() {
        asm volatile("bar.sync 1, %0;" ::"n"(NTHREADS) : "memory");
    }
};

template <int DT, int NT, class Sync = SyncAll>
struct GenericLane {
    using Tr = Traits<DT>;
    static constexpr int E = Tr::E;
    static constexpr int NW = NT / 32;

    GenericSmem<NT>& sm;
    const void* row;
    int V;
    bool vec_ok;
    int nvec, R, nchunks;
    int tid, lane, warp;
    double lmax, inv_tau;
    TypPred tp;

    __device__ GenericLane(GenericSmem<NT>& s, const void* row_, int V_, bool vec_ok_)
        : sm(s), row(row_), V(V_), vec_ok(vec_ok_) {
        tp.on = 0; tp.mu = 0.0; tp.T = 0; tp.need = 0; tp.eq_mode = 0;
        tid = threadIdx.x;
        lane = tid & 31;
        warp = tid >> 5;
        nvec = (V + E - 1) / E;
        const int rows32 = (nvec + 31) / 32;
        R = (rows32 + MAXCH - 1) / MAXCH;
        nchunks = (rows32 + R - 1) / R;
    }

    __device__ __forceinline__ void chunk_keys(int ci, int r, uint32_t (&k)[E], int& base) const {
        const int vi = (ci * R + r) * 32 + lane;
        base = vi * E;
        if (vi < nvec) {
            load_vec_keys<DT>(row, V, vi, vec_ok, k);
        } else {
#pragma unroll
            for (int e = 0; e < E; ++e) k[e] = Tr::KEY_NINF;
        }
    }

    // index-order rank, among the elements equal to p.T, of this lane's first one
    __device__ __forceinline__ int lane_rank0(const uint32_t (&k)[E], const Pred& p, int& tie_run) const {
        if (p.eq_mode != 2) return 0;
        int cnt = 0;
#pragma unroll
        for (int e = 0; e < E; ++e) cnt += (k[e] == p.T);
        const int incl = warp_incl_scan_i(cnt, lane);
        const int rank0 = tie_run + incl - cnt;
        tie_run += __shfl_sync(FULL, incl, 31);
        return rank0;
    }

    __device__ __forceinline__ unsigned kept_bits(const uint32_t (&k)[E], const Pred& p, int rank0) const {
        unsigned m = 0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (k[e] > p.T) {
                m |= 1u << e;
            } else if (k[e] == p.T) {
                if (p.eq_mode == 1 || (p.eq_mode == 2 && rank0 < p.need)) m |= 1u << e;
                ++rank0;
            }
        }
        return m;
    }

    __device__ __forceinline__ double mass(uint32_t key) const {
        return exp_nonpos(((double)Tr::value_f(key) - lmax) * inv_tau, sm.exp_tbl);
    }

    // Does chunk ci hold mass?  (Not to be read off the scanned sums: the scan adds lane totals in
    // another order than the running sums inside a lane, so sum[ci+1] > sum[ci] can hold by an ulp
    // for an empty chunk at a lane boundary.)
    __device__ __forceinline__ bool has_mass(int ci) const { return (sm.chunk_has[ci >> 5] >> (ci & 31)) & 1u; }
    __device__ __forceinline__ void clear_has() {
        for (int i = tid; i < MAXCH / 32; i += NT) sm.chunk_has[i] = 0u;
        Sync::sync();
    }
    __device__ __forceinline__ void put_chunk(int ci, double local) {      // lane 0 of the chunk's warp
        sm.chunk_sum[ASX_AT(ci, MAXCH + 1, 82)] = local;
        if (local > 0.0) red_shared_or(&sm.chunk_has[ci >> 5], 1u << (ci & 31));
    }

    // typical cut: order key of a token, larger = nearer the mean scaled logit
    __device__ __forceinline__ unsigned long long tkey(uint32_t key) const {
        const double y = ((double)Tr::value_f(key) - lmax) * inv_tau;
        return ~(unsigned long long)__double_as_longlong(fabs(y - tp.mu));
    }
    // kept elements of this lane's vector under the top-k / nucleus predicate and, if on, the
    // typical cut; tie_run / tie_run2 carry the index-order ranks of the two kinds of ties
    __device__ __forceinline__ unsigned kept_all(const uint32_t (&k)[E], const Pred& p, int& tie_run, int& tie_run2) const {
        const int rank0 = lane_rank0(k, p, tie_run);
        unsigned bits = kept_bits(k, p, rank0);
        if (!tp.on) return bits;
        unsigned gt = 0, eqm = 0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (bits & (1u << e)) {
                const unsigned long long t = tkey(k[e]);
                if (t > tp.T) gt |= 1u << e;
                else if (t == tp.T) eqm |= 1u << e;
            }
        }
        if (tp.eq_mode == 1) return gt | eqm;
        if (tp.eq_mode == 2) {
            const int cnt = __popc(eqm);
            const int incl = warp_incl_scan_i(cnt, lane);
            int rank = tie_run2 + incl - cnt;
            tie_run2 += __shfl_sync(FULL, incl, 31);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                if (eqm & (1u << e)) {
                    if (rank < tp.need) gt |= 1u << e;
                    ++rank;
                }
            }
        }
        return gt;
    }

    // exclusive scan of a[0..n), n >= 1, in place by warp 0; a[n] receives the total
    template <typename T>
    __device__ void scan_exclusive(T* a, int n) {
        if (warp == 0) {
            const int per = (n + 31) / 32;
            const int b = min(lane * per, n), e = min(b + per, n);
            T s = 0;
            for (int i = b; i < e; ++i) s += a[i];
            T incl = s;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const T u = __shfl_up_sync(FULL, incl, o);
                if (lane >= o) incl += u;
            }
            T run = __shfl_up_sync(FULL, incl, 1);
            if (lane == 0) run = 0;
            for (int i = b; i < e; ++i) {
                const T v = a[i];
                a[i] = run;
                run += v;
            }
            // the total continues the same running sum as the prefixes, so that
            // a[i+1] > a[i] exactly when element i added something
            if (e == n && b < n) a[n] = run;
        }
        Sync::sync();
    }

    // chunk_eq[ci] <- number of elements equal to T in chunks before ci
    __device__ void tie_prepass(uint32_t T) {
        for (int ci = warp; ci < nchunks; ci += NW) {
            int cnt = 0;
            for (int r = 0; r < R; ++r) {
                uint32_t k[E];
                int base;
                chunk_keys(ci, r, k, base);
#pragma unroll
                for (int e = 0; e < E; ++e) cnt += (k[e] == T);
            }
            cnt = warp_sum_i(cnt);
            if (lane == 0) sm.chunk_eq[ASX_AT(ci, MAXCH + 1, 83)] = cnt;
        }
        Sync::sync();
        scan_exclusive(sm.chunk_eq, nchunks);
    }

    // chunk_sum[ci] <- mass of the kept elements of chunk ci
    __device__ void sum_pass(const Pred& p) {
        clear_has();
        for (int ci = warp; ci < nchunks; ci += NW) {
            int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[ci] : 0;
            int tie_run2 = (tp.on && tp.eq_mode == 2) ? sm.chunk_eq2[ci] : 0;
            double local = 0.0;
            for (int r = 0; r < R; ++r) {
                uint32_t k[E];
                int base;
                chunk_keys(ci, r, k, base);
                const unsigned bits = kept_all(k, p, tie_run, tie_run2);
#pragma unroll
                for (int e = 0; e < E; ++e)
                    if (bits & (1u << e)) local += mass(k[e]);
            }
            local = warp_sum_d(local);
            if (lane == 0) put_chunk(ci, local);
        }
        Sync::sync();
    }

    // histogram of digit (key >> shift) & 255 over kept elements whose key matches
    // `prefix` on `mask`; counts always, masses if MASS
    template <bool MASS>
    __device__ void hist_pass(const Pred& p, uint32_t prefix, uint32_t mask, int shift) {
        for (int i = tid; i < 256 * HIST_REP; i += NT) {
            sm.hist_cnt[i] = 0;
            sm.hist_mass[i] = 0.0;
        }
        const int rep = lane & (HIST_REP - 1);
        Sync::sync();
        // Each thread gathers runs of equal digits in registers and touches shared memory only
        // when the digit changes: the leading digits of a row fall into a handful of bins, and
        // a shared-memory fp64 add is a compare-and-swap loop that such crowding serialises.
        // (Merging across the warp first -- one add per distinct digit among 32 lanes -- was
        // tried and is 2-3x slower: the lower digits are all different.)
        int cur_d = -1, cur_n = 0;
        double cur_m = 0.0;
        for (int ci = warp; ci < nchunks; ci += NW) {
            int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[ci] : 0;
            for (int r = 0; r < R; ++r) {
                uint32_t k[E];
                int base;
                chunk_keys(ci, r, k, base);
                const int rank0 = lane_rank0(k, p, tie_run);
                const unsigned bits = kept_bits(k, p, rank0);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if ((bits & (1u << e)) && (k[e] & mask) == prefix) {
                        const int d = (k[e] >> shift) & 255;
                        if (d != cur_d) {
                            if (cur_n) {
                                atomicAdd(&sm.hist_cnt[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 80)], cur_n);
                                if (MASS) atomicAdd(&sm.hist_mass[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 81)], cur_m);
                            }
                            cur_d = d; cur_n = 0; cur_m = 0.0;
                        }
                        ++cur_n;
                        if (MASS) cur_m += mass(k[e]);
                    }
                }
            }
        }
        if (cur_n) {
            atomicAdd(&sm.hist_cnt[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 80)], cur_n);
            if (MASS) atomicAdd(&sm.hist_mass[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 81)], cur_m);
        }
        Sync::sync();
    }

    // Largest non-empty digit d with (acc + weight of digits >= d) >= target; if none
    // (rounding), the smallest non-empty digit.  Outputs through shared memory:
    // b_i[0] = d, b_i[1] = acc_cnt + count(digits > d), b_i[2] = count(d),
    // b_d[0] = acc_mass + mass(digits > d).
    template <bool MASS>
    __device__ void choose_digit(int acc_cnt, double acc_mass, int k_target, double m_target) {
        if (warp == 0) {
            int c[8];
            double m[8];
            int lc = 0;
            double lm = 0.0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                c[e] = 0;
                m[e] = 0.0;
#pragma unroll
                for (int r = 0; r < HIST_REP; ++r) {
                    c[e] += sm.hist_cnt[(lane * 8 + e) * HIST_REP + r];
                    if (MASS) m[e] += sm.hist_mass[(lane * 8 + e) * HIST_REP + r];
                }
                lc += c[e];
                lm += m[e];
            }
            const int suf_c = warp_suffix_i(lc, lane);
            const double suf_m = MASS ? warp_suffix_d(lm, lane) : 0.0;
            int above_c = __shfl_down_sync(FULL, suf_c, 1);
            double above_m = __shfl_down_sync(FULL, suf_m, 1);
            if (lane == 31) { above_c = 0; above_m = 0.0; }
            int best = -1, best_above_c = 0, best_c = 0;
            double best_above_m = 0.0, best_m = 0.0;
            int low = -1, low_above_c = 0, low_c = 0;
            double low_above_m = 0.0, low_m = 0.0;
            int run_c = above_c;
            double run_m = above_m;
#pragma unroll
            for (int e = 7; e >= 0; --e) {
                if (c[e] > 0) {
                    const bool ok = MASS ? (acc_mass + (run_m + m[e]) >= m_target)
                                         : (acc_cnt + run_c + c[e] >= k_target);
                    if (ok && best < 0) {
                        best = lane * 8 + e; best_above_c = run_c; best_above_m = run_m; best_c = c[e]; best_m = m[e];
                    }
                    low = lane * 8 + e; low_above_c = run_c; low_above_m = run_m; low_c = c[e]; low_m = m[e];
                }
                run_c += c[e];
                run_m += m[e];
            }
            const unsigned bal = __ballot_sync(FULL, best >= 0);
            int src;
            if (bal) {
                src = 31 - __clz(bal);
            } else {
                const unsigned bal2 = __ballot_sync(FULL, low >= 0);
                src = bal2 ? (__ffs(bal2) - 1) : 0;
                best = low; best_above_c = low_above_c; best_above_m = low_above_m; best_c = low_c; best_m = low_m;
            }
            best_m = __shfl_sync(FULL, best_m, src);
            best = __shfl_sync(FULL, best, src);
            best_above_c = __shfl_sync(FULL, best_above_c, src);
            best_above_m = __shfl_sync(FULL, best_above_m, src);
            best_c = __shfl_sync(FULL, best_c, src);
            if (lane == 0) {
                sm.b_i[0] = best < 0 ? 0 : best;
                sm.b_i[1] = acc_cnt + best_above_c;
                sm.b_i[2] = best_c;
                sm.b_d[0] = acc_mass + best_above_m;
                sm.b_d[1] = best_m;
            }
        }
        Sync::sync();
    }

    __device__ LaneResult fail(double c_in, int status) {
        LaneResult r;
        r.token = -1; r.status = status; r.n_kept = 0; r.code_out = c_in; r.p_tok = 0.0; r.cdf_lo = 0.0;
        return r;
    }

    // ------------------------------------------------------------------ no cut: every finite token kept
    // Lean version of the same steps for lanes without top-k / nucleus on 16-byte aligned rows:
    // a packed NaN-propagating max pass, then masses straight from the float values.
    __device__ __forceinline__ void chunk_floats(int ci, int r, float (&x)[E], int& base) const {
        using P = Pass<DT>;
        const int vi = (ci * R + r) * 32 + lane;
        base = vi * E;
        if (vi < nvec && base + E <= V) {
            const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) + (size_t)base * Tr::BYTES);
            P::floats(q, x);
        } else {
#pragma unroll
            for (int e = 0; e < E; ++e)
                x[e] = (vi < nvec && base + e < V) ? P::load_f(row, base + e) : __uint_as_float(0xFF800000u);
        }
    }

    __device__ __noinline__ LaneResult run_nocut(double c_in, double inv_tau_) {
        using P = Pass<DT>;
        inv_tau = inv_tau_;
        fill_exp_table(sm.exp_tbl, tid);
        double c = c_in;
        const bool code_bad = !(c >= 0.0 && c <= 1.0);
        if (c == 1.0) c = ASX_ONE_BELOW;
        // ---- 1. maximum (NaN and +inf propagate into it)
        typename P::Acc acc = P::init();
        float vmn = __uint_as_float(0x7F800000u);                    // the row's minimum, for the plain case below
        const int nvf = (V * Tr::BYTES) >> 4;
        for (int vi = tid; vi < nvf; vi += NT) {
            const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) + (size_t)vi * 16);
            P::merge(acc, P::reduce(q));
            vmn = fminf(vmn, P::vmin(q));
        }
        for (int j = nvf * E + tid; j < V; j += NT) {
            P::fold_scalar(acc, row, j);
            vmn = fminf(vmn, P::load_f(row, j));
        }
        uint32_t k0, k1;
        P::keys(acc, k0, k1);
        uint32_t kmax = warp_max_u(max(k0, k1));
        uint32_t kmin = warp_min_u(P::key_of_f(vmn));
        if (lane == 0) { sm.red_u[warp] = kmax; sm.red_u2[warp] = kmin; }
        if (tid == 0) sm.b_i[2] = 0;
        Sync::sync();
        kmax = 0; kmin = 0xFFFFFFFFu;
        for (int w = 0; w < NW; ++w) { kmax = max(kmax, sm.red_u[w]); kmin = min(kmin, sm.red_u2[w]); }
        if (code_bad || kmax >= Tr::KEY_PINF || kmax <= Tr::KEY_NINF) {
            Sync::sync();
            return fail(c_in, ST_NUMERIC);
        }
        lmax = (double)Tr::value_f(kmax);
        const double s64 = inv_tau * 0x1.71547652b82fep+6;          // 64 log2(e) / temp
        const double c64 = -lmax * s64;
        // The plain case -- no masked token, and no mass below 2^-1000 of the largest: every token
        // is kept and the exponential needs no underflow guard, which shortens the loop that every
        // logit of every step goes through.
        const bool plain = kmin > Tr::KEY_NINF && fma((double)Tr::value_f(kmin), s64, c64) >= -64000.0;
        // ---- 2. per-chunk masses in index order
        clear_has();
        int nfin = 0;
        for (int ci = warp; ci < nchunks; ci += NW) {
            double local = 0.0;
            for (int r = 0; r < R; ++r) {
                float x[E];
                int base;
                chunk_floats(ci, r, x, base);
                if (plain && base + E <= V) {        // (a vector reaching past V holds -inf padding: guarded)
#pragma unroll
                    for (int e = 0; e < E; ++e) local += exp2_64th<false>(fma((double)x[e], s64, c64), sm.exp_tbl);
                } else {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        local += exp2_64th(fma((double)x[e], s64, c64), sm.exp_tbl);
                        nfin += (x[e] > __uint_as_float(0xFF800000u));
                    }
                }
            }
            local = warp_sum_d(local);
            if (lane == 0) put_chunk(ci, local);
        }
        nfin = warp_sum_i(nfin);
        if (lane == 0) atomicAdd(&sm.b_i[2], nfin);
        Sync::sync();
        scan_exclusive(sm.chunk_sum, nchunks);
        // ---- 3. the chunk, then the element, whose interval holds c * Z
        const double Z = sm.chunk_sum[nchunks];
        const double t = c * Z;
        const int n_kept = plain ? V : sm.b_i[2];
        if (tid == 0) { sm.b_i[0] = INT_MAX; sm.b_i[1] = -1; }
        Sync::sync();
        for (int ci = tid; ci < nchunks; ci += NT) {
            if (has_mass(ci)) {
                atomicMax(&sm.b_i[1], ci);
                if (t < sm.chunk_sum[ci + 1]) atomicMin(&sm.b_i[0], ci);
            }
        }
        Sync::sync();
        const bool force_last = (sm.b_i[0] == INT_MAX);
        const int cstar = force_last ? sm.b_i[1] : sm.b_i[0];
        if (warp == 0) {
            double run = sm.chunk_sum[cstar];
            int last_idx = -1;
            double last_S = 0.0, last_e = 1.0;
            int tok = -1;
            double tok_S = 0.0, tok_e = 1.0;
            for (int r = 0; r < R && tok < 0; ++r) {
                float x[E];
                int base;
                chunk_floats(cstar, r, x, base);
                double ev[E];
                double local = 0.0;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    ev[e] = exp2_64th(fma((double)x[e], s64, c64), sm.exp_tbl);
                    local += ev[e];
                }
                const double incl = warp_incl_scan_d(local, lane);
                double excl = __shfl_up_sync(FULL, incl, 1);
                if (lane == 0) excl = 0.0;
                int pick = -1;
                double pick_S = 0.0, pick_e = 1.0;
                double S = run + excl;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if (ev[e] > 0.0) {
                        if (pick < 0 && t < S + ev[e]) { pick = base + e; pick_S = S; pick_e = ev[e]; }
                        last_idx = base + e; last_S = S; last_e = ev[e];
                        S += ev[e];
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
                }
                run += __shfl_sync(FULL, incl, 31);
            }
            if (tok < 0) {   // rounding at the top end: the last token with mass in the chunk
                const unsigned best = warp_max_u((unsigned)(last_idx + 1));
                const unsigned bal = __ballot_sync(FULL, (unsigned)(last_idx + 1) == best);
                const int L = __ffs(bal) - 1;
                tok = __shfl_sync(FULL, last_idx, L);
                tok_S = __shfl_sync(FULL, last_S, L);
                tok_e = __shfl_sync(FULL, last_e, L);
            }
            if (lane == 0) {
                double cn = (t - tok_S) / tok_e;
                if (!(cn >= 0.0)) cn = 0.0;
                if (cn > ASX_ONE_BELOW) cn = ASX_ONE_BELOW;
                LaneResult r;
                r.token = tok; r.status = tok < 0 ? ST_NUMERIC : ST_OK; r.n_kept = n_kept;
                r.code_out = tok < 0 ? c_in : cn;
                r.p_tok = tok_e / Z;
                r.cdf_lo = tok_S / Z;
                sm.res = r;
            }
        }
        Sync::sync();
        const LaneResult out = sm.res;
        Sync::sync();
        return out;
    }

    // The typical cut among the elements kept by `p` (whose masses' scan is in chunk_sum): sets tp.
    __device__ void typical_cut(const Pred& p, double typical_p, int& n_kept) {
        const double Z1 = sm.chunk_sum[nchunks];
        Sync::sync();
        // mean scaled logit under the distribution: mu = sum e_j y_j / Z1  (= ln Z1 - H)
        double acc = 0.0;
        for (int ci = warp; ci < nchunks; ci += NW) {
            int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[ci] : 0, unused = 0;
            for (int r = 0; r < R; ++r) {
                uint32_t k[E];
                int base;
                chunk_keys(ci, r, k, base);
                const unsigned bits = kept_all(k, p, tie_run, unused);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if (bits & (1u << e)) {
                        const double y = ((double)Tr::value_f(k[e]) - lmax) * inv_tau;
                        const double m = exp_nonpos(y, sm.exp_tbl);
                        if (m > 0.0) acc += m * y;
                    }
                }
            }
        }
        acc = warp_sum_d(acc);
        if (lane == 0) sm.red_d[warp] = acc;
        Sync::sync();
        double tot = 0.0;
        for (int w = 0; w < NW; ++w) tot += sm.red_d[w];
        Sync::sync();
        tp.mu = tot / Z1;
        // mass-weighted radix select on the 64-bit order key, 8 bits at a time
        const double target = typical_p * Z1;
        unsigned long long prefix = 0, mask = 0;
        int acc_c = 0, eq = 0;
        double acc_m = 0.0, eq_m = 0.0;
        const int rep = lane & (HIST_REP - 1);
        for (int shift = 56; shift >= 0; shift -= 8) {
            for (int i = tid; i < 256 * HIST_REP; i += NT) { sm.hist_cnt[i] = 0; sm.hist_mass[i] = 0.0; }
            Sync::sync();
            int cur_d = -1, cur_n = 0;
            double cur_m = 0.0;
            for (int ci = warp; ci < nchunks; ci += NW) {
                int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[ci] : 0, unused = 0;
                for (int r = 0; r < R; ++r) {
                    uint32_t k[E];
                    int base;
                    chunk_keys(ci, r, k, base);
                    const unsigned bits = kept_all(k, p, tie_run, unused);
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        if (bits & (1u << e)) {
                            const unsigned long long t = tkey(k[e]);
                            if ((t & mask) == prefix) {
                                const int d = (int)((t >> shift) & 255ull);
                                if (d != cur_d) {
                                    if (cur_n) {
                                        atomicAdd(&sm.hist_cnt[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 80)], cur_n);
                                        atomicAdd(&sm.hist_mass[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 81)], cur_m);
                                    }
                                    cur_d = d; cur_n = 0; cur_m = 0.0;
                                }
                                ++cur_n;
                                cur_m += mass(k[e]);
                            }
                        }
                    }
                }
            }
            if (cur_n) {
                atomicAdd(&sm.hist_cnt[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 80)], cur_n);
                atomicAdd(&sm.hist_mass[ASX_AT(cur_d * HIST_REP + rep, 256 * HIST_REP, 81)], cur_m);
            }
            Sync::sync();
            choose_digit<true>(acc_c, acc_m, 0, target);
            prefix |= (unsigned long long)sm.b_i[0] << shift;
            mask |= 0xFFull << shift;
            acc_c = sm.b_i[1];
            eq = sm.b_i[2];
            acc_m = sm.b_d[0];
            eq_m = sm.b_d[1];
            Sync::sync();
        }
        // `eq` kept elements share the threshold key (equal logits: equal masses): take the fewest
        // of them, lowest indices first, that bring the mass to the target
        const double e_P = eq_m / (double)eq;
        long long r = (long long)ceil((target - acc_m) / e_P);
        if (r < 1) r = 1;
        if (r > eq) r = eq;
        while (r > 1 && acc_m + (double)(r - 1) * e_P >= target) --r;
        while (r < eq && acc_m + (double)r * e_P < target) ++r;
        // ties at the threshold, per chunk, among the elements kept so far
        for (int ci = warp; ci < nchunks; ci += NW) {
            int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[ci] : 0, unused = 0;
            int cnt = 0;
            for (int rr = 0; rr < R; ++rr) {
                uint32_t k[E];
                int base;
                chunk_keys(ci, rr, k, base);
                const unsigned bits = kept_all(k, p, tie_run, unused);
#pragma unroll
                for (int e = 0; e < E; ++e)
                    if ((bits & (1u << e)) && tkey(k[e]) == prefix) ++cnt;
            }
            cnt = warp_sum_i(cnt);
            if (lane == 0) sm.chunk_eq2[ci] = cnt;
        }
        Sync::sync();
        scan_exclusive(sm.chunk_eq2, nchunks);
        tp.T = prefix;
        tp.need = (int)r;
        tp.eq_mode = ((int)r < eq) ? 2 : 1;
        tp.on = 1;
        n_kept = acc_c + (int)r;
    }

    // ------------------------------------------------------------------ nucleus through value bins
    // The nucleus threshold of a row without a top-k, for nuclei of any width, in two passes over
    // the row instead of the radix select's five with fp64 masses:
    //   B. counts of the elements in WB bins by depth below the row maximum, d = (l_max - l) / temp
    //      in octaves, 128 bins per octave over 24 octaves and one bin for the rest (integer
    //      additions to shared memory are native; fp32 ones are compare-and-swap loops).  The
    //      binning is a monotone function of the key: every key of a bin is above every key of the
    //      next.  A bin's count times the masses at its two edges bounds its mass from both sides,
    //      so the cumulative bounds bracket the bin in which the nucleus ends: bins [b_hi, b_lo].
    //   C. exact fp64 masses: elements above the bracket are kept (their masses go to the chunk
    //      sums right away), elements below it only add to Z, the bracket's elements (<= WCAP) are
    //      listed and ranked exactly (key descending, index ascending).  The first rank at which the
    //      exact prefix reaches top_p * Z closes the kept set.
    // Every decision is taken on exact fp64 sums; the bins only say where to look.  Whatever they
    // cannot settle (a bracket with more than WCAP elements or reaching the last bin, a prefix within
    // rounding of the target) returns 0 and the radix select decides.
    static constexpr int WB = 3072;
    static constexpr int WCAP = 1024;
    bool bins = true;                          // false: always the radix select

    __device__ __forceinline__ float wdepth(uint32_t key, float lmax_f, float s2) const {
        return (lmax_f - Tr::value_f(key)) * s2;
    }
    // exclusive scan of one value per thread over the block, thread order; `total` to every thread
    __device__ __forceinline__ double block_excl_scan_d(double v, double& total) {
        const double incl = warp_incl_scan_d(v, lane);
        if (lane == 31) sm.red_d[warp] = incl;
        Sync::sync();
        double off = 0.0;
        total = 0.0;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            if (w < warp) off += sm.red_d[w];
            total += sm.red_d[w];
        }
        Sync::sync();
        return off + (incl - v);
    }
    __device__ __forceinline__ int block_excl_scan_i(int v, int& total) {
        const int incl = warp_incl_scan_i(v, lane);
        if (lane == 31) sm.red_i[warp] = incl;
        Sync::sync();
        int off = 0;
        total = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            if (w < warp) off += sm.red_i[w];
            total += sm.red_i[w];
        }
        Sync::sync();
        return off + (incl - v);
    }
    __device__ __forceinline__ int chunk_of_index(int idx) const { return (idx / E) / (32 * R); }

    // Bins of one counting pass: `nfine` bins of 1 / scale octaves each over depths from d0 down; the
    // bracket is bins bhi..blo.
    struct WBracket {
        float d0, scale;
        int nfine;
        int bhi, blo;
    };
    // bin of an element at depth d >= d0, or nfine for what lies past the bins
    __device__ __forceinline__ static int wbin(float d, const WBracket& w) {
        const float rel = (d - w.d0) * w.scale;
        return rel < (float)w.nfine ? (int)rel : w.nfine;
    }
    // upper edge (smallest depth) of bin b
    __device__ __forceinline__ static float wedge(int b, const WBracket& w) { return w.d0 + (float)b / w.scale; }
    // class of an element at depth d: 0 above the bracket (kept), 1 inside it, 2 below it; through the
    // very expression that filled the bins, so that counts and classes agree element by element
    __device__ __forceinline__ static int wclass(float d, const WBracket& w) {
        if (d < w.d0) return 0;
        const int b = wbin(d, w);
        return b < w.bhi ? 0 : (b <= w.blo ? 1 : 2);
    }

    __device__ int nucleus_by_bins(double top_p, int nfin_in, Pred& p, int& n_kept) {
        int nfin = nfin_in;                          // < 0: not known yet, the first level counts it
        // This object lives in local memory (its member functions are called out of line), and a store
        // through a shared-memory pointer may alias it as far as the compiler can tell: members used in
        // the loops would be loaded again after every such store.  Locals of the same names shadow them
        // here and stay in registers.
        GenericSmem<NT>& sm = this->sm;
        const void* const row = this->row;
        const int V = this->V, nvec = this->nvec, R = this->R, nchunks = this->nchunks;
        const bool vec_ok = this->vec_ok;
        const int tid = this->tid, lane = this->lane, warp = this->warp;
        const double lmax = this->lmax, inv_tau = this->inv_tau;
        const double* const exp_tbl = sm.exp_tbl;
        double* const chunk_sum = sm.chunk_sum;
        unsigned* const chunk_has = sm.chunk_has;
        auto mass = [&](uint32_t key) -> double { return exp_nonpos(((double)Tr::value_f(key) - lmax) * inv_tau, exp_tbl); };
        auto put_chunk = [&](int ci, double local) {
            chunk_sum[ASX_AT(ci, MAXCH + 1, 82)] = local;
            if (local > 0.0) red_shared_or(&chunk_has[ci >> 5], 1u << (ci & 31));
        };
        auto chunk_of_index = [&](int idx) -> int { return (idx / E) / (32 * R); };
        int* wbc = reinterpret_cast<int*>(sm.hist_mass);                        // WB counts; later
        unsigned long long* wcand = reinterpret_cast<unsigned long long*>(sm.hist_mass);   // WCAP composites
        unsigned long long* acc_hi = reinterpret_cast<unsigned long long*>(sm.hist_cnt);   // MAXCH fixed-point sums
        unsigned long long* acc_lo = reinterpret_cast<unsigned long long*>(sm.chunk_eq);   // (chunk_eq + chunk_eq2)
        static_assert(sizeof(sm.hist_mass) + sizeof(sm.hist_cnt) >= WB * 4 && sizeof(sm.hist_mass) >= WCAP * 8,
                      "bins and list share the histograms' space");
        static_assert(sizeof(sm.hist_cnt) >= MAXCH * 8 && 2 * sizeof(sm.chunk_eq) >= MAXCH * 8 + 8, "fixed-point sums");
        const float lmax_f = (float)lmax;
        const float s2 = (float)(inv_tau * 1.4426950408889634);

        // ---- B. bin counts, at most twice: 128 bins per octave from the maximum down; if the bracket
        //         that gives holds more elements than the list, its range again with finer bins
        WBracket wb;
        wb.d0 = 0.f; wb.scale = 128.f; wb.nfine = WB; wb.bhi = 0; wb.blo = 0;
        // elements above d0 / past the bins: bounds of their mass, their number
        double base_lo = 0.0, base_hi = 0.0, Zf = 0.0;
        int base_c = 0, tail_c = 0;
        int n_in = 0, n_br = 0;
        for (int level = 0;; ++level) {
            for (int i = tid; i < WB; i += NT) wbc[i] = 0;
            Sync::sync();
            int deep = 0;                              // past the bins: counted in a register, they are many
            const int nall = wb.nfine;
            // fp32 masses in registers, four partial sums: of every element (first level: that is Z to
            // 4e-5), of the elements above the window (second level)
            float msum[4] = {0.f, 0.f, 0.f, 0.f};
            {
                constexpr int U = 4;                   // loads in flight per thread
                for (int v0 = tid; v0 < nvec; v0 += U * NT) {
                    uint32_t k[U][E];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int vi = v0 + u * NT;
                        if (vi < nvec) {
                            load_vec_keys<DT>(row, V, vi, vec_ok, k[u]);
                        } else {
#pragma unroll
                            for (int e = 0; e < E; ++e) k[u][e] = Tr::KEY_NINF;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            if (k[u][e] > Tr::KEY_NINF) {
                                const float d = wdepth(k[u][e], lmax_f, s2);
                                if (level == 0 || d < wb.d0) msum[e & 3] += ex2_approx(-d);
                                if (d >= wb.d0) {
                                    const int b = wbin(d, wb);
                                    if (b < nall) red_shared_add(&wbc[b], 1);
                                    else ++deep;
                                }
                            }
                        }
                    }
                }
            }
            {
                double msum_all;
                (void)block_excl_scan_d(((double)msum[0] + (double)msum[1]) + ((double)msum[2] + (double)msum[3]), msum_all);
                if (level == 0) {
                    // (the first level's bins end 24 octaves down; the elements past them are only counted)
                    int all_deep;
                    (void)block_excl_scan_i(deep, all_deep);
                    tail_c = all_deep;
                    Zf = msum_all;
                } else {
                    base_lo = msum_all * (1.0 - 1e-4);
                    base_hi = msum_all * (1.0 + 1e-4);
                }
            }
            Sync::sync();
            // Cumulative bounds in bin order, a run of consecutive bins per thread.  An element of
            // bin b has its mass in (2^-edge(b+1), 2^-edge(b)], edge(b) = d0 + b / scale; the factor
            // 1e-3 covers the rounding of d.  b_hi: first bin at which the upper bound of the mass so
            // far reaches the lowest possible target; b_lo: first bin at which the lower bound
            // reaches the highest possible target.
            constexpr int PERB = (WB + NT - 1) / NT;
            const int b0 = min(tid * PERB, nall), b1 = min(b0 + PERB, nall);
            double s_lo = 0.0, s_hi = 0.0;
            int s_c = 0;
            for (int b = b0; b < b1; ++b) {
                const int c = wbc[b];
                s_hi += (double)c * (double)ex2_approx(-wedge(b, wb));
                s_lo += (double)c * (double)ex2_approx(-wedge(b + 1, wb));
                s_c += c;
            }
            double tot_lo, tot_hi;
            int tot_c;
            const double run_lo0 = base_lo + block_excl_scan_d(s_lo, tot_lo);
            const double run_hi0 = base_hi + block_excl_scan_d(s_hi, tot_hi);
            const int run_c0 = base_c + block_excl_scan_i(s_c, tot_c);
            const double Z_lo = Zf * (1.0 - 1e-4), Z_hi = Zf * (1.0 + 1e-4);      // (the fp32 sum of every mass)
            if (nfin < 0) nfin = base_c + tot_c + tail_c;
            if (base_c + tot_c + tail_c != nfin) return 0;
            if (tid == 0) { sm.b_i[0] = INT_MAX; sm.b_i[1] = INT_MAX; sm.b_i[2] = -1; sm.b_i[3] = -1; }
            Sync::sync();
            const double t_lo = top_p * Z_lo * (1.0 - 1e-3), t_hi = top_p * Z_hi * (1.0 + 1e-3);
            {
                double r_lo = run_lo0, r_hi = run_hi0;
                int first_hi = INT_MAX, first_lo = INT_MAX, last = -1;
                for (int b = b0; b < b1; ++b) {
                    const int c = wbc[b];
                    if (c > 0) {
                        r_hi += (double)c * (double)ex2_approx(-wedge(b, wb));
                        r_lo += (double)c * (double)ex2_approx(-wedge(b + 1, wb));
                        if (first_hi == INT_MAX && r_hi >= t_lo) first_hi = b;
                        if (first_lo == INT_MAX && r_lo >= t_hi) first_lo = b;
                        last = b;
                    }
                }
                if (first_hi != INT_MAX) atomicMin(&sm.b_i[0], first_hi);
                if (first_lo != INT_MAX) atomicMin(&sm.b_i[1], first_lo);
                if (last >= 0) atomicMax(&sm.b_i[2], last);
            }
            Sync::sync();
            const int bhi = sm.b_i[0];
            int blo = sm.b_i[1];
            const int last_bin = sm.b_i[2];
            Sync::sync();
            if (bhi == INT_MAX) return 0;               // the nucleus ends past the bins
            if (blo == INT_MAX) {
                if (tail_c > 0) return 0;               // ... or may do so
                blo = last_bin;                         // the target sits at the very end of the mass
            }
            // counts at the bracket's two ends
            {
                int c_run = run_c0;
                for (int b = b0; b < b1; ++b) {
                    if (b == bhi) sm.b_i[2] = c_run;
                    c_run += wbc[b];
                    if (b == blo) sm.b_i[3] = c_run;
                }
            }
            Sync::sync();
            n_in = sm.b_i[2];
            const int thru_c = sm.b_i[3];
            n_br = thru_c - n_in;
            Sync::sync();                               // the bins are dead from here
            if (thru_c < 0 || blo < bhi || n_br < 1) return 0;
            wb.bhi = bhi;
            wb.blo = blo;
            if (n_br <= WCAP) break;
            if (level == 1) return 0;
            // finer bins over the bracket's range: the largest power-of-two scale under which it fits
            const float w_lo = wedge(bhi, wb), w_hi = wedge(blo + 1, wb);
            const float width = w_hi - w_lo;
            float sc = 1.f;
            while (width * (sc * 2.f) <= (float)WB && sc < 16777216.f) sc *= 2.f;
            if (sc <= wb.scale) return 0;               // (cannot be refined)
            tail_c = nfin - thru_c;
            base_c = n_in;                              // (their mass: summed in the next pass)
            wb.d0 = w_lo;
            wb.scale = sc;
            wb.nfine = (int)ceilf(width * sc);          // exactly the bracket's range
            wb.bhi = 0; wb.blo = 0;
        }

        // The classes as key thresholds (the class is a monotone function of the key): K0 the smallest
        // key above the bracket, K1 the smallest key not below it; two integer compares per element
        // instead of the depth arithmetic.
        uint32_t K0, K1;
        {
            auto first_key = [&](int cls_max) -> uint32_t {     // smallest key of class <= cls_max
                if (wclass(wdepth(row_kmax, lmax_f, s2), wb) > cls_max) return row_kmax + 1u;
                uint32_t lo = Tr::KEY_NINF + 1u, hi = row_kmax;   // class(hi) <= cls_max
                while (lo < hi) {
                    const uint32_t mid = lo + ((hi - lo) >> 1);
                    if (wclass(wdepth(mid, lmax_f, s2), wb) <= cls_max) hi = mid; else lo = mid + 1u;
                }
                return hi;
            };
            K0 = first_key(0);
            K1 = first_key(1);
        }

        // ---- C. exact masses: chunk sums of the elements above the bracket, Z's part below it,
        //         the bracket's elements listed
        clear_has();
        if (tid == 0) sm.b_u[0] = 0u;
        for (int i = tid; i < MAXCH; i += NT) { acc_hi[i] = 0ull; acc_lo[i] = 0ull; }
        Sync::sync();
        float below_f[4] = {0.f, 0.f, 0.f, 0.f};     // four partial sums: a few hundred terms each
        if (warp < nchunks) {
            const int nq = ((nchunks - warp + NW - 1) / NW) * R;      // this warp's vectors, chunk by chunk
            auto vi_of = [&](int q) -> int { return ((warp + (q / R) * NW) * R + q % R) * 32 + lane; };
            auto fetch = [&](int q, uint4& raw, bool& is_raw) {
                is_raw = false;
                if (q < nq) {
                    const int vi = vi_of(q);
                    if (vec_ok && (vi + 1) * E <= V) {
                        raw = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) + (size_t)vi * 16);
                        is_raw = true;
                    }
                }
            };
            constexpr int G = 4;                          // vectors in flight per lane
            double local = 0.0;
            for (int q0 = 0; q0 < nq; q0 += G) {
                uint4 raw[G];
                bool is_raw[G];
#pragma unroll
                for (int g = 0; g < G; ++g) fetch(q0 + g, raw[g], is_raw[g]);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const int q = q0 + g;
                    if (q < nq) {
                        const int vi = vi_of(q);
                        uint32_t k[E];
                        if (is_raw[g]) {
                            Tr::unpack(raw[g], k);
                        } else if (vi < nvec) {
                            load_vec_keys<DT>(row, V, vi, vec_ok, k);
                        } else {
#pragma unroll
                            for (int e = 0; e < E; ++e) k[e] = Tr::KEY_NINF;
                        }
                        unsigned in_mask = 0;
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            const uint32_t ke = k[e];
                            if (ke >= K0) {
                                in_mask |= 1u << e;
                            } else if (ke >= K1) {
                                const unsigned slot = atom_shared_add(&sm.b_u[0], 1u);
                                if (slot < (unsigned)WCAP)
                                    wcand[slot] = ((unsigned long long)ke << 32) | (uint32_t)~(uint32_t)(vi * E + e);
                            } else if (ke > Tr::KEY_NINF) {
                                below_f[e & 3] += ex2_approx(-wdepth(ke, lmax_f, s2));   // fp32 first: see the decision below
                            }
                        }
                        // fp64 masses of the kept ones, one per round: a lane rarely has more than one in a
                        // vector, and the warp runs as many rounds as its busiest lane
                        while (in_mask) {
                            const int e0 = __ffs(in_mask) - 1;
                            in_mask &= in_mask - 1;
                            uint32_t ks = k[0];
#pragma unroll
                            for (int e = 1; e < E; ++e) if (e0 == e) ks = k[e];
                            local += mass(ks);
                        }
                        if (q % R == R - 1) {
                            local = warp_sum_d(local);
                            if (lane == 0) put_chunk(warp + (q / R) * NW, local);
                            local = 0.0;
                        }
                    }
                }
            }
        }
        double below = ((double)below_f[0] + (double)below_f[1]) + ((double)below_f[2] + (double)below_f[3]);
        below = warp_sum_d(below);
        if (lane == 0) sm.red_d[warp] = below;
        Sync::sync();
        if ((int)sm.b_u[0] != n_br) return 0;           // (cannot happen: same function of the same keys)
        double S_out = 0.0;
#pragma unroll
        for (int w = 0; w < NW; ++w) S_out += sm.red_d[w];
        // S_in by warp 0, lanes over the chunks in a fixed order
        if (warp == 0) {
            double s_in = 0.0;
            for (int ci = lane; ci < nchunks; ci += 32) s_in += sm.chunk_sum[ci];
            s_in = warp_sum_d(s_in);
            if (lane == 0) sm.b_d[2] = s_in;
        }
        // ---- the bracket's elements in rank order: bitonic sort, descending, padded with zeros
        int P = 32;
        while (P < n_br) P <<= 1;
        for (int i = n_br + tid; i < P; i += NT) wcand[i] = 0ull;
        Sync::sync();
        for (int kk = 2; kk <= P; kk <<= 1) {
            for (int j = kk >> 1; j > 0; j >>= 1) {
                for (int i = tid; i < P / 2; i += NT) {
                    const int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1)), hi = lo | j;
                    const bool desc = (lo & kk) == 0;
                    const unsigned long long x = wcand[lo], y = wcand[hi];
                    if ((x < y) == desc) { wcand[lo] = y; wcand[hi] = x; }
                }
                Sync::sync();
            }
        }
        const double S_in = sm.b_d[2];
        // exact prefix masses in rank order: `per` consecutive ranks per thread
        const int per = (P + NT - 1) / NT;               // 1..4
        double mloc[4] = {0.0, 0.0, 0.0, 0.0};
        double lsum = 0.0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = tid * per + i;
            if (i < per && j < n_br) { mloc[i] = mass((uint32_t)(wcand[j] >> 32)); lsum += mloc[i]; }
        }
        const double wincl = warp_incl_scan_d(lsum, lane);
        if (lane == 31) sm.red_d[warp] = wincl;
        if (tid == 0) { sm.b_i[0] = INT_MAX; sm.b_i[1] = 0; sm.b_i[2] = 0; }
        Sync::sync();
        double off = 0.0, S_br = 0.0;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            if (w < warp) off += sm.red_d[w];
            S_br += sm.red_d[w];
        }
        double before[4];
        {
            double run = S_in + (off + (wincl - lsum));  // exact prefix before this thread's ranks
#pragma unroll
            for (int i = 0; i < 4; ++i) { before[i] = run; run += mloc[i]; }
        }
        // The part of Z below the bracket came from fp32 masses (relative error under 4e-5): good
        // enough unless a prefix lies that close to the target; then that part is summed again in
        // fp64 and the decision repeated.  Within rounding of fp64 sums the radix select decides.
        double out_tol = S_out * 4e-5;
        int r;
        double pre_r, incl_r;
        uint32_t T;
        for (int attempt = 0;; ++attempt) {
            const double Z = (S_in + S_br) + S_out;
            const double target = top_p * Z;
            const double tol = Z * 1e-13 + top_p * out_tol;
            Sync::sync();
            if (tid == 0) sm.b_i[0] = INT_MAX;
            Sync::sync();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = tid * per + i;
                if (i < per && j < n_br && before[i] + mloc[i] >= target) atomicMin(&sm.b_i[0], j);
            }
            Sync::sync();
            r = sm.b_i[0];
            bool again = (r == INT_MAX);         // the sums do not reach the target inside the bracket
            if (!again) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int j = tid * per + i;
                    if (i < per && j == r) {
                        sm.b_d[0] = before[i];
                        sm.b_d[1] = before[i] + mloc[i];
                        sm.b_u[1] = (uint32_t)(wcand[j] >> 32);
                    }
                }
                Sync::sync();
                pre_r = sm.b_d[0]; incl_r = sm.b_d[1]; T = sm.b_u[1];
                again = incl_r - target < tol || target - pre_r < tol;
            }
            if (!again) break;
            if (attempt == 1 || out_tol == 0.0) return 0;
            // the masses below the bracket once more, in fp64 (below 2^-40 of the maximum an fp32
            // mass is exact enough by any count)
            double ex = 0.0;
            constexpr int U = 4;
            for (int v0 = tid; v0 < nvec; v0 += U * NT) {
                uint32_t k[U][E];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int vi = v0 + u * NT;
                    if (vi < nvec) {
                        load_vec_keys<DT>(row, V, vi, vec_ok, k[u]);
                    } else {
#pragma unroll
                        for (int e = 0; e < E; ++e) k[u][e] = Tr::KEY_NINF;
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        if (k[u][e] > Tr::KEY_NINF && k[u][e] < K1) {
                            const float d = wdepth(k[u][e], lmax_f, s2);
                            ex += d < 40.f ? mass(k[u][e]) : (double)ex2_approx(-d);
                        }
                    }
                }
            }
            ex = warp_sum_d(ex);
            Sync::sync();
            if (lane == 0) sm.red_d[warp] = ex;
            Sync::sync();
            S_out = 0.0;
#pragma unroll
            for (int w = 0; w < NW; ++w) S_out += sm.red_d[w];
            out_tol = 0.0;
        }
        Sync::sync();
        if (tid == 0) { sm.b_i[1] = 0; sm.b_i[2] = 0; }
        Sync::sync();
        {
            int eq = 0, need = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = tid * per + i;
                if (i < per && j < n_br && (uint32_t)(wcand[j] >> 32) == T) { ++eq; need += (j <= r); }
            }
            eq = warp_sum_i(eq);
            need = warp_sum_i(need);
            if (lane == 0 && eq) { atomicAdd(&sm.b_i[1], eq); atomicAdd(&sm.b_i[2], need); }
        }
        // ---- kept elements of the bracket join their chunks' sums: two 64-bit fixed-point parts per
        //      chunk, so that the sums do not depend on the order in which the additions arrive
        const double m_top = mass((uint32_t)(wcand[0] >> 32));
        const int ex_top = ((int)(__double2hiint(m_top) >> 20) & 0x7FF) - 1023;     // m_top in [2^ex, 2^(ex+1))
        const double sc = __hiloint2double((1023 + 50 - ex_top) << 20, 0);          // m_top * sc in [2^50, 2^51)
        const bool sc_ok = m_top > 0.0 && ex_top > -900;
        if (sc_ok) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = tid * per + i;
                if (i < per && j <= r && j < n_br) {
                    const double f = mloc[i] * sc;                                   // < 2^51
                    const unsigned long long hi = (unsigned long long)f;             // (truncates)
                    const unsigned long long lo = (unsigned long long)((f - (double)hi) * 4503599627370496.0);   // * 2^52
                    const int ci = chunk_of_index((int)~(uint32_t)wcand[j]);
                    red_shared_add(&acc_hi[ci], hi);
                    red_shared_add(&acc_lo[ci], lo);
                }
            }
        }
        Sync::sync();
        if (!sc_ok) return 0;
        const int eq_all = sm.b_i[1], need_all = sm.b_i[2];
        for (int ci = tid; ci < nchunks; ci += NT) {
            const unsigned long long hi = acc_hi[ci], lo = acc_lo[ci];
            if (hi | lo) {
                const double add = ((double)hi + (double)lo * (1.0 / 4503599627370496.0)) / sc;
                sm.chunk_sum[ci] += add;
                if (add > 0.0) red_shared_or(&sm.chunk_has[ci >> 5], 1u << (ci & 31));
            }
        }
        Sync::sync();
        p.T = T;
        p.need = need_all;
        p.eq_mode = need_all < eq_all ? 2 : 1;
        n_kept = n_in + r + 1;
        if (p.eq_mode == 2) {
            // chunk_eq[ci] <- elements equal to T in the chunks before ci: all of them are in the list
            for (int ci = tid; ci <= nchunks; ci += NT) sm.chunk_eq[ci] = 0;
            Sync::sync();
            for (int j = tid; j < n_br; j += NT)
                if ((uint32_t)(wcand[j] >> 32) == T) atomicAdd(&sm.chunk_eq[chunk_of_index((int)~(uint32_t)wcand[j])], 1);
            Sync::sync();
            scan_exclusive(sm.chunk_eq, nchunks);
        }
        scan_exclusive(sm.chunk_sum, nchunks);
        return 1;
    }

    // pass 1: the row's largest key, whether it is a usable row, its finite count
    __device__ int extremes(unsigned& kmax_out, int& nfin_out) {
        GenericSmem<NT>& sm = this->sm;              // (locals: see nucleus_by_bins)
        const void* const row = this->row;
        const int V = this->V, nvec = this->nvec, tid = this->tid, lane = this->lane, warp = this->warp;
        const bool vec_ok = this->vec_ok;
        unsigned kmax = 0, kmin = 0xFFFFFFFFu;
        int nfin = 0;
        {
            constexpr int U = 4;                       // loads in flight per thread
            for (int v0 = tid; v0 < nvec; v0 += U * NT) {
                uint32_t k[U][E];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int vi = v0 + u * NT;
                    if (vi < nvec) {
                        load_vec_keys<DT>(row, V, vi, vec_ok, k[u]);
                    } else {
#pragma unroll
                        for (int e = 0; e < E; ++e) k[u][e] = Tr::KEY_NINF;   // (a masked token: allowed, not counted)
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        kmax = max(kmax, k[u][e]);
                        kmin = min(kmin, k[u][e]);
                        nfin += (k[u][e] > Tr::KEY_NINF);
                    }
                }
            }
        }
        kmax = warp_max_u(kmax);
        kmin = warp_min_u(kmin);
        nfin = warp_sum_i(nfin);
        if (lane == 0) { sm.red_u[warp] = kmax; sm.red_u2[warp] = kmin; sm.red_i[warp] = nfin; }
        Sync::sync();
        kmax = 0; kmin = 0xFFFFFFFFu; nfin = 0;
        for (int w = 0; w < NW; ++w) {
            kmax = max(kmax, sm.red_u[w]);
            kmin = min(kmin, sm.red_u2[w]);
            nfin += sm.red_i[w];
        }
        Sync::sync();
        kmax_out = kmax;
        nfin_out = nfin;
        if (kmin < Tr::KEY_NINF || kmax >= Tr::KEY_PINF || kmax == Tr::KEY_NINF) return ST_NUMERIC;
        return ST_OK;
    }

    // A caller that has already been over the row (every element finite or masked, not all masked)
    // hands over its largest key; the nucleus through bins then starts without pass 1.
    bool have_kmax = false;
    uint32_t known_kmax = 0;
    uint32_t row_kmax = 0;                     // the row's largest key, once known

    // Steps 1-4 of the general routine: the kept set as a predicate `p`, its size, and in
    // chunk_sum the exclusive scan of the kept masses per chunk (chunk_sum[nchunks] = Z).
    // Needs inv_tau set and the exp table filled; returns ST_OK or ST_NUMERIC.
    __device__ __forceinline__ int prepare(int top_k, double top_p, Pred& p, int& n_kept, double typical_p = 1.0) {
        const bool nucleus_only = top_k <= 0 && top_p > 0.0 && top_p < 1.0 && !(typical_p > 0.0 && typical_p < 1.0);
        unsigned kmax = 0;
        int nfin = -1;
        if (bins && nucleus_only && have_kmax) {
            // ---- nucleus without a top-k, maximum known: the value bins settle most rows in two passes
            lmax = (double)Tr::value_f(known_kmax);
            row_kmax = known_kmax;
            if (nucleus_by_bins(top_p, nfin, p, n_kept)) return ST_OK;
            Sync::sync();
        }
        // ---- 1. extremes and finite count
        if (extremes(kmax, nfin) != ST_OK) return ST_NUMERIC;
        lmax = (double)Tr::value_f(kmax);
        row_kmax = kmax;

        p.T = Tr::KEY_NINF; p.need = 0; p.eq_mode = 0;     // every finite logit
        n_kept = nfin;

        // ---- 2. top-k
        if (top_k > 0 && top_k < nfin) {
            uint32_t prefix = 0, mask = 0;
            int acc = 0, eq = 0;
            for (int shift = Tr::KEYBITS - 8; shift >= 0; shift -= 8) {
                hist_pass<false>(p, prefix, mask, shift);
                choose_digit<false>(acc, 0.0, top_k, 0.0);
                prefix |= (uint32_t)sm.b_i[0] << shift;
                mask |= 0xFFu << shift;
                acc = sm.b_i[1];
                eq = sm.b_i[2];
                Sync::sync();
            }
            p.T = prefix;
            p.need = top_k - acc;
            p.eq_mode = (p.need < eq) ? 2 : 1;
            n_kept = top_k;
            if (p.eq_mode == 2) tie_prepass(p.T);
        }

        // ---- nucleus without a top-k: the value bins settle most rows in two passes
        if (bins && !have_kmax && !(top_k > 0 && top_k < nfin) && top_p > 0.0 && top_p < 1.0 && !(typical_p > 0.0 && typical_p < 1.0)) {
            if (nucleus_by_bins(top_p, nfin, p, n_kept)) return ST_OK;
            Sync::sync();
            p.T = Tr::KEY_NINF; p.need = 0; p.eq_mode = 0;
            n_kept = nfin;
        }

        // ---- 3. masses of the kept set
        sum_pass(p);
        scan_exclusive(sm.chunk_sum, nchunks);

        // ---- 3b. locally typical cut on the distribution over the survivors (it takes the
        //          nucleus's place): tokens ordered by |y - mu| ascending, mu = sum p_j y_j
        if (typical_p > 0.0 && typical_p < 1.0) {
            typical_cut(p, typical_p, n_kept);
            sum_pass(p);
            scan_exclusive(sm.chunk_sum, nchunks);
            return ST_OK;
        }

        // ---- 4. nucleus on the distribution renormalised over the survivors
        if (top_p > 0.0 && top_p < 1.0) {
            const double target = top_p * sm.chunk_sum[nchunks];
            Sync::sync();
            uint32_t prefix = 0, mask = 0;
            int acc_c = 0, eq = 0;
            double acc_m = 0.0;
            for (int shift = Tr::KEYBITS - 8; shift >= 0; shift -= 8) {
                hist_pass<true>(p, prefix, mask, shift);
                choose_digit<true>(acc_c, acc_m, 0, target);
                prefix |= (uint32_t)sm.b_i[0] << shift;
                mask |= 0xFFu << shift;
                acc_c = sm.b_i[1];
                eq = sm.b_i[2];
                acc_m = sm.b_d[0];
                Sync::sync();
            }
            // `eq` kept elements share the threshold key and the same mass e_P: take the
            // fewest of them (lowest indices) that bring the mass to the target
            const double e_P = mass(prefix);
            long long r = (long long)ceil((target - acc_m) / e_P);
            if (r < 1) r = 1;
            if (r > eq) r = eq;
            while (r > 1 && acc_m + (double)(r - 1) * e_P >= target) --r;
            while (r < eq && acc_m + (double)r * e_P < target) ++r;
            const int n_new = acc_c + (int)r;
            if (n_new != n_kept) {
                const bool same_ranked = (prefix == p.T && p.eq_mode == 2);
                if ((int)r < eq) {
                    p.eq_mode = 2;
                    p.need = (int)r;
                } else if (prefix != p.T) {
                    p.eq_mode = 1;
                }
                p.T = prefix;
                n_kept = n_new;
                if (p.eq_mode == 2 && !same_ranked) tie_prepass(p.T);
                sum_pass(p);
                scan_exclusive(sm.chunk_sum, nchunks);
            }
        }

        return ST_OK;
    }

    __device__ __noinline__ LaneResult run(double c_in, double inv_tau_, int top_k, double top_p, double typical_p = 1.0) {
        const bool typical = typical_p > 0.0 && typical_p < 1.0;
        if (top_k <= 0 && !(top_p > 0.0 && top_p < 1.0) && !typical && vec_ok) return run_nocut(c_in, inv_tau_);
        inv_tau = inv_tau_;
        fill_exp_table(sm.exp_tbl, tid);
        double c = c_in;
        const bool code_bad = !(c >= 0.0 && c <= 1.0);
        if (c == 1.0) c = ASX_ONE_BELOW;
        Pred p;
        int n_kept;
        if (prepare(top_k, top_p, p, n_kept, typical_p) != ST_OK || code_bad) return fail(c_in, ST_NUMERIC);

        // ---- 5/6. locate the chunk, then the element
        const double Z = sm.chunk_sum[nchunks];
        const double t = c * Z;
        if (tid == 0) { sm.b_i[0] = INT_MAX; sm.b_i[1] = -1; }
        Sync::sync();
        for (int ci = tid; ci < nchunks; ci += NT) {
            if (has_mass(ci)) {
                atomicMax(&sm.b_i[1], ci);
                if (t < sm.chunk_sum[ci + 1]) atomicMin(&sm.b_i[0], ci);
            }
        }
        Sync::sync();
        const bool force_last = (sm.b_i[0] == INT_MAX);
        const int cstar = force_last ? sm.b_i[1] : sm.b_i[0];

        if (warp == 0) {
            double run = sm.chunk_sum[ASX_AT(cstar, MAXCH + 1, 84)];
            int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[cstar] : 0;
            int tie_run2 = (tp.on && tp.eq_mode == 2) ? sm.chunk_eq2[cstar] : 0;
            int last_idx = -1;
            double last_S = 0.0, last_e = 1.0;
            int tok = -1;
            double tok_S = 0.0, tok_e = 1.0;
            for (int r = 0; r < R && tok < 0; ++r) {
                uint32_t k[E];
                int base;
                chunk_keys(cstar, r, k, base);
                const unsigned bits = kept_all(k, p, tie_run, tie_run2);
                double ev[E];
                double local = 0.0;
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    ev[e] = (bits & (1u << e)) ? mass(k[e]) : 0.0;
                    local += ev[e];
                }
                const double incl = warp_incl_scan_d(local, lane);
                double excl = __shfl_up_sync(FULL, incl, 1);
                if (lane == 0) excl = 0.0;
                int pick = -1;
                double pick_S = 0.0, pick_e = 1.0;
                if (bits) {
                    double S = run + excl;
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        if (bits & (1u << e)) {
                            if (pick < 0 && t < S + ev[e]) { pick = base + e; pick_S = S; pick_e = ev[e]; }
                            last_idx = base + e; last_S = S; last_e = ev[e];
                            S += ev[e];
                        }
                    }
                }
                const bool cross = !force_last && bits && (t < run + incl);
                const unsigned bal = __ballot_sync(FULL, cross);
                if (bal) {
                    const int L = __ffs(bal) - 1;
                    if (pick < 0) { pick = last_idx; pick_S = last_S; pick_e = last_e; }
                    tok = __shfl_sync(FULL, pick, L);
                    tok_S = __shfl_sync(FULL, pick_S, L);
                    tok_e = __shfl_sync(FULL, pick_e, L);
                }
                run += __shfl_sync(FULL, incl, 31);
            }
            if (tok < 0) {   // rounding at the top end: the last kept element of the chunk
                const unsigned best = warp_max_u((unsigned)(last_idx + 1));
                const unsigned bal = __ballot_sync(FULL, (unsigned)(last_idx + 1) == best);
                const int L = __ffs(bal) - 1;
                tok = __shfl_sync(FULL, last_idx, L);
                tok_S = __shfl_sync(FULL, last_S, L);
                tok_e = __shfl_sync(FULL, last_e, L);
            }
            if (lane == 0) {
                double cn = (t - tok_S) / tok_e;
                if (!(cn >= 0.0)) cn = 0.0;
                if (cn > ASX_ONE_BELOW) cn = ASX_ONE_BELOW;
                LaneResult r;
                r.token = tok; r.status = tok < 0 ? ST_NUMERIC : ST_OK; r.n_kept = n_kept;
                r.code_out = tok < 0 ? c_in : cn;
                r.p_tok = tok_e / Z;
                r.cdf_lo = tok_S / Z;
                sm.res = r;
            }
        }
        Sync::sync();
        const LaneResult out = sm.res;
        Sync::sync();
        return out;
    }

    // One step with an extended-precision code: the token that owns cell `tcell` of the 2^32 cells
    // of this step's CDF over the kept set (any cut), with its cells in sm.xp_lo / sm.xp_hi.
    __device__ __noinline__ LaneResult run_xp(unsigned long long tcell, double inv_tau_, int top_k, double top_p) {
        inv_tau = inv_tau_;
        fill_exp_table(sm.exp_tbl, tid);
        Pred p;
        int n_kept;
        if (prepare(top_k, top_p, p, n_kept) != ST_OK) return fail(0.0, ST_NUMERIC);
        if (warp == 0) {
            const double Z = sm.chunk_sum[nchunks];
            const double K = 4294967296.0 / Z;
            int last_c = -1;
            for (int ci = lane; ci < nchunks; ci += 32)
                if (has_mass(ci)) last_c = ci;
            last_c = (int)warp_max_u((unsigned)(last_c + 1)) - 1;
            int tok = -1;
            unsigned long long plo = 0, phi = 0;
            double pe = 1.0;
            if (last_c >= 0) {
                int first = INT_MAX;
                for (int ci = lane; ci <= last_c; ci += 32) {
                    const unsigned long long fe = ci == last_c ? XP_TOP : xp_cell(sm.chunk_sum[ci + 1], K);
                    if (fe > tcell && has_mass(ci)) first = min(first, ci);
                }
                const int cstar = (int)warp_min_u((unsigned)first);
                const unsigned long long Fend = cstar == last_c ? XP_TOP : xp_cell(sm.chunk_sum[cstar + 1], K);
                // masses of sub-row r of the chunk (kept elements only)
                auto sub_masses = [&](int r, int& tie_run, double (&ev)[E], int& base) {
                    uint32_t k[E];
                    chunk_keys(cstar, r, k, base);
                    const int rank0 = lane_rank0(k, p, tie_run);
                    const unsigned bits = kept_bits(k, p, rank0);
#pragma unroll
                    for (int e = 0; e < E; ++e) ev[e] = (bits & (1u << e)) ? mass(k[e]) : 0.0;
                };
                // the last sub-row of the chunk that holds mass
                int r_last = 0;
                {
                    int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[cstar] : 0;
                    for (int r = 0; r < R; ++r) {
                        double ev[E];
                        int base;
                        sub_masses(r, tie_run, ev, base);
                        double local = 0.0;
#pragma unroll
                        for (int e = 0; e < E; ++e) local += ev[e];
                        if (__ballot_sync(FULL, local > 0.0)) r_last = r;
                    }
                }
                double run = sm.chunk_sum[cstar];
                // the chunk starts in the cell where the chunk with mass before it ended
                int prev_c = -1;
                for (int ci = lane; ci < cstar; ci += 32)
                    if (has_mass(ci)) prev_c = ci;
                prev_c = (int)warp_max_u((unsigned)(prev_c + 1)) - 1;
                unsigned long long carry = prev_c < 0 ? 0ull : xp_cell(sm.chunk_sum[prev_c + 1], K);
                int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[cstar] : 0;
                for (int r = 0; r <= r_last && tok < 0; ++r) {
                    double ev[E];
                    int base;
                    sub_masses(r, tie_run, ev, base);
                    int pk = 0;
                    const int L = xp_subrow<E>(ev, lane, K, tcell, r == r_last, Fend, run, carry, pk, plo, phi, pe);
                    if (L >= 0) tok = __shfl_sync(FULL, base, L) + pk;
                }
            }
            if (lane == 0) {
                LaneResult r;
                r.token = tok; r.status = tok < 0 ? ST_NUMERIC : ST_OK; r.n_kept = n_kept;
                r.code_out = 0.0;
                r.p_tok = pe / sm.chunk_sum[nchunks];
                r.cdf_lo = (double)plo * (1.0 / 4294967296.0);
                sm.xp_lo = plo; sm.xp_hi = phi;
                sm.res = r;
            }
        }
        Sync::sync();
        const LaneResult out = sm.res;
        Sync::sync();
        return out;
    }

    // interval_of for lanes without top-k / nucleus on 16-byte aligned rows: a packed max pass,
    // then one pass that sums every mass and, separately, the masses below the token.
    __device__ __noinline__ LaneResult interval_nocut(int tok, double inv_tau_) {
        using P = Pass<DT>;
        inv_tau = inv_tau_;
        fill_exp_table(sm.exp_tbl, tid);
        typename P::Acc acc = P::init();
        float vmn = __uint_as_float(0x7F800000u);
        const int nvf = (V * Tr::BYTES) >> 4;
        for (int vi = tid; vi < nvf; vi += NT) {
            const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) + (size_t)vi * 16);
            P::merge(acc, P::reduce(q));
            vmn = fminf(vmn, P::vmin(q));
        }
        for (int j = nvf * E + tid; j < V; j += NT) {
            P::fold_scalar(acc, row, j);
            vmn = fminf(vmn, P::load_f(row, j));
        }
        uint32_t k0, k1;
        P::keys(acc, k0, k1);
        uint32_t kmax = warp_max_u(max(k0, k1));
        uint32_t kmin = warp_min_u(P::key_of_f(vmn));
        if (lane == 0) { sm.red_u[warp] = kmax; sm.red_u2[warp] = kmin; }
        Sync::sync();
        kmax = 0; kmin = 0xFFFFFFFFu;
        for (int w = 0; w < NW; ++w) { kmax = max(kmax, sm.red_u[w]); kmin = min(kmin, sm.red_u2[w]); }
        if (kmax >= Tr::KEY_PINF || kmax <= Tr::KEY_NINF) {
            Sync::sync();
            return fail(0.0, ST_NUMERIC);
        }
        lmax = (double)Tr::value_f(kmax);
        const double s64 = inv_tau * 0x1.71547652b82fep+6;          // 64 log2(e) / temp
        const double c64 = -lmax * s64;
        // plain rows (no masked token, nothing below 2^-1000 of the largest mass): no underflow guard,
        // every token counts, and whole vectors on one side of the token need no per-element test
        const bool plain = kmin > Tr::KEY_NINF && fma((double)Tr::value_f(kmin), s64, c64) >= -64000.0;
        double all = 0.0, below = 0.0, e_tok = 0.0;
        int has = 0, nfin = 0;
        for (int vi = tid; vi < nvec; vi += NT) {
            float x[E];
            const int base = vi * E;
            if (plain && base + E <= V && (base + E <= tok || base > tok)) {
                const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) + (size_t)base * Tr::BYTES);
                P::floats(q, x);
                double vsum = 0.0;
#pragma unroll
                for (int e = 0; e < E; ++e) vsum += exp2_64th<false>(fma((double)x[e], s64, c64), sm.exp_tbl);
                all += vsum;
                if (base < tok) below += vsum;
                nfin += E;
                continue;
            }
            if (base + E <= V) {
                const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) + (size_t)base * Tr::BYTES);
                P::floats(q, x);
            } else {
#pragma unroll
                for (int e = 0; e < E; ++e)
                    x[e] = (base + e < V) ? P::load_f(row, base + e) : __uint_as_float(0xFF800000u);
            }
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const double m = exp2_64th(fma((double)x[e], s64, c64), sm.exp_tbl);
                const bool fin = x[e] > __uint_as_float(0xFF800000u);
                all += m;
                nfin += fin;
                if (base + e < tok) below += m;
                if (base + e == tok && fin) { e_tok = m; has = 1; }
            }
        }
        all = warp_sum_d(all);
        below = warp_sum_d(below);
        e_tok = warp_sum_d(e_tok);
        has = warp_sum_i(has);
        nfin = warp_sum_i(nfin);
        if (lane == 0) {
            sm.hist_mass[warp] = all;
            sm.hist_mass[NW + warp] = below;
            sm.hist_mass[2 * NW + warp] = e_tok;
            sm.hist_cnt[warp] = has;
            sm.hist_cnt[NW + warp] = nfin;
        }
        Sync::sync();
        LaneResult r;
        {
            double Z = 0.0, S = 0.0, et = 0.0;
            int h = 0, n = 0;
            for (int w = 0; w < NW; ++w) {
                Z += sm.hist_mass[w];
                S += sm.hist_mass[NW + w];
                et += sm.hist_mass[2 * NW + w];
                h += sm.hist_cnt[w];
                n += sm.hist_cnt[NW + w];
            }
            const bool kept = h > 0;
            r.token = kept ? tok : -1; r.status = kept ? ST_OK : ST_NUMERIC; r.n_kept = n;
            r.code_out = 0.0;
            r.p_tok = et / Z;
            r.cdf_lo = S / Z;
        }
        Sync::sync();
        return r;
    }

    // The other direction of one step (the codebook of Sec. 4.1 read from token to interval):
    // for a given token, cdf_lo = F_{tok-1} and p_tok under the same modified distribution.
    // A token outside the kept set (probability zero) gives ST_NUMERIC.
    __device__ __noinline__ LaneResult interval_of(int tok, double inv_tau_, int top_k, double top_p) {
        if (top_k <= 0 && !(top_p > 0.0 && top_p < 1.0) && vec_ok) return interval_nocut(tok, inv_tau_);
        inv_tau = inv_tau_;
        fill_exp_table(sm.exp_tbl, tid);
        Pred p;
        int n_kept;
        if (prepare(top_k, top_p, p, n_kept) != ST_OK) return fail(0.0, ST_NUMERIC);
        const double Z = sm.chunk_sum[nchunks];
        const int vi_tok = tok / E;
        const int cstar = (vi_tok >> 5) / R;
        if (warp == 0) {
            double below = 0.0, e_tok = 0.0;
            int has = 0;
            int tie_run = (p.eq_mode == 2) ? sm.chunk_eq[cstar] : 0;
            for (int r = 0; r < R; ++r) {
                if ((cstar * R + r) * 32 * E > tok) break;      // warp-uniform: rows past the token
                uint32_t k[E];
                int base;
                chunk_keys(cstar, r, k, base);
                const int rank0 = lane_rank0(k, p, tie_run);
                const unsigned bits = kept_bits(k, p, rank0);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if (bits & (1u << e)) {
                        const double m = mass(k[e]);
                        if (base + e < tok) below += m;
                        if (base + e == tok) { e_tok = m; has = 1; }
                    }
                }
            }
            below = warp_sum_d(below);
            e_tok = warp_sum_d(e_tok);      // one lane holds it, the others add zero
            has = warp_sum_i(has);
            if (lane == 0) {
                LaneResult r;
                const bool kept = has > 0;
                r.token = kept ? tok : -1; r.status = kept ? ST_OK : ST_NUMERIC; r.n_kept = n_kept;
                r.code_out = 0.0;
                r.p_tok = e_tok / Z;
                r.cdf_lo = (sm.chunk_sum[cstar] + below) / Z;
                sm.res = r;
            }
        }
        Sync::sync();
        const LaneResult out = sm.res;
        Sync::sync();
        return out;
    }
};

}  // namespace asx

// Streaming decode step: one CTA per lane for any vocabulary size, no inter-CTA
// communication (lanes are independent: Remark after Proposition 1).
//
// CTA = 8 consumer warps + 1 producer warp.  The producer's lane 0 feeds a ring of
// 16 KB shared-memory stages with bulk async copies (TMA, each into this CTA only; `full`
// mbarrier per stage carries the byte count, `empty` mbarrier per stage collects
// one arrival per consumer warp), running ahead across rows, so HBM reads never
// wait for compute.  Consumers see each row exactly once (Algorithm 1 needs every
// conditional probability once):
//   resident rows (row <= ring): all stages land, one NaN-propagating max pass,
//       one threshold T0, one hit pass from shared memory;
//   streamed rows (row > ring): each 16 KB slice goes shared memory -> registers,
//       the stage is released at once, the slice is folded into the running
//       max and tested against the current T0; T0 is recomputed at slices
//       0, 1, 2, 4, 8, ... and only ever rises.
// T0 is a lower bound on the K0-th largest logit: each warp takes the m-th
// largest (m = ceil(K0 / 8)) of its 64 per-thread subset maxima (warp_select16),
// and T0 is the smallest of the 8 warp values, so at least K0 elements
// are >= T0.  The hot loop costs one packed max and one compare per 16-byte
// vector; a vector holding an element >= T0 is copied (warp-aggregated, one
// atomic per warp) to a small list.  Once per row the listed vectors are
// searched for elements >= the FINAL T0, which also discards what earlier,
// lower thresholds let in.  The epilogue is exact and fp64 on those candidates
// only: rank by (value desc, index asc), top-k, masses, nucleus prefix, index
// order, CDF prefix, crossing, rescale (Algorithm 1: w_i, (m, M),
// c <- (c - m)/(M - m)).  For nucleus-only lanes the masses of everything else
// are summed in fp32 (they only enter the nucleus target top_p * Z1).  Lanes the
// list cannot decide (a nucleus deeper than the list can be made, too many ties)
// are marked and served by deferred_lanes_kernel, launched right after this kernel:
// GenericLane on the row in global memory (L2), four CTAs per SM.
#pragma once
#include "as_staged.cuh"

namespace asx {

constexpr int SK_NT = 256;                 // consumer threads
constexpr int SK_NW = SK_NT / 32;          // consumer warps
constexpr int SK_THREADS = SK_NT + 32;     // + producer warp
constexpr int SK_CAP = 512;                // candidate (element) capacity per lane
constexpr int SK_STAGE_VEC = 1024;         // 16-byte vectors per stage (16 KB)
constexpr int SK_STAGE_BYTES = SK_STAGE_VEC * 16;
constexpr int SK_VPT = SK_STAGE_VEC / SK_NT;   // vectors per consumer thread per slice
constexpr int SK_MAXSTAGES = 12;
constexpr int SK_RES_STAGES = 6;           // rows of up to this many stages (96 KB) stay resident
constexpr int SK_K0_RESIDENT = 256;        // largest top_k served by the list, resident rows
constexpr int SK_K0_STREAMED = 96;         // ... streamed rows (hits grow like K0 ln(V / K0))
constexpr int SK_KP = 48;                  // K0 for nucleus-only lanes

using SyncC = SyncNamed<SK_NT>;

// CAPV: hit-vector capacity per lane (1024 lets three CTAs share an SM; fp32 rows need 2048)
template <int CAPV>
struct StreamSmemT {
    unsigned long long full_bar[SK_MAXSTAGES];
    unsigned long long empty_bar[SK_MAXSTAGES];
    union {
        struct {
            union {
                uint4 cvec[CAPV];                       // hit vectors (dead once extracted)
                struct {
                    unsigned long long srt[SK_CAP + 4];    // candidates by rank
                    double e[SK_CAP];                      // mass by rank
                } rk;
            } v;
            int cidx[CAPV];                             // vector index of each hit vector
            unsigned long long cand[SK_CAP + 4];           // (key << 32) | ~index, any order
        } ep;
    } u;
    double exp_tbl[64];
    double red_d[SK_NW];
    unsigned wmax[2][SK_NW];
    unsigned wsel[2][SK_NW];
    double list_mass;    // epilogue: total mass of the ranked list (nucleus lanes)
    int vec_count;
    int cand_count;
    int poisoned;        // a bounded wait ran out: stop issuing / stop waiting
    unsigned long long xp_lo, xp_hi;   // extended-precision steps: the chosen token's cells
    int prod_done;       // the copy-issuing thread has left; prod_st / prod_round say what it armed
    unsigned prod_st, prod_round;
    int b_i[4];
};

// Programmatic dependent launch.  allow_next: the next kernel on the stream may begin its own
// set-up while this grid still runs.  wait_prev: returns once the kernel before this one has
// completed and its writes are visible (at once if this launch does not overlap anything).
__device__ __forceinline__ void pdl_allow_next() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prev() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// m-th largest (1-based) of the 64 16-bit keys held two per lane, by a search on the value, two
// bits per step: the largest v with count(keys >= v) >= m (0 if fewer than m keys are positive).
// Up to SEL_PEEL_MAX the maximum is taken off the top m times instead.
constexpr int SEL_PEEL_MAX = 12;
__device__ __forceinline__ uint32_t warp_select16(uint32_t a16, uint32_t b16, int m, uint32_t lo16 = 0) {
    // Only an answer above lo16 (the threshold already in force) is of use, and it cannot exceed the
    // warp's maximum: search the bits below their common prefix.  0 = no bound above lo16.
    if (m <= SEL_PEEL_MAX) {
        // small m: take the maximum off the top m times (one redux and one ballot per round, against
        // six ballots per two bits of the search below); duplicates count once each, as they must
        uint32_t v = 0;
#pragma unroll 1
        for (int r = 0; r < m; ++r) {
            const uint32_t mx = max(a16, b16);
            v = warp_max_u(mx);
            if (v <= lo16) return 0;             // (also: fewer than m positive keys)
            const int owner = __ffs(__ballot_sync(FULL, mx == v)) - 1;
            if ((int)(threadIdx.x & 31) == owner) { if (a16 == v) a16 = 0; else b16 = 0; }
        }
        return v;
    }
    const uint32_t hi16 = warp_max_u(max(a16, b16));
    if (hi16 <= lo16) return 0;
    int nb = 32 - __clz(lo16 ^ hi16);            // differing low bits
    nb = (nb + 1) & ~1;                          // two bits per step
    uint32_t res = nb >= 16 ? 0u : (hi16 >> nb) << nb;
    if (res) {
        const int n0 = __popc(__ballot_sync(FULL, a16 >= res)) + __popc(__ballot_sync(FULL, b16 >= res));
        if (n0 < m) return 0;                    // the m-th largest lies below the common prefix
    }
#pragma unroll 1
    for (int bit = nb - 2; bit >= 0; bit -= 2) {
        const uint32_t c1 = res | (1u << bit), c2 = res | (2u << bit), c3 = res | (3u << bit);
        const int n1 = __popc(__ballot_sync(FULL, a16 >= c1)) + __popc(__ballot_sync(FULL, b16 >= c1));
        const int n2 = __popc(__ballot_sync(FULL, a16 >= c2)) + __popc(__ballot_sync(FULL, b16 >= c2));
        const int n3 = __popc(__ballot_sync(FULL, a16 >= c3)) + __popc(__ballot_sync(FULL, b16 >= c3));
        res = n3 >= m ? c3 : n2 >= m ? c2 : n1 >= m ? c1 : res;
    }
    return res;
}

// Exact decode on a candidate list src[0..C) (composites, any order); dst is scratch of C + 4
// entries.  depth_key: every element of the row with key >= depth_key is in the list, so ranks
// are exact down to that key.  Returns false if the list cannot decide the lane (uniformly in all
// threads); `out` is set in thread 0 only.
template <int DT, int NT, class Sync, class StreamSmem, bool XP = false>
__device__ __noinline__ bool epilogue_ranked(StreamSmem& sm, unsigned long long* src, unsigned long long* dst,
                                             double* e, int C, uint32_t depth_key, double c, double lmax,
                                             double inv_tau, int top_k, double top_p, double tail,
                                             LaneResult& out, unsigned long long tcell = 0) {
    using Tr = Traits<DT>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // (src[C..C+3] are zero: the caller zero-fills the array before collecting candidates)
    // ---- ranks by (value desc, index asc): composites are distinct -> a permutation; each
    //      thread also computes the mass of its own candidate and stores it by rank
    //      A short list is shared out G threads to a candidate (G a power of two, the G threads
    //      adjacent lanes of one warp): each counts a G-th of the list, the counts are added by
    //      shuffles, one of them stores the composite and another the mass.
    const int kmax = (top_k > 0 && top_k < C) ? top_k : C;
    const bool topk_only = !(top_p < 1.0);
    {
        const int G = C <= NT / 8 ? 8 : C <= NT / 4 ? 4 : C <= NT / 2 ? 2 : 1;
        const int sub = tid & (G - 1);
        for (int i0 = 0; i0 < C; i0 += NT / G) {
            const int i = i0 + tid / G;
            const bool valid = i < C;
            const unsigned long long ci = valid ? src[i] : ~0ull;
            int r = 0;
#pragma unroll 1
            for (int j = sub * 4; j < C; j += G * 4)
                r += (src[j] > ci) + (src[j + 1] > ci) + (src[j + 2] > ci) + (src[j + 3] > ci);
            for (int o = G >> 1; o > 0; o >>= 1) r += __shfl_xor_sync(FULL, r, o);
            if (valid) {
                // with a top-k alone nothing past rank kmax is looked at again: zeros there, which
                // the index loop below relies on
                if (sub == 0) dst[ASX_AT(r, SK_CAP + 4, 10)] = (topk_only && r >= kmax) ? 0ull : ci;
                if (sub == (G > 1 ? 1 : 0))
                    e[ASX_AT(r, SK_CAP, 11)] = exp_nonpos(((double)Tr::value_f((uint32_t)(ci >> 32)) - lmax) * inv_tau, sm.exp_tbl);
            }
        }
    }
    ASX_MARK(6);
    if (tid < 4) dst[C + tid] = 0ull;             // ~0 = index 0xFFFFFFFF: never "smaller"
    Sync::sync();
    int n_final, ok;
    if (top_p < 1.0) {
        if (warp == 0) {
            // prefix masses in rank order: nucleus on the distribution renormalised over the survivors
            int nf = kmax, okw = 1;
            const int per = (kmax + 31) / 32;
            const int b = min(lane * per, kmax), en = min(b + per, kmax);
            double s = 0.0;
            for (int r = b; r < en; ++r) s += e[r];
            const double incl = warp_incl_scan_d(s, lane);
            const double total = __shfl_sync(FULL, incl, 31);
            if (lane == 0) sm.list_mass = total;
            const double target = top_p * (total + tail);
            double run = __shfl_up_sync(FULL, incl, 1);
            if (lane == 0) run = 0.0;
            int below = 0;
            for (int r = b; r < en; ++r) { run += e[r]; below += (run < target); }
            below = warp_sum_i(below);
            if (below >= kmax) {
                if (top_k == 0) okw = 0;       // nucleus-only: it reaches past the list
            } else {
                nf = below + 1;
            }
            if (okw && (uint32_t)(dst[ASX_AT(nf - 1, SK_CAP + 4, 12)] >> 32) < depth_key) okw = 0;   // cut below the exact depth
            __syncwarp();
            if (lane == 0) {
                sm.b_i[0] = nf; sm.b_i[1] = okw;
                // entries past the kept ranks must not count in the index loop
                if (nf < C) { dst[nf] = 0ull; dst[nf + 1] = 0ull; dst[nf + 2] = 0ull; dst[nf + 3] = 0ull; }
            }
        }
        Sync::sync();
        n_final = sm.b_i[0];
        ok = sm.b_i[1];
    } else {
        // top-k only: the answer follows from kmax alone, every thread sees it; the entries past
        // the kept ranks were stored as zeros
        n_final = kmax;
        ok = ((uint32_t)(dst[ASX_AT(kmax - 1, SK_CAP + 4, 13)] >> 32) >= depth_key) ? 1 : 0;
    }
    ASX_MARK(7);
    if (ok) {
        // ---- index order among the kept: src is free now, it receives (index << 32) | rank
        const int G = n_final <= NT / 8 ? 8 : n_final <= NT / 4 ? 4 : n_final <= NT / 2 ? 2 : 1;
        const int sub = tid & (G - 1);
        for (int r0 = 0; r0 < n_final; r0 += NT / G) {
            const int r = r0 + tid / G;
            const bool valid = r < n_final;
            const uint32_t idx = valid ? ~(uint32_t)dst[r] : 0u;
            int ir = 0;
#pragma unroll 1
            for (int q = sub * 4; q < n_final; q += G * 4)
                ir += (~(uint32_t)dst[q] < idx) + (~(uint32_t)dst[q + 1] < idx) +
                      (~(uint32_t)dst[q + 2] < idx) + (~(uint32_t)dst[q + 3] < idx);
            for (int o = G >> 1; o > 0; o >>= 1) ir += __shfl_xor_sync(FULL, ir, o);
            if (valid && sub == 0) src[ASX_AT(ir, SK_CAP + 4, 14)] = ((unsigned long long)idx << 32) | (uint32_t)r;
        }
        Sync::sync();
        ASX_MARK(8);
        if (XP && warp == 0) {
            // extended-precision step: the token that owns the code's cell among the kept tokens in
            // index order; its cells go to sm.xp_lo / sm.xp_hi
            const int per = (n_final + 31) / 32;
            const int b = min(lane * per, n_final), en = min(b + per, n_final);
            int pidx = 0;
            unsigned long long plo = 0, phi = 0;
            double pe = 1.0, Z = 1.0;
            const int L = xp_span(b, en, [&](int i) { return e[(uint32_t)src[i]]; }, lane, tcell, pidx, plo, phi, pe, Z);
            if (lane == 0) {
                LaneResult r;
                r.token = L >= 0 ? (int)(src[pidx] >> 32) : -1;
                r.status = L >= 0 ? ST_OK : ST_NUMERIC; r.n_kept = n_final; r.code_out = 0.0;
                r.p_tok = pe / Z; r.cdf_lo = (double)plo * (1.0 / 4294967296.0);
                sm.xp_lo = plo; sm.xp_hi = phi;
                out = r;
            }
        } else if (warp == 0) {
            // lane l owns index-order positions [b, en); up to 4 masses are kept in registers
            const int per = (n_final + 31) / 32;
            const int b = min(lane * per, n_final), en = min(b + per, n_final);
            double ev4[4] = {0.0, 0.0, 0.0, 0.0};
            double s = 0.0;
            if (per <= 4) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (b + k < en) { ev4[k] = e[ASX_AT((uint32_t)src[b + k], SK_CAP, 15)]; s += ev4[k]; }
            } else {
                for (int i = b; i < en; ++i) s += e[ASX_AT((uint32_t)src[i], SK_CAP, 16)];
            }
            const double incl = warp_incl_scan_d(s, lane);
            double run = __shfl_up_sync(FULL, incl, 1);
            if (lane == 0) run = 0.0;
            // Z continues the same running sum as the prefixes: run + (elements in order)
            double zrun = run;
            if (per <= 4) {
#pragma unroll
                for (int k = 0; k < 4; ++k) if (b + k < en) zrun += ev4[k];
            } else {
                for (int i = b; i < en; ++i) zrun += e[(uint32_t)src[i]];
            }
            const double Z = __shfl_sync(FULL, zrun, (n_final - 1) / per);
            const double tt = c * Z;
            int pick = -1;
            double pS = 0.0, pe = 1.0;
            if (per <= 4) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (b + k < en) {
                        const double ev = ev4[k];
                        if (pick < 0 && (tt < run + ev || b + k == n_final - 1)) { pick = b + k; pS = run; pe = ev; }
                        run += ev;
                    }
                }
            } else {
                for (int i = b; i < en; ++i) {
                    const double ev = e[(uint32_t)src[i]];
                    if (pick < 0 && (tt < run + ev || i == n_final - 1)) { pick = i; pS = run; pe = ev; }
                    run += ev;
                }
            }
            const unsigned bal = __ballot_sync(FULL, pick >= 0);
            const int L = __ffs(bal) - 1;
            pick = __shfl_sync(FULL, pick, L);
            pS = __shfl_sync(FULL, pS, L);
            pe = __shfl_sync(FULL, pe, L);
            // the three divisions on three lanes
            const double num = lane == 0 ? (tt - pS) : lane == 1 ? pe : pS;
            const double den = lane == 0 ? pe : Z;
            const double quo = num / den;
            const double p_tok = __shfl_sync(FULL, quo, 1), cdf_lo = __shfl_sync(FULL, quo, 2);
            if (lane == 0) {
                double cn = quo;
                if (!(cn >= 0.0)) cn = 0.0;
                if (cn > ASX_ONE_BELOW) cn = ASX_ONE_BELOW;
                LaneResult r;
                r.token = (int)(src[ASX_AT(pick, SK_CAP + 4, 17)] >> 32); r.status = ST_OK; r.n_kept = n_final; r.code_out = cn;
                r.p_tok = p_tok; r.cdf_lo = cdf_lo;
                out = r;
            }
        }
    }
    ASX_MARK(9);
    ASX_MARK(10);
    // No barrier here: the result lives in thread 0, which is also the one that writes it out, and
    // every caller passes a block barrier before shared memory is written again.
    return ok != 0;
}

// One more pass over a 16-byte aligned row in global memory, f(vector, vector index), thread t
// taking vectors t, t + 256, ...  Each thread keeps D asynchronous 16-byte copies in flight into
// slots of its own in `staging` (D * 256 vectors of shared memory that are dead meanwhile): with a
// single load per thread in flight a lone CTA is latency-bound, and holding more loads in
// registers would cost the whole kernel registers.
template <int D, class F>
__device__ __forceinline__ void reread_row(uint4* staging, const char* row, int nvec_full, F&& f) {
    const int tid = threadIdx.x;
    const uint4* rv = reinterpret_cast<const uint4*>(row);
    uint4* mine = staging + tid;
    const uint32_t mine_s = smem_u32(mine);
    auto copy = [&](int slot, int v) {
        if (v < nvec_full)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(mine_s + slot * (SK_NT * 16)), "l"(rv + v) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");     // one group per step, empty or not
    };
#pragma unroll
    for (int d = 0; d < D; ++d) copy(d, tid + d * SK_NT);
    int slot = 0;
    for (int v = tid; v < nvec_full; v += SK_NT) {
        asm volatile("cp.async.wait_group %0;" ::"n"(D - 1) : "memory");
        const uint4 q = mine[ASX_AT(slot, D, 60) * SK_NT];
        f(q, v);
        copy(slot, v + D * SK_NT);                 // after f: the slot's value has been consumed
        slot = slot + 1 == D ? 0 : slot + 1;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Nucleus-only lane whose nucleus reaches below the exact depth of the list (key >= t0key).
// The row is read again from global memory (it was just streamed, so mostly from L2):
//   1. the elements below the old threshold are counted into bins over y = (x - max) * scale2,
//      128 bins per unit of log2 mass, 8 units deep (a list of a few hundred candidates never
//      reaches further down, and the fewer elements fall into the window, the fewer shared-memory
//      atomics the pass costs; counts only: integer additions to shared memory are native, fp32
//      ones are compare-and-swap loops);
//   2. the bins are taken from the top until the mass they hold at the least (count times the
//      mass at the bin's lower edge) covers what the nucleus still lacks, with a margin: that
//      gives a lower threshold t1 below which no nucleus token can lie, if the candidates still
//      fit the list;
//   3. everything >= t1 is collected afresh, the rest summed in fp32, and the exact epilogue
//      runs again.  Returns false if the window or the list capacity does not suffice.
constexpr int DP_NB = 1024;
constexpr float DP_BINS_PER_UNIT = 128.f;
template <int DT, class StreamSmem, bool XP = false>
__device__ __noinline__ bool deepen_nucleus(StreamSmem& sm, int V, float scale2, double inv_tau, double top_p,
                                            const char* row, uint32_t gmax, float t0f, double tailsum, double c,
                                            LaneResult& r, unsigned long long tcell = 0) {
    using Tr = Traits<DT>;
    using P = Pass<DT>;
    constexpr int E = Tr::E;
    constexpr int NT = SK_NT;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nvec_full = (V * Tr::BYTES) >> 4;           // whole 16-byte vectors
    const float lmaxf = Tr::value_f(gmax);
    const float y0 = (t0f - lmaxf) * scale2;
    int* hcnt = reinterpret_cast<int*>(sm.u.ep.v.cvec) + DP_NB;        // (the staging area starts past 2 * DP_NB words)
    const double list_mass = sm.list_mass;
    {
        // every token that could still join weighs less than the old threshold does: if even that many
        // of them as the list has room for cannot cover what the nucleus lacks, the pass is pointless
        const double lacking = top_p * (list_mass + tailsum) - list_mass;
        const double room = (double)(SK_CAP - 8 - sm.cand_count);
        if (lacking > room * (double)ex2_approx(y0) * 1.001) { ASX_COUNT(2); return false; }
    }
    SyncC::sync();                                         // the epilogue's arrays are dead
    for (int i = tid; i < DP_NB; i += NT) hcnt[i] = 0;
    if (tid == 0) sm.cand_count = 0;
    for (int i = tid; i < SK_CAP + 4; i += NT) sm.u.ep.cand[i] = 0ull;
    SyncC::sync();
    auto visit = [&](auto&& f) {                           // f(x, index) over the whole row
        // staging: the hit-vector list past the histogram
        constexpr int D = (int)((sizeof(sm.u.ep.v.cvec) - DP_NB * 8) / (NT * 16));
        static_assert(D >= 2, "the list is too small to stage a re-read");
        reread_row<D>(sm.u.ep.v.cvec + DP_NB / 2, row, nvec_full, [&](const uint4& q, int v) {
            float x[E];
            P::floats(q, x);
#pragma unroll
            for (int e = 0; e < E; ++e) f(x[e], v * E + e);
        });
        for (int j = nvec_full * E + tid; j < V; j += NT) f(Tr::value_f(Tr::load_key(row, j)), j);
    };
    // ---- 1. histogram below the old threshold
    visit([&](float x, int) {
        if (x < t0f) {
            const float y = (x - lmaxf) * scale2;
            const float d = (y0 - y) * DP_BINS_PER_UNIT;
            if (d < (float)DP_NB) {
                const int bin = (int)d;
                red_shared_add(&hcnt[ASX_AT(bin, DP_NB, 20)], 1);
            }
        }
    });
    SyncC::sync();
    // ---- 2. lowest bin needed
    if (warp == 0) {
        const double target = top_p * (list_mass + tailsum);
        const double need = (target - list_mass) * 1.002 + 1e-7 * target;
        constexpr int PER = DP_NB / 32;
        // least mass of an element of bin i: at the bin's lower edge, y0 - (i + 1) / 128
        auto least = [&](int i) -> double { return (double)hcnt[i] * (double)ex2_approx(y0 - (float)(i + 1) / DP_BINS_PER_UNIT); };
        double m = 0.0;
        int n = 0;
        for (int i = 0; i < PER; ++i) { m += least(lane * PER + i); n += hcnt[lane * PER + i]; }
        const double mi = warp_incl_scan_d(m, lane);
        const int ni = warp_incl_scan_i(n, lane);
        double run = mi - m;
        int cnt = ni - n;
        int found = -1, found_cnt = 0;
        for (int i = 0; i < PER; ++i) {
            run += least(lane * PER + i);
            cnt += hcnt[lane * PER + i];
            if (found < 0 && run >= need) { found = lane * PER + i; found_cnt = cnt; }
        }
        const unsigned bal = __ballot_sync(FULL, found >= 0);
        int bin = -1, below = 0;
        if (bal) {
            const int L = __ffs(bal) - 1;
            bin = __shfl_sync(FULL, found, L);
            below = __shfl_sync(FULL, found_cnt, L);
        }
        if (lane == 0) { sm.b_i[0] = bin; sm.b_i[1] = below; }
    }
    SyncC::sync();
    const int bin = sm.b_i[0];
    const int old_count = sm.b_i[2];
    if (bin < 0) { ASX_COUNT(1); return false; }
    if (sm.b_i[1] + old_count > SK_CAP - 8) { ASX_COUNT(2); return false; }
    const float t1f = lmaxf + (y0 - (float)(bin + 1) / DP_BINS_PER_UNIT - 2e-3f) / scale2;
    uint32_t depth_key = P::key_of_f(t1f);
    if (Tr::value_f(depth_key) < t1f) depth_key += 1;     // smallest key whose value is >= t1
    SyncC::sync();
    // ---- 3. collect afresh.  The mass outside the new list is the old one less the tokens that
    //         join now (those below the old threshold): an exponential for a few hundred elements,
    //         not for the whole row again.
    float joined = 0.f;
    visit([&](float x, int j) {
        if (x >= t1f) {
            const uint32_t key = P::key_of_f(x);
            if (key > Tr::KEY_NINF) {
                const int slot = atomicAdd(&sm.cand_count, 1);
                if (slot < SK_CAP) sm.u.ep.cand[ASX_AT(slot, SK_CAP + 4, 30)] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)j;
                if (x < t0f) joined += ex2_approx((x - lmaxf) * scale2);
            }
        }
    });
    const double td = warp_sum_d((double)joined);
    if (lane == 0) sm.red_d[warp] = td;
    SyncC::sync();
    double tsum = tailsum;
#pragma unroll
    for (int w = 0; w < SK_NW; ++w) tsum -= sm.red_d[w];
    if (tsum < 0.0) tsum = 0.0;
    const int C = sm.cand_count;
    if (C <= 0 || C > SK_CAP || !(tsum == tsum) || !(tsum < 1e300)) { ASX_COUNT(3); return false; }
    const bool ok2 = epilogue_ranked<DT, NT, SyncC, StreamSmem, XP>(sm, sm.u.ep.cand, sm.u.ep.v.rk.srt, sm.u.ep.v.rk.e, C, depth_key, c,
                                                        (double)lmaxf, inv_tau, 0, top_p, tsum, r, tcell);
    if (!ok2) ASX_COUNT(4);
    return ok2;
}

// A lane whose hit vectors outgrew the list: the threshold is still exact (it comes from the
// subset maxima, not from the list), so one more pass over the row (just streamed, mostly in
// L2) takes the candidates >= t0key directly and sums the rest against `ref` in fp32.
// Returns this thread's share of that sum; the caller's barrier completes the list.
template <int DT, class StreamSmem>
__device__ __noinline__ float recollect_row(StreamSmem& sm, int V, const char* row, float t0f, uint32_t t0key,
                                            float ref, float scale2) {
    using Tr = Traits<DT>;
    using P = Pass<DT>;
    constexpr int E = Tr::E;
    const int tid = threadIdx.x;
    const int nvec_full = (V * Tr::BYTES) >> 4;
    float tail = 0.f;
    auto take = [&](float x, int j) {
        bool hit = false;
        if (x >= t0f) {
            const uint32_t key = P::key_of_f(x);
            if (key >= t0key && key > Tr::KEY_NINF) {
                hit = true;
                const int slot = atomicAdd(&sm.cand_count, 1);
                if (slot < SK_CAP) sm.u.ep.cand[ASX_AT(slot, SK_CAP + 4, 30)] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)j;
            }
        }
        if (!hit) tail += ex2_approx((x - ref) * scale2);
    };
    constexpr int D = (int)(sizeof(sm.u.ep.v.cvec) / (SK_NT * 16)) < 8 ? (int)(sizeof(sm.u.ep.v.cvec) / (SK_NT * 16)) : 8;
    reread_row<D>(sm.u.ep.v.cvec, row, nvec_full, [&](const uint4& q, int v) {   // the list is dead: staging
        float x[E];
        P::floats(q, x);
#pragma unroll
        for (int e = 0; e < E; ++e) take(x[e], v * E + e);
    });
    for (int j = nvec_full * E + tid; j < V; j += SK_NT) take(Tr::value_f(Tr::load_key(row, j)), j);
    return tail;
}

// UA builds also serve rows that do not start on a 16-byte boundary (a pitch or base pointer that
// is only element-aligned): such a row is copied from the boundary below its start, the `lead`
// elements in front of it are masked to -inf in the first vector, and every token index shifts
// by `lead`.  The bytes in front belong to the same 16-byte granule as the row's first element,
// so the copy never leaves mapped memory; past its end nothing beyond whole granules inside the
// row is copied.  Calls whose rows are all aligned use the build without this.
template <int DT>
__device__ __forceinline__ void mask_lead(uint4& q, int lead) {
    uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (DT == DT_BF16) {
            if (2 * i < lead) w[i] = (w[i] & 0xFFFF0000u) | 0xFF80u;
            if (2 * i + 1 < lead) w[i] = (w[i] & 0x0000FFFFu) | 0xFF800000u;
        } else if (i < lead) {
            w[i] = 0xFF800000u;
        }
    }
    q = make_uint4(w[0], w[1], w[2], w[3]);
}

// Token of a lane that the streaming kernel leaves to deferred_lanes_kernel (never seen by a caller).
constexpr int LANE_DEFERRED = -2;

// One lane's outputs (thread 0 of the CTA that decided it).  XP: the decoder state is narrowed to the
// token's cells [xp_lo, xp_hi) and refilled with digits of the code.
template <bool GATHER, bool XP>
__device__ __forceinline__ void finish_lane(const StepArgs& a, int ln, const LaneResult& r, int path,
                                            unsigned long long xp_lo, unsigned long long xp_hi) {
    if (XP) {
        a.tokens[(size_t)ln * a.tok_stride] = r.token;
        if (r.status == ST_OK) {         // narrow the interval to the token's cells, shift digits in
            XpState xs;
            xs.range = a.xp_state[(size_t)ln * 4]; xs.code = a.xp_state[(size_t)ln * 4 + 1];
            xs.q = a.xp_state[(size_t)ln * 4 + 2]; xs.packed = a.xp_state[(size_t)ln * 4 + 3];
            xp_advance(xs, xp_lo, xp_hi, (unsigned)a.xp_N);
            a.xp_state[(size_t)ln * 4] = xs.range; a.xp_state[(size_t)ln * 4 + 1] = xs.code;
            a.xp_state[(size_t)ln * 4 + 2] = xs.q; a.xp_state[(size_t)ln * 4 + 3] = xs.packed;
        } else if (a.diag.lane_status) {
            a.diag.lane_status[ln] = r.status;
        }
    } else if (GATHER) {
        a.tokens[(size_t)ln * a.tok_stride] = r.token;
        a.codes_out[ln] = r.code_out;
        if (a.diag.lane_status && r.status != ST_OK) a.diag.lane_status[ln] = r.status;
    } else {
        write_result(a, ln, r, path);
    }
}

// The lanes the streaming kernel left undecided (token == LANE_DEFERRED), through the general
// routine on their rows in global memory (just streamed: mostly in L2).  Launched after every
// launch of the streaming kernel, with the same arguments; CTA b looks at lanes b, b + grid, ...
// and leaves at once where none is marked.  `stage_bytes` > 0: the row fits that much dynamic shared
// memory and is copied there first (from the 16-byte boundary below its start), so that the routine's
// passes run from shared memory.
constexpr int DL_NT = 256;
constexpr int DL_STAGE_MAX = 96 * 1024 + 32;     // rows up to 96 KB are staged
template <int DT, bool GATHER, bool XP>
__global__ void __launch_bounds__(DL_NT, 4) deferred_lanes_kernel(const StepArgs a, const int stage_bytes) {
    using Tr = Traits<DT>;
    __shared__ GenericSmem<DL_NT> sm;
    extern __shared__ uint4 dl_stage[];
    pdl_allow_next();
    pdl_wait_prev();
    {
        // this CTA's lanes looked at side by side, one per thread: usually none is marked, and a walk
        // through them one dependent load after the other would be the whole cost of this kernel
        int any = 0;
        for (long long ln = blockIdx.x + (long long)threadIdx.x * gridDim.x; ln < a.lanes; ln += (long long)DL_NT * gridDim.x)
            any |= a.tokens[(size_t)ln * (GATHER ? a.tok_stride : 1)] == LANE_DEFERRED;
        if (!__syncthreads_or(any)) return;
    }
    for (int ln = blockIdx.x; ln < a.lanes; ln += gridDim.x) {
        if (a.tokens[(size_t)ln * (GATHER ? a.tok_stride : 1)] != LANE_DEFERRED) continue;    // (uniform over the CTA)
        const int ri = GATHER ? a.row_idx[(size_t)ln * a.idx_stride] : ln;
        const char* row = reinterpret_cast<const char*>(a.logits) + (size_t)ri * (size_t)a.ld * Tr::BYTES;
        if (stage_bytes > 0) {
            const int lead = (int)(reinterpret_cast<uintptr_t>(row) & 15);
            const uint4* src = reinterpret_cast<const uint4*>(row - lead);
            const int nfull = (lead + a.V * Tr::BYTES) >> 4;                 // whole 16-byte vectors
            for (int i = threadIdx.x; i < nfull; i += DL_NT) dl_stage[i] = src[i];
            // (the ragged end byte by byte: reading its whole vector could cross the end of the allocation)
            char* dst = reinterpret_cast<char*>(dl_stage);
            for (int i = (nfull << 4) + threadIdx.x; i < lead + a.V * Tr::BYTES; i += DL_NT) dst[i] = (row - lead)[i];
            __syncthreads();
            row = dst + lead;
        }
        const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
        GenericLane<DT, DL_NT> g(sm, row, a.V, vec_ok);
        g.bins = !a.radix_nucleus;
        LaneResult r;
        if (XP) {
            XpState xs = {XP_RANGE_TOP, 0ull, 0ull, 0ull};
            xs.range = a.xp_state[(size_t)ln * 4]; xs.code = a.xp_state[(size_t)ln * 4 + 1];
            r = g.run_xp(xp_target(xs), a.inv_tau, a.top_k, a.top_p);      // (the state was checked by the streaming kernel)
        } else {
            r = g.run(lane_code(a, ln), a.inv_tau, a.top_k, a.top_p);
        }
        if (threadIdx.x == 0) finish_lane<GATHER, XP>(a, ln, r, PATH_GENERAL, sm.xp_lo, sm.xp_hi);
        __syncthreads();
    }
}

template <int DT, int CAPV, int MINB, bool UA = false, bool GATHER = false, bool XP = false>
__global__ void __launch_bounds__(SK_THREADS, MINB) step_stream_kernel(const StepArgs a, const int stages) {
    using StreamSmem = StreamSmemT<CAPV>;
    constexpr int SK_CAPV = CAPV;
    using Tr = Traits<DT>;
    using P = Pass<DT>;
    constexpr int NT = SK_NT;
    constexpr int E = Tr::E;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    StreamSmem& sm = *reinterpret_cast<StreamSmem*>(smem_raw);
    unsigned char* ring = smem_raw + ((sizeof(StreamSmem) + 127) & ~(size_t)127);
    const uint4* ringv = reinterpret_cast<const uint4*>(ring);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    ASX_MARK(13);
    ASX_SPAN(0);
    ASX_CTA(0);
    const int V = a.V;
    const int row_bytes = (V + (UA ? E - 1 : 0)) * Tr::BYTES;          // UA: the longest a row gets with its lead
    const int bulk_bytes = row_bytes & ~15;
    const int bulk_vec = bulk_bytes >> 4;
    const int tail_elems = (row_bytes - bulk_bytes) / Tr::BYTES;      // < E
    const int nsl = (bulk_vec + SK_STAGE_VEC - 1) / SK_STAGE_VEC;      // slices per row
    const bool resident = nsl <= stages;
    const int S = resident ? max(nsl, 1) : stages;                     // ring length in use

    // GATHER: the row comes from a table through an index; lanes without a usable index sit out
    auto lane_row = [&](int ln) -> int { return GATHER ? a.row_idx[(size_t)ln * a.idx_stride] : ln; };
    auto lane_active = [&](int ln) -> bool {
        if (!GATHER) return true;
        const int i = lane_row(ln);
        return i >= 0 && i != a.eos && i < a.rows;
    };
    auto row_of = [&](int ln) -> const char* {
        return reinterpret_cast<const char*>(a.logits) + (size_t)lane_row(ln) * (size_t)a.ld * Tr::BYTES;
    };
    auto staged_ok = [&](int ln) -> bool { return UA || (reinterpret_cast<uintptr_t>(row_of(ln)) & 15) == 0; };
    auto lead_of = [&](int ln) -> int {
        return UA ? (int)((reinterpret_cast<uintptr_t>(row_of(ln)) & 15) / Tr::BYTES) : 0;
    };
    // one row's own geometry (UA: it depends on the row's lead)
    auto geom = [&](int lead, int& bb, int& bv, int& te, int& ns) {
        const int rb = (V + lead) * Tr::BYTES;
        bb = rb & ~15;
        bv = bb >> 4;
        te = (rb - bb) / Tr::BYTES;
        ns = (bv + SK_STAGE_VEC - 1) / SK_STAGE_VEC;
    };

    // The producer lane initialises the barriers of the stages in use and starts the first copies
    // before the block-wide barrier, so the first row is in flight while the rest of the CTA sets up.
    const bool is_producer = (warp == SK_NW && lane == 0);
    unsigned p_st = 0, p_round = 0;               // producer: slices issued so far = p_round * S + p_st
    int ln_issue = blockIdx.x;                    // producer: lane whose slices come next
    int s_issue = 0;
    auto issue_some = [&](bool first_row_only) -> bool {   // false: a bounded wait ran out
        for (; ln_issue < a.lanes; ln_issue += gridDim.x, s_issue = 0) {
            if (GATHER && !lane_active(ln_issue)) continue;
            if (!staged_ok(ln_issue)) continue;
            int bulk_bytes_i = bulk_bytes, nsl_i = nsl;
            const int lead_i = lead_of(ln_issue);
            if (UA) { int bv, te; geom(lead_i, bulk_bytes_i, bv, te, nsl_i); }
            const char* src = row_of(ln_issue) - lead_i * Tr::BYTES;
            for (; s_issue < nsl_i; ++s_issue, p_st = (p_st + 1 == (unsigned)S ? (++p_round, 0u) : p_st + 1)) {
                const int st = (int)p_st;
                if (p_round >= 1) {               // the stage must have been drained by every consumer warp
                    if (first_row_only) return true;
                    if (*(volatile int*)&sm.poisoned) return false;
                    if (!mbar_wait_bounded(smem_u32(&sm.empty_bar[st]), (p_round - 1) & 1, a.wait_cycles)) {
                        *(volatile int*)&sm.poisoned = 1;
                        return false;
                    }
                }
                const uint32_t bytes = (uint32_t)min(SK_STAGE_BYTES, bulk_bytes_i - s_issue * SK_STAGE_BYTES);
                const uint32_t bar = smem_u32(&sm.full_bar[st]);
                if (a.debug_no_copy) return false;    // (time-out test: nothing is armed, nothing is in flight)
                mbar_expect_tx(bar, bytes);
                bulk_g2s(smem_u32(ring + (size_t)st * SK_STAGE_BYTES), src + (size_t)s_issue * SK_STAGE_BYTES, bytes, bar);
            }
            if (first_row_only) { ln_issue += gridDim.x; s_issue = 0; return true; }
        }
        return true;
    };
    // Set-up that touches no global memory comes first: it may run while the kernel before this
    // one on the stream is still draining.  Everything after pdl_wait_prev() sees that kernel's
    // writes (logits, codes, the previous step's tokens in a decode loop).
    pdl_allow_next();
    if (is_producer) {
        for (int i = 0; i < S; ++i) {
            mbar_init(smem_u32(&sm.full_bar[i]), 1);
            mbar_init(smem_u32(&sm.empty_bar[i]), SK_NW);
        }
        fence_mbar_init();
        sm.poisoned = 0;
        sm.prod_done = 0;
    }
    fill_exp_table(sm.exp_tbl, tid);
    pdl_wait_prev();
    if (is_producer) issue_some(true);            // fills the ring without waiting
    __syncthreads();

    // =========================== producer warp ===========================
    if (warp == SK_NW) {
        if (lane == 0) {
            issue_some(false);
            // what has been armed, for the consumers' drain should a wait run out
            sm.prod_st = p_st;
            sm.prod_round = p_round;
            __threadfence_block();
            *(volatile int*)&sm.prod_done = 1;
        }
        return;
    }
    // =========================== consumer warps ===========================
    const bool want_tail = (a.top_k == 0);        // nucleus-only: masses of non-candidates in fp32
    const int K0 = a.top_k > 0 ? a.top_k : SK_KP;
    const int m_sel = (K0 + SK_NW - 1) / SK_NW;
    const float scale2 = a.scale2;
    const uint32_t ninf_word = (DT == DT_BF16) ? 0xFF80FF80u : 0xFF800000u;
    // consumer's position in the ring: the slice counter g is kept as stage (g mod S) and phase
    // parity ((g / S) & 1) and advanced by additions; a division by S per use cost more
    // instructions than the work between two uses
    unsigned g_st = 0, g_par = 0;
    auto stage_of = [&](int off) -> unsigned { const unsigned st = g_st + off; return st >= (unsigned)S ? st - S : st; };
    auto advance = [&](int n) { g_st += n; if (g_st >= (unsigned)S) { g_st -= S; g_par ^= 1u; } };   // n <= S
    int thr_calls = 0;

    // block step: max so far and (optionally) threshold from the subset maxima held in `acc`;
    // one barrier: the exchange slots are double-buffered between consecutive calls
    auto threshold = [&](const typename P::Acc& acc, uint32_t& gmax, uint32_t& t0key, bool want_sel, uint32_t lo_key) {
        uint32_t k0, k1;
        P::keys(acc, k0, k1);
        const uint32_t wm = warp_max_u(max(k0, k1));
#ifdef ASX_PROFILE
        const long long tq0 = clock64();
#endif
        const uint32_t ws = want_sel ? warp_select16(P::key16(k0), P::key16(k1), m_sel, P::key16(lo_key)) : 0u;
#ifdef ASX_PROFILE
        const long long tq1 = clock64();
#endif
        const int buf = thr_calls & 1;
        ++thr_calls;
        if (lane == 0) { sm.wmax[buf][warp] = wm; sm.wsel[buf][warp] = ws; }
        SyncC::sync();
#ifdef ASX_PROFILE
        if (blockIdx.x == 0 && tid == 0) { g_asx_marks[28] += tq1 - tq0; g_asx_marks[29] += clock64() - tq1; g_asx_marks[30] += 1; }
#endif
        gmax = 0;
        uint32_t t16 = 0xFFFFFFFFu;
#pragma unroll
        for (int w = 0; w < SK_NW; ++w) { gmax = max(gmax, sm.wmax[buf][w]); t16 = min(t16, sm.wsel[buf][w]); }
        t0key = max(P::key_from16(t16), Tr::KEY_NINF);
    };
    // SK_VPT vectors of one thread against the threshold.  Per vector: one packed max (shared with
    // the running max when do_merge) and one compare.  Hit vectors are copied to the list: one
    // ballot per vector position, one atomic per warp and position that has hits.  Nucleus-only
    // lanes also sum 2^((x - ref) * scale2) over the vectors that are not listed.
    auto slice_pass = [&](const uint4 (&q)[SK_VPT], int vec0, unsigned valid, bool do_merge, typename P::Acc& acc,
                          float t0f, float ref, float& tail) {
        unsigned hm = 0;
#pragma unroll
        for (int j = 0; j < SK_VPT; ++j) {
            const typename P::Acc part = P::reduce(q[j]);
            if (do_merge) P::merge(acc, part);
            const bool hit = ((valid >> j) & 1u) && P::part_max(part) >= t0f;
            hm |= (hit ? 1u : 0u) << j;
            if (want_tail) {
                float x[E];
                P::floats(q[j], x);
                float sacc = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) sacc += ex2_approx((x[e] - ref) * scale2);
                tail += hit ? 0.f : sacc;
            }
        }
        if (__any_sync(FULL, hm != 0)) {
            // one slot reservation per warp and slice: ballots per vector position, then a single atomic
            unsigned bal[SK_VPT];
            int total = 0;
#pragma unroll
            for (int j = 0; j < SK_VPT; ++j) {
                bal[j] = __ballot_sync(FULL, (hm >> j) & 1u);
                total += __popc(bal[j]);
            }
            int base = 0;
            if (lane == 0) base = atomicAdd(&sm.vec_count, total);
            base = __shfl_sync(FULL, base, 0);
#pragma unroll
            for (int j = 0; j < SK_VPT; ++j) {
                if ((hm >> j) & 1u) {
                    const int slot = base + __popc(bal[j] & ((1u << lane) - 1u));
                    if (slot < SK_CAPV) {
                        sm.u.ep.v.cvec[ASX_AT(slot, SK_CAPV, 40)] = q[j];
                        sm.u.ep.cidx[ASX_AT(slot, SK_CAPV, 41)] = vec0 + j * NT;
                    }
                }
                base += __popc(bal[j]);
            }
        }
    };

    // Elements of one vector that pass the final threshold -> candidate list, token index base + e.
    // One slot reservation per vector: a reservation per element made up to E dependent atomic round
    // trips per warp pass (the hits of a warp's lanes sit at different e), which cost more than the
    // passes over the row.  With with_tail the other elements join the fp32 tail.
    auto push_vec = [&](const uint4& q, int base, float t0f, uint32_t t0key, bool with_tail, float ref, float& tail) {
        float x[E];
        P::floats(q, x);
        if (!with_tail) {
            // lean form: one float compare per element; the exact key test and the reservation run
            // only for the one or two elements that pass (~55 instructions per vector against ~170)
            unsigned m = 0;
#pragma unroll
            for (int e = 0; e < E; ++e) m |= (x[e] >= t0f ? 1u : 0u) << e;
#pragma unroll 1
            while (m) {
                const int e = __ffs(m) - 1;
                m &= m - 1;
                float xe = x[0];
#pragma unroll
                for (int k = 1; k < E; ++k) xe = (e == k) ? x[k] : xe;
                const uint32_t key = P::key_of_f(xe);
                if (key >= t0key && key > Tr::KEY_NINF) {
                    const int slot = atomicAdd(&sm.cand_count, 1);
                    if (slot < SK_CAP) sm.u.ep.cand[ASX_AT(slot, SK_CAP + 4, 31)] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)(base + e);
                }
            }
            return;
        }
        unsigned em = 0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            bool hit = false;
            if (x[e] >= t0f) {
                const uint32_t key = P::key_of_f(x[e]);
                hit = key >= t0key && key > Tr::KEY_NINF;
            }
            em |= (hit ? 1u : 0u) << e;
            if (with_tail && !hit) tail += ex2_approx((x[e] - ref) * scale2);
        }
        if (em) {
            int slot = atomicAdd(&sm.cand_count, __popc(em));
#pragma unroll
            for (int e = 0; e < E; ++e) {
                if ((em >> e) & 1u) {
                    if (slot < SK_CAP)
                        sm.u.ep.cand[ASX_AT(slot, SK_CAP + 4, 32)] = ((unsigned long long)P::key_of_f(x[e]) << 32) | (uint32_t)~(uint32_t)(base + e);
                    ++slot;
                }
            }
        }
    };

    for (int ln = blockIdx.x; ln < a.lanes; ln += gridDim.x) {
        if (GATHER && !lane_active(ln)) continue;
        // the code is first looked at just before the epilogue: its 8-byte load queues behind the
        // row copies of the whole grid, and an earlier use would hold up the passes over the row
        const double c_in = XP ? 0.5 : lane_code(a, ln);
        const char* row = row_of(ln);
        const int lead = lead_of(ln);
        int bulk_bytes_l = bulk_bytes, bulk_vec_l = bulk_vec, tail_elems_l = tail_elems, nsl_l = nsl;
        if (UA) geom(lead, bulk_bytes_l, bulk_vec_l, tail_elems_l, nsl_l);
        const char* vrow = row - lead * Tr::BYTES;     // where the copies start

        // Lanes the candidate list cannot decide are left to the kernel that follows this one on the
        // stream (deferred_lanes_kernel: the general routine): their token is set to LANE_DEFERRED and
        // nothing else of theirs is written.  The general routine is not part of this kernel: even out
        // of line its register needs weighed on the allocation of the streaming passes (2-10 % of
        // their time), and the lanes that need it are spread over the whole machine that way.
        LaneResult r;
        int path = PATH_COMPACT;
        bool decided = false;
        bool whole_row = false;                 // a row that would have to be kept whole (no usable cut)

        if (tid == 0) { sm.vec_count = 0; sm.cand_count = 0; }
        // the candidate array starts zeroed: entries past the count rank below every candidate,
        // which the epilogue's 4-wide rank loop relies on
        for (int i = tid; i < SK_CAP + 4; i += NT) sm.u.ep.cand[i] = 0ull;

        // ragged end of the row (< 16 bytes): one padded vector read straight from global memory
        uint4 qt = make_uint4(ninf_word, ninf_word, ninf_word, ninf_word);
        if (tail_elems_l > 0 && tid == 0) {
            uint32_t w[4];
            // (a row shorter than a granule has its lead in this vector: those elements stay masked)
            const int skip = (UA && bulk_vec_l == 0) ? lead : 0;
            if (DT == DT_BF16) {
                const unsigned short* src = reinterpret_cast<const unsigned short*>(vrow + bulk_bytes_l);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t lo = (2 * i >= skip && 2 * i < tail_elems_l) ? src[2 * i] : 0xFF80u;
                    const uint32_t hi = (2 * i + 1 >= skip && 2 * i + 1 < tail_elems_l) ? src[2 * i + 1] : 0xFF80u;
                    w[i] = lo | (hi << 16);
                }
            } else {
                const uint32_t* src = reinterpret_cast<const uint32_t*>(vrow + bulk_bytes_l);
#pragma unroll
                for (int i = 0; i < 4; ++i) w[i] = (i >= skip && i < tail_elems_l) ? src[i] : 0xFF800000u;
            }
            qt = make_uint4(w[0], w[1], w[2], w[3]);
        }

        typename P::Acc acc = P::init();
        uint32_t gmax = 0, t0key = Tr::KEY_NINF;
        float tail = 0.f;
        float ref = 0.f;             // exponent reference of the fp32 tail
        float t0f = 0.f;
        const bool cut = a.fast && (a.top_k > 0 || a.top_p < 1.0);

        auto wait_full = [&](int off) {            // slice g + off, off < S
            if (*(volatile int*)&sm.poisoned) return;
            const unsigned par = g_par ^ (g_st + off >= (unsigned)S ? 1u : 0u);
            if (!mbar_wait_bounded(smem_u32(&sm.full_bar[stage_of(off)]), par, a.wait_cycles)) *(volatile int*)&sm.poisoned = 1;
        };
        auto release = [&](int off) {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.empty_bar[stage_of(off)]));
        };
        auto load_slice = [&](const uint4* sv, int nv, uint4 (&q)[SK_VPT]) -> unsigned {
            unsigned valid = 0;
#pragma unroll
            for (int j = 0; j < SK_VPT; ++j) {
                const int v = j * NT + tid;
                const bool ok = v < nv;
                valid |= (ok ? 1u : 0u) << j;
                q[j] = ok ? sv[ASX_AT(v, SK_STAGE_VEC, 51)] : make_uint4(ninf_word, ninf_word, ninf_word, ninf_word);
            }
            return valid;
        };

        ASX_MARK(0);
        ASX_CTA(1);
        if (resident) {
            // ---- all stages land; max pass from shared memory.  Each vector's own maximum stays
            //      in a register, so the hit test after the threshold needs no second pass.
            float pm[SK_RES_STAGES * SK_VPT];
#pragma unroll
            for (int s = 0; s < SK_RES_STAGES; ++s) {
                if (s < nsl_l) {
                    wait_full(s);
                    ASX_MARK(1);
                    uint4 q[SK_VPT];
                    const unsigned valid = load_slice(ringv + (size_t)stage_of(s) * SK_STAGE_VEC,
                                                      min(SK_STAGE_VEC, bulk_vec_l - s * SK_STAGE_VEC), q);
                    if (UA && s == 0 && tid == 0 && lead) {
                        // the elements in front of the row: masked here and in the ring (this thread
                        // alone reads that vector again; the next bulk copy into the stage is
                        // ordered after the store by the proxy fence)
                        mask_lead<DT>(q[0], lead);
                        reinterpret_cast<uint4*>(ring)[(size_t)g_st * SK_STAGE_VEC] = q[0];
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    }
#pragma unroll
                    for (int j = 0; j < SK_VPT; ++j) {
                        const typename P::Acc part = P::reduce(q[j]);
                        P::merge(acc, part);
                        // NaN for vectors past the row: they must not pass any threshold, not even
                        // -inf (a row with fewer than K0 elements), or the hit loop below would read
                        // stages that do not exist
                        pm[s * SK_VPT + j] = ((valid >> j) & 1u) ? P::part_max(part) : __uint_as_float(0x7FC00000u);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < SK_VPT; ++j) pm[s * SK_VPT + j] = __uint_as_float(0x7FC00000u);
                }
            }
            if (tid == 0) P::merge(acc, P::reduce(qt));
            ASX_MARK(2);
            ASX_CTA(2);
            threshold(acc, gmax, t0key, cut, 0u);
            ASX_MARK(3);
            ASX_CTA(3);
            const bool bad = gmax >= Tr::KEY_PINF || gmax <= Tr::KEY_NINF;
            if (bad) {
                r = failed_lane(c_in, ST_NUMERIC);
                decided = true;
                for (int s = 0; s < nsl_l; ++s) release(s);
            } else if (!cut) {
                // (launches of this kernel always carry a cut it can serve; a row without one is deferred)
                whole_row = true;
                for (int s = 0; s < nsl_l; ++s) release(s);
            } else {
                ref = Tr::value_f(gmax);
                t0f = Tr::value_f(t0key);
                if (!want_tail) {
                    // the threshold is final here: vectors whose maximum passes give their elements
                    // straight to the candidate list
                    unsigned hm = 0;
#pragma unroll
                    for (int i = 0; i < SK_RES_STAGES * SK_VPT; ++i) hm |= (pm[i] >= t0f ? 1u : 0u) << i;
#pragma unroll 1
                    while (hm) {
                        const int i = __ffs(hm) - 1;
                        hm &= hm - 1;
                        const int s = i / SK_VPT, v = (i % SK_VPT) * NT + tid;
                        const uint4 q = ringv[ASX_AT((size_t)stage_of(s) * SK_STAGE_VEC + v, (size_t)S * SK_STAGE_VEC, 50)];
                        float unused = 0.f;
                        push_vec(q, (s * SK_STAGE_VEC + v) * E - lead, t0f, t0key, false, ref, unused);
                    }
                } else {
#pragma unroll 1
                    for (int s = 0; s < nsl_l; ++s) {
                        uint4 q[SK_VPT];
                        const unsigned valid = load_slice(ringv + (size_t)stage_of(s) * SK_STAGE_VEC,
                                                          min(SK_STAGE_VEC, bulk_vec_l - s * SK_STAGE_VEC), q);
                        slice_pass(q, s * SK_STAGE_VEC + tid, valid, false, acc, t0f, ref, tail);
                    }
                }
                for (int s = 0; s < nsl_l; ++s) release(s);     // the producer may refill: next row
            }
        } else {
            // ---- streamed: slice -> registers -> stage released; T0 at slices 0, 1, 2, 4, 8, ...
            int refresh_at = 1;
#ifdef ASX_PROFILE
            long long pw = 0, pl = 0, pt = 0, pc = 0, tt0;
#define ASX_ACC(var) do { const long long tt1 = clock64(); var += tt1 - tt0; tt0 = tt1; } while (0)
            tt0 = clock64();
#else
#define ASX_ACC(var) do {} while (0)
#endif
#pragma unroll 1
            for (int s = 0; s < nsl_l; ++s, advance(1)) {
                wait_full(0);
                ASX_ACC(pw);
                uint4 q[SK_VPT];
                const unsigned valid = load_slice(ringv + (size_t)g_st * SK_STAGE_VEC,
                                                  min(SK_STAGE_VEC, bulk_vec_l - s * SK_STAGE_VEC), q);
                release(0);
                if (UA && s == 0 && tid == 0 && lead) mask_lead<DT>(q[0], lead);
                ASX_ACC(pl);
                if (s == 0) {
#pragma unroll
                    for (int j = 0; j < SK_VPT; ++j) P::merge(acc, P::reduce(q[j]));
                }
                if (s == 0 || s == refresh_at) {
                    uint32_t gm, t0new;
                    threshold(acc, gm, t0new, true, t0key);
                    t0key = max(t0key, t0new);
                    t0f = Tr::value_f(t0key);
                    if (s == 0) ref = Tr::value_f(min(max(gm, Tr::KEY_NINF + 1), Tr::KEY_PINF - 1));
                    if (s == refresh_at) refresh_at <<= 1;
                }
                ASX_ACC(pt);
                slice_pass(q, s * SK_STAGE_VEC + tid, valid, s > 0, acc, t0f, ref, tail);
                ASX_ACC(pc);
            }
#ifdef ASX_PROFILE
            if (blockIdx.x == 0 && tid == 0) { g_asx_marks[24] = pw; g_asx_marks[25] = pl; g_asx_marks[26] = pt; g_asx_marks[27] = pc; }
#endif
            if (tid == 0) P::merge(acc, P::reduce(qt));
            // final max.  Lanes with a top-k also take the threshold that the whole row's subset maxima
            // give (the last refresh saw half the row): fewer candidates to rank, and every element
            // >= it sits in a listed vector, listed under an earlier, lower threshold.  Nucleus-only lanes
            // keep the lower one: their list must reach as deep as the nucleus, and a shallower list sends
            // more of them through the deepening pass (measured: 1024 x 128256 f32 228 -> 275 us).
            uint32_t t0last;
            threshold(acc, gmax, t0last, a.top_k > 0, t0key);
            if (a.top_k > 0) {
                t0key = max(t0key, t0last);
                t0f = Tr::value_f(t0key);
            }
            const bool bad = gmax >= Tr::KEY_PINF || gmax <= Tr::KEY_NINF;
            if (bad) {
                r = failed_lane(c_in, ST_NUMERIC);
                decided = true;
            }
        }

        // ---- hit vectors -> candidates >= the final threshold; the rest of them joins the tail
        ASX_MARK(4);
        // (rows that fit the ring with a top-k push their candidates directly: nothing is listed)
        const bool listed = !(resident && cut && !want_tail);
        if (listed) SyncC::sync();
        const int nvh = listed ? sm.vec_count : 0;
        bool list_ok = !decided && !whole_row && nvh <= SK_CAPV;
        if (list_ok) {
            for (int i = tid; i < nvh; i += NT) {
                const uint4 q = sm.u.ep.v.cvec[ASX_AT(i, SK_CAPV, 42)];
                // most listed vectors came in under an earlier, lower threshold
                if (!want_tail && !(P::part_max(P::reduce(q)) >= t0f)) continue;
                push_vec(q, sm.u.ep.cidx[i] * E - lead, t0f, t0key, want_tail, ref, tail);
            }
            // the ragged last vector lives in thread 0's registers
            if (tail_elems_l > 0 && tid == 0) push_vec(qt, bulk_vec_l * E - lead, t0f, t0key, want_tail, ref, tail);
        }
        if (!list_ok && !decided && !whole_row && nvh > SK_CAPV && !(UA && lead) && !*(volatile int*)&sm.poisoned) {
            // more hit vectors than the list holds: take the candidates in one more pass, against
            // the threshold that the whole row's subset maxima give now
            ASX_COUNT(8);
            uint32_t gm2, t0new;
            threshold(acc, gm2, t0new, true, t0key);
            t0key = max(t0key, t0new);
            t0f = Tr::value_f(t0key);
            tail = recollect_row<DT, StreamSmem>(sm, V, row, t0f, t0key, ref, scale2);
            list_ok = true;
        }
        double tailsum = 0.0;
        if (want_tail) {
            const double td = warp_sum_d((double)tail);
            if (lane == 0) sm.red_d[warp] = td;
        }
        SyncC::sync();                      // candidates complete; cvec is dead from here on
        if (want_tail) {
#pragma unroll
            for (int w = 0; w < SK_NW; ++w) tailsum += sm.red_d[w];
        }
        const int C = sm.cand_count;
        list_ok = list_ok && C > 0 && C <= SK_CAP;
        const double lmax = (double)Tr::value_f(gmax);
        // the tail was summed against `ref` (<= lmax); bring it to the true maximum
        if (want_tail) tailsum *= exp_nonpos(((double)ref - lmax) * a.inv_tau, sm.exp_tbl);
        ASX_MARK(5);
        ASX_CTA(5);
#ifdef ASX_PROFILE
        if (blockIdx.x == 0 && tid == 0) { g_asx_marks[20] = nvh; g_asx_marks[21] = C; }
#endif
        const double c = c_in == 1.0 ? ASX_ONE_BELOW : c_in;
        XpState xs = {XP_RANGE_TOP, 0ull, 0ull, 0ull};
        unsigned long long tcell = 0;
        if (XP) {            // the lane's code comes as the state of an arithmetic decoder
            xs.range = a.xp_state[(size_t)ln * 4]; xs.code = a.xp_state[(size_t)ln * 4 + 1];
            if (!xp_state_ok(xs)) { if (!decided) r = failed_lane(c_in, ST_NUMERIC); decided = true; xs.range = XP_RANGE_TOP; xs.code = 0ull; }
            tcell = xp_target(xs);
        }
        if (*(volatile int*)&sm.poisoned) {
            r = failed_lane(c_in, ST_TIMEOUT);
            decided = true;
        } else if (!decided && !(c_in >= 0.0 && c_in <= 1.0)) {
            r = failed_lane(c_in, ST_NUMERIC);
            decided = true;
        } else if (list_ok && (!want_tail || (tailsum == tailsum && tailsum < 1e300))) {
            decided = epilogue_ranked<DT, NT, SyncC, StreamSmem, XP>(sm, sm.u.ep.cand, sm.u.ep.v.rk.srt, sm.u.ep.v.rk.e, C, t0key, c,
                                                         lmax, a.inv_tau, a.top_k, a.top_p, tailsum, r, tcell);
        }
        if (!decided && want_tail && list_ok && !(UA && lead) && !*(volatile int*)&sm.poisoned) {
            // the nucleus reaches below the exact depth of the list: lower the threshold once
            ASX_COUNT(0);
            if (tid == 0) sm.b_i[2] = C;
            decided = deepen_nucleus<DT, StreamSmem, XP>(sm, V, scale2, a.inv_tau, a.top_p, row, gmax, t0f, tailsum, c, r, tcell);
        }
        if (!decided) {
            ASX_COUNT(5);
            if (nvh > SK_CAPV) ASX_COUNT(6);
            if (sm.cand_count > SK_CAP) ASX_COUNT(7);
        }
        if (resident) advance(nsl_l);
        if (tid == 0) {
            if (!decided) a.tokens[(size_t)ln * (GATHER ? a.tok_stride : 1)] = LANE_DEFERRED;
            else finish_lane<GATHER, XP>(a, ln, r, path, sm.xp_lo, sm.xp_hi);
        }
        SyncC::sync();
        ASX_MARK(12);
        ASX_CTA(6);
    }
    if (tid == 0 && *(volatile int*)&sm.poisoned) {
        // A wait ran out.  Copies armed before that may still be in flight into this CTA's shared
        // memory: the CTA does not leave before each armed stage has landed or its own bounded
        // wait has run out as well.  (The copy-issuing thread stops at its next wait once it sees
        // the flag, and says what it had armed.)
        const long long t0 = clock64();
        while (!*(volatile int*)&sm.prod_done && clock64() - t0 <= 2 * a.wait_cycles + 1000000) { }
        if (*(volatile int*)&sm.prod_done) {
            __threadfence_block();
            const unsigned pst = sm.prod_st, prd = sm.prod_round;
            for (unsigned st = 0; st < (unsigned)S; ++st) {
                const int rnd = (int)prd - (st < pst ? 0 : 1);       // the last round that armed this stage
                if (rnd >= 0 && !mbar_wait_bounded(smem_u32(&sm.full_bar[st]), (unsigned)rnd & 1u, a.wait_cycles)) break;
            }
        }
    }
    ASX_MARK(14);
    ASX_SPAN(2);
    ASX_CTA(7);
}

}  // namespace asx

// Streaming decode step: one CTA per lane for any vocabulary size, no inter-CTA
// communication (lanes are independent: Remark after Proposition 1).
//
// CTA = 8 consumer warps + 1 producer warp.  The producer's lane 0 feeds a ring of
// 16 KB shared-memory stages with bulk async copies (TMA, non-multicast; `full`
// mbarrier per stage carries the byte count, `empty` mbarrier per stage collects
// one arrival per consumer warp), running ahead across rows, so HBM reads never
// wait for compute.  Consumers see each row exactly once (Algorithm 1 needs every
// conditional probability once):
//   resident rows (row <= ring): all stages land, one NaN-propagating max pass,
//       one threshold T0, one compaction pass from shared memory;
//   streamed rows (row > ring): each 16 KB slice goes shared memory -> registers,
//       the stage is released at once, the slice is folded into the running
//       max and compacted against the current T0; T0 is recomputed at slices
//       0, 1, 2, 4, 8, ... and only ever rises.
// T0 is a lower bound on the K0-th largest logit: each warp takes the m-th
// largest (m = ceil(K0 / 8)) of its 64 per-thread subset maxima by a 16-step
// ballot search, and T0 is the smallest of the 8 warp values, so at least K0
// elements are >= T0.  Every element >= T0 is appended to a candidate list.
// The epilogue is exact and fp64 on that list only: bitonic sort by (value desc,
// index asc), top-k, masses, nucleus prefix, sort by index, CDF prefix,
// crossing, rescale (Algorithm 1: w_i, (m, M), c <- (c - m)/(M - m)).
// For nucleus-only lanes the masses of non-candidates are summed in fp32 (they
// only enter the nucleus target top_p * Z1).  Lanes the list cannot decide
// (too many candidates, nucleus deeper than the list, unaligned rows) go to
// GenericLane, which reads the row from global memory (L2).
#pragma once
#include "as_staged.cuh"

namespace asx {

constexpr int SK_NT = 256;                 // consumer threads
constexpr int SK_NW = SK_NT / 32;          // consumer warps
constexpr int SK_THREADS = SK_NT + 32;     // + producer warp
constexpr int SK_CAP = 1024;               // candidate capacity per lane
constexpr int SK_STAGE_VEC = 1024;         // 16-byte vectors per stage (16 KB)
constexpr int SK_STAGE_BYTES = SK_STAGE_VEC * 16;
constexpr int SK_VPT = SK_STAGE_VEC / SK_NT;   // vectors per consumer thread per slice
constexpr int SK_MAXSTAGES = 12;
constexpr int SK_K0_MAX = 128;             // largest top_k served by the candidate list
constexpr int SK_KP = 96;                  // K0 for nucleus-only lanes

using SyncC = SyncNamed<SK_NT>;

struct StreamSmem {
    unsigned long long full_bar[SK_MAXSTAGES];
    unsigned long long empty_bar[SK_MAXSTAGES];
    union {
        struct {
            unsigned long long cand[SK_CAP];    // (key << 32) | ~index
            unsigned long long isort[SK_CAP];   // (index << 32) | rank
            double e[SK_CAP];                   // mass by rank
        } ep;
        GenericSmem<SK_NT> gen;
    } u;
    double exp_tbl[64];
    double red_d[SK_NW];
    unsigned wmax[SK_NW];
    unsigned wsel[SK_NW];
    int cand_count;
    int poisoned;        // a bounded wait ran out: stop issuing / stop waiting
    int b_i[4];
    LaneResult res;
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// m-th largest (1-based) of the 64 16-bit keys held two per lane, by binary search on the
// value: the largest v with count(keys >= v) >= m.
__device__ __forceinline__ uint32_t warp_select16(uint32_t a16, uint32_t b16, int m) {
    uint32_t res = 0;
#pragma unroll
    for (int bit = 15; bit >= 0; --bit) {
        const uint32_t cand = res | (1u << bit);
        const int cnt = __popc(__ballot_sync(FULL, a16 >= cand)) + __popc(__ballot_sync(FULL, b16 >= cand));
        if (cnt >= m) res = cand;
    }
    return res;
}

// bitonic sort of a[0..P) (P a power of two) by NT threads; DESC: largest first
template <int NT, class Sync, bool DESC>
__device__ void bitonic_sort(unsigned long long* a, int P, int tid) {
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < P; i += NT) {
                const int ixj = i ^ j;
                if (ixj > i) {
                    const unsigned long long x = a[i], y = a[ixj];
                    const bool first_big = ((i & k) == 0) == DESC;   // this pair wants the larger first
                    if ((x < y) == first_big) { a[i] = y; a[ixj] = x; }
                }
            }
            Sync::sync();
        }
    }
}

// Exact decode on the candidate list.  t0_final: every element of the row with key >= t0_final is
// in the list, so ranks are exact down to that key.  Returns false if the list cannot decide.
template <int DT, int NT, class Sync>
__device__ bool epilogue_sorted(StreamSmem& sm, int C, uint32_t t0_final, double c, double lmax,
                                double inv_tau, int top_k, double top_p, double tail, LaneResult& out) {
    using Tr = Traits<DT>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long* cand = sm.u.ep.cand;
    unsigned long long* isort = sm.u.ep.isort;
    double* e = sm.u.ep.e;
    int P = 32;
    while (P < C) P <<= 1;
    for (int i = C + tid; i < P; i += NT) cand[i] = 0ull;     // sorts after every real candidate
    Sync::sync();
    bitonic_sort<NT, Sync, true>(cand, P, tid);
    const int kmax = (top_k > 0 && top_k < C) ? top_k : C;
    for (int r = tid; r < kmax; r += NT)
        e[r] = exp_nonpos(((double)Tr::value_f((uint32_t)(cand[r] >> 32)) - lmax) * inv_tau, sm.exp_tbl);
    Sync::sync();
    if (warp == 0) {
        // prefix masses in rank order: nucleus on the distribution renormalised over the survivors
        const int per = (kmax + 31) / 32;
        const int b = min(lane * per, kmax), en = min(b + per, kmax);
        double s = 0.0;
        for (int r = b; r < en; ++r) s += e[r];
        const double incl = warp_incl_scan_d(s, lane);
        const double total = __shfl_sync(FULL, incl, 31);
        int n_final = kmax, ok = 1;
        if (top_p < 1.0) {
            const double target = top_p * (total + tail);
            double run = __shfl_up_sync(FULL, incl, 1);
            if (lane == 0) run = 0.0;
            int below = 0;
            for (int r = b; r < en; ++r) { run += e[r]; below += (run < target); }
            below = warp_sum_i(below);
            if (below >= kmax) {
                if (top_k == 0) ok = 0;        // nucleus-only: it reaches past the list
            } else {
                n_final = below + 1;
            }
        }
        if (lane == 0) { sm.b_i[0] = n_final; sm.b_i[1] = ok; }
    }
    Sync::sync();
    const int n_final = sm.b_i[0];
    if (!sm.b_i[1]) return false;
    if ((uint32_t)(cand[n_final - 1] >> 32) < t0_final) return false;   // cut below the exact depth
    int P2 = 32;
    while (P2 < n_final) P2 <<= 1;
    for (int i = tid; i < P2; i += NT)
        isort[i] = i < n_final ? (((unsigned long long)(~(uint32_t)cand[i])) << 32) | (uint32_t)i : ~0ull;
    Sync::sync();
    bitonic_sort<NT, Sync, false>(isort, P2, tid);
    if (warp == 0) {
        const int per = (n_final + 31) / 32;
        const int b = min(lane * per, n_final), en = min(b + per, n_final);
        double s = 0.0;
        for (int i = b; i < en; ++i) s += e[(uint32_t)isort[i]];
        const double incl = warp_incl_scan_d(s, lane);
        double run = __shfl_up_sync(FULL, incl, 1);
        if (lane == 0) run = 0.0;
        double zrun = run;                       // Z continues the same running sum as the prefixes
        for (int i = b; i < en; ++i) zrun += e[(uint32_t)isort[i]];
        const double Z = __shfl_sync(FULL, zrun, (n_final - 1) / per);
        const double t = c * Z;
        int pick = -1;
        double pS = 0.0, pe = 1.0;
        for (int i = b; i < en; ++i) {
            const double ev = e[(uint32_t)isort[i]];
            if (pick < 0 && (t < run + ev || i == n_final - 1)) { pick = i; pS = run; pe = ev; }
            run += ev;
        }
        const unsigned bal = __ballot_sync(FULL, pick >= 0);
        const int L = __ffs(bal) - 1;
        pick = __shfl_sync(FULL, pick, L);
        pS = __shfl_sync(FULL, pS, L);
        pe = __shfl_sync(FULL, pe, L);
        if (lane == 0) {
            double cn = (t - pS) / pe;
            if (!(cn >= 0.0)) cn = 0.0;
            if (cn > ASX_ONE_BELOW) cn = ASX_ONE_BELOW;
            LaneResult r;
            r.token = (int)(isort[pick] >> 32); r.status = ST_OK; r.n_kept = n_final; r.code_out = cn;
            r.p_tok = pe / Z; r.cdf_lo = pS / Z;
            sm.res = r;
        }
    }
    Sync::sync();
    out = sm.res;
    return true;
}

template <int DT>
__global__ void __launch_bounds__(SK_THREADS) step_stream_kernel(const StepArgs a, const int stages) {
    using Tr = Traits<DT>;
    using P = Pass<DT>;
    constexpr int E = Tr::E;
    constexpr int NT = SK_NT;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    StreamSmem& sm = *reinterpret_cast<StreamSmem*>(smem_raw);
    unsigned char* ring = smem_raw + ((sizeof(StreamSmem) + 127) & ~(size_t)127);
    const uint4* ringv = reinterpret_cast<const uint4*>(ring);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int V = a.V;
    const int row_bytes = V * Tr::BYTES;
    const int bulk_bytes = row_bytes & ~15;
    const int bulk_vec = bulk_bytes >> 4;
    const int tail_elems = (row_bytes - bulk_bytes) / Tr::BYTES;      // < E
    const int nsl = (bulk_vec + SK_STAGE_VEC - 1) / SK_STAGE_VEC;      // slices per row
    const bool resident = nsl <= stages;
    const int S = resident ? max(nsl, 1) : stages;                     // ring length in use

    if (tid == 0) {
        for (int i = 0; i < SK_MAXSTAGES; ++i) {
            mbar_init(smem_u32(&sm.full_bar[i]), 1);
            mbar_init(smem_u32(&sm.empty_bar[i]), SK_NW);
        }
        fence_mbar_init();
        sm.poisoned = 0;
    }
    fill_exp_table(sm.exp_tbl, tid);
    __syncthreads();

    auto row_of = [&](int ln) -> const char* {
        return reinterpret_cast<const char*>(a.logits) + (size_t)ln * (size_t)a.ld * Tr::BYTES;
    };
    auto staged_ok = [&](int ln) -> bool { return (reinterpret_cast<uintptr_t>(row_of(ln)) & 15) == 0; };

    // =========================== producer warp ===========================
    if (warp == SK_NW) {
        if (lane == 0) {
            unsigned g = 0;                       // slices issued so far (ring position)
            for (int ln = blockIdx.x; ln < a.lanes; ln += gridDim.x) {
                if (!staged_ok(ln)) continue;
                const char* src = row_of(ln);
                for (int s = 0; s < nsl; ++s, ++g) {
                    const int st = g % S;
                    if (g >= (unsigned)S) {       // the stage must have been drained by every consumer warp
                        if (*(volatile int*)&sm.poisoned) return;
                        if (!mbar_wait_bounded(smem_u32(&sm.empty_bar[st]), ((g / S) - 1) & 1)) {
                            *(volatile int*)&sm.poisoned = 1;
                            return;
                        }
                    }
                    const uint32_t bytes = (uint32_t)min(SK_STAGE_BYTES, bulk_bytes - s * SK_STAGE_BYTES);
                    const uint32_t bar = smem_u32(&sm.full_bar[st]);
                    fence_proxy_async();
                    mbar_expect_tx(bar, bytes);
                    bulk_g2s(smem_u32(ring + (size_t)st * SK_STAGE_BYTES), src + (size_t)s * SK_STAGE_BYTES, bytes, bar);
                }
            }
        }
        return;
    }

    // =========================== consumer warps ===========================
    const bool want_tail = (a.top_k == 0);        // nucleus-only: masses of non-candidates in fp32
    const int K0 = a.top_k > 0 ? a.top_k : SK_KP;
    const int m_sel = (K0 + SK_NW - 1) / SK_NW;
    unsigned g = 0;

    // block step: max so far and threshold from the subset maxima held in `acc`
    auto threshold = [&](const typename P::Acc& acc, uint32_t& gmax, uint32_t& t0key) {
        uint32_t k0, k1;
        P::keys(acc, k0, k1);
        const uint32_t wm = warp_max_u(max(k0, k1));
        const uint32_t ws = warp_select16(P::key16(k0), P::key16(k1), m_sel);
        SyncC::sync();                           // previous readers of wmax / wsel are done
        if (lane == 0) { sm.wmax[warp] = wm; sm.wsel[warp] = ws; }
        SyncC::sync();
        gmax = 0;
        uint32_t t16 = 0xFFFFFFFFu;
#pragma unroll
        for (int w = 0; w < SK_NW; ++w) { gmax = max(gmax, sm.wmax[w]); t16 = min(t16, sm.wsel[w]); }
        t0key = max(P::key_from16(t16), Tr::KEY_NINF);
    };
    // compaction of one vector: candidates to the list, the rest to the fp32 tail
    auto compact = [&](const uint4& q, int vec_index, uint32_t t0key, float t0f, float ref, float& tail) {
        if (!want_tail) {
            if (P::vmax(q) >= t0f) {
                float x[E];
                P::floats(q, x);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    if (x[e] >= t0f) {
                        const uint32_t key = P::key_of_f(x[e]);
                        if (key >= t0key && key > Tr::KEY_NINF) {
                            const int slot = atomicAdd(&sm.cand_count, 1);
                            if (slot < SK_CAP)
                                sm.u.ep.cand[slot] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)(vec_index * E + e);
                        }
                    }
                }
            }
        } else {
            float x[E];
            P::floats(q, x);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const float ev = ex2_approx((x[e] - ref) * a.scale2);
                bool pushed = false;
                if (x[e] >= t0f) {
                    const uint32_t key = P::key_of_f(x[e]);
                    if (key >= t0key && key > Tr::KEY_NINF) {
                        pushed = true;
                        const int slot = atomicAdd(&sm.cand_count, 1);
                        if (slot < SK_CAP)
                            sm.u.ep.cand[slot] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)(vec_index * E + e);
                    }
                }
                tail += pushed ? 0.f : ev;
            }
        }
    };

    for (int ln = blockIdx.x; ln < a.lanes; ln += gridDim.x) {
        const double c_in = a.codes[ln];
        double c = c_in;
        const bool code_bad = !(c >= 0.0 && c <= 1.0);
        if (c == 1.0) c = ASX_ONE_BELOW;
        const char* row = row_of(ln);

        if (!staged_ok(ln)) {        // unaligned row: general routine from global memory
            GenericLane<DT, NT, SyncC> gl(sm.u.gen, row, V, false);
            const LaneResult r = gl.run(c_in, a.inv_tau, a.top_k, a.top_p);
            if (tid == 0) write_result(a, ln, r, PATH_GENERAL);
            continue;
        }
        if (tid == 0) sm.cand_count = 0;

        // ragged end of the row (< 16 bytes): one padded vector read straight from global memory
        uint4 qt = make_uint4(0, 0, 0, 0);
        if (tail_elems > 0 && tid == 0) {
            uint32_t w[4];
            if (DT == DT_BF16) {
                const unsigned short* src = reinterpret_cast<const unsigned short*>(row + bulk_bytes);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t lo = (2 * i < tail_elems) ? src[2 * i] : 0xFF80u;
                    const uint32_t hi = (2 * i + 1 < tail_elems) ? src[2 * i + 1] : 0xFF80u;
                    w[i] = lo | (hi << 16);
                }
            } else {
                const uint32_t* src = reinterpret_cast<const uint32_t*>(row + bulk_bytes);
#pragma unroll
                for (int i = 0; i < 4; ++i) w[i] = (i < tail_elems) ? src[i] : 0xFF800000u;
            }
            qt = make_uint4(w[0], w[1], w[2], w[3]);
        }

        typename P::Acc acc = P::init();
        uint32_t gmax = 0, t0key = Tr::KEY_NINF;
        float tail = 0.f;
        float ref = 0.f;             // exponent reference of the fp32 tail
        bool timed_out = false;
        const bool cut = a.fast && (a.top_k > 0 || a.top_p < 1.0);

        auto wait_full = [&](unsigned gg) {
            if (*(volatile int*)&sm.poisoned) { timed_out = true; return; }
            if (!mbar_wait_bounded(smem_u32(&sm.full_bar[gg % S]), (gg / S) & 1)) {
                timed_out = true;
                *(volatile int*)&sm.poisoned = 1;
            }
        };
        auto release = [&](unsigned gg) {
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sm.empty_bar[gg % S]));
        };

        if (resident) {
            // ---- all stages land; max pass from shared memory
            for (int s = 0; s < nsl; ++s) {
                wait_full(g + s);
                const int nv = min(SK_STAGE_VEC, bulk_vec - s * SK_STAGE_VEC);
                const uint4* sv = ringv + (size_t)((g + s) % S) * SK_STAGE_VEC;
#pragma unroll
                for (int j = 0; j < SK_VPT; ++j) {
                    const int v = j * NT + tid;
                    if (v < nv) P::fold(acc, sv[v]);
                }
            }
            if (tail_elems > 0 && tid == 0) P::fold(acc, qt);
            threshold(acc, gmax, t0key);
            const bool bad = code_bad || gmax >= Tr::KEY_PINF || gmax <= Tr::KEY_NINF;
            if (bad || !cut) {
                LaneResult r;
                if (bad) {
                    r = failed_lane(c_in, ST_NUMERIC);
                } else {
                    // no cut: every token is kept; the general routine scans the row in shared memory
                    if (tail_elems > 0 && tid < tail_elems) {
                        if (DT == DT_BF16)
                            reinterpret_cast<unsigned short*>(ring + bulk_bytes)[tid] =
                                reinterpret_cast<const unsigned short*>(row + bulk_bytes)[tid];
                        else
                            reinterpret_cast<uint32_t*>(ring + bulk_bytes)[tid] =
                                reinterpret_cast<const uint32_t*>(row + bulk_bytes)[tid];
                    }
                    SyncC::sync();
                    GenericLane<DT, NT, SyncC> gl(sm.u.gen, ring, V, true);
                    r = gl.run(c_in, a.inv_tau, a.top_k, a.top_p);
                }
                for (int s = 0; s < nsl; ++s) release(g + s);
                g += nsl;
                if (tid == 0) write_result(a, ln, r, bad ? PATH_COMPACT : PATH_GENERAL);
                continue;
            }
            ref = Tr::value_f(gmax);
            const float t0f = Tr::value_f(t0key);
            for (int s = 0; s < nsl; ++s) {
                const int nv = min(SK_STAGE_VEC, bulk_vec - s * SK_STAGE_VEC);
                const uint4* sv = ringv + (size_t)((g + s) % S) * SK_STAGE_VEC;
#pragma unroll
                for (int j = 0; j < SK_VPT; ++j) {
                    const int v = j * NT + tid;
                    if (v < nv) compact(sv[v], s * SK_STAGE_VEC + v, t0key, t0f, ref, tail);
                }
            }
            if (tail_elems > 0 && tid == 0) compact(qt, bulk_vec, t0key, t0f, ref, tail);
            for (int s = 0; s < nsl; ++s) release(g + s);     // the producer may refill: next row
            g += nsl;
        } else {
            // ---- streamed: slice -> registers -> stage released; T0 at slices 0, 1, 2, 4, 8, ...
            int refresh_at = 1;
            float t0f = 0.f;
            for (int s = 0; s < nsl; ++s, ++g) {
                wait_full(g);
                const int nv = min(SK_STAGE_VEC, bulk_vec - s * SK_STAGE_VEC);
                const uint4* sv = ringv + (size_t)(g % S) * SK_STAGE_VEC;
                uint4 q[SK_VPT];
#pragma unroll
                for (int j = 0; j < SK_VPT; ++j) {
                    const int v = j * NT + tid;
                    q[j] = (v < nv) ? sv[v] : make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
                }
                if (DT == DT_F32) {
#pragma unroll
                    for (int j = 0; j < SK_VPT; ++j)
                        if (j * NT + tid >= nv) q[j] = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
                }
                release(g);
                if (s == 0) {
#pragma unroll
                    for (int j = 0; j < SK_VPT; ++j) P::fold(acc, q[j]);
                }
                if (s == 0 || s == refresh_at) {
                    uint32_t gm, t0new;
                    threshold(acc, gm, t0new);
                    t0key = max(t0key, t0new);
                    t0f = Tr::value_f(t0key);
                    if (s == 0) ref = Tr::value_f(min(max(gm, Tr::KEY_NINF + 1), Tr::KEY_PINF - 1));
                    if (s == refresh_at) refresh_at <<= 1;
                }
                if (s > 0) {
#pragma unroll
                    for (int j = 0; j < SK_VPT; ++j) P::fold(acc, q[j]);
                }
#pragma unroll
                for (int j = 0; j < SK_VPT; ++j) {
                    const int v = j * NT + tid;
                    if (v < nv) compact(q[j], s * SK_STAGE_VEC + v, t0key, t0f, ref, tail);
                }
            }
            if (tail_elems > 0 && tid == 0) {
                P::fold(acc, qt);
                compact(qt, bulk_vec, t0key, t0f, ref, tail);
            }
            uint32_t t0unused;
            threshold(acc, gmax, t0unused);       // final max (t0key keeps the value candidates were taken with)
            const bool bad = code_bad || gmax >= Tr::KEY_PINF || gmax <= Tr::KEY_NINF;
            if (bad) {
                if (tid == 0) write_result(a, ln, failed_lane(c_in, ST_NUMERIC), PATH_COMPACT);
                continue;
            }
        }

        // ---- candidate list complete: tail mass, then the exact epilogue
        double tailsum = 0.0;
        if (want_tail) {
            const double td = warp_sum_d((double)tail);
            SyncC::sync();
            if (lane == 0) sm.red_d[warp] = td;
            SyncC::sync();
#pragma unroll
            for (int w = 0; w < SK_NW; ++w) tailsum += sm.red_d[w];
        } else {
            SyncC::sync();
        }
        (void)timed_out;                          // a wait that ran out has set sm.poisoned
        const double lmax = (double)Tr::value_f(gmax);
        // the tail was summed against `ref` (<= lmax); bring it to the true maximum
        if (want_tail) tailsum *= exp_nonpos(((double)ref - lmax) * a.inv_tau, sm.exp_tbl);
        const int C = sm.cand_count;
        LaneResult r;
        bool done = false;
        if (*(volatile int*)&sm.poisoned) {
            r = failed_lane(c_in, ST_TIMEOUT);
            done = true;
        } else if (C > 0 && C <= SK_CAP && (!want_tail || (tailsum == tailsum && tailsum < 1e300))) {
            done = epilogue_sorted<DT, NT, SyncC>(sm, C, t0key, c, lmax, a.inv_tau, a.top_k, a.top_p, tailsum, r);
        }
        const int path = done ? PATH_COMPACT : PATH_GENERAL;
        if (!done) {
            SyncC::sync();
            GenericLane<DT, NT, SyncC> gl(sm.u.gen, row, V, true);
            r = gl.run(c_in, a.inv_tau, a.top_k, a.top_p);
        }
        if (tid == 0) write_result(a, ln, r, path);
        SyncC::sync();
    }
}

}  // namespace asx

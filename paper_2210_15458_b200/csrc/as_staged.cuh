// Staged decode step: the HBM-bound path.
//
// One CTA (CS = 1) or one thread-block cluster of CS CTAs owns a lane at a time
// and loops over lanes (persistent grid).  Per lane:
//   load    the row (or this CTA's 1/CS slice of it) is brought into shared
//           memory ONCE by bulk async copies (TMA, 8 KB each, one mbarrier per
//           copy) -- the only HBM read of the step (Algorithm 1 needs each
//           conditional probability once);
//   pass 1  as the copies land: NaN-propagating max, kept as two disjoint
//           "subset maxima" per thread;
//   cut     when a top-k / nucleus cut is active, a lower bound T0 on the value
//           of the K0-th largest logit is taken from the subset maxima (the
//           K0-th largest of M maxima of disjoint subsets is below at least K0
//           elements), ranks exchange max and T0 through distributed shared
//           memory;
//   pass 2  from shared memory: every element >= T0 is appended to the lane
//           leader's candidate list (a few dozen to a few hundred entries); for
//           nucleus-only lanes the same pass also sums exp() of the rest in
//           fp32 (the deep tail only enters the nucleus target top_p * Z1);
//   next    the next lane's copies are issued, so they overlap the epilogue;
//   epilogue (leader CTA) exact, fp64, on the candidate list only: ranks by
//           (value desc, index asc), top-k, masses, nucleus prefix, index-order
//           prefix, crossing, rescale (Algorithm 1's w_i, (m, M), c <- (c-m)/(M-m)).
// Anything the compaction cannot serve (unaligned rows, too many candidates, a
// nucleus reaching beyond the candidates, no cut at all) goes to GenericLane.
#pragma once
#include "as_generic.cuh"
#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace asx {

constexpr int ST_NT = 512;             // threads per CTA
constexpr int ST_CAP = 512;            // candidate capacity per lane
constexpr int ST_CHUNK_VEC = ST_NT;    // 16-byte vectors per bulk copy: one per thread
constexpr int ST_CHUNK_BYTES = ST_CHUNK_VEC * 16;
constexpr int ST_MAXCHUNK = 27;        // 27 * 8 KB = 216 KB
constexpr int ST_M = 2 * ST_NT;        // subset maxima per CTA
constexpr int ST_KP = 256;             // candidates aimed at for nucleus-only lanes
constexpr long long ST_WAIT_CYCLES = 2000000000LL;   // ~1 s: default bound on any mbarrier wait

// Phase timestamps of CTA 0 for profiling builds (-DASX_PROFILE); compiled out otherwise.
#ifdef ASX_PROFILE
__device__ long long g_asx_marks[32];
__device__ unsigned long long g_asx_counts[16];
__device__ unsigned long long g_asx_span[4];      // first / last CTA start, first / last CTA end (globaltimer, ns)
__device__ __forceinline__ void asx_span(int i) {
    if (threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        atomicMin(&g_asx_span[i], t);
        atomicMax(&g_asx_span[i + 1], t);
    }
}
#define ASX_SPAN(i) asx_span(i)
__device__ unsigned long long g_asx_cta[1024][8];  // per-CTA phase times of its first lane (globaltimer, ns)
__device__ __forceinline__ void asx_cta(int i) {
    if (threadIdx.x == 0 && blockIdx.x < 1024) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_asx_cta[blockIdx.x][i] = t;
    }
}
#define ASX_CTA(i) asx_cta(i)
#define ASX_MARK(i) do { if (blockIdx.x == 0 && threadIdx.x == 0) g_asx_marks[i] = clock64(); } while (0)
#define ASX_COUNT(i) do { if (threadIdx.x == 0) atomicAdd(&g_asx_counts[i], 1ull); } while (0)
#else
#define ASX_MARK(i) do {} while (0)
#define ASX_COUNT(i) do {} while (0)
#define ASX_SPAN(i) do {} while (0)
#define ASX_CTA(i) do {} while (0)
#endif

struct DiagOut {
    double* p_tok;
    double* cdf_lo;
    int* n_kept;
    int* lane_status;
    int* path;
};
constexpr int PATH_COMPACT = 0;
constexpr int PATH_GENERAL = 1;

struct StepArgs {
    const void* logits;
    const double* codes;
    int* tokens;
    double* codes_out;
    DiagOut diag;
    long long ld;
    double inv_tau;
    double top_p;
    float scale2;      // log2(e) / temp, for the fp32 tail
    int lanes;
    int V;
    int top_k;
    int fast;          // 1: try the compaction path for lanes with a cut
    // lat_N > 0: the codes are the lattice itself, lane i taking c = (lat_j0 + i + lat_u) / lat_N
    // mod 1 (the same fp64 expression as the lattice kernel), and `codes` is not read
    int lat_N;
    int lat_j0;
    double lat_u;
    // Row gather (builds with GATHER; the decode loop over a table): lane ln reads row
    // row_idx[ln * idx_stride] of `logits`; a lane whose index is negative, equal to `eos` or
    // not below `rows` is skipped altogether (nothing read, nothing written).  Tokens go to
    // tokens[ln * tok_stride].
    const int* row_idx;
    int idx_stride;
    int tok_stride;
    int eos;
    int rows;
    int radix_nucleus;        // 1: the general routine finds every nucleus by its radix select
    // extended-precision decode (builds with XP): the lanes' decoder states [lanes, 4], read and
    // written in place, and the lattice size that drives their digit source
    unsigned long long* xp_state;
    int xp_N;
    // bound on every mbarrier wait, in clock cycles; when it runs out the lane reports ST_TIMEOUT
    long long wait_cycles;
    // test of the time-out path only: the copy-issuing thread issues nothing, so every wait runs out
    int debug_no_copy;
};

__device__ __forceinline__ double lane_code(const StepArgs& a, int ln) {
    if (a.lat_N > 0) {
        double c = ((double)(a.lat_j0 + ln) + a.lat_u) / (double)a.lat_N;
        if (c >= 1.0) c -= 1.0;
        return c;
    }
    return a.codes[ln];
}

// ---------------------------------------------------------------------------
// PTX wrappers: mbarrier + bulk async copy global -> shared
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// dst, src 16-byte aligned, bytes a multiple of 16; completes on `bar`; the copy lands in this CTA only
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// waits for the phase with the given parity; gives up after `limit` clock cycles
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                     " selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (clock64() - t0 > limit) return false;
    }
}
// ---------------------------------------------------------------------------
// shared memory
// ---------------------------------------------------------------------------
struct EpiSmem {
    double e[ST_CAP];                 // mass by rank
    double e_idx[ST_CAP];             // mass by index order
    int tok_idx[ST_CAP];              // token by index order
    unsigned short order[ST_CAP];     // rank -> candidate slot
};

template <int NT>
struct StagedSmem {
    unsigned long long bars[ST_MAXCHUNK + 1];
    unsigned long long cand[ST_CAP];  // (key << 32) | ~index : larger = ranks earlier
    union {
        EpiSmem ep;
        GenericSmem<NT> gen;
    } u;
    unsigned submax[ST_M];
    int hist[256];
    double exp_tbl[64];
    unsigned xch_max[8];
    unsigned xch_t0[8];
    int xch_flag[8];
    double xch_tail[8];
    double red_d[NT / 32];
    unsigned red_u[NT / 32];
    int cand_count;
    int b_i[4];
    LaneResult res;
};

__device__ __forceinline__ void write_result(const StepArgs& a, int ln, const LaneResult& r, int path) {
    if (a.diag.path) a.diag.path[ln] = path;
    a.tokens[ln] = r.token;
    a.codes_out[ln] = r.code_out;
    if (a.diag.p_tok) a.diag.p_tok[ln] = r.p_tok;
    if (a.diag.cdf_lo) a.diag.cdf_lo[ln] = r.cdf_lo;
    if (a.diag.n_kept) a.diag.n_kept[ln] = r.n_kept;
    if (a.diag.lane_status) a.diag.lane_status[ln] = r.status;
}

__device__ __forceinline__ LaneResult failed_lane(double c_in, int status) {
    LaneResult r;
    r.token = -1; r.status = status; r.n_kept = 0; r.code_out = c_in; r.p_tok = 0.0; r.cdf_lo = 0.0;
    return r;
}

// K-th largest (1-based) of the upper 16 key bits of sm.submax[0..ST_M): two 8-bit radix
// passes.  K <= ST_M.  All threads of the CTA call it; the result is uniform.
template <int DT, int NT>
__device__ uint32_t select_kth16(StagedSmem<NT>& sm, int K) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t prefix = 0;
    int remaining = K;
#pragma unroll 1
    for (int shift = 8; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += NT) sm.hist[i] = 0;
        __syncthreads();
        for (int m = tid; m < ST_M; m += NT) {
            const uint32_t k16 = Pass<DT>::key16(sm.submax[m]);
            if (shift == 8 || (k16 >> 8) == prefix) atomicAdd(&sm.hist[(k16 >> shift) & 255], 1);
        }
        __syncthreads();
        if (warp == 0) {
            int c[8], lc = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) { c[e] = sm.hist[lane * 8 + e]; lc += c[e]; }
            const int suf = warp_suffix_i(lc, lane);
            int above = __shfl_down_sync(FULL, suf, 1);
            if (lane == 31) above = 0;
            int best = -1, best_above = 0, run = above;
#pragma unroll
            for (int e = 7; e >= 0; --e) {
                if (best < 0 && c[e] > 0 && run + c[e] >= remaining) { best = lane * 8 + e; best_above = run; }
                run += c[e];
            }
            const unsigned bal = __ballot_sync(FULL, best >= 0);
            const int src = bal ? 31 - __clz(bal) : 0;
            best = __shfl_sync(FULL, best, src);
            best_above = __shfl_sync(FULL, best_above, src);
            if (lane == 0) { sm.b_i[0] = best < 0 ? 0 : best; sm.b_i[1] = best_above; }
        }
        __syncthreads();
        remaining -= sm.b_i[1];
        prefix = (shift == 8) ? (uint32_t)sm.b_i[0] : ((prefix << 8) | (uint32_t)sm.b_i[0]);
        __syncthreads();
    }
    return prefix;
}

// Exact decode on the candidate list of the leader CTA.  Returns false if the list cannot
// decide the lane (nucleus-only lane whose nucleus reaches past the candidates).
template <int DT, int NT>
__device__ bool epilogue(StagedSmem<NT>& sm, int C, double c, double c_in, double lmax, double inv_tau,
                         int top_k, double top_p, double tail, LaneResult& out) {
    using Tr = Traits<DT>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    EpiSmem& ep = sm.u.ep;
    // ranks by (value desc, index asc): composites are distinct, so ranks are a permutation
    for (int i = tid; i < C; i += NT) {
        const unsigned long long ci = sm.cand[i];
        int r = 0;
        for (int j = 0; j < C; ++j) r += (sm.cand[j] > ci);
        ep.order[ASX_AT(r, ST_CAP, 91)] = (unsigned short)i;
    }
    __syncthreads();
    ASX_MARK(8);
    const int kmax = (top_k > 0 && top_k < C) ? top_k : C;
    for (int r = tid; r < kmax; r += NT) {
        const uint32_t key = (uint32_t)(sm.cand[ep.order[r]] >> 32);
        ep.e[r] = exp_nonpos(((double)Tr::value_f(key) - lmax) * inv_tau, sm.exp_tbl);
    }
    __syncthreads();
    ASX_MARK(9);
    // nucleus on the distribution renormalised over the survivors: prefix masses in rank order
    if (warp == 0) {
        const int per = (kmax + 31) / 32;
        const int b = min(lane * per, kmax), e = min(b + per, kmax);
        double s = 0.0;
        for (int r = b; r < e; ++r) s += ep.e[r];
        const double incl = warp_incl_scan_d(s, lane);
        const double total = __shfl_sync(FULL, incl, 31);
        int n_final = kmax;
        int ok = 1;
        if (top_p < 1.0) {
            const double target = top_p * (total + tail);
            double run = __shfl_up_sync(FULL, incl, 1);
            if (lane == 0) run = 0.0;
            int below = 0;                     // ranks whose inclusive prefix is still under the target
            for (int r = b; r < e; ++r) { run += ep.e[r]; below += (run < target); }
            below = warp_sum_i(below);
            if (below >= kmax) {
                // never reached: with a tail outside the list the nucleus extends beyond it
                if (tail > 0.0 || top_k == 0) ok = 0;
                n_final = kmax;
            } else {
                n_final = below + 1;
            }
        }
        if (lane == 0) { sm.b_i[0] = n_final; sm.b_i[1] = ok; }
    }
    __syncthreads();
    ASX_MARK(10);
    const int n_final = sm.b_i[0];
    if (!sm.b_i[1]) return false;
    // index order among the kept
    for (int r = tid; r < n_final; r += NT) {
        const uint32_t idx = ~(uint32_t)sm.cand[ep.order[r]];
        int ir = 0;
        for (int q = 0; q < n_final; ++q) ir += (~(uint32_t)sm.cand[ep.order[q]] < idx);
        ep.e_idx[ASX_AT(ir, ST_CAP, 92)] = ep.e[r];
        ep.tok_idx[ASX_AT(ir, ST_CAP, 93)] = (int)idx;
    }
    __syncthreads();
    ASX_MARK(11);
    if (warp == 0) {
        const int per = (n_final + 31) / 32;
        const int b = min(lane * per, n_final), e = min(b + per, n_final);
        double s = 0.0;
        for (int i = b; i < e; ++i) s += ep.e_idx[i];
        const double incl = warp_incl_scan_d(s, lane);
        double run = __shfl_up_sync(FULL, incl, 1);
        if (lane == 0) run = 0.0;
        // Z continues the same running sum as the prefixes (last non-empty lane)
        double zrun = run;
        for (int i = b; i < e; ++i) zrun += ep.e_idx[i];
        const int last_lane = (n_final - 1) / per;
        const double Z = __shfl_sync(FULL, zrun, last_lane);
        const double t = c * Z;
        int pick = -1;
        double pS = 0.0, pe = 1.0;
        for (int i = b; i < e; ++i) {
            const double ev = ep.e_idx[i];
            if (pick < 0 && t < run + ev) { pick = i; pS = run; pe = ev; }
            if (i == n_final - 1 && pick < 0) { pick = i; pS = run; pe = ev; }   // top end
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
            r.token = ep.tok_idx[pick]; r.status = ST_OK; r.n_kept = n_final; r.code_out = cn;
            r.p_tok = pe / Z; r.cdf_lo = pS / Z;
            sm.res = r;
        }
    }
    __syncthreads();
    out = sm.res;
    (void)c_in;
    return true;
}

template <int DT, int CS>
__global__ void __launch_bounds__(ST_NT, 1) step_staged_kernel(const StepArgs a) {
    using Tr = Traits<DT>;
    using P = Pass<DT>;
    constexpr int E = Tr::E;
    constexpr int NT = ST_NT;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    StagedSmem<NT>& sm = *reinterpret_cast<StagedSmem<NT>*>(smem_raw);
    unsigned char* rowbuf = smem_raw + ((sizeof(StagedSmem<NT>) + 127) & ~(size_t)127);
    const uint4* rowv = reinterpret_cast<const uint4*>(rowbuf);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (CS > 1) ? (int)cluster.block_rank() : 0;
    const int cluster_id = blockIdx.x / CS, nclusters = gridDim.x / CS;

    const int V = a.V;
    const int nvec = (V + E - 1) / E;
    const int slice_vec = (nvec + CS - 1) / CS;
    const int v0 = min(crank * slice_vec, nvec), v1 = min(v0 + slice_vec, nvec);
    const int my_nvec = v1 - v0;
    const int elem0 = v0 * E, elem1 = min(V, v1 * E);
    const int my_bytes = (elem1 - elem0) * Tr::BYTES;
    const int bulk_bytes = my_bytes & ~15;
    const int bulk_vec = bulk_bytes >> 4;
    const int tail_elems = (my_bytes - bulk_bytes) / Tr::BYTES;   // < E, only on the last slice
    const int nchunk = (bulk_bytes + ST_CHUNK_BYTES - 1) / ST_CHUNK_BYTES;

    if (tid == 0) {
        for (int i = 0; i < ST_MAXCHUNK; ++i) mbar_init(smem_u32(&sm.bars[i]), 1);
        fence_mbar_init();
    }
    if (tid == 0) sm.b_i[3] = 0;
    fill_exp_table(sm.exp_tbl, tid);
    __syncthreads();
    if (CS > 1) cluster.sync();     // every CTA of the cluster is resident before remote writes

    uint32_t phase = 0;             // completed uses of the mbarriers
    bool poisoned = false;          // a bounded wait ran out: stop issuing copies

    auto row_of = [&](int ln) -> const char* {
        return reinterpret_cast<const char*>(a.logits) + (size_t)ln * (size_t)a.ld * Tr::BYTES;
    };
    auto staged_ok = [&](int ln) -> bool { return (reinterpret_cast<uintptr_t>(row_of(ln)) & 15) == 0; };
    // bring this CTA's slice of lane ln's row into shared memory
    auto issue = [&](int ln) {
        const char* src = row_of(ln) + (size_t)elem0 * Tr::BYTES;
        if (tid == 0 && !poisoned && !a.debug_no_copy) {
            fence_proxy_async();
            for (int i = 0; i < nchunk; ++i) {
                const uint32_t bytes = (uint32_t)min(ST_CHUNK_BYTES, bulk_bytes - i * ST_CHUNK_BYTES);
                const uint32_t bar = smem_u32(&sm.bars[i]);
                mbar_expect_tx(bar, bytes);
                bulk_g2s(smem_u32(rowbuf + (size_t)i * ST_CHUNK_BYTES), src + (size_t)i * ST_CHUNK_BYTES, bytes, bar);
            }
        }
        if (tail_elems > 0) {        // ragged end of the row: plain loads, padded with masked tokens
            if (tid < E) {
                if (DT == DT_BF16) {
                    unsigned short* d = reinterpret_cast<unsigned short*>(rowbuf + bulk_bytes);
                    d[tid] = tid < tail_elems ? reinterpret_cast<const unsigned short*>(src + bulk_bytes)[tid]
                                              : (unsigned short)0xFF80u;
                } else {
                    uint32_t* d = reinterpret_cast<uint32_t*>(rowbuf + bulk_bytes);
                    d[tid] = tid < tail_elems ? reinterpret_cast<const uint32_t*>(src + bulk_bytes)[tid] : 0xFF800000u;
                }
            }
            __syncthreads();
        }
    };

    int ln = cluster_id;
    if (ln < a.lanes && staged_ok(ln)) issue(ln);

    for (int it = 0; ln < a.lanes; ln += nclusters, ++it) {
        const int leader = (CS > 1) ? (it % CS) : 0;
        const bool is_leader = (crank == leader);
        const int nxt = ln + nclusters;
        const double c_in = lane_code(a, ln);
        double c = c_in;
        const bool code_bad = !(c >= 0.0 && c <= 1.0);
        if (c == 1.0) c = ASX_ONE_BELOW;

        if (!staged_ok(ln)) {       // unaligned row: the general routine reads it from global memory
            if (is_leader) {
                GenericLane<DT, NT> g(sm.u.gen, row_of(ln), V, false);
                g.bins = !a.radix_nucleus;
                const LaneResult r = g.run(c_in, a.inv_tau, a.top_k, a.top_p);
                if (tid == 0) write_result(a, ln, r, PATH_GENERAL);
            }
            if (nxt < a.lanes && staged_ok(nxt)) issue(nxt);
            continue;
        }

        // ---------------- pass 1: max, as the copies land
        ASX_MARK(0);
        typename P::Acc acc = P::init();
        bool timed_out = poisoned;
        for (int i = 0; i < nchunk; ++i) {
            if (!poisoned && !timed_out && !mbar_wait_bounded(smem_u32(&sm.bars[i]), phase & 1, a.wait_cycles)) timed_out = true;
            const int v = i * ST_CHUNK_VEC + tid;
            if (v < bulk_vec) P::fold(acc, rowv[v]);
        }
        ++phase;
        ASX_MARK(1);
        if (tail_elems > 0 && tid == 0) P::fold(acc, rowv[bulk_vec]);
        uint32_t k0, k1;
        P::keys(acc, k0, k1);
        sm.submax[2 * tid] = k0;
        sm.submax[2 * tid + 1] = k1;
        uint32_t cmax = warp_max_u(max(k0, k1));
        const unsigned any_to = __ballot_sync(FULL, timed_out);
        if (lane == 0) { sm.red_u[warp] = cmax; if (any_to) sm.b_i[3] = 1; }
        if (tid == 0 && is_leader) sm.cand_count = 0;
        __syncthreads();
        cmax = 0;
        for (int w = 0; w < NT / 32; ++w) cmax = max(cmax, sm.red_u[w]);
        const bool cut = a.fast && (a.top_k > 0 || a.top_p < 1.0);
        ASX_MARK(2);
        uint32_t t0key = Tr::KEY_NINF;
        if (cut) {
            const int K0 = a.top_k > 0 ? a.top_k : ST_KP;
            const int K0r = (K0 + CS - 1) / CS;
            if (K0r <= ST_M) t0key = P::key_from16(select_kth16<DT, NT>(sm, K0r));
        }
        ASX_MARK(3);
        int flag = sm.b_i[3];
        __syncthreads();
        if (tid == 0) sm.b_i[3] = 0;
        if (flag) poisoned = true;

        // ---------------- exchange over the cluster
        uint32_t gmax = cmax, gt0 = t0key;
        if (CS > 1) {
            if (tid < CS) {
                StagedSmem<NT>* peer = cluster.map_shared_rank(&sm, tid);
                peer->xch_max[crank] = cmax;
                peer->xch_t0[crank] = t0key;
                peer->xch_flag[crank] = flag;
            }
            cluster.sync();
            gmax = 0; gt0 = 0xFFFFFFFFu; flag = 0;
            for (int r = 0; r < CS; ++r) {
                gmax = max(gmax, sm.xch_max[r]);
                gt0 = min(gt0, sm.xch_t0[r]);
                flag |= sm.xch_flag[r];
            }
        }
        if (flag || code_bad || gmax >= Tr::KEY_PINF || gmax <= Tr::KEY_NINF) {
            // timeout, bad code, NaN / +inf (NaN-propagating max), or nothing but -inf
            if (is_leader && tid == 0) write_result(a, ln, failed_lane(c_in, flag ? ST_TIMEOUT : ST_NUMERIC), PATH_COMPACT);
            if (CS > 1) cluster.sync();          // peers are done with this row's exchange slots
            else __syncthreads();
            if (nxt < a.lanes && staged_ok(nxt)) issue(nxt);
            continue;
        }
        ASX_MARK(4);
        const double lmax = (double)Tr::value_f(gmax);
        gt0 = max(gt0, Tr::KEY_NINF);            // a bound below every finite key means "all of them"

        if (!cut) {
            // no cut: every token is kept; the general routine scans the whole row
            if (CS == 1) {
                GenericLane<DT, NT> g(sm.u.gen, rowbuf, V, true);
                g.bins = !a.radix_nucleus;
                const LaneResult r = g.run(c_in, a.inv_tau, a.top_k, a.top_p);
                if (tid == 0) write_result(a, ln, r, PATH_GENERAL);
            } else {
                cluster.sync();
                if (is_leader) {
                    GenericLane<DT, NT> g(sm.u.gen, row_of(ln), V, true);
                    g.bins = !a.radix_nucleus;
                    const LaneResult r = g.run(c_in, a.inv_tau, a.top_k, a.top_p);
                    if (tid == 0) write_result(a, ln, r, PATH_GENERAL);
                }
            }
            if (nxt < a.lanes && staged_ok(nxt)) issue(nxt);
            continue;
        }

        // ---------------- pass 2: compaction (+ fp32 tail mass for nucleus-only lanes)
        StagedSmem<NT>* lead = (CS > 1) ? cluster.map_shared_rank(&sm, leader) : &sm;
        const float t0f = Tr::value_f(gt0);
        const bool want_tail = (a.top_k == 0);
        const float lmaxf = Tr::value_f(gmax);
        float tail = 0.f;
        for (int v = tid; v < my_nvec; v += NT) {
            const uint4 q = rowv[ASX_AT(v, ST_MAXCHUNK * ST_CHUNK_VEC, 94)];
            if (!want_tail) {
                if (P::vmax(q) >= t0f) {
                    float x[E];
                    P::floats(q, x);
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const uint32_t key = P::key_of_f(x[e]);
                        if (x[e] >= t0f && key >= gt0 && key > Tr::KEY_NINF) {
                            const int slot = atomicAdd(&lead->cand_count, 1);
                            if (slot < ST_CAP)
                                lead->cand[ASX_AT(slot, ST_CAP, 90)] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)((v0 + v) * E + e);
                        }
                    }
                }
            } else {
                float x[E];
                P::floats(q, x);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const float ev = ex2_approx((x[e] - lmaxf) * a.scale2);
                    bool pushed = false;
                    if (x[e] >= t0f) {
                        const uint32_t key = P::key_of_f(x[e]);
                        if (key >= gt0 && key > Tr::KEY_NINF) {
                            pushed = true;
                            const int slot = atomicAdd(&lead->cand_count, 1);
                            if (slot < ST_CAP)
                                lead->cand[ASX_AT(slot, ST_CAP, 90)] = ((unsigned long long)key << 32) | (uint32_t)~(uint32_t)((v0 + v) * E + e);
                        }
                    }
                    tail += pushed ? 0.f : ev;
                }
            }
        }
        ASX_MARK(5);
        if (want_tail) {
            double td = warp_sum_d((double)tail);
            if (lane == 0) sm.red_d[warp] = td;
            __syncthreads();
            if (tid == 0) {
                td = 0.0;
                for (int w = 0; w < NT / 32; ++w) td += sm.red_d[w];
                lead->xch_tail[crank] = td;
            }
        }
        if (CS > 1) cluster.sync();
        else __syncthreads();

        // ---------------- next lane's copies overlap the epilogue
        ASX_MARK(6);
        if (nxt < a.lanes && staged_ok(nxt)) issue(nxt);
        ASX_MARK(7);

        // ---------------- epilogue on the leader
        if (is_leader) {
            const int C = sm.cand_count;
            double tailsum = 0.0;
            if (want_tail) for (int r = 0; r < CS; ++r) tailsum += sm.xch_tail[r];
            LaneResult r;
            bool done = false;
            if (C <= ST_CAP && C > 0)
                done = epilogue<DT, NT>(sm, C, c, c_in, lmax, a.inv_tau, a.top_k, a.top_p, tailsum, r);
            if (!done) {
                __syncthreads();
                GenericLane<DT, NT> g(sm.u.gen, row_of(ln), V, true);
                g.bins = !a.radix_nucleus;
                r = g.run(c_in, a.inv_tau, a.top_k, a.top_p);
            }
            if (tid == 0) write_result(a, ln, r, done ? PATH_COMPACT : PATH_GENERAL);
            __syncthreads();
        }
        ASX_MARK(12);
    }
    if (poisoned && tid == 0 && !a.debug_no_copy) {
        // copies issued before the wait ran out may still be in flight: give them one more bounded wait
        for (int i = 0; i < nchunk; ++i) mbar_wait_bounded(smem_u32(&sm.bars[i]), (phase - 1) & 1, a.wait_cycles);
    }
    if (CS > 1) cluster.sync();     // no CTA leaves while a peer may still write into its shared memory
}

}  // namespace asx

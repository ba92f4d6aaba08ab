// C-ABI entry points (see include/arith_sampling.h) and the kernels behind them.
#include "../../include/arith_sampling.h"
#include "as_stream.cuh"
#include "as_nocut.cuh"
#include "as_metrics.cuh"

#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>

namespace asx {

// ---------------------------------------------------------------------------
// host-side state
// ---------------------------------------------------------------------------
static thread_local char g_err[512] = "";
// launch-shape overrides (as_tune): each is read once per launch; relaxed atomics make a
// concurrent as_tune well-defined (a launch sees the old or the new value)
struct Tune {
    std::atomic<int> v{0};
    operator int() const { return v.load(std::memory_order_relaxed); }
    void operator=(int x) { v.store(x, std::memory_order_relaxed); }
};
static Tune g_tune_path, g_tune_cluster, g_tune_ctas, g_tune_stages, g_tune_minb, g_tune_serial,
    g_tune_wait_kcycles, g_tune_no_copy, g_tune_radix_nucleus;

static long long wait_cycles_now() {
    const int k = g_tune_wait_kcycles;
    return k > 0 ? (long long)k * 1000 : ST_WAIT_CYCLES;
}

static int set_err(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

static int cuda_fail(cudaError_t e, const char* what) {
    return set_err(AS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

struct DeviceInfo {
    int sms = 0;
    bool ok = false;
};
static DeviceInfo g_dev[64];

static int device_info(const DeviceInfo** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return set_err(AS_ERR_CUDA, "device ordinal %d out of range", dev);
    if (!g_dev[dev].ok) {
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        g_dev[dev].sms = sms;
        g_dev[dev].ok = true;
    }
    *out = &g_dev[dev];
    return AS_OK;
}

using DiagPtrs = DiagOut;

// ---------------------------------------------------------------------------
// staged step kernel: launch shape
// ---------------------------------------------------------------------------
constexpr size_t SMEM_OPTIN_MAX = 232448;   // 227 KB per CTA on sm_100

static size_t staged_fixed_bytes() { return (sizeof(StagedSmem<ST_NT>) + 127) & ~(size_t)127; }

template <int DT, int CS>
static int launch_staged(const StepArgs& a, size_t smem, int sms, int want_per_sm, cudaStream_t st) {
    static size_t attr_set[64] = {0};
    static int max_clusters[64] = {0};
    static size_t max_clusters_smem[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    auto kern = step_staged_kernel<DT, CS>;
    cudaError_t e;
    if (attr_set[dev] < smem) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_OPTIN_MAX - 1024));
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(max dynamic shared memory)");
        attr_set[dev] = SMEM_OPTIN_MAX;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(ST_NT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (max_clusters_smem[dev] != smem) {       // resident clusters for this shape (cached)
        cfg.gridDim = dim3(CS * sms);
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) return cuda_fail(e, "cudaOccupancyMaxActiveClusters");
        if (n < 1) return set_err(AS_ERR_CUDA, "staged kernel does not fit (cluster %d, %zu bytes shared)", CS, smem);
        max_clusters[dev] = n;
        max_clusters_smem[dev] = smem;
    }
    int nclusters = max_clusters[dev];
    if (want_per_sm > 0) {
        const long long cap = (long long)want_per_sm * sms / CS;
        if (cap >= 1 && cap < nclusters) nclusters = (int)cap;
    }
    if (nclusters > a.lanes) nclusters = a.lanes;
    cfg.gridDim = dim3(nclusters * CS);
    e = cudaLaunchKernelEx(&cfg, kern, a);
    if (e != cudaSuccess) return cuda_fail(e, "staged step kernel launch");
    return AS_OK;
}

template <int DT, int CAPV, int MINB, bool UA, bool GATHER = false, bool XP = false>
static int launch_stream_ua(const StepArgs& a, int stages, int sms, int want_per_sm, cudaStream_t st) {
    static bool attr_set[64] = {false};
    static int per_sm_cache[64][SK_MAXSTAGES + 1] = {{0}};
    int dev = 0;
    cudaGetDevice(&dev);
    auto kern = step_stream_kernel<DT, CAPV, MINB, UA, GATHER, XP>;
    cudaError_t e;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_OPTIN_MAX - 1024));
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(max dynamic shared memory)");
        attr_set[dev] = true;
    }
    const size_t fixed = (sizeof(StreamSmemT<CAPV>) + 127) & ~(size_t)127;
    const size_t smem = fixed + (size_t)stages * SK_STAGE_BYTES;
    if (per_sm_cache[dev][stages] == 0) {
        int n = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, SK_THREADS, smem);
        if (e != cudaSuccess) return cuda_fail(e, "cudaOccupancyMaxActiveBlocksPerMultiprocessor");
        if (n < 1) return set_err(AS_ERR_CUDA, "streaming kernel does not fit (%zu bytes shared)", smem);
        per_sm_cache[dev][stages] = n;
    }
    int per_sm = per_sm_cache[dev][stages];
    if (want_per_sm > 0 && want_per_sm < per_sm) per_sm = want_per_sm;
    long long grid = (long long)per_sm * sms;
    if (grid > a.lanes) grid = a.lanes;
    // Launched so that it may start while the kernel before it on the stream drains, if that
    // kernel allows it (this kernel does, at its start): launch latency, CTA set-up and barrier
    // initialisation then overlap the predecessor's tail.  The kernel waits for the predecessor's
    // completion (griddepcontrol.wait) before it touches global memory, so results are the same.
    // Only for launches of one row per CTA, where the launch gap is a tenth of the time: early
    // CTAs take the slots that free up first, which bunches the low block indices on few SMs, and
    // in a launch of several rows per CTA those are the CTAs with one row more (1024 x 256000:
    // 138 -> 144 us with the overlap, 256 x 32000: 13.3 -> 12.75 us).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(SK_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (!g_tune_serial && grid == a.lanes) ? 1 : 0;
    e = cudaLaunchKernelEx(&cfg, kern, a, stages);
    if (e != cudaSuccess) return cuda_fail(e, "streaming step kernel launch");
    // the lanes it leaves undecided: the general routine, four CTAs per SM, set up while the
    // streaming kernel drains
    cudaLaunchConfig_t cfd = {};
    long long gd = 4LL * sms;
    if (gd > a.lanes) gd = a.lanes;
    cfd.gridDim = dim3((unsigned)gd);
    cfd.blockDim = dim3(DL_NT);
    cfd.dynamicSmemBytes = 0;
    cfd.stream = st;
    cfd.attrs = attr;
    cfd.numAttrs = g_tune_serial ? 0 : 1;
    // rows of up to 96 KB are staged in shared memory (two CTAs per SM then)
    static bool dl_attr_set[64] = {false};
    auto dkern = deferred_lanes_kernel<DT, GATHER, XP>;
    if (!dl_attr_set[dev]) {
        e = cudaFuncSetAttribute(dkern, cudaFuncAttributeMaxDynamicSharedMemorySize, DL_STAGE_MAX);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(deferred lanes kernel)");
        dl_attr_set[dev] = true;
    }
    const long long row_span = (long long)a.V * (DT == DT_BF16 ? 2 : 4) + 15 + 16;
    const int stage_bytes = row_span <= DL_STAGE_MAX ? (int)(row_span & ~15LL) : 0;
    cfd.dynamicSmemBytes = (size_t)stage_bytes;
    e = cudaLaunchKernelEx(&cfd, dkern, a, stage_bytes);
    if (e != cudaSuccess) return cuda_fail(e, "deferred lanes kernel launch");
    return AS_OK;
}

// rows that all start on 16-byte boundaries take the plain build; otherwise the build that
// copies each row from the boundary below its start
template <int DT, int CAPV, int MINB>
static int launch_stream(const StepArgs& a, bool unaligned, int stages, int sms, int want_per_sm, cudaStream_t st) {
    if (a.row_idx && a.xp_state) return launch_stream_ua<DT, CAPV, MINB, true, true, true>(a, stages, sms, want_per_sm, st);
    if (a.row_idx) return launch_stream_ua<DT, CAPV, MINB, true, true>(a, stages, sms, want_per_sm, st);   // table rows: any alignment
    return unaligned ? launch_stream_ua<DT, CAPV, MINB, true>(a, stages, sms, want_per_sm, st)
                     : launch_stream_ua<DT, CAPV, MINB, false>(a, stages, sms, want_per_sm, st);
}

template <int DT>
static int launch_staged_cs(int cs, const StepArgs& a, size_t smem, int sms, int per_sm, cudaStream_t st) {
    switch (cs) {
        case 1: return launch_staged<DT, 1>(a, smem, sms, per_sm, st);
        case 2: return launch_staged<DT, 2>(a, smem, sms, per_sm, st);
        case 4: return launch_staged<DT, 4>(a, smem, sms, per_sm, st);
        default: return launch_staged<DT, 8>(a, smem, sms, per_sm, st);
    }
}

// Lanes without a cut on 16-byte aligned rows of up to 96 KB: groups of 256 threads, each with a
// row buffer in shared memory (as_nocut.cuh).  AS_ERR_UNSUPPORTED (no message): not for that kernel.
template <int DT, int MODE>
static int launch_nocut_dm(NocutArgs& a, double temp, int sms, cudaStream_t st) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    auto kern = nocut_kernel<DT, MODE>;
    cudaError_t e;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_OPTIN_MAX - 1024));
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(max dynamic shared memory)");
        attr_set[dev] = true;
    }
    const size_t row_stride = (((size_t)a.V * Traits<DT>::BYTES) + 127) & ~(size_t)127;
    int groups = (int)((SMEM_OPTIN_MAX - 1024 - nc_fixed_bytes()) / row_stride);
    if (groups > NC_MAXG) groups = NC_MAXG;
    if (groups < 1) return AS_ERR_UNSUPPORTED;
    a.use_table = (DT == DT_BF16 && temp >= NC_MIN_TEMP) ? 1 : 0;
    a.wait_cycles = wait_cycles_now();
    a.debug_no_copy = g_tune_no_copy;
    long long grid = ((long long)a.lanes + groups - 1) / groups;
    if (grid > sms) grid = sms;
    const size_t smem = nc_fixed_bytes() + (size_t)groups * row_stride;
    kern<<<(unsigned)grid, groups * NC_GT, smem, st>>>(a, groups, (int)row_stride);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "no-cut kernel launch");
    return AS_OK;
}

template <int MODE>
static int launch_nocut(NocutArgs& a, int dtype, double temp, int sms, cudaStream_t st) {
    const size_t esz = dtype == AS_F32 ? 4 : 2;
    if (g_tune_path != 0) return AS_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(a.data) & 15) != 0 || (((size_t)a.ld * esz) & 15) != 0) return AS_ERR_UNSUPPORTED;
    if ((size_t)a.V * esz > (size_t)NC_MAXROW) return AS_ERR_UNSUPPORTED;
    return dtype == AS_F32 ? launch_nocut_dm<DT_F32, MODE>(a, temp, sms, st) : launch_nocut_dm<DT_BF16, MODE>(a, temp, sms, st);
}

// ---------------------------------------------------------------------------
// kernels
// ---------------------------------------------------------------------------
constexpr int GEN_NT = 512;

__global__ void lattice_kernel(int N, double u, double* __restrict__ codes) {
    // Definition "Arithmetic sampling" (Sec. 4.2), spacing 1/N: c_j = (j + u)/N mod 1
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j < N) {
        double c = ((double)j + u) / (double)N;
        if (c >= 1.0) c -= 1.0;
        codes[j] = c;
    }
}

// The code sets as the paper prints them (Sec. 4.2): variant 1 = (i/(N+1) + b) mod 1, the Definition
// "Arithmetic sampling"; variant 2 = i/(N+1), the naive codebook; i = 1..N, codes[i-1] = c_i.
__global__ void lattice_variant_kernel(int N, double b, int variant, double* __restrict__ codes) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x + 1;
    if (i <= N) {
        double c = (double)i / (double)(N + 1);
        if (variant == 1) {
            c += b;
            if (c >= 1.0) c -= 1.0;
        }
        codes[i - 1] = c;
    }
}

template <int DT>
__global__ void __launch_bounds__(GEN_NT)
step_generic_kernel(const void* __restrict__ logits, int lanes, int V, long long ld,
                    const double* codes, int lat_N, int lat_j0, double lat_u, double inv_tau, int top_k,
                    double top_p, double typical_p, int* __restrict__ tokens, double* codes_out, DiagPtrs diag, int radix_nucleus) {
    __shared__ GenericSmem<GEN_NT> sm;
    for (int ln = blockIdx.x; ln < lanes; ln += gridDim.x) {
        const char* row = reinterpret_cast<const char*>(logits) + (size_t)ln * (size_t)ld * Traits<DT>::BYTES;
        const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
        double c;
        if (lat_N > 0) {            // the lattice itself (same expression as lattice_kernel)
            c = ((double)(lat_j0 + ln) + lat_u) / (double)lat_N;
            if (c >= 1.0) c -= 1.0;
        } else {
            c = codes[ln];
        }
        GenericLane<DT, GEN_NT> g(sm, row, V, vec_ok);
        g.bins = !radix_nucleus;
        const LaneResult r = g.run(c, inv_tau, top_k, top_p, typical_p);
        if (threadIdx.x == 0) {
            tokens[ln] = r.token;
            codes_out[ln] = r.code_out;
            if (diag.p_tok) diag.p_tok[ln] = r.p_tok;
            if (diag.cdf_lo) diag.cdf_lo[ln] = r.cdf_lo;
            if (diag.n_kept) diag.n_kept[ln] = r.n_kept;
            if (diag.lane_status) diag.lane_status[ln] = r.status;
            if (diag.path) diag.path[ln] = PATH_GENERAL;
        }
    }
}

// Algorithm 1's REPEAT ... UNTIL loop for one lane per CTA over a bigram table.
// Lane state comes either from (start, N, u) [codes_in == nullptr] or from
// (prev, codes_in).
template <int DT>
__global__ void __launch_bounds__(GEN_NT)
decode_generic_kernel(const void* __restrict__ table, int V, long long ld,
                      const int* __restrict__ start_or_prev, const double* __restrict__ codes_in,
                      int lanes, int N, double u, int T, int eos, double inv_tau, int top_k,
                      double top_p, int* __restrict__ seq, int* __restrict__ len,
                      double* __restrict__ codes_final, int* __restrict__ lane_status) {
    __shared__ GenericSmem<GEN_NT> sm;
    for (int ln = blockIdx.x; ln < lanes; ln += gridDim.x) {
        int prev;
        double c;
        if (codes_in) {
            prev = start_or_prev[ln];
            c = codes_in[ln];
        } else {
            prev = start_or_prev[ln / N];
            c = ((double)(ln % N) + u) / (double)N;
            if (c >= 1.0) c -= 1.0;
        }
        int n = 0, status = ST_OK;
        for (int t = 0; t < T; ++t) {
            if (prev < 0 || prev >= V) { status = ST_NUMERIC; break; }
            const char* row = reinterpret_cast<const char*>(table) + (size_t)prev * (size_t)ld * Traits<DT>::BYTES;
            const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
            GenericLane<DT, GEN_NT> g(sm, row, V, vec_ok);
            const LaneResult r = g.run(c, inv_tau, top_k, top_p);
            if (r.status != ST_OK) { status = r.status; break; }
            if (threadIdx.x == 0) seq[(size_t)ln * T + t] = r.token;
            n = t + 1;
            c = r.code_out;
            prev = r.token;
            if (r.token == eos) break;
        }
        for (int t = n + (int)threadIdx.x; t < T; t += GEN_NT) seq[(size_t)ln * T + t] = -1;
        if (threadIdx.x == 0) {
            len[ln] = n;
            if (codes_final) codes_final[ln] = c;
            if (lane_status) lane_status[ln] = status;
        }
    }
}

// Sequence -> interval (the codebook of Sec. 4.1 in the other direction): one CTA per lane walks
// the lane's tokens; lo gathers width * F_{i-1}, width multiplies by p_i.
template <int DT>
__global__ void __launch_bounds__(GEN_NT)
encode_generic_kernel(const void* __restrict__ table, int V, long long ld, const int* __restrict__ prev0,
                      const int* __restrict__ seq, const int* __restrict__ len, int lanes, int T,
                      double inv_tau, int top_k, double top_p, double* __restrict__ lo_out,
                      double* __restrict__ width_out, int* __restrict__ lane_status) {
    __shared__ GenericSmem<GEN_NT> sm;
    for (int ln = blockIdx.x; ln < lanes; ln += gridDim.x) {
        int prev = prev0[ln];
        const int n = min(len[ln], T);
        double lo = 0.0, comp = 0.0, width = 1.0;
        int status = ST_OK;
        for (int t = 0; t < n; ++t) {
            const int tok = seq[(size_t)ln * T + t];
            if (prev < 0 || prev >= V || tok < 0 || tok >= V) { status = -1; break; }   // AS_ERR_INVALID_ARG
            const char* row = reinterpret_cast<const char*>(table) + (size_t)prev * (size_t)ld * Traits<DT>::BYTES;
            const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
            GenericLane<DT, GEN_NT> g(sm, row, V, vec_ok);
            const LaneResult r = g.interval_of(tok, inv_tau, top_k, top_p);
            if (r.status != ST_OK) { status = r.status; break; }
            // compensated running sum: the terms shrink geometrically with t
            const double term = width * r.cdf_lo;
            const double s = lo + term;
            comp += (fabs(lo) >= fabs(term)) ? (lo - s) + term : (term - s) + lo;
            lo = s;
            width *= r.p_tok;
            prev = tok;
        }
        if (threadIdx.x == 0) {
            lo_out[ln] = lo + comp;
            width_out[ln] = width;
            if (lane_status) lane_status[ln] = status;
        }
    }
}

// Extended-precision codes: decoder state of the lattice codes (j + u)/N, j = j0 .. j0 + count - 1,
// one copy per start token.  U = floor(u 2^53); A = j 2^53 + U; the first 53 binary digits of the
// code are A div N, all further ones come from the long division of A mod N by N.
__global__ void xp_state_kernel(int N, unsigned long long U, int j0, int count, int S, unsigned long long* __restrict__ state) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const unsigned __int128 A = ((unsigned __int128)(unsigned long long)(j0 + i) << 53) + U;
    XpState s;
    s.range = XP_RANGE_TOP;
    s.code = 0;
    s.q = (unsigned long long)(A / (unsigned long long)N);
    s.packed = (53ull << 32) | (unsigned long long)(A % (unsigned long long)N);
    s.code = xp_next_bits(s, 32, (unsigned)N);
    s.code = (s.code << 31) | xp_next_bits(s, 31, (unsigned)N);
    for (int g = 0; g < S; ++g) {
        unsigned long long* o = state + ((size_t)g * count + i) * 4;
        o[0] = s.range; o[1] = s.code; o[2] = s.q; o[3] = s.packed;
    }
}

// Algorithm 1's loop with extended-precision codes, one CTA per lane, any cut (general routine).
template <int DT>
__global__ void __launch_bounds__(GEN_NT)
decode_xp_generic_kernel(const void* __restrict__ table, int V, long long ld, const int* __restrict__ prev_in,
                         unsigned long long* __restrict__ state, int lanes, int N, int T, int eos, double inv_tau,
                         int top_k, double top_p, int* __restrict__ seq, int* __restrict__ len,
                         int* __restrict__ lane_status) {
    __shared__ GenericSmem<GEN_NT> sm;
    for (int ln = blockIdx.x; ln < lanes; ln += gridDim.x) {
        XpState xs;
        xs.range = state[(size_t)ln * 4]; xs.code = state[(size_t)ln * 4 + 1];
        xs.q = state[(size_t)ln * 4 + 2]; xs.packed = state[(size_t)ln * 4 + 3];
        int prev = prev_in[ln];
        int n = 0, status = ST_OK;
        for (int t = 0; t < T; ++t) {
            if (prev < 0 || prev >= V || !xp_state_ok(xs)) { status = ST_NUMERIC; break; }
            const char* row = reinterpret_cast<const char*>(table) + (size_t)prev * (size_t)ld * Traits<DT>::BYTES;
            const bool vec_ok = (reinterpret_cast<uintptr_t>(row) & 15) == 0;
            GenericLane<DT, GEN_NT> g(sm, row, V, vec_ok);
            const LaneResult r = g.run_xp(xp_target(xs), inv_tau, top_k, top_p);
            if (r.status != ST_OK) { status = r.status; break; }
            xp_advance(xs, sm.xp_lo, sm.xp_hi, (unsigned)N);
            if (threadIdx.x == 0) seq[(size_t)ln * T + t] = r.token;
            n = t + 1;
            prev = r.token;
            if (r.token == eos) break;
        }
        for (int t = n + (int)threadIdx.x; t < T; t += GEN_NT) seq[(size_t)ln * T + t] = -1;
        __syncthreads();
        if (threadIdx.x == 0) {
            len[ln] = n;
            state[(size_t)ln * 4] = xs.range; state[(size_t)ln * 4 + 1] = xs.code;
            state[(size_t)ln * 4 + 2] = xs.q; state[(size_t)ln * 4 + 3] = xs.packed;
            if (lane_status) lane_status[ln] = status;
        }
    }
}

// Decode loop as one launch of the streaming kernel per step (lanes with a top-k / nucleus cut):
// set-up and wrap-up.  The state lives in the caller's outputs: the codes in codes_final, the
// previous token in the sequence itself (column t-1; for step 0 the start tokens are parked in
// `len`, which the wrap-up overwrites), a finished lane being one whose previous entry is the
// padding or EOS.
__global__ void decode_setup_kernel(const int* __restrict__ start_or_prev, const double* __restrict__ codes_in,
                                    int lanes, int N, double u, int V, int T, int* __restrict__ idx0,
                                    double* __restrict__ codes, int* __restrict__ seq, int* __restrict__ lane_status) {
    const size_t total = (size_t)lanes * T;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) seq[i] = -1;
    for (int ln = blockIdx.x * blockDim.x + threadIdx.x; ln < lanes; ln += gridDim.x * blockDim.x) {
        int prev;
        double c;
        if (codes_in) {
            prev = start_or_prev[ln];
            c = codes_in[ln];
        } else {
            prev = start_or_prev[ln / N];
            c = ((double)(ln % N) + u) / (double)N;
            if (c >= 1.0) c -= 1.0;
        }
        const bool ok = prev >= 0 && prev < V;
        idx0[ln] = ok ? prev : -1;
        if (codes) codes[ln] = c;
        if (lane_status) lane_status[ln] = ok ? ST_OK : ST_NUMERIC;
    }
}

__global__ void decode_wrapup_kernel(const int* __restrict__ seq, int lanes, int T, int* __restrict__ len) {
    for (int ln = blockIdx.x * blockDim.x + threadIdx.x; ln < lanes; ln += gridDim.x * blockDim.x) {
        int n = 0;
        while (n < T && seq[(size_t)ln * T + n] >= 0) ++n;
        len[ln] = n;
    }
}

// ---------------------------------------------------------------------------
// argument checks
// ---------------------------------------------------------------------------
static int check_scalars(int dtype, int V, long long ld, double temp, double top_p) {
    if (dtype != AS_F32 && dtype != AS_BF16) return set_err(AS_ERR_INVALID_ARG, "unknown dtype %d", dtype);
    if (V < 1) return set_err(AS_ERR_INVALID_ARG, "V = %d must be >= 1", V);
    if (V > AS_MAX_V) return set_err(AS_ERR_UNSUPPORTED, "V = %d exceeds AS_MAX_V = %d", V, AS_MAX_V);
    if (ld < V) return set_err(AS_ERR_INVALID_ARG, "ld = %lld is smaller than V = %d", ld, V);
    if (!(temp > 0.0) || std::isinf(temp)) return set_err(AS_ERR_INVALID_ARG, "temp must be positive and finite");
    if (std::isnan(top_p)) return set_err(AS_ERR_INVALID_ARG, "top_p is NaN");
    return AS_OK;
}

static int check_data(const void* data, int dtype) {
    if (!data) return set_err(AS_ERR_INVALID_ARG, "logits/table pointer is NULL");
    const uintptr_t a = reinterpret_cast<uintptr_t>(data);
    if (a % (dtype == AS_F32 ? 4 : 2)) return set_err(AS_ERR_INVALID_ARG, "logits/table pointer is not element-aligned");
    return AS_OK;
}

static int grid_for(int lanes, int sms, int per_sm) {
    const long long cap = (long long)sms * per_sm;
    return (int)(lanes < cap ? lanes : cap);
}

}  // namespace asx

using namespace asx;

extern "C" {

int as_version(void) { return 1000; }

#ifdef ASX_PROFILE
// profiling builds only: copies CTA 0's phase timestamps of the last staged launch
int as_debug_marks(long long* h_out) {
    return cudaMemcpyFromSymbol(h_out, g_asx_marks, sizeof(long long) * 32) == cudaSuccess ? AS_OK : AS_ERR_CUDA;
}
int as_debug_span(unsigned long long* h_out, int reset) {
    unsigned long long init[4] = {~0ull, 0ull, ~0ull, 0ull};
    if (reset) return cudaMemcpyToSymbol(g_asx_span, init, sizeof(init)) == cudaSuccess ? AS_OK : AS_ERR_CUDA;
    return cudaMemcpyFromSymbol(h_out, g_asx_span, sizeof(init)) == cudaSuccess ? AS_OK : AS_ERR_CUDA;
}
int as_debug_cta(unsigned long long* h_out) {
    return cudaMemcpyFromSymbol(h_out, g_asx_cta, sizeof(unsigned long long) * 1024 * 8) == cudaSuccess ? AS_OK : AS_ERR_CUDA;
}
int as_debug_counts(unsigned long long* h_out) {
    return cudaMemcpyFromSymbol(h_out, g_asx_counts, sizeof(unsigned long long) * 16) == cudaSuccess ? AS_OK : AS_ERR_CUDA;
}
#endif

#ifdef AS_BOUNDS_CHECK
// checked builds only: the record of out-of-range indices (failures, first site, its index, its
// bound) since the last reset
int as_debug_bounds(int* h_out4, int reset) {
    int zero[4] = {0, 0, 0, 0};
    if (h_out4 && cudaMemcpyFromSymbol(h_out4, g_asx_bounds, sizeof(zero)) != cudaSuccess) return AS_ERR_CUDA;
    if (reset && cudaMemcpyToSymbol(g_asx_bounds, zero, sizeof(zero)) != cudaSuccess) return AS_ERR_CUDA;
    return AS_OK;
}
#endif

const char* as_last_error(void) { return g_err; }

int as_tune(int key, int value) {
    switch (key) {
        case AS_TUNE_STEP_PATH:
            if (value < 0 || value > 2) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_STEP_PATH takes 0, 1 or 2");
            g_tune_path = value;
            return AS_OK;
        case AS_TUNE_CLUSTER:
            if (value != 0 && value != 1 && value != 2 && value != 4 && value != 8)
                return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_CLUSTER takes 0, 1, 2, 4 or 8");
            g_tune_cluster = value;
            return AS_OK;
        case AS_TUNE_CTAS_PER_SM:
            if (value < 0 || value > 32) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_CTAS_PER_SM takes 0..32");
            g_tune_ctas = value;
            return AS_OK;
        case AS_TUNE_MIN_CTAS:
            if (value != 0 && value != 2 && value != 3) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_MIN_CTAS takes 0, 2 or 3");
            g_tune_minb = value;
            return AS_OK;
        case AS_TUNE_SERIAL_LAUNCH:
            if (value != 0 && value != 1) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_SERIAL_LAUNCH takes 0 or 1");
            g_tune_serial = value;
            return AS_OK;
        case AS_TUNE_STAGES:
            if (value < 0 || value == 1 || value > SK_MAXSTAGES) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_STAGES takes 0 or 2..12");
            g_tune_stages = value;
            return AS_OK;
        case AS_TUNE_WAIT_KCYCLES:
            if (value < 0) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_WAIT_KCYCLES takes 0 (default) or a positive count of 1000 cycles");
            g_tune_wait_kcycles = value;
            return AS_OK;
        case AS_TUNE_DEBUG_NO_COPY:
            if (value != 0 && value != 1) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_DEBUG_NO_COPY takes 0 or 1");
            g_tune_no_copy = value;
            return AS_OK;
        case AS_TUNE_RADIX_NUCLEUS:
            if (value != 0 && value != 1) return set_err(AS_ERR_INVALID_ARG, "AS_TUNE_RADIX_NUCLEUS takes 0 or 1");
            g_tune_radix_nucleus = value;
            return AS_OK;
        default:
            return set_err(AS_ERR_INVALID_ARG, "unknown tuning key %d", key);
    }
}

int as_lattice_codes(int N, double u, double* d_codes, void* stream) {
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (!(u >= 0.0 && u < 1.0)) return set_err(AS_ERR_INVALID_ARG, "shift u must lie in [0,1)");
    if (!d_codes) return set_err(AS_ERR_INVALID_ARG, "d_codes is NULL");
    const DeviceInfo* di;
    int rc = device_info(&di);
    if (rc != AS_OK) return rc;
    lattice_kernel<<<(N + 255) / 256, 256, 0, (cudaStream_t)stream>>>(N, u, d_codes);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "lattice kernel launch");
    return AS_OK;
}

int as_lattice_codes_variant(int N, double b, int variant, double* d_codes, void* stream) {
    if (variant == AS_LATTICE_SHIFTED) return as_lattice_codes(N, b, d_codes, stream);
    if (variant != AS_LATTICE_PAPER_DEFINITION && variant != AS_LATTICE_NAIVE)
        return set_err(AS_ERR_INVALID_ARG, "unknown lattice variant %d", variant);
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (variant == AS_LATTICE_PAPER_DEFINITION && !(b >= 0.0 && b < 1.0))
        return set_err(AS_ERR_INVALID_ARG, "shift b must lie in [0,1)");
    if (!d_codes) return set_err(AS_ERR_INVALID_ARG, "d_codes is NULL");
    const DeviceInfo* di;
    int rc = device_info(&di);
    if (rc != AS_OK) return rc;
    lattice_variant_kernel<<<(N + 255) / 256, 256, 0, (cudaStream_t)stream>>>(N, b, variant, d_codes);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "lattice kernel launch");
    return AS_OK;
}

}  // extern "C"

// The streaming kernel for one step: one CTA per lane; rows of up to 6 stages (96 KB) stay resident
// in the ring.  Sets a.fast.  AS_ERR_UNSUPPORTED (no message): this step is not for that kernel.
static int launch_streaming(StepArgs& a, int dtype, bool unaligned, int sms, cudaStream_t st) {
    // lanes without a cut keep every token: nothing to compact, and the general kernel's lean loop
    // (512 threads, four CTAs per SM) serves them 20 % faster than a detour through the ring
    if (a.top_k <= 0 && !(a.top_p < 1.0)) return AS_ERR_UNSUPPORTED;
    const int E = dtype == AS_F32 ? 4 : 8;
    const bool off_grid = unaligned || a.row_idx != nullptr;
    const size_t row_bytes = (size_t)((a.V + (off_grid ? E - 1 : 0) + E - 1) / E) * 16;
    const int nsl = (int)((row_bytes + SK_STAGE_BYTES - 1) / SK_STAGE_BYTES);
    // rows of up to SK_RES_STAGES stages stay resident unless a smaller ring is asked for
    const bool resident = nsl <= SK_RES_STAGES && !(g_tune_stages > 0 && g_tune_stages < nsl);
    a.fast = (a.top_k > 0 && a.top_k <= (resident ? SK_K0_RESIDENT : SK_K0_STREAMED)) || (a.top_k == 0 && a.top_p < 1.0);
    if (!a.fast) return AS_ERR_UNSUPPORTED;       // (a top-k beyond the candidate list: the general kernels)
    int stages = resident ? (nsl < 1 ? 1 : nsl) : (g_tune_stages > 0 ? g_tune_stages : 3);
    if (!resident && stages >= nsl) stages = nsl - 1;
    if (dtype == AS_F32) {
        if (!resident && g_tune_minb != 2)
            return launch_stream<DT_F32, 1536, 3>(a, unaligned, stages < 2 ? stages : 2, sms, g_tune_ctas, st);
        return launch_stream<DT_F32, 2048, 2>(a, unaligned, stages, sms, g_tune_ctas, st);
    }
    // bf16 rows that stream: a 1024-entry hit list and <= 72 registers let three CTAs share an SM
    if (!resident && g_tune_minb != 2)
        return launch_stream<DT_BF16, 1024, 3>(a, unaligned, stages < 3 ? stages : 3, sms, g_tune_ctas, st);
    return launch_stream<DT_BF16, 2048, 2>(a, unaligned, stages, sms, g_tune_ctas, st);
}

// as_step and as_step_lattice: lat_N = 0 reads d_codes, lat_N > 0 forms the lattice codes in the kernel
static int step_common(const void* d_logits, int dtype, int lanes, int V, long long ld, const double* d_codes,
                       int lat_N, int lat_j0, double lat_u, double temp, int top_k, double top_p,
                       int32_t* d_tokens, double* d_codes_out, const as_step_diag* diag, void* stream,
                       double typical_p = 1.0) {
    if (lanes < 0) return set_err(AS_ERR_INVALID_ARG, "lanes = %d must be >= 0", lanes);
    int rc = check_scalars(dtype, V, ld, temp, top_p);
    if (rc != AS_OK) return rc;
    if (lanes == 0) return AS_OK;
    if ((rc = check_data(d_logits, dtype)) != AS_OK) return rc;
    if ((!d_codes && lat_N == 0) || !d_tokens || !d_codes_out) return set_err(AS_ERR_INVALID_ARG, "codes / tokens / codes_out pointer is NULL");
    const DeviceInfo* di;
    rc = device_info(&di);
    if (rc != AS_OK) return rc;
    DiagPtrs dp = {nullptr, nullptr, nullptr, nullptr, nullptr};
    if (diag) dp = {diag->d_p_tok, diag->d_cdf_lo, diag->d_n_kept, diag->d_lane_status, diag->d_path};
    if (top_k < 0 || top_k >= V) top_k = 0;
    if (!(top_p > 0.0 && top_p < 1.0)) top_p = 1.0;
    if (std::isnan(typical_p)) return set_err(AS_ERR_INVALID_ARG, "typical_p is NaN");
    const bool typical = typical_p > 0.0 && typical_p < 1.0;
    if (!typical) typical_p = 1.0;
    if (typical && top_p < 1.0) return set_err(AS_ERR_INVALID_ARG, "a step takes a nucleus (top_p) or a typical cut (typical_p), not both");
    const double inv_tau = 1.0 / temp;
    cudaStream_t st = (cudaStream_t)stream;
    StepArgs a;
    a.logits = d_logits; a.codes = d_codes; a.tokens = d_tokens; a.codes_out = d_codes_out; a.diag = dp;
    a.ld = ld; a.inv_tau = inv_tau; a.top_p = top_p; a.scale2 = (float)(1.4426950408889634 / temp);
    a.lanes = lanes; a.V = V; a.top_k = top_k;
    a.lat_N = lat_N; a.lat_j0 = lat_j0; a.lat_u = lat_u;
    a.row_idx = nullptr; a.idx_stride = 1; a.tok_stride = 1; a.eos = -1; a.rows = 0;
    a.xp_state = nullptr; a.xp_N = 0;
    a.wait_cycles = wait_cycles_now(); a.debug_no_copy = g_tune_no_copy; a.radix_nucleus = g_tune_radix_nucleus;
    const int E = dtype == AS_F32 ? 4 : 8;
    const size_t esz = dtype == AS_F32 ? 4 : 2;
    // some row starts off a 16-byte boundary: it is read from the boundary below, up to E-1 elements longer
    const bool unaligned = (reinterpret_cast<uintptr_t>(d_logits) & 15) != 0 || (((size_t)ld * esz) & 15) != 0;
    const size_t row_bytes = (size_t)((V + (unaligned && g_tune_path == 0 ? E - 1 : 0) + E - 1) / E) * 16;
    if (g_tune_path == 0 && !typical) {
        rc = launch_streaming(a, dtype, unaligned, di->sms, st);
        if (rc != AS_ERR_UNSUPPORTED) return rc;
    }
    if (top_k == 0 && !(top_p < 1.0) && !typical) {
        NocutArgs n = {};
        n.data = d_logits; n.ld = ld; n.V = V; n.lanes = lanes; n.inv_tau = inv_tau;
        n.codes = d_codes; n.lat_N = lat_N; n.lat_j0 = lat_j0; n.lat_u = lat_u;
        n.tokens = d_tokens; n.codes_out = d_codes_out; n.diag = dp;
        rc = launch_nocut<NC_STEP>(n, dtype, temp, di->sms, st);
        if (rc != AS_ERR_UNSUPPORTED) return rc;
    }
    if (g_tune_path == 2 && !typical) {
        // cluster kernel: the row split over CS CTAs' shared memory
        int cs = g_tune_cluster;
        if (cs == 0) cs = row_bytes <= 80 * 1024 ? 1 : row_bytes <= 160 * 1024 ? 2 : row_bytes <= 320 * 1024 ? 4 : 8;
        const size_t slice_bytes = (((row_bytes / 16) + cs - 1) / cs) * 16;
        const size_t smem = staged_fixed_bytes() + slice_bytes + 16;
        if (smem <= SMEM_OPTIN_MAX - 1024 && slice_bytes <= (size_t)ST_MAXCHUNK * ST_CHUNK_BYTES) {
            a.fast = (top_k > 0 && top_k <= 300) || (top_k == 0 && top_p < 1.0);
            return dtype == AS_F32 ? launch_staged_cs<DT_F32>(cs, a, smem, di->sms, g_tune_ctas, st)
                                   : launch_staged_cs<DT_BF16>(cs, a, smem, di->sms, g_tune_ctas, st);
        }
    }
    const int grid = grid_for(lanes, di->sms, g_tune_ctas > 0 ? g_tune_ctas : 4);
    if (dtype == AS_F32)
        step_generic_kernel<DT_F32><<<grid, GEN_NT, 0, st>>>(d_logits, lanes, V, ld, d_codes, lat_N, lat_j0, lat_u, inv_tau, top_k, top_p, typical_p, d_tokens, d_codes_out, dp, (int)g_tune_radix_nucleus);
    else
        step_generic_kernel<DT_BF16><<<grid, GEN_NT, 0, st>>>(d_logits, lanes, V, ld, d_codes, lat_N, lat_j0, lat_u, inv_tau, top_k, top_p, typical_p, d_tokens, d_codes_out, dp, (int)g_tune_radix_nucleus);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "step kernel launch");
    return AS_OK;
}

extern "C" {

int as_step(const void* d_logits, int dtype, int lanes, int V, long long ld, const double* d_codes,
            double temp, int top_k, double top_p, int32_t* d_tokens, double* d_codes_out,
            const as_step_diag* diag, void* stream) {
    return step_common(d_logits, dtype, lanes, V, ld, d_codes, 0, 0, 0.0, temp, top_k, top_p, d_tokens,
                       d_codes_out, diag, stream);
}

int as_step_typical(const void* d_logits, int dtype, int lanes, int V, long long ld, const double* d_codes,
                    double temp, int top_k, double typical_p, int32_t* d_tokens, double* d_codes_out,
                    const as_step_diag* diag, void* stream) {
    return step_common(d_logits, dtype, lanes, V, ld, d_codes, 0, 0, 0.0, temp, top_k, 1.0, d_tokens,
                       d_codes_out, diag, stream, typical_p);
}

int as_step_lattice(const void* d_logits, int dtype, int lanes, int V, long long ld, int N, double u, int j0,
                    double temp, int top_k, double top_p, int32_t* d_tokens, double* d_codes_out,
                    const as_step_diag* diag, void* stream) {
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (!(u >= 0.0 && u < 1.0)) return set_err(AS_ERR_INVALID_ARG, "shift u must lie in [0,1)");
    if (j0 < 0 || lanes < 0 || (long long)j0 + lanes > N)
        return set_err(AS_ERR_INVALID_ARG, "lanes j0 .. j0+lanes-1 = %d .. %lld must lie in [0, N = %d)", j0, (long long)j0 + lanes - 1, N);
    return step_common(d_logits, dtype, lanes, V, ld, nullptr, N, j0, u, temp, top_k, top_p, d_tokens,
                       d_codes_out, diag, stream);
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

size_t as_step_host_work_bytes(int dtype, int lanes, long long ld) {
    if (lanes < 0 || ld < 0 || (dtype != AS_F32 && dtype != AS_BF16)) return 0;
    const size_t esz = dtype == AS_F32 ? 4 : 2;
    // the rows are staged at a pitch rounded up to 16 bytes (see as_step_host)
    return align256((size_t)lanes * ((((size_t)ld * esz) + 15) & ~(size_t)15)) + 2 * align256((size_t)lanes * 8) +
           2 * align256((size_t)lanes * 4) + 256;
}

int as_step_host(const void* h_logits, int dtype, int lanes, int V, long long ld, const double* h_codes,
                 double temp, int top_k, double top_p, int32_t* h_tokens, double* h_codes_out,
                 int32_t* h_lane_status, void* d_work, size_t work_bytes, void* stream) {
    if (lanes < 0) return set_err(AS_ERR_INVALID_ARG, "lanes = %d must be >= 0", lanes);
    int rc = check_scalars(dtype, V, ld, temp, top_p);
    if (rc != AS_OK) return rc;
    if (lanes == 0) return AS_OK;
    if ((rc = check_data(h_logits, dtype)) != AS_OK) return rc;
    if (!h_codes || !h_tokens || !h_codes_out) return set_err(AS_ERR_INVALID_ARG, "host codes / tokens / codes_out pointer is NULL");
    if (!d_work || (reinterpret_cast<uintptr_t>(d_work) & 255)) return set_err(AS_ERR_INVALID_ARG, "d_work must be a 256-byte aligned device pointer");
    if (work_bytes < as_step_host_work_bytes(dtype, lanes, ld)) return set_err(AS_ERR_INVALID_ARG, "work_bytes is smaller than as_step_host_work_bytes()");
    const size_t esz = dtype == AS_F32 ? 4 : 2;
    // A host pitch that is not a multiple of 16 bytes would leave every other row unaligned and
    // send it through the general routine; the copy can place the rows at an aligned pitch for free.
    const bool repitch = (((size_t)ld * esz) & 15) != 0;
    const size_t dpitch = repitch ? ((((size_t)V * esz) + 15) & ~(size_t)15) : (size_t)ld * esz;
    const long long d_ld = (long long)(dpitch / esz);
    const size_t nlog = (size_t)lanes * ((((size_t)ld * esz) + 15) & ~(size_t)15);
    char* w = reinterpret_cast<char*>(d_work);
    void* d_logits = w;                 w += align256(nlog);
    double* d_codes = (double*)w;       w += align256((size_t)lanes * 8);
    double* d_codes_out = (double*)w;   w += align256((size_t)lanes * 8);
    int32_t* d_tokens = (int32_t*)w;    w += align256((size_t)lanes * 4);
    int32_t* d_status = (int32_t*)w;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    // the last row may be shorter than ld in the caller's buffer: copy lanes-1 full pitches + V
    const size_t ncopy = ((size_t)(lanes - 1) * (size_t)ld + (size_t)V) * esz;
    if (repitch)
        e = cudaMemcpy2DAsync(d_logits, dpitch, h_logits, (size_t)ld * esz, (size_t)V * esz, (size_t)lanes,
                              cudaMemcpyHostToDevice, st);
    else
        e = cudaMemcpyAsync(d_logits, h_logits, ncopy, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e, "copy logits to device");
    if ((e = cudaMemcpyAsync(d_codes, h_codes, (size_t)lanes * 8, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e, "copy codes to device");
    as_step_diag dg = {nullptr, nullptr, nullptr, d_status, nullptr};
    rc = as_step(d_logits, dtype, lanes, V, d_ld, d_codes, temp, top_k, top_p, d_tokens, d_codes_out, &dg, stream);
    if (rc != AS_OK) {
        // the copies above are queued on the work buffer: do not hand it back while they run
        cudaStreamSynchronize(st);
        return rc;
    }
    if ((e = cudaMemcpyAsync(h_tokens, d_tokens, (size_t)lanes * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e, "copy tokens to host");
    if ((e = cudaMemcpyAsync(h_codes_out, d_codes_out, (size_t)lanes * 8, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e, "copy codes to host");
    if (h_lane_status && (e = cudaMemcpyAsync(h_lane_status, d_status, (size_t)lanes * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e, "copy status to host");
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(e, "stream synchronize");
    return AS_OK;
}

// ---------------------------------------------------------------------------
// as_step_host_static: the work buffer lives in the library
// ---------------------------------------------------------------------------
// Device memory reserved at load time on every GPU that loads this library.  In host code the
// name below is only a handle for the runtime, not a device address: the address a kernel or a
// copy can use comes from cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_static_work[AS_STATIC_WORK_BYTES];
static void* g_static_work_addr[64] = {nullptr};

static int static_work_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return set_err(AS_ERR_CUDA, "device ordinal %d out of range", dev);
    if (!g_static_work_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_work);      // this device is current
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static work buffer)");
        if (!p) return set_err(AS_ERR_CUDA, "static work buffer has no device address");
        g_static_work_addr[dev] = p;
    }
    *out = g_static_work_addr[dev];
    return AS_OK;
}

int as_step_host_static(const void* h_logits, int dtype, int lanes, int V, long long ld, const double* h_codes,
                        double temp, int top_k, double top_p, int32_t* h_tokens, double* h_codes_out,
                        int32_t* h_lane_status, void* stream) {
    if (lanes < 0) return set_err(AS_ERR_INVALID_ARG, "lanes = %d must be >= 0", lanes);
    int rc = check_scalars(dtype, V, ld, temp, top_p);
    if (rc != AS_OK) return rc;
    if (lanes == 0) return AS_OK;
    const size_t need = as_step_host_work_bytes(dtype, lanes, ld);
    if (need == 0 || need > (size_t)AS_STATIC_WORK_BYTES)
        return set_err(AS_ERR_UNSUPPORTED,
                       "this step needs %zu bytes of device work space, the built-in buffer holds %zu "
                       "(AS_STATIC_WORK_BYTES): use as_step_host with your own buffer, or fewer lanes per call",
                       need, (size_t)AS_STATIC_WORK_BYTES);
    void* work = nullptr;
    rc = static_work_address(&work);
    if (rc != AS_OK) return rc;
    return as_step_host(h_logits, dtype, lanes, V, ld, h_codes, temp, top_k, top_p, h_tokens, h_codes_out,
                        h_lane_status, work, (size_t)AS_STATIC_WORK_BYTES, stream);
}

static int decode_common(const void* d_table, int dtype, int V, long long ld, const int32_t* d_tok,
                         const double* d_codes_in, int lanes, int N, double u, int T, int eos,
                         double temp, int top_k, double top_p, int32_t* d_seq, int32_t* d_len,
                         double* d_codes_final, int32_t* d_lane_status, void* stream) {
    int rc = check_scalars(dtype, V, ld, temp, top_p);
    if (rc != AS_OK) return rc;
    if (T < 0) return set_err(AS_ERR_INVALID_ARG, "T = %d must be >= 0", T);
    if (lanes == 0) return AS_OK;
    if ((rc = check_data(d_table, dtype)) != AS_OK) return rc;
    if (!d_tok) return set_err(AS_ERR_INVALID_ARG, "start / prev token pointer is NULL");
    if (!d_len || (!d_seq && T > 0)) return set_err(AS_ERR_INVALID_ARG, "seq / len pointer is NULL");
    const DeviceInfo* di;
    rc = device_info(&di);
    if (rc != AS_OK) return rc;
    if (top_k < 0 || top_k >= V) top_k = 0;
    if (!(top_p > 0.0 && top_p < 1.0)) top_p = 1.0;
    const double inv_tau = 1.0 / temp;
    cudaStream_t st = (cudaStream_t)stream;
    if ((top_k > 0 || top_p < 1.0) && g_tune_path == 0 && d_codes_final && T > 0) {
        // lanes with a cut: one launch of the streaming kernel per step, rows gathered from the table
        StepArgs a;
        a.logits = d_table; a.codes = d_codes_final; a.codes_out = d_codes_final;
        a.diag = {nullptr, nullptr, nullptr, d_lane_status, nullptr};
        a.ld = ld; a.inv_tau = inv_tau; a.top_p = top_p; a.scale2 = (float)(1.4426950408889634 / temp);
        a.lanes = lanes; a.V = V; a.top_k = top_k;
        a.lat_N = 0; a.lat_j0 = 0; a.lat_u = 0.0;
        a.rows = V;
        a.xp_state = nullptr; a.xp_N = 0;
        a.wait_cycles = wait_cycles_now(); a.debug_no_copy = g_tune_no_copy; a.radix_nucleus = g_tune_radix_nucleus;
        cudaError_t e;
        bool served = true;
        for (int t = 0; t < T && served; ++t) {
            a.tokens = d_seq + t; a.tok_stride = T;
            a.row_idx = t == 0 ? d_len : d_seq + (t - 1);
            a.idx_stride = t == 0 ? 1 : T;
            a.eos = (t == 0 || eos < 0) ? -1 : eos;          // a start token may equal EOS
            if (t == 0) {
                // is this a step for the streaming kernel at all?  (decided before anything is written)
                StepArgs probe = a;
                const int E = dtype == AS_F32 ? 4 : 8;
                const size_t row_bytes = (size_t)((V + E - 1 + E - 1) / E) * 16;
                const int nsl = (int)((row_bytes + SK_STAGE_BYTES - 1) / SK_STAGE_BYTES);
                const bool resident = nsl <= SK_RES_STAGES && !(g_tune_stages > 0 && g_tune_stages < nsl);
                probe.fast = (top_k > 0 && top_k <= (resident ? SK_K0_RESIDENT : SK_K0_STREAMED)) || (top_k == 0 && top_p < 1.0);
                if (!probe.fast) { served = false; break; }
                const int sg = grid_for(lanes, di->sms, 8);
                decode_setup_kernel<<<sg, 256, 0, st>>>(d_tok, d_codes_in, lanes, N, u, V, T, d_len, d_codes_final, d_seq, d_lane_status);
                if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "decode set-up kernel launch");
            }
            rc = launch_streaming(a, dtype, true, di->sms, st);
            if (rc != AS_OK) return rc == AS_ERR_UNSUPPORTED ? set_err(AS_ERR_CUDA, "streaming kernel refused a decode step") : rc;
        }
        if (served) {
            decode_wrapup_kernel<<<grid_for(lanes, di->sms, 8), 256, 0, st>>>(d_seq, lanes, T, d_len);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "decode wrap-up kernel launch");
            return AS_OK;
        }
    }
    if (top_k == 0 && !(top_p < 1.0)) {
        NocutArgs n = {};
        n.data = d_table; n.ld = ld; n.V = V; n.lanes = lanes; n.inv_tau = inv_tau;
        n.tok_in = d_tok; n.codes_in = d_codes_in; n.N = N; n.u = u; n.T = T; n.eos = eos;
        n.seq = d_seq; n.len = d_len; n.codes_final = d_codes_final; n.lane_status = d_lane_status;
        rc = launch_nocut<NC_DECODE>(n, dtype, temp, di->sms, st);
        if (rc != AS_ERR_UNSUPPORTED) return rc;
    }
    const int grid = grid_for(lanes, di->sms, g_tune_ctas > 0 ? g_tune_ctas : 4);
    if (dtype == AS_F32)
        decode_generic_kernel<DT_F32><<<grid, GEN_NT, 0, st>>>(d_table, V, ld, d_tok, d_codes_in, lanes, N, u, T, eos, inv_tau, top_k, top_p, d_seq, d_len, d_codes_final, d_lane_status);
    else
        decode_generic_kernel<DT_BF16><<<grid, GEN_NT, 0, st>>>(d_table, V, ld, d_tok, d_codes_in, lanes, N, u, T, eos, inv_tau, top_k, top_p, d_seq, d_len, d_codes_final, d_lane_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "decode kernel launch");
    return AS_OK;
}

int as_decode_bigram(const void* d_table, int dtype, int V, long long ld, const int32_t* d_start, int S,
                     int N, double u, int T, int eos, double temp, int top_k, double top_p,
                     int32_t* d_seq, int32_t* d_len, double* d_codes_final, int32_t* d_lane_status,
                     void* stream) {
    if (S < 0) return set_err(AS_ERR_INVALID_ARG, "S = %d must be >= 0", S);
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (!(u >= 0.0 && u < 1.0)) return set_err(AS_ERR_INVALID_ARG, "shift u must lie in [0,1)");
    if ((long long)S * N > 0x7FFFFFFFLL) return set_err(AS_ERR_UNSUPPORTED, "S*N exceeds 2^31-1 lanes");
    return decode_common(d_table, dtype, V, ld, d_start, nullptr, S * N, N, u, T, eos, temp, top_k, top_p,
                         d_seq, d_len, d_codes_final, d_lane_status, stream);
}

int as_decode_bigram_codes(const void* d_table, int dtype, int V, long long ld, const int32_t* d_prev,
                           const double* d_codes_in, int lanes, int T, int eos, double temp, int top_k,
                           double top_p, int32_t* d_seq, int32_t* d_len, double* d_codes_final,
                           int32_t* d_lane_status, void* stream) {
    if (lanes < 0) return set_err(AS_ERR_INVALID_ARG, "lanes = %d must be >= 0", lanes);
    if (!d_codes_in) return set_err(AS_ERR_INVALID_ARG, "d_codes_in is NULL");
    return decode_common(d_table, dtype, V, ld, d_prev, d_codes_in, lanes, 1, 0.0, T, eos, temp, top_k, top_p,
                         d_seq, d_len, d_codes_final, d_lane_status, stream);
}

int as_encode_bigram(const void* d_table, int dtype, int V, long long ld, const int32_t* d_prev,
                     const int32_t* d_seq, const int32_t* d_len, int lanes, int T, double temp,
                     int top_k, double top_p, double* d_lo, double* d_width, int32_t* d_lane_status,
                     void* stream) {
    if (lanes < 0) return set_err(AS_ERR_INVALID_ARG, "lanes = %d must be >= 0", lanes);
    if (T < 0) return set_err(AS_ERR_INVALID_ARG, "T = %d must be >= 0", T);
    int rc = check_scalars(dtype, V, ld, temp, top_p);
    if (rc != AS_OK) return rc;
    if (lanes == 0) return AS_OK;
    if ((rc = check_data(d_table, dtype)) != AS_OK) return rc;
    if (!d_prev || !d_len || !d_lo || !d_width) return set_err(AS_ERR_INVALID_ARG, "d_prev, d_len, d_lo or d_width is NULL");
    if (T > 0 && !d_seq) return set_err(AS_ERR_INVALID_ARG, "d_seq is NULL");
    const DeviceInfo* di;
    rc = device_info(&di);
    if (rc != AS_OK) return rc;
    if (top_k < 0 || top_k >= V) top_k = 0;
    if (!(top_p > 0.0 && top_p < 1.0)) top_p = 1.0;
    const double inv_tau = 1.0 / temp;
    cudaStream_t st = (cudaStream_t)stream;
    if (top_k == 0 && !(top_p < 1.0)) {
        NocutArgs n = {};
        n.data = d_table; n.ld = ld; n.V = V; n.lanes = lanes; n.inv_tau = inv_tau;
        n.tok_in = d_prev; n.seq_in = d_seq; n.len_in = d_len; n.T = T;
        n.lo_out = d_lo; n.width_out = d_width; n.lane_status = d_lane_status;
        rc = launch_nocut<NC_ENCODE>(n, dtype, temp, di->sms, st);
        if (rc != AS_ERR_UNSUPPORTED) return rc;
    }
    const int grid = grid_for(lanes, di->sms, g_tune_ctas > 0 ? g_tune_ctas : 4);
    if (dtype == AS_F32)
        encode_generic_kernel<DT_F32><<<grid, GEN_NT, 0, st>>>(d_table, V, ld, d_prev, d_seq, d_len, lanes, T, inv_tau, top_k, top_p, d_lo, d_width, d_lane_status);
    else
        encode_generic_kernel<DT_BF16><<<grid, GEN_NT, 0, st>>>(d_table, V, ld, d_prev, d_seq, d_len, lanes, T, inv_tau, top_k, top_p, d_lo, d_width, d_lane_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "encode kernel launch");
    return AS_OK;
}

int as_ngram_diversity(const int32_t* d_seq, const int32_t* d_len, int S, int N, int T,
                       int64_t* d_unique, int64_t* d_total, double* d_div, void* stream) {
    if (S < 0) return set_err(AS_ERR_INVALID_ARG, "S = %d must be >= 0", S);
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (T < 0) return set_err(AS_ERR_INVALID_ARG, "T = %d must be >= 0", T);
    if ((long long)N * T > AS_NGRAM_MAX_ITEMS)
        return set_err(AS_ERR_UNSUPPORTED, "N * T = %lld exceeds AS_NGRAM_MAX_ITEMS = %d", (long long)N * T, AS_NGRAM_MAX_ITEMS);
    if (S == 0) return AS_OK;
    if (!d_len || !d_unique || !d_total || !d_div || (!d_seq && T > 0))
        return set_err(AS_ERR_INVALID_ARG, "d_seq, d_len, d_unique, d_total or d_div is NULL");
    const DeviceInfo* di;
    int rc = device_info(&di);
    if (rc != AS_OK) return rc;
    const int items = N * T;
    int cap = 64;
    while (cap < 2 * items) cap <<= 1;
    const size_t smem = sizeof(int) * ((size_t)items + N + cap);
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaGetDevice(&dev);
    cudaError_t e;
    if (!attr_set[dev]) {
        e = cudaFuncSetAttribute(ngram_diversity_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(SMEM_OPTIN_MAX - 1024));
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(max dynamic shared memory)");
        attr_set[dev] = true;
    }
    if (smem > SMEM_OPTIN_MAX - 1024) return set_err(AS_ERR_UNSUPPORTED, "group of %d x %d tokens does not fit shared memory", N, T);
    const int grid = S < di->sms * 2 ? S : di->sms * 2;
    ngram_diversity_kernel<<<grid, NG_NT, smem, (cudaStream_t)stream>>>(d_seq, d_len, S, N, T, cap,
                                                                        reinterpret_cast<long long*>(d_unique),
                                                                        reinterpret_cast<long long*>(d_total), d_div);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "n-gram diversity kernel launch");
    return AS_OK;
}

int as_reward_mean(const int32_t* d_seq, const int32_t* d_len, int S, int N, int T, const double* d_r, int V,
                   double* d_lane_reward, double* d_mean, int32_t* d_group_status, void* stream) {
    if (S < 0) return set_err(AS_ERR_INVALID_ARG, "S = %d must be >= 0", S);
    if (N < 1 || N > AS_REWARD_MAX_N) return set_err(AS_ERR_INVALID_ARG, "N = %d must lie in [1, %d]", N, AS_REWARD_MAX_N);
    if (T < 0) return set_err(AS_ERR_INVALID_ARG, "T = %d must be >= 0", T);
    if (V < 1) return set_err(AS_ERR_INVALID_ARG, "V = %d must be >= 1", V);
    if (S == 0) return AS_OK;
    if (!d_len || !d_r || !d_mean || (!d_seq && T > 0))
        return set_err(AS_ERR_INVALID_ARG, "d_seq, d_len, d_r or d_mean is NULL");
    const DeviceInfo* di;
    int rc = device_info(&di);
    if (rc != AS_OK) return rc;
    const int grid = S < di->sms * 8 ? S : di->sms * 8;
    reward_mean_kernel<<<grid, RM_NT, sizeof(double) * (size_t)N, (cudaStream_t)stream>>>(
        d_seq, d_len, S, N, T, d_r, V, d_lane_reward, d_mean, d_group_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "reward mean kernel launch");
    return AS_OK;
}

int as_xp_lattice_state(int N, double u, int j0, int count, int S, uint64_t* d_state, void* stream) {
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (!(u >= 0.0 && u < 1.0)) return set_err(AS_ERR_INVALID_ARG, "shift u must lie in [0,1)");
    if (j0 < 0 || count < 0 || (long long)j0 + count > N)
        return set_err(AS_ERR_INVALID_ARG, "codes j0 .. j0+count-1 must lie in [0, N = %d)", N);
    if (S < 0) return set_err(AS_ERR_INVALID_ARG, "S = %d must be >= 0", S);
    if (count == 0 || S == 0) return AS_OK;
    if (!d_state) return set_err(AS_ERR_INVALID_ARG, "d_state is NULL");
    const DeviceInfo* di;
    int rc = device_info(&di);
    if (rc != AS_OK) return rc;
    const unsigned long long U = (unsigned long long)std::floor(u * 9007199254740992.0);   // floor(u 2^53), exact
    xp_state_kernel<<<(count + 127) / 128, 128, 0, (cudaStream_t)stream>>>(N, U, j0, count, S,
                                                                            reinterpret_cast<unsigned long long*>(d_state));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "extended-precision state kernel launch");
    return AS_OK;
}

int as_decode_bigram_xp(const void* d_table, int dtype, int V, long long ld, const int32_t* d_prev,
                        uint64_t* d_state, int lanes, int N, int T, int eos, double temp, int top_k,
                        double top_p, int32_t* d_seq, int32_t* d_len, int32_t* d_lane_status, void* stream) {
    if (lanes < 0) return set_err(AS_ERR_INVALID_ARG, "lanes = %d must be >= 0", lanes);
    if (N < 1) return set_err(AS_ERR_INVALID_ARG, "N = %d must be >= 1", N);
    if (T < 0) return set_err(AS_ERR_INVALID_ARG, "T = %d must be >= 0", T);
    int rc = check_scalars(dtype, V, ld, temp, top_p);
    if (rc != AS_OK) return rc;
    if (lanes == 0) return AS_OK;
    if ((rc = check_data(d_table, dtype)) != AS_OK) return rc;
    if (!d_prev || !d_state || !d_len || (!d_seq && T > 0))
        return set_err(AS_ERR_INVALID_ARG, "d_prev, d_state, d_seq or d_len is NULL");
    const DeviceInfo* di;
    rc = device_info(&di);
    if (rc != AS_OK) return rc;
    if (top_k < 0 || top_k >= V) top_k = 0;
    if (!(top_p > 0.0 && top_p < 1.0)) top_p = 1.0;
    const double inv_tau = 1.0 / temp;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long* state = reinterpret_cast<unsigned long long*>(d_state);
    if (top_k == 0 && !(top_p < 1.0)) {
        NocutArgs n = {};
        n.data = d_table; n.ld = ld; n.V = V; n.lanes = lanes; n.inv_tau = inv_tau;
        n.tok_in = d_prev; n.N = N; n.T = T; n.eos = eos;
        n.seq = d_seq; n.len = d_len; n.lane_status = d_lane_status; n.xp_state = state;
        rc = launch_nocut<NC_DECODE_XP>(n, dtype, temp, di->sms, st);
        if (rc != AS_ERR_UNSUPPORTED) return rc;
    }
    if ((top_k > 0 || top_p < 1.0) && g_tune_path == 0 && T > 0) {
        // lanes with a cut: one launch of the streaming kernel per step, rows gathered from the table,
        // the states advanced in place (as the fp64 loop does with its codes)
        StepArgs a;
        a.logits = d_table; a.codes = nullptr; a.codes_out = nullptr;
        a.diag = {nullptr, nullptr, nullptr, d_lane_status, nullptr};
        a.ld = ld; a.inv_tau = inv_tau; a.top_p = top_p; a.scale2 = (float)(1.4426950408889634 / temp);
        a.lanes = lanes; a.V = V; a.top_k = top_k;
        a.lat_N = 0; a.lat_j0 = 0; a.lat_u = 0.0;
        a.rows = V;
        a.xp_state = state; a.xp_N = N;
        a.wait_cycles = wait_cycles_now(); a.debug_no_copy = g_tune_no_copy; a.radix_nucleus = g_tune_radix_nucleus;
        const int E = dtype == AS_F32 ? 4 : 8;
        const size_t row_bytes = (size_t)((V + E - 1 + E - 1) / E) * 16;
        const int nsl = (int)((row_bytes + SK_STAGE_BYTES - 1) / SK_STAGE_BYTES);
        const bool resident = nsl <= SK_RES_STAGES && !(g_tune_stages > 0 && g_tune_stages < nsl);
        const bool fast = (top_k > 0 && top_k <= (resident ? SK_K0_RESIDENT : SK_K0_STREAMED)) || (top_k == 0 && top_p < 1.0);
        if (resident || fast) {
            cudaError_t e;
            decode_setup_kernel<<<grid_for(lanes, di->sms, 8), 256, 0, st>>>(d_prev, nullptr, lanes, 1, 0.0, V, T, d_len, nullptr, d_seq, d_lane_status);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "decode set-up kernel launch");
            for (int t = 0; t < T; ++t) {
                a.tokens = d_seq + t; a.tok_stride = T;
                a.row_idx = t == 0 ? d_len : d_seq + (t - 1);
                a.idx_stride = t == 0 ? 1 : T;
                a.eos = (t == 0 || eos < 0) ? -1 : eos;
                rc = launch_streaming(a, dtype, true, di->sms, st);
                if (rc != AS_OK) return rc == AS_ERR_UNSUPPORTED ? set_err(AS_ERR_CUDA, "streaming kernel refused a decode step") : rc;
            }
            decode_wrapup_kernel<<<grid_for(lanes, di->sms, 8), 256, 0, st>>>(d_seq, lanes, T, d_len);
            if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "decode wrap-up kernel launch");
            return AS_OK;
        }
    }
    const int grid = grid_for(lanes, di->sms, g_tune_ctas > 0 ? g_tune_ctas : 4);
    if (dtype == AS_F32)
        decode_xp_generic_kernel<DT_F32><<<grid, GEN_NT, 0, st>>>(d_table, V, ld, d_prev, state, lanes, N, T, eos, inv_tau, top_k, top_p, d_seq, d_len, d_lane_status);
    else
        decode_xp_generic_kernel<DT_BF16><<<grid, GEN_NT, 0, st>>>(d_table, V, ld, d_prev, state, lanes, N, T, eos, inv_tau, top_k, top_p, d_seq, d_len, d_lane_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "extended-precision decode kernel launch");
    return AS_OK;
}

}  // extern "C"

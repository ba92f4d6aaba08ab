// Shared device helpers: order-preserving integer keys for bf16 / fp32 logits,
// an fp64 exp for non-positive arguments, warp scans and reductions.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace asx {

constexpr int DT_F32 = 0;
constexpr int DT_BF16 = 1;

constexpr int ST_OK = 0;
constexpr int ST_TIMEOUT = -4;
constexpr int ST_NUMERIC = -5;

// Checked builds (-DAS_BOUNDS_CHECK): every index into a ring stage, a hit or candidate list, a
// rank array, a histogram, a chunk array, the mass table or a row buffer goes through ASX_AT.  An
// index outside [0, n) is recorded (the count of failures and the first one's site, index and
// bound) and replaced by 0, so that the access stays in bounds: nothing traps, and the host reads
// the record after the launch.  In ordinary builds ASX_AT(i, n, site) is just i.
#ifdef AS_BOUNDS_CHECK
__device__ int g_asx_bounds[4];
__device__ __forceinline__ bool asx_in(long long i, long long n, int site) {
    if (i >= 0 && i < n) return true;
    if (atomicAdd(&g_asx_bounds[0], 1) == 0) {
        g_asx_bounds[1] = site;
        g_asx_bounds[2] = (int)i;
        g_asx_bounds[3] = (int)n;
    }
    return false;
}
#define ASX_AT(i, n, site) (asx_in((long long)(i), (long long)(n), (site)) ? (i) : 0)
#else
#define ASX_AT(i, n, site) (i)
#endif

// Largest double below 1: rescaled codes are clamped into [0, ONE_BELOW].
#define ASX_ONE_BELOW 0x1.fffffffffffffp-1

// ---------------------------------------------------------------------------
// Keys: an unsigned integer whose order equals the order of the stored float
// (the two zeros share one key).  -inf maps to KEY_NINF (masked token); anything below it is a negative NaN,
// anything >= KEY_PINF is +inf or a positive NaN.
// ---------------------------------------------------------------------------
template <int DT> struct Traits;

template <> struct Traits<DT_F32> {
    static constexpr int E = 4;            // elements per 16-byte vector
    static constexpr int BYTES = 4;
    static constexpr int KEYBITS = 32;
    static constexpr uint32_t KEY_NINF = 0x007FFFFFu;
    static constexpr uint32_t KEY_PINF = 0xFF800000u;
    // (-0.0 gets the key of +0.0: the two compare equal, so they must tie and fall to the index)
    __device__ __forceinline__ static uint32_t key_of(uint32_t bits) {
        if (bits == 0x80000000u) bits = 0u;
        return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
    }
    __device__ __forceinline__ static float value_f(uint32_t key) {
        uint32_t bits = (key & 0x80000000u) ? (key ^ 0x80000000u) : ~key;
        return __uint_as_float(bits);
    }
    __device__ __forceinline__ static void unpack(const uint4& q, uint32_t (&k)[4]) {
        k[0] = key_of(q.x); k[1] = key_of(q.y); k[2] = key_of(q.z); k[3] = key_of(q.w);
    }
    __device__ __forceinline__ static uint32_t load_key(const void* row, long long j) {
        return key_of(reinterpret_cast<const uint32_t*>(row)[j]);
    }
};

template <> struct Traits<DT_BF16> {
    static constexpr int E = 8;
    static constexpr int BYTES = 2;
    static constexpr int KEYBITS = 16;
    static constexpr uint32_t KEY_NINF = 0x007Fu;
    static constexpr uint32_t KEY_PINF = 0xFF80u;
    __device__ __forceinline__ static uint32_t key_of(uint32_t b16) {
        if (b16 == 0x8000u) b16 = 0u;                   // -0.0 ties with +0.0
        return (b16 & 0x8000u) ? (~b16 & 0xFFFFu) : (b16 | 0x8000u);
    }
    __device__ __forceinline__ static float value_f(uint32_t key) {
        uint32_t bits = (key & 0x8000u) ? (key ^ 0x8000u) : (~key & 0xFFFFu);
        return __uint_as_float(bits << 16);
    }
    __device__ __forceinline__ static void unpack(const uint4& q, uint32_t (&k)[8]) {
        k[0] = key_of(q.x & 0xFFFFu); k[1] = key_of(q.x >> 16);
        k[2] = key_of(q.y & 0xFFFFu); k[3] = key_of(q.y >> 16);
        k[4] = key_of(q.z & 0xFFFFu); k[5] = key_of(q.z >> 16);
        k[6] = key_of(q.w & 0xFFFFu); k[7] = key_of(q.w >> 16);
    }
    __device__ __forceinline__ static uint32_t load_key(const void* row, long long j) {
        return key_of(reinterpret_cast<const uint16_t*>(row)[j]);
    }
};

// Keys of the E elements of vector `vi` of a row (element base vi*E); elements
// at or past V read as masked.  `vec_ok`: the row start is 16-byte aligned.
template <int DT>
__device__ __forceinline__ void load_vec_keys(const void* row, int V, int vi, bool vec_ok,
                                              uint32_t (&k)[Traits<DT>::E]) {
    using Tr = Traits<DT>;
    const int base = vi * Tr::E;
    if (vec_ok && base + Tr::E <= V) {
        const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(row) +
                                                        (size_t)base * Tr::BYTES);
        Tr::unpack(q, k);
    } else {
#pragma unroll
        for (int e = 0; e < Tr::E; ++e)
            k[e] = (base + e < V) ? Tr::load_key(row, base + e) : Tr::KEY_NINF;
    }
}

// ---------------------------------------------------------------------------
// exp(y) for y <= 0 in fp64: y = (64 n + j) ln2/64 + f, |f| <= ln2/128;
// exp(y) = 2^n * 2^(j/64) * exp(f), exp(f) by a degree-5 polynomial
// (truncation ~3e-17).  tbl[j] = 2^(j/64).  Arguments below -700 return 0.
// ---------------------------------------------------------------------------
// exp(y) for |y| <= 700 or so (no range check: the result's exponent is formed by integer addition)
__device__ __forceinline__ double exp_core(double y, const double* __restrict__ tbl) {
    const double MAGIC = 6755399441055744.0;          // 1.5 * 2^52: rounds to integer
    double r = fma(y, 0x1.71547652b82fep+6, MAGIC);    // y * 64/ln2
    const int k = __double2loint(r);
    r -= MAGIC;
    double f = fma(r, -0x1.62e42fe000000p-7, y);       // ln2/64, high part (24 low bits zero)
    f = fma(r, -0x1.f473de6af278fp-36, f);             // ln2/64, low part
    double p = fma(f, 1.0 / 120.0, 1.0 / 24.0);
    p = fma(p, f, 1.0 / 6.0);
    p = fma(p, f, 0.5);
    p = fma(p, f, 1.0);
    p = fma(p, f, 1.0);
    const double v = tbl[k & 63] * p;
    const int n = k >> 6;                              // floor((64n+j)/64)
    return __hiloint2double(__double2hiint(v) + (n << 20), __double2loint(v));
}
__device__ __forceinline__ double exp_nonpos(double y, const double* __restrict__ tbl) {
    if (!(y >= -700.0)) return 0.0;
    return exp_core(y, tbl);
}

// 2^(j/64), j = 0..63, correctly rounded.
__device__ const double ASX_T64[64] = {
    0x1.0000000000000p+0, 0x1.02c9a3e778061p+0, 0x1.059b0d3158574p+0, 0x1.0874518759bc8p+0,
    0x1.0b5586cf9890fp+0, 0x1.0e3ec32d3d1a2p+0, 0x1.11301d0125b51p+0, 0x1.1429aaea92de0p+0,
    0x1.172b83c7d517bp+0, 0x1.1a35beb6fcb75p+0, 0x1.1d4873168b9aap+0, 0x1.2063b88628cd6p+0,
    0x1.2387a6e756238p+0, 0x1.26b4565e27cddp+0, 0x1.29e9df51fdee1p+0, 0x1.2d285a6e4030bp+0,
    0x1.306fe0a31b715p+0, 0x1.33c08b26416ffp+0, 0x1.371a7373aa9cbp+0, 0x1.3a7db34e59ff7p+0,
    0x1.3dea64c123422p+0, 0x1.4160a21f72e2ap+0, 0x1.44e086061892dp+0, 0x1.486a2b5c13cd0p+0,
    0x1.4bfdad5362a27p+0, 0x1.4f9b2769d2ca7p+0, 0x1.5342b569d4f82p+0, 0x1.56f4736b527dap+0,
    0x1.5ab07dd485429p+0, 0x1.5e76f15ad2148p+0, 0x1.6247eb03a5585p+0, 0x1.6623882552225p+0,
    0x1.6a09e667f3bcdp+0, 0x1.6dfb23c651a2fp+0, 0x1.71f75e8ec5f74p+0, 0x1.75feb564267c9p+0,
    0x1.7a11473eb0187p+0, 0x1.7e2f336cf4e62p+0, 0x1.82589994cce13p+0, 0x1.868d99b4492edp+0,
    0x1.8ace5422aa0dbp+0, 0x1.8f1ae99157736p+0, 0x1.93737b0cdc5e5p+0, 0x1.97d829fde4e50p+0,
    0x1.9c49182a3f090p+0, 0x1.a0c667b5de565p+0, 0x1.a5503b23e255dp+0, 0x1.a9e6b5579fdbfp+0,
    0x1.ae89f995ad3adp+0, 0x1.b33a2b84f15fbp+0, 0x1.b7f76f2fb5e47p+0, 0x1.bcc1e904bc1d2p+0,
    0x1.c199bdd85529cp+0, 0x1.c67f12e57d14bp+0, 0x1.cb720dcef9069p+0, 0x1.d072d4a07897cp+0,
    0x1.d5818dcfba487p+0, 0x1.da9e603db3285p+0, 0x1.dfc97337b9b5fp+0, 0x1.e502ee78b3ff6p+0,
    0x1.ea4afa2a490dap+0, 0x1.efa1bee615a27p+0, 0x1.f50765b6e4540p+0, 0x1.fa7c1819e90d8p+0};

// Copies the table into shared memory (divergent indices make a constant-bank
// read serialise; a shared-memory read does not).  Caller synchronises after.
__device__ __forceinline__ void fill_exp_table(double* tbl, int tid) {
    if (tid < 64) tbl[tid] = ASX_T64[tid];
}

// Additions to shared memory without a return value, on the shared-space address: through a
// pointer whose address space the compiler cannot see they would be issued as generic atomics,
// which take tens of cycles per lane on shared memory.
__device__ __forceinline__ void red_shared_add(float* p, float v) {
    asm volatile("red.shared.add.f32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "f"(v) : "memory");
}
__device__ __forceinline__ void red_shared_add(int* p, int v) {
    asm volatile("red.shared.add.s32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v) : "memory");
}
__device__ __forceinline__ void red_shared_or(unsigned* p, unsigned v) {
    asm volatile("red.shared.or.b32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned atom_shared_add(unsigned* p, unsigned v) {
    unsigned old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void red_shared_add(unsigned long long* p, unsigned long long v) {
    asm volatile("red.shared.add.u64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "l"(v) : "memory");
}

// ---------------------------------------------------------------------------
// Warp primitives (all 32 lanes active).
// ---------------------------------------------------------------------------
constexpr unsigned FULL = 0xFFFFFFFFu;

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}
// 32-bit integer reductions: one redux.sync instruction each instead of five shuffle steps
__device__ __forceinline__ int warp_sum_i(int v) { return __reduce_add_sync(FULL, v); }
__device__ __forceinline__ unsigned warp_max_u(unsigned v) { return __reduce_max_sync(FULL, v); }
__device__ __forceinline__ unsigned warp_min_u(unsigned v) { return __reduce_min_sync(FULL, v); }
// inclusive scans over lanes 0..31 in lane order
__device__ __forceinline__ double warp_incl_scan_d(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double u = __shfl_up_sync(FULL, v, o);
        if (lane >= o) v += u;
    }
    return v;
}
__device__ __forceinline__ int warp_incl_scan_i(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(FULL, v, o);
        if (lane >= o) v += u;
    }
    return v;
}
// inclusive suffix sums: lane l gets the sum over lanes >= l
__device__ __forceinline__ double warp_suffix_d(double v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double u = __shfl_down_sync(FULL, v, o);
        if (lane + o < 32) v += u;
    }
    return v;
}
__device__ __forceinline__ int warp_suffix_i(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_down_sync(FULL, v, o);
        if (lane + o < 32) v += u;
    }
    return v;
}

// ---------------------------------------------------------------------------
// 2^(t/64) for t <= 0 in fp64, t given in units of 1/64 (t = (x - max)/temp * 64 log2 e):
// t = 64 n + j + f, |f| <= 1/2;  2^(t/64) = 2^n * 2^(j/64) * exp(f ln2/64), the last factor by a
// degree-5 polynomial (truncation ~3e-17).  One fused multiply-add upstream forms t, so the
// whole evaluation is 10 fp64 operations.  Arguments below -64000 (2^-1000) return 0.
// ---------------------------------------------------------------------------
template <bool GUARD = true>
__device__ __forceinline__ double exp2_64th(double t, const double* __restrict__ tbl) {
    if (GUARD && !(t >= -64000.0)) return 0.0;     // (without the guard the caller vouches for t >= -64000)
    const double MAGIC = 6755399441055744.0;
    double r = t + MAGIC;
    const int k = __double2loint(r);
    r -= MAGIC;
    const double f = t - r;
    const double L = 0x1.62e42fefa39efp-7;               // ln2 / 64
    double p = fma(f, L * L * L * L * L / 120.0, L * L * L * L / 24.0);
    p = fma(p, f, L * L * L / 6.0);
    p = fma(p, f, L * L / 2.0);
    p = fma(p, f, L);
    p = fma(p, f, 1.0);
    const double v = tbl[k & 63] * p;
    const int n = k >> 6;
    return __hiloint2double(__double2hiint(v) + (n << 20), __double2loint(v));
}

// ---------------------------------------------------------------------------
// Packed NaN-propagating maxima and float views of one 16-byte vector.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t min_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float max_nan_f32(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}
__device__ __forceinline__ float ex2_approx(float y) {
    float d;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(d) : "f"(y));
    return d;
}

template <int DT> struct Pass;
template <> struct Pass<DT_BF16> {
    // running NaN-propagating max, two bf16 lanes packed in one register
    struct Acc { uint32_t m; };
    __device__ static Acc init() { return Acc{0xFF80FF80u}; }            // (-inf, -inf)
    __device__ static void fold(Acc& a, const uint4& q) {
        a.m = max_nan_bf16x2(a.m, max_nan_bf16x2(max_nan_bf16x2(q.x, q.y), max_nan_bf16x2(q.z, q.w)));
    }
    // NaN-propagating max of one vector, kept packed; merged into the running max and
    // reused for the "any element >= threshold" test
    __device__ static Acc reduce(const uint4& q) {
        return Acc{max_nan_bf16x2(max_nan_bf16x2(q.x, q.y), max_nan_bf16x2(q.z, q.w))};
    }
    __device__ static void merge(Acc& a, const Acc& b) { a.m = max_nan_bf16x2(a.m, b.m); }
    __device__ static void fold_scalar(Acc& a, const void* row, long long j) {
        const uint32_t b = reinterpret_cast<const uint16_t*>(row)[j];
        a.m = max_nan_bf16x2(a.m, b | (b << 16));
    }
    __device__ static float load_f(const void* row, long long j) {
        return __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(row)[j] << 16);
    }
    __device__ static float part_max(const Acc& b) {
        return fmaxf(__uint_as_float(b.m << 16), __uint_as_float(b.m & 0xFFFF0000u));
    }
    __device__ static void keys(const Acc& a, uint32_t& k0, uint32_t& k1) {
        k0 = Traits<DT_BF16>::key_of(a.m & 0xFFFFu);
        k1 = Traits<DT_BF16>::key_of(a.m >> 16);
    }
    __device__ static uint32_t key16(uint32_t key) { return key; }
    __device__ static uint32_t key_from16(uint32_t k16) { return k16; }
    __device__ static void floats(const uint4& q, float (&x)[8]) {
        x[0] = __uint_as_float(q.x << 16); x[1] = __uint_as_float(q.x & 0xFFFF0000u);
        x[2] = __uint_as_float(q.y << 16); x[3] = __uint_as_float(q.y & 0xFFFF0000u);
        x[4] = __uint_as_float(q.z << 16); x[5] = __uint_as_float(q.z & 0xFFFF0000u);
        x[6] = __uint_as_float(q.w << 16); x[7] = __uint_as_float(q.w & 0xFFFF0000u);
    }
    // max of the 8 elements (no NaN present any more)
    __device__ static float vmax(const uint4& q) {
        const uint32_t m = max_nan_bf16x2(max_nan_bf16x2(q.x, q.y), max_nan_bf16x2(q.z, q.w));
        return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    }
    __device__ static uint32_t key_of_f(float x) { return Traits<DT_BF16>::key_of(__float_as_uint(x) >> 16); }
    // min of the 8 elements (NaN-free data; a NaN is caught by the max pass)
    __device__ static float vmin(const uint4& q) {
        const uint32_t m = min_bf16x2(min_bf16x2(q.x, q.y), min_bf16x2(q.z, q.w));
        return fminf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    }
};
template <> struct Pass<DT_F32> {
    struct Acc { float a, b; };
    __device__ static Acc init() { return Acc{__uint_as_float(0xFF800000u), __uint_as_float(0xFF800000u)}; }
    __device__ static void fold(Acc& s, const uint4& q) {
        s.a = max_nan_f32(s.a, max_nan_f32(__uint_as_float(q.x), __uint_as_float(q.z)));
        s.b = max_nan_f32(s.b, max_nan_f32(__uint_as_float(q.y), __uint_as_float(q.w)));
    }
    __device__ static Acc reduce(const uint4& q) {
        return Acc{max_nan_f32(__uint_as_float(q.x), __uint_as_float(q.z)),
                   max_nan_f32(__uint_as_float(q.y), __uint_as_float(q.w))};
    }
    __device__ static void merge(Acc& s, const Acc& b) { s.a = max_nan_f32(s.a, b.a); s.b = max_nan_f32(s.b, b.b); }
    __device__ static void fold_scalar(Acc& s, const void* row, long long j) {
        s.a = max_nan_f32(s.a, reinterpret_cast<const float*>(row)[j]);
    }
    __device__ static float load_f(const void* row, long long j) { return reinterpret_cast<const float*>(row)[j]; }
    __device__ static float part_max(const Acc& b) { return fmaxf(b.a, b.b); }
    __device__ static void keys(const Acc& s, uint32_t& k0, uint32_t& k1) {
        k0 = Traits<DT_F32>::key_of(__float_as_uint(s.a));
        k1 = Traits<DT_F32>::key_of(__float_as_uint(s.b));
    }
    __device__ static uint32_t key16(uint32_t key) { return key >> 16; }
    __device__ static uint32_t key_from16(uint32_t k16) { return k16 << 16; }   // rounds the bound down
    __device__ static void floats(const uint4& q, float (&x)[4]) {
        x[0] = __uint_as_float(q.x); x[1] = __uint_as_float(q.y);
        x[2] = __uint_as_float(q.z); x[3] = __uint_as_float(q.w);
    }
    __device__ static float vmax(const uint4& q) {
        return fmaxf(fmaxf(__uint_as_float(q.x), __uint_as_float(q.y)),
                     fmaxf(__uint_as_float(q.z), __uint_as_float(q.w)));
    }
    __device__ static uint32_t key_of_f(float x) { return Traits<DT_F32>::key_of(__float_as_uint(x)); }
    __device__ static float vmin(const uint4& q) {
        return fminf(fminf(__uint_as_float(q.x), __uint_as_float(q.y)),
                     fminf(__uint_as_float(q.z), __uint_as_float(q.w)));
    }
};

// ---------------------------------------------------------------------------
// Extended-precision codes: Algorithm 1's c <- (c - m)/(M - m) in exact arithmetic, as the
// step of an arithmetic decoder.  A lane's state is four 64-bit words: the current interval
// has `range` units, in (2^62, 2^63]; `code` < range is the code's offset in it; `q` holds the
// not yet consumed bits of the code's first 53 binary digits, `packed` = (their number << 32)
// | the remainder of the long division that yields all further digits of the rational code
// (j + u)/N.  One step cuts the interval into 2^32 cells of r = range >> 32 units; the cell
// t = min(code / r, 2^32 - 1) holds the code; token j owns the cells [F(P_j), F(P_{j+1})) with
// P the prefix sums of the kept masses in index order and F(P) = floor(P * 2^32 / Z), the last
// token with mass ending at 2^32 (it also takes the range mod 2^32 units left over).
// ---------------------------------------------------------------------------
constexpr unsigned long long XP_TOP = 0x100000000ull;           // 2^32 cells
constexpr unsigned long long XP_RANGE_TOP = 1ull << 63;
constexpr unsigned long long XP_RANGE_LOW = 1ull << 62;

struct XpState {
    unsigned long long range, code, q, packed;
};

__device__ __forceinline__ unsigned long long xp_cell(double P, double K) {
    const double f = P * K;
    return f >= 4294967296.0 ? XP_TOP : (unsigned long long)f;
}
__device__ __forceinline__ bool xp_state_ok(const XpState& s) {
    return s.range > XP_RANGE_LOW && s.range <= XP_RANGE_TOP && s.code < s.range;
}
__device__ __forceinline__ unsigned long long xp_target(const XpState& s) {
    const unsigned long long t = s.code / (s.range >> 32);
    return t > 0xFFFFFFFFull ? 0xFFFFFFFFull : t;
}
// the next k <= 32 binary digits of the code, most significant first
__device__ __forceinline__ unsigned long long xp_next_bits(XpState& s, int k, unsigned N) {
    unsigned long long out = 0;
    int nq = (int)(s.packed >> 32);
    unsigned long long rem = s.packed & 0xFFFFFFFFull;
    const int take = k < nq ? k : nq;
    if (take > 0) {
        nq -= take;
        out = (s.q >> nq) & ((1ull << take) - 1ull);
        s.q &= nq ? ((1ull << nq) - 1ull) : 0ull;
        k -= take;
    }
    if (k > 0) {
        const unsigned long long x = rem << k;            // rem < N < 2^31, k <= 32
        out = (out << k) | (x / N);
        rem = x % N;
    }
    s.packed = ((unsigned long long)nq << 32) | rem;
    return out;
}
// the chosen token owns the cells [lo, hi): narrow the interval to it and shift digits in
__device__ __forceinline__ void xp_advance(XpState& s, unsigned long long lo, unsigned long long hi, unsigned N) {
    const unsigned long long r = s.range >> 32;
    s.code -= r * lo;
    s.range = hi == XP_TOP ? s.range - r * lo : r * (hi - lo);
    int shift = __clzll((long long)(s.range - 1)) - 1;    // range -> (2^62, 2^63]
    while (shift > 0) {
        const int k = shift < 32 ? shift : 32;
        s.code = (s.code << k) | xp_next_bits(s, k, N);
        s.range <<= k;
        shift -= k;
    }
}

// One sub-row of the chunk that holds the code's cell: lane l has the masses ev[0..E) of E
// consecutive tokens, lanes in index order.  `run` is the fp64 prefix before the sub-row,
// `carry` the cell where it starts (both uniform, both advanced here).  The cell where a lane's
// last token with mass ends is computed once and handed on, so that neighbouring tokens always
// meet in the same cell whatever the rounding of the sums; the chunk's last token with mass
// (in the sub-row flagged is_last) ends at Fend.  Returns the lane that holds the token (its
// element pk, cells [plo, phi), mass pe) or -1; uniform.
template <int E>
__device__ __forceinline__ int xp_subrow(const double (&ev)[E], int lane, double K, unsigned long long tcell,
                                         bool is_last, unsigned long long Fend, double& run,
                                         unsigned long long& carry, int& pk, unsigned long long& plo,
                                         unsigned long long& phi, double& pe) {
    double local = 0.0;
    int klast = -1;
#pragma unroll
    for (int k = 0; k < E; ++k) { local += ev[k]; if (ev[k] > 0.0) klast = k; }
    const double incl = warp_incl_scan_d(local, lane);
    double excl = __shfl_up_sync(FULL, incl, 1);
    if (lane == 0) excl = 0.0;
    const unsigned massive = __ballot_sync(FULL, local > 0.0);
    const double run_next = run + __shfl_sync(FULL, incl, 31);
    if (!massive) { run = run_next; return -1; }
    const int Llast = 31 - __clz(massive);
    const unsigned long long endc = (is_last && lane == Llast) ? Fend : xp_cell(run + incl, K);
    const unsigned before = massive & ((1u << lane) - 1u);
    const unsigned long long prev_end = __shfl_sync(FULL, endc, before ? 31 - __clz(before) : 0);
    unsigned long long lo = before ? prev_end : carry;
    int pick = -1;
    unsigned long long mylo = 0, myhi = 0;
    double mye = 1.0;
    double S = run + excl;
#pragma unroll
    for (int k = 0; k < E; ++k) {
        if (ev[k] > 0.0) {
            unsigned long long hi;
            if (k == klast) {
                hi = endc;
            } else {
                S += ev[k];
                hi = xp_cell(S, K);
            }
            if (pick < 0 && hi > tcell) { pick = k; mylo = lo; myhi = hi; mye = ev[k]; }
            lo = hi;
        }
    }
    carry = __shfl_sync(FULL, endc, Llast);
    run = run_next;
    const unsigned bal = __ballot_sync(FULL, pick >= 0);
    if (!bal) return -1;
    const int L = __ffs(bal) - 1;
    pk = __shfl_sync(FULL, pick, L);
    plo = __shfl_sync(FULL, mylo, L);
    phi = __shfl_sync(FULL, myhi, L);
    pe = __shfl_sync(FULL, mye, L);
    return L;
}

// The same selection over one list of tokens in index order, lane l owning the positions [b, en)
// (masses through ev(i)); the list is the whole kept set: it starts at cell 0 and its last token
// with mass ends at 2^32.  Returns the owning lane (position pidx, cells [plo, phi), mass pe) or -1;
// Z receives the total mass.  Uniform.
template <class F>
__device__ __forceinline__ int xp_span(int b, int en, F&& ev, int lane, unsigned long long tcell, int& pidx,
                                       unsigned long long& plo, unsigned long long& phi, double& pe, double& Z) {
    double local = 0.0;
    int klast = -1;
    for (int i = b; i < en; ++i) {
        const double m = ev(i);
        local += m;
        if (m > 0.0) klast = i;
    }
    const double incl = warp_incl_scan_d(local, lane);
    double excl = __shfl_up_sync(FULL, incl, 1);
    if (lane == 0) excl = 0.0;
    Z = __shfl_sync(FULL, incl, 31);
    const unsigned massive = __ballot_sync(FULL, local > 0.0);
    if (!massive) return -1;
    const double K = 4294967296.0 / Z;
    const int Llast = 31 - __clz(massive);
    const unsigned long long endc = lane == Llast ? XP_TOP : xp_cell(incl, K);
    const unsigned before = massive & ((1u << lane) - 1u);
    const unsigned long long prev_end = __shfl_sync(FULL, endc, before ? 31 - __clz(before) : 0);
    unsigned long long lo = before ? prev_end : 0ull;
    int pick = -1;
    unsigned long long mylo = 0, myhi = 0;
    double mye = 1.0;
    double S = excl;
    for (int i = b; i < en; ++i) {
        const double m = ev(i);
        if (m > 0.0) {
            unsigned long long hi;
            if (i == klast) {
                hi = endc;
            } else {
                S += m;
                hi = xp_cell(S, K);
            }
            if (pick < 0 && hi > tcell) { pick = i; mylo = lo; myhi = hi; mye = m; }
            lo = hi;
        }
    }
    const unsigned bal = __ballot_sync(FULL, pick >= 0);
    if (!bal) return -1;
    const int L = __ffs(bal) - 1;
    pidx = __shfl_sync(FULL, pick, L);
    plo = __shfl_sync(FULL, mylo, L);
    phi = __shfl_sync(FULL, myhi, L);
    pe = __shfl_sync(FULL, mye, L);
    return L;
}

// Result of one decode step for one lane, identical in every thread of the CTA.
struct LaneResult {
    int token;
    int status;
    int n_kept;
    double code_out;
    double p_tok;
    double cdf_lo;
};

}  // namespace asx

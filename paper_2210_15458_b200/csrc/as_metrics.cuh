// What is computed from a group of N decoded sequences: the n-gram diversity score of
// Sec. 5.1 and the sample-mean estimator of Sec. 4.2.  Integer and reduction work on
// sequences that are already on the device, one CTA per group.
#pragma once
#include "as_common.cuh"

namespace asx {

constexpr int NG_NT = 512;
constexpr int NG_MAX_ITEMS = 16384;      // N * T of one group: tokens and hash slots share 227 KB

__device__ __forceinline__ uint32_t ng_hash(const int* s, int n) {
    uint32_t h = 0x9E3779B9u;
    for (int k = 0; k < n; ++k) {
        h = (h ^ (uint32_t)s[k]) * 0x85EBCA6Bu;
        h ^= h >> 13;
    }
    h *= 0xC2B2AE35u;
    return h ^ (h >> 16);
}

// d = sum_{n=1..4} unique_n / total_n per group (Sec. 5.1, "Diverse beam generation").
// The group's tokens sit in shared memory; the distinct n-grams are counted with an
// open-addressing table whose slots hold the position (lane * T + t, plus one) of the first
// n-gram that claimed them, so that equality is decided on the tokens themselves: the count is
// exact, and it does not depend on which thread wins a slot.  Every probe loop is bounded by
// the table size, which is at least twice the number of n-grams.
__global__ void __launch_bounds__(NG_NT)
ngram_diversity_kernel(const int* __restrict__ seq, const int* __restrict__ len, int S, int N, int T, int cap,
                       long long* __restrict__ unique, long long* __restrict__ total, double* __restrict__ div) {
    extern __shared__ int ng_smem[];
    const int items = N * T;
    int* toks = ng_smem;                 // [items]
    int* lens = toks + items;            // [N]
    int* table = lens + N;               // [cap], cap a power of two
    __shared__ int cnt[2];
    const int tid = threadIdx.x, lane = tid & 31;
    const int mask = cap - 1;
    for (int g = blockIdx.x; g < S; g += gridDim.x) {
        __syncthreads();
        for (int i = tid; i < N; i += NG_NT) lens[i] = min(max(len[(size_t)g * N + i], 0), T);
        for (int i = tid; i < items; i += NG_NT) toks[i] = seq[(size_t)g * items + i];
        double dsum = 0.0;
        for (int n = 1; n <= 4; ++n) {
            __syncthreads();
            for (int i = tid; i < cap; i += NG_NT) table[i] = 0;
            if (tid < 2) cnt[tid] = 0;
            __syncthreads();
            int uniq = 0, tot = 0;
            for (int item = tid; item < items; item += NG_NT) {
                const int i = item / T, t = item - i * T;
                if (t + n > lens[i]) continue;
                ++tot;
                const int* me = toks + item;
                uint32_t h = ng_hash(me, n) & mask;
                for (int probe = 0; probe < cap; ++probe) {
                    int cur = *(volatile int*)&table[h];
                    if (cur == 0) {
                        cur = atomicCAS(&table[h], 0, item + 1);
                        if (cur == 0) { ++uniq; break; }
                    }
                    const int* other = toks + (cur - 1);
                    bool eq = true;
                    for (int k = 0; k < n; ++k) eq = eq && (other[k] == me[k]);
                    if (eq) break;
                    h = (h + 1) & mask;
                }
            }
            uniq = warp_sum_i(uniq);
            tot = warp_sum_i(tot);
            if (lane == 0) { atomicAdd(&cnt[0], uniq); atomicAdd(&cnt[1], tot); }
            __syncthreads();
            if (tid == 0) {
                const int u = cnt[0], m = cnt[1];
                unique[(size_t)g * 4 + n - 1] = u;
                total[(size_t)g * 4 + n - 1] = m;
                if (m > 0) dsum += (double)u / (double)m;
            }
        }
        if (tid == 0) div[g] = dsum;
    }
}

// (1/N) sum_i s(x_i) with s(x) = sum_{t < len} r[x_t] per group of N lanes (Sec. 4.2, the
// proposition on the estimator's unbiasedness and consistency).  One warp per lane at a time;
// the group's mean is summed in lane order by one thread, so the result does not depend on timing.
constexpr int RM_NT = 256;
__global__ void __launch_bounds__(RM_NT)
reward_mean_kernel(const int* __restrict__ seq, const int* __restrict__ len, int S, int N, int T,
                   const double* __restrict__ r, int V, double* __restrict__ lane_reward,
                   double* __restrict__ mean, int* __restrict__ group_status) {
    extern __shared__ double rm_s[];          // [N]
    __shared__ int bad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int g = blockIdx.x; g < S; g += gridDim.x) {
        __syncthreads();
        if (tid == 0) bad = 0;
        __syncthreads();
        for (int i = warp; i < N; i += RM_NT / 32) {
            const size_t ln = (size_t)g * N + i;
            const int L = min(max(len[ln], 0), T);
            double s = 0.0;
            int b = 0;
            for (int t = lane; t < L; t += 32) {
                const int tok = seq[ln * T + t];
                if (tok < 0 || tok >= V) b = 1;
                else s += r[tok];
            }
            s = warp_sum_d(s);
            b = warp_sum_i(b);
            if (lane == 0) {
                rm_s[i] = s;
                if (lane_reward) lane_reward[ln] = s;
                if (b) bad = 1;
            }
        }
        __syncthreads();
        if (tid == 0) {
            double acc = 0.0, comp = 0.0;           // compensated, in lane order
            for (int i = 0; i < N; ++i) {
                const double x = rm_s[i], t2 = acc + x;
                comp += (fabs(acc) >= fabs(x)) ? (acc - t2) + x : (x - t2) + acc;
                acc = t2;
            }
            mean[g] = (acc + comp) / (double)N;
            if (group_status) group_status[g] = bad ? -1 : 0;   // AS_ERR_INVALID_ARG : AS_OK
        }
    }
}

}  // namespace asx

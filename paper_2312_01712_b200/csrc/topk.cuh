// Block-level streaming top-k over 64-bit keys (distance bits in the high word, id or index in
// the low word).  Distances are non-negative fp32 (or +inf), so the unsigned order of the keys
// is the lexicographic (distance, id) order the search returns (paper Sec. 2.1: the query "sorts
// the results and selects the top-k"; ties by ascending id is this library's rule).
//
// Protocol, all threads of the CTA taking part:
//   topk_init(...)                                   once
//   repeat: every thread calls topk_push for at most one... R candidates in total per round,
//           then topk_round_end(..., R) which compacts when the next round could overflow
//   topk_finalize(...)                               sorted keys in buf[0..min(cnt,k))
#pragma once

#include <stdint.h>

#include "common.cuh"

namespace ivfpq {

constexpr unsigned long long kKeyPad = 0x7F800000FFFFFFFFull;  // (+inf, id -1): sorts after every real key

struct TopkState {
    unsigned long long* buf;  // [kTopkCap] shared memory
    int* cnt;                 // shared
    unsigned long long* tau;  // shared: a candidate is kept only if key < *tau
};

__device__ __forceinline__ unsigned long long make_key(float dist, uint32_t low) {
    return ((unsigned long long)__float_as_uint(dist) << 32) | (unsigned long long)low;
}

__device__ __forceinline__ void topk_init(const TopkState& t) {
    if (threadIdx.x == 0) {
        *t.cnt = 0;
        *t.tau = kKeyPad;
    }
    __syncthreads();
}

// Returns false when the buffer was full (caller raises the overflow flag; cannot happen when
// the round protocol is respected).
__device__ __forceinline__ bool topk_push(const TopkState& t, unsigned long long key) {
    int pos = atomicAdd(t.cnt, 1);
    if (pos < kTopkCap) {
        t.buf[pos] = key;
        return true;
    }
    return false;
}

// Ascending bitonic sort of buf[0..n2), n2 a power of two.
__device__ inline void bitonic_sort(unsigned long long* buf, int n2) {
    for (int size = 2; size <= n2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int i = threadIdx.x; i < (n2 >> 1); i += blockDim.x) {
                int lo = 2 * i - (i & (stride - 1));
                int hi = lo + stride;
                bool asc = (lo & size) == 0;
                unsigned long long a = buf[lo], b = buf[hi];
                if ((a > b) == asc) {
                    buf[lo] = b;
                    buf[hi] = a;
                }
            }
        }
    }
    __syncthreads();
}

// Sort what is buffered, keep the k best, tighten the threshold.
__device__ inline void topk_compact(const TopkState& t, int k) {
    __syncthreads();
    int n = min(*t.cnt, kTopkCap);
    int n2 = 2;
    while (n2 < n) n2 <<= 1;
    for (int i = n + threadIdx.x; i < n2; i += blockDim.x) t.buf[i] = ~0ull;
    bitonic_sort(t.buf, n2);
    if (threadIdx.x == 0) {
        *t.cnt = min(n, k);
        if (n >= k) *t.tau = t.buf[k - 1];
    }
    __syncthreads();
}

// Call after a round in which at most `round_items` pushes happened CTA-wide; `next_items` is the
// upper bound for the next round.
__device__ __forceinline__ void topk_round_end(const TopkState& t, int k, int next_items) {
    __syncthreads();
    const int c = *t.cnt;
    __syncthreads();  // nobody may push again before every thread has read the same count
    if (c + next_items > kTopkCap) topk_compact(t, k);
}

__device__ __forceinline__ void topk_finalize(const TopkState& t, int k) { topk_compact(t, k); }

}  // namespace ivfpq

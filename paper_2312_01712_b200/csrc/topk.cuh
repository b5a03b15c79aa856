// Block-level streaming top-k over 64-bit keys (distance bits in the high word, id or index in
// the low word).  Distances are non-negative fp32 (or +inf), so the unsigned order of the keys
// is the lexicographic (distance, id) order the search returns (paper Sec. 2.1: the query "sorts
// the results and selects the top-k"; ties by ascending id is this library's rule).
//
// Candidates whose key is below the current threshold are appended to a shared-memory buffer.
// When the buffer fills up, topk_select keeps the k smallest keys with a most-significant-digit
// radix selection (8-bit digits, shared-memory histogram) and tightens the threshold; nothing is
// sorted until topk_finalize, which orders only the k survivors.
#pragma once

#include <stdint.h>

#include "common.cuh"

namespace ivfpq {

constexpr unsigned long long kKeyPad = 0x7F800000FFFFFFFFull;  // (+inf, id -1): sorts after every real key
constexpr int kTopkHistInts = 264;                             // 256 bins + 3 result words, padded

struct TopkState {
    unsigned long long* buf;  // [kTopkCap] shared memory
    int* cnt;                 // shared
    unsigned long long* tau;  // shared: a candidate is kept only if key < *tau
    int* hist;                // [kTopkHistInts] shared
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

// Returns false when the buffer was full (the caller raises the overflow flag; cannot happen
// when the fill protocol of the caller is respected).
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

// Keeps the k smallest keys of the buffer (unordered) and sets the threshold to an exclusive
// upper bound of the kept keys.  No-op when at most k keys are buffered.  NT = threads per CTA.
template <int NT>
__device__ inline void topk_select(const TopkState& t, int k) {
    constexpr int kPerThread = (kTopkCap + NT - 1) / NT;
    __syncthreads();
    const int n = min(*t.cnt, kTopkCap);
    if (n <= k) return;  // uniform over the CTA
    const int tid = threadIdx.x;
    unsigned long long prefix = 0;  // high digits of the k-th smallest key found so far
    int need = k;                   // rank of the wanted key among the keys that share the prefix
    int shift = 56;
    for (;; shift -= 8) {
        for (int i = tid; i < 256; i += NT) t.hist[i] = 0;
        __syncthreads();
        for (int i0 = 0; i0 < n; i0 += NT) {  // whole warps iterate together (warp-aggregated counting)
            const int i = i0 + tid;
            int digit = -1;
            if (i < n) {
                const unsigned long long key = t.buf[i];
                if (shift == 56 || (key >> (shift + 8)) == (prefix >> (shift + 8)))
                    digit = (int)((key >> shift) & 255ull);
            }
            const unsigned peers = __match_any_sync(0xFFFFFFFFu, digit);
            if (digit >= 0 && (tid & 31) == __ffs(peers) - 1) atomicAdd(&t.hist[digit], __popc(peers));
        }
        __syncthreads();
        if (tid < 32) {  // first warp: locate the bin that holds rank `need`
            int local[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                local[j] = t.hist[tid * 8 + j];
                sum += local[j];
            }
            int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (tid >= o) incl += v;
            }
            int excl = incl - sum;
            if (excl < need && need <= incl) {
                int below = excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (below < need && need <= below + local[j]) {
                        t.hist[256] = tid * 8 + j;
                        t.hist[257] = below;
                        t.hist[258] = local[j];
                    }
                    below += local[j];
                }
            }
        }
        __syncthreads();
        const int digit = t.hist[256], below = t.hist[257], inbin = t.hist[258];
        prefix |= (unsigned long long)digit << shift;
        need -= below;
        if (inbin == need || shift == 0) break;  // every key of this bin is kept
        // the next pass clears bins 0..255 only after this barrier-separated read of 256..258
    }
    const unsigned long long bound = ((prefix >> shift) + 1ull) << shift;  // exclusive; no real key has top byte 0xFF
    unsigned long long mine[kPerThread];
    bool keep[kPerThread];
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        const int i = tid + j * NT;
        mine[j] = i < n ? t.buf[i] : ~0ull;
        keep[j] = mine[j] < bound;
    }
    __syncthreads();
    if (tid == 0) {
        *t.cnt = 0;
        *t.tau = bound;
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kPerThread; ++j)
        if (keep[j]) t.buf[atomicAdd(t.cnt, 1)] = mine[j];
    __syncthreads();
}

// Final ordering: the k smallest keys, ascending, in buf[0..min(cnt, k)).
template <int NT>
__device__ inline void topk_finalize(const TopkState& t, int k) {
    topk_select<NT>(t, k);
    __syncthreads();
    const int n = min(*t.cnt, kTopkCap);
    int n2 = 2;
    while (n2 < n) n2 <<= 1;
    for (int i = n + threadIdx.x; i < n2; i += NT) t.buf[i] = ~0ull;
    bitonic_sort(t.buf, n2);
    if (threadIdx.x == 0 && n > k) *t.cnt = k;
    __syncthreads();
}

// End of a round in which at most `next_items` further pushes can happen CTA-wide before the
// next call: selects when the buffer could overflow.
template <int NT>
__device__ __forceinline__ void topk_round_end(const TopkState& t, int k, int next_items) {
    __syncthreads();
    const int c = *t.cnt;
    __syncthreads();  // nobody may push again before every thread has read the same count
    if (c + next_items > kTopkCap) topk_select<NT>(t, k);
}

}  // namespace ivfpq

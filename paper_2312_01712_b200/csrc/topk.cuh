// Block-level streaming top-k over 64-bit keys (distance bits in the high word, id or index in
// the low word).  Distances are non-negative fp32 (or +inf), so the unsigned order of the keys
// is the lexicographic (distance, id) order the search returns (the final ranking of all visited
// points, paper Sec. 2.1, last paragraph; ties by ascending id is this library's rule).
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

// Which threads cooperate in a selection: the whole CTA by default; a kernel whose warps have
// different roles passes a policy with its own thread numbering and named barrier.
struct CtaGroup {
    __device__ __forceinline__ static int tid() { return threadIdx.x; }
    __device__ __forceinline__ static void sync() { __syncthreads(); }
};

// Keys of values that may be negative (the inner-product path ranks by -similarity): an
// order-preserving map of every fp32 to uint32 takes the place of the raw bits; -0 counts as +0.
constexpr unsigned long long kKeyPadSigned = 0xFF800000FFFFFFFFull;  // ordered_bits(+inf), id -1
__device__ __forceinline__ uint32_t ordered_bits(float v) {
    const uint32_t u = __float_as_uint(__fadd_rn(v, 0.0f));
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o);
}

struct TopkState {
    unsigned long long* buf;  // [kTopkCap] shared memory
    int* cnt;                 // shared
    unsigned long long* tau;  // shared: a candidate is kept only if key < *tau
    int* hist;                // [kTopkHistInts] shared
    unsigned long long pad = kKeyPad;  // the key that sorts after every real key (kKeyPadSigned for ordered_bits keys)
};

__device__ __forceinline__ unsigned long long make_key(float dist, uint32_t low) {
    return ((unsigned long long)__float_as_uint(dist) << 32) | (unsigned long long)low;
}

__device__ __forceinline__ void topk_init(const TopkState& t) {
    if (threadIdx.x == 0) {
        *t.cnt = 0;
        *t.tau = t.pad;
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
template <int NT, class G = CtaGroup, int CAP = kTopkCap>
__device__ inline void topk_select(const TopkState& t, int k) {
    constexpr int kPerThread = (CAP + NT - 1) / NT;
    G::sync();
    const int n = min(*t.cnt, CAP);
    if (n <= k) return;  // uniform over the CTA
    const int tid = G::tid();
    unsigned long long prefix = 0;  // high digits of the k-th smallest key found so far
    int need = k;                   // rank of the wanted key among the keys that share the prefix
    int shift = 56;
    for (;; shift -= 8) {
        for (int i = tid; i < 256; i += NT) t.hist[i] = 0;
        G::sync();
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
        G::sync();
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
        G::sync();
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
    G::sync();
    if (tid == 0) {
        *t.cnt = 0;
        *t.tau = bound;
    }
    G::sync();
#pragma unroll
    for (int j = 0; j < kPerThread; ++j)
        if (keep[j]) t.buf[atomicAdd(t.cnt, 1)] = mine[j];
    G::sync();
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

// ---------------------------------------------------------------------------------------------
// Quick compaction and ranked output (used by the persistent scan kernels).
//
// Between two compactions any valid threshold will do, so the buffer is not reduced to exactly
// k keys: one histogram pass over the distance bits (kQuickBins bins spread evenly between the
// smallest and the largest buffered distance) finds the first bin boundary below which at least
// k keys lie; those keys are kept and the boundary becomes the threshold.  Only the final answer
// is exact: the few survivors are ranked by counting, for each key, the keys below it, and
// written straight to their output slots.
//
// `qs` is an int array of kQuickWords words of shared memory that is all zero between calls
// except qs[kQuickBins] (running minimum, kept at 0xFFFFFFFF): topk_quick_init sets this up.
// NT = threads of the group G (at least kQuickBins, whole warps).
// ---------------------------------------------------------------------------------------------
constexpr int kQuickBins = 256;
constexpr int kQuickWords = kQuickBins + 40;  // + min, max, result (2), warp sums (up to 32)

template <int NT, class G = CtaGroup>
__device__ __forceinline__ void topk_quick_init(int* qs) {
    for (int i = G::tid(); i < kQuickWords; i += NT) qs[i] = (i == kQuickBins) ? -1 : 0;
    G::sync();
}

// Keeps the keys below a bin boundary chosen so that at least k survive; sets the threshold to
// that boundary.  No-op when at most k keys are buffered.  With REFINE, while more than `keep_max`
// keys would survive because the boundary bin is crowded (distances bunched together, as the banded
// distances of the sparsity-aware search are, or many keys sharing one distance), that bin is split
// again: by finer distance bits, then by the low word of the key.
// Falls back to the exact selection when the histogram cannot separate the distances (e.g. all
// equal).  Must be called by all threads of the group; contains barriers.
template <int NT, class G = CtaGroup, int CAP = kTopkCap, bool REFINE = false>
__device__ inline void topk_quick_compact(const TopkState& t, int k, int* qs, int keep_max = 0) {
    constexpr int kPerThread = (CAP + NT - 1) / NT;
    constexpr int B = kQuickBins;
    static_assert(NT >= B && NT % 32 == 0, "one bin per thread of the first B threads");
    G::sync();
    const int n = min(*t.cnt, CAP);
    if (n <= k) return;  // uniform over the group
    const int tid = G::tid();
    unsigned* uq = reinterpret_cast<unsigned*>(qs);
    unsigned long long mine[kPerThread];
    unsigned lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        const int i = tid + j * NT;
        mine[j] = i < n ? t.buf[i] : ~0ull;
        if (i < n) {
            const unsigned h = (unsigned)(mine[j] >> 32);
            lo = min(lo, h);
            hi = max(hi, h);
        }
    }
    lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    hi = __reduce_max_sync(0xFFFFFFFFu, hi);
    if ((tid & 31) == 0) {
        atomicMin(&uq[B], lo);
        atomicMax(&uq[B + 1], hi);
    }
    G::sync();
    lo = uq[B];
    hi = uq[B + 1];
    const unsigned range = hi - lo;
    int shift = 0;  // smallest shift with (range >> shift) < B
    if (range >= (unsigned)B) shift = (32 - __clz(range)) - (31 - __clz(B));

    // One histogram pass over the keys that `binof` maps to a bin in [0, B): returns the bin that
    // holds the key of rank `need` among them, the inclusive count up to that bin and the bin's own
    // count.  Leaves the shared words in their between-calls state again.
    int bin = 0, incl_total = 0, bin_count = 0;
    auto hist_pass = [&](auto binof, int need) {
#pragma unroll
        for (int j = 0; j < kPerThread; ++j) {
            const int i = tid + j * NT;
            const int b = i < n ? binof(mine[j]) : -1;
            if (b >= 0) atomicAdd(&qs[b], 1);
        }
        G::sync();
        const int v = tid < B ? qs[tid] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if ((tid & 31) >= o) incl += x;
        }
        if (tid < B && (tid & 31) == 31) qs[B + 4 + (tid >> 5)] = incl;
        if (tid == 0) qs[B + 2] = -1;
        G::sync();
        if (tid < B) {
            int before = 0;
            for (int w = 0; w < (tid >> 5); ++w) before += qs[B + 4 + w];
            incl += before;
            if (incl - v < need && need <= incl) {  // exactly one thread: its bin holds the wanted rank
                qs[B + 2] = tid;
                qs[B + 3] = incl;
                qs[B + 36] = v;
            }
        }
        G::sync();
        bin = qs[B + 2];
        incl_total = qs[B + 3];
        bin_count = qs[B + 36];
        G::sync();  // everybody has read the result and the warp sums
        if (tid < B) qs[tid] = 0;
        if (tid < kQuickWords - B) qs[B + tid] = (tid == 0) ? -1 : 0;
        G::sync();
    };
    // bins of the distance bits: (distance - base) >> sh, when that is below B
    auto dist_bin = [&](unsigned base, int sh) {
        return [=](unsigned long long key) {
            const unsigned h = (unsigned)(key >> 32);
            if (h < base) return -1;
            const unsigned b = (h - base) >> sh;
            return b < (unsigned)B ? (int)b : -1;
        };
    };

    hist_pass(dist_bin(lo, shift), k);
    int below = incl_total - bin_count;   // keys in the bins before the boundary bin
    unsigned base = lo;                   // first distance of the boundary bin is base + (bin << sh)
    int sh = shift;
    // exclusive bound on the keys that stay
    unsigned long long bound = ((unsigned long long)base + ((unsigned long long)(bin + 1) << sh)) << 32;
    bool ok = bin >= 0;
    if (REFINE) {
        // narrow the distance bits while the boundary bin is crowded
        for (int level = 0; level < 3 && ok && below + bin_count > keep_max && sh > 0; ++level) {
            base += (unsigned)bin << sh;
            sh = sh > 8 ? sh - 8 : 0;
            hist_pass(dist_bin(base, sh), k - below);
            ok = bin >= 0;
            below += incl_total - bin_count;
            bound = ((unsigned long long)base + ((unsigned long long)(bin + 1) << sh)) << 32;
        }
        if (ok && below + bin_count > keep_max && bin_count > 1 && sh == 0) {
            // many keys share one distance (base + bin): split that group by the low word (the id)
            const unsigned tie = base + (unsigned)bin;
            unsigned ilo = 0xFFFFFFFFu, ihi = 0u;
#pragma unroll
            for (int j = 0; j < kPerThread; ++j) {
                const int i = tid + j * NT;
                if (i < n && (unsigned)(mine[j] >> 32) == tie) {
                    ilo = min(ilo, (unsigned)mine[j]);
                    ihi = max(ihi, (unsigned)mine[j]);
                }
            }
            ilo = __reduce_min_sync(0xFFFFFFFFu, ilo);
            ihi = __reduce_max_sync(0xFFFFFFFFu, ihi);
            if ((tid & 31) == 0) {
                atomicMin(&uq[B], ilo);
                atomicMax(&uq[B + 1], ihi);
            }
            G::sync();
            ilo = uq[B];
            ihi = uq[B + 1];
            G::sync();
            if (tid == 0) {
                uq[B] = 0xFFFFFFFFu;
                uq[B + 1] = 0u;
            }
            const unsigned irange = ihi - ilo;
            int ish = 0;
            if (irange >= (unsigned)B) ish = (32 - __clz(irange)) - (31 - __clz(B));
            G::sync();
            hist_pass([=](unsigned long long key) {
                return (unsigned)(key >> 32) == tie ? (int)(((unsigned)key - ilo) >> ish) : -1;
            }, k - below);
            ok = bin >= 0;
            below += incl_total - bin_count;
            const unsigned long long next_id = (unsigned long long)ilo + ((unsigned long long)(bin + 1) << ish);
            bound = next_id > 0xFFFFFFFFull ? ((unsigned long long)tie + 1ull) << 32 : ((unsigned long long)tie << 32) | next_id;
        }
    }
    const int kept = below + bin_count;
    if (!ok || kept >= n) {  // uniform: nothing would be dropped
        topk_select<NT, G, CAP>(t, k);  // uses the same shared words as its histogram
        topk_quick_init<NT, G>(qs);
        return;
    }
    if (tid == 0) {
        *t.cnt = 0;
        *t.tau = bound < t.pad ? bound : t.pad;
    }
    G::sync();
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
        const bool keep = mine[j] < bound;  // the filler ~0 never passes
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, keep);
        if (bal != 0) {
            int base = 0;
            if ((tid & 31) == 0) base = atomicAdd(t.cnt, __popc(bal));
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            if (keep) t.buf[base + __popc(bal & ((1u << (tid & 31)) - 1u))] = mine[j];
        }
    }
    G::sync();
}

// Rank of every buffered key among the n buffered keys (n <= kTopkCap), by counting; calls
// emit(rank, key) for the keys of rank < k.  Equal keys are ordered by buffer position, so ranks
// are distinct.  All threads of the group must call it; the buffer must be complete (barrier
// before).
template <int NT, class G = CtaGroup, class Emit>
__device__ __forceinline__ void topk_emit_ranked(const TopkState& t, int n, int k, Emit emit) {
    const int tid = G::tid();
    if (n * 2 <= NT) {
        // S consecutive lanes share a key and split the comparisons
        int S = 2;
        while (S < 32 && n * (S * 2) <= NT) S *= 2;
        const int i = tid / S, part = tid & (S - 1);
        int rank = 0;
        const unsigned long long me = i < n ? t.buf[i] : 0ull;
        if (i < n)
            for (int j = part; j < n; j += S) {
                const unsigned long long o = t.buf[j];
                rank += (o < me || (o == me && j < i)) ? 1 : 0;
            }
        for (int o = 1; o < S; o <<= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
        if (i < n && part == 0 && rank < k) emit(rank, me);
    } else {
        for (int i = tid; i < n; i += NT) {
            const unsigned long long me = t.buf[i];
            int rank = 0;
            for (int j = 0; j < n; ++j) {
                const unsigned long long o = t.buf[j];
                rank += (o < me || (o == me && j < i)) ? 1 : 0;
            }
            if (rank < k) emit(rank, me);
        }
    }
}

}  // namespace ivfpq

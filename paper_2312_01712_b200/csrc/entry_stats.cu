// Entry usage and locality statistics of the neighbours of a query (paper Sec. 3.2 "Sparsity of
// Codebook Entries Used by Top-k Neighbors", Sec. 3.3 "Spatial Locality of Codebook Entries Used by
// Top-k Neighbors"): per (query, subspace) the number of distinct codebook entries its neighbours
// are encoded with, and a histogram of how close those entries are to the query's residual
// projection (rank 0 = the closest entry).  An analysis tool for calibrating radii, not a step of
// the search.
//
// One CTA per query, one warp per (neighbour, subspace) pair at a time: the lanes split the
// codebook's entries, evaluate the squared distance with the search's arithmetic and count the
// entries ordered before the neighbour's own entry ((distance, entry number) ascending); lane 0
// adds one to the global histogram.  Used entries are marked in a shared bit set and counted at
// the end.  The codebook comes through L2 (at most 64 KB per subspace).
#include "common.cuh"

namespace ivfpq {

namespace {

constexpr int kStatThreads = 256;

__global__ void __launch_bounds__(kStatThreads) entry_stats_kernel(
    const float* __restrict__ cent, const float* __restrict__ cb, const int64_t* __restrict__ list_off,
    const uint8_t* __restrict__ codes, const float* __restrict__ queries, const int64_t* __restrict__ nbr, int d,
    int nlist, int nsub, int dsub, int ksub, int k, int64_t ntotal, int32_t* __restrict__ usage,
    unsigned long long* __restrict__ rank_hist, int* __restrict__ status) {
    __shared__ uint32_t used[IVFPQ_MAX_NSUB * 8];
    __shared__ int list_of[IVFPQ_MAX_K];   // the list of every neighbour, -1 = skip
    const int64_t q = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < nsub * 8; i += kStatThreads) used[i] = 0;
    for (int j = tid; j < k; j += kStatThreads) {
        const int64_t x = nbr[q * k + j];
        int c = -1;
        if (x >= ntotal) {
            atomicOr(status, kFlagBadList);
        } else if (x >= 0) {
            int lo = 0, hi = nlist;   // the last list whose offset is <= x
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (list_off[mid] <= x) lo = mid; else hi = mid;
            }
            c = lo;
        }
        list_of[j] = c;
    }
    __syncthreads();
    const float* qv = queries + q * d;
    for (int w = warp; w < k * nsub; w += kStatThreads / 32) {
        const int j = w / nsub, s = w - j * nsub;
        const int c = list_of[j];
        if (c < 0) continue;   // uniform over the warp
        const int64_t x = nbr[q * k + j];
        const int own = codes[x * nsub + s];
        if (own >= ksub) {
            if (lane == 0) atomicOr(status, kFlagBadList);
            continue;
        }
        const float* qs = qv + s * dsub;
        const float* cs = cent + (int64_t)c * d + s * dsub;
        const float* es = cb + (int64_t)s * ksub * dsub;
        auto dist_to = [&](int e) {
            float d2 = 0.0f;
            for (int t = 0; t < dsub; ++t) {
                const float u = __fsub_rn(__fsub_rn(qs[t], cs[t]), __ldg(es + (int64_t)e * dsub + t));
                d2 = __fmaf_rn(u, u, d2);
            }
            return d2;
        };
        const float mine = dist_to(own);
        int before = 0;
        for (int e = lane; e < ksub; e += 32) {
            const float v = dist_to(e);
            before += (v < mine || (v == mine && e < own)) ? 1 : 0;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, o);
        if (lane == 0) {
            atomicAdd(rank_hist + (int64_t)s * ksub + before, 1ull);
            atomicOr(&used[s * 8 + (own >> 5)], 1u << (own & 31));
        }
    }
    __syncthreads();
    for (int s = tid; s < nsub; s += kStatThreads) {
        int n = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) n += __popc(used[s * 8 + i]);
        usage[q * nsub + s] = n;
    }
}

}  // namespace

cudaError_t launch_entry_stats(const ivfpq_index* ix, const uint8_t* codes, const float* queries, int64_t nq,
                               const int64_t* nbr, int k, int32_t* usage, unsigned long long* rank_hist, int* status,
                               cudaStream_t st) {
    entry_stats_kernel<<<(unsigned)nq, kStatThreads, 0, st>>>(ix->cent, ix->cb, ix->list_off, codes, queries, nbr, ix->d,
                                                              ix->nlist, ix->nsub, ix->dsub, ix->ksub, k, ix->ntotal,
                                                              usage, rank_hist, status);
    return cudaGetLastError();
}

}  // namespace ivfpq

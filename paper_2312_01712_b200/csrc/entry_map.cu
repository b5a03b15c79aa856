// Load-time construction of the inverted index from codebook entries to search points (paper
// Sec. 5.1, Algorithm 1, the `Map` output: for every cluster, subspace and entry, the points of
// that cluster whose projection in that subspace is encoded with that entry).  The sparsity-aware
// list scan (scan16x8_map.cu) walks it to visit only the points behind selected entries
// (Sec. 5.3, paragraph after Algorithm 2).
//
// Layout.  Every inverted list is cut into chunks of at most kMapChunk points (the per-point
// accumulators of one chunk fit the scan kernel's shared memory); positions are chunk-local and
// fit 16 bits.  For the chunk whose first point has the global index g0 (index into the
// list-contiguous id array) and which holds n points:
//   map_pos[16 * g0 + s * n + first + i], i in [0, count), with
//   first | count << 16 = map_off[(chunk * 16 + s) * 256 + e]
// are the positions (0 .. n-1, in no particular order) of the points whose code in subspace s is e.
// chunk_first[list] is the number of chunks before the list's first one.
#include "common.cuh"

namespace ivfpq {

namespace {

// One CTA per (list, subspace); it walks the list's chunks.
__global__ void __launch_bounds__(256) entry_map_kernel(const uint8_t* __restrict__ codes,
                                                        const int64_t* __restrict__ list_off,
                                                        const int32_t* __restrict__ chunk_first, int nsub,
                                                        uint32_t* __restrict__ map_off, uint16_t* __restrict__ map_pos) {
    __shared__ int hist[256];
    __shared__ int cursor[256];
    __shared__ int wsum[8];
    const int list = blockIdx.x;
    const int s = blockIdx.y;
    const int tid = threadIdx.x;
    const int64_t p0 = list_off[list];
    const int64_t len = list_off[list + 1] - p0;
    const int nch = (int)((len + kMapChunk - 1) / kMapChunk);
    for (int ch = 0; ch < nch; ++ch) {
        const int64_t g0 = p0 + (int64_t)ch * kMapChunk;
        const int n = (int)(len - (int64_t)ch * kMapChunk < kMapChunk ? len - (int64_t)ch * kMapChunk : kMapChunk);
        hist[tid] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += 256) atomicAdd(&hist[codes[(g0 + i) * nsub + s]], 1);
        __syncthreads();
        // exclusive prefix sum over the 256 bins
        const int v = hist[tid];
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if ((tid & 31) >= o) incl += x;
        }
        if ((tid & 31) == 31) wsum[tid >> 5] = incl;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < (tid >> 5); ++w) before += wsum[w];
        const int excl = before + incl - v;
        cursor[tid] = excl;
        map_off[((size_t)(chunk_first[list] + ch) * nsub + s) * 256 + tid] = (uint32_t)excl | ((uint32_t)v << 16);
        __syncthreads();
        uint16_t* dst = map_pos + (size_t)g0 * nsub + (size_t)s * n;
        for (int i = tid; i < n; i += 256) dst[atomicAdd(&cursor[codes[(g0 + i) * nsub + s]], 1)] = (uint16_t)i;
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_entry_map(const ivfpq_index* ix, const uint8_t* codes, cudaStream_t st) {
    if (!ix->map_pos || ix->ntotal == 0) return cudaSuccess;
    entry_map_kernel<<<dim3((unsigned)ix->nlist, (unsigned)ix->nsub), 256, 0, st>>>(
        codes, ix->list_off, ix->chunk_first, ix->nsub, const_cast<uint32_t*>(ix->map_off),
        const_cast<uint16_t*>(ix->map_pos));
    return cudaGetLastError();
}

}  // namespace ivfpq

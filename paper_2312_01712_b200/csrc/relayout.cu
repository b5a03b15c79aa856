// Load-time re-layout of the PQ codes into the device layout the list scan streams.
//
// Source: codes[ntotal][nsub] bytes, list-contiguous (the conventional IVFPQ encoding, paper
// Sec. 2.1 "Product Quantization", step 4).  Destination: every inverted list is padded to whole
// blocks of 32 points; inside a block the code bytes are stored as 4-byte words, word-major
// across the 32 points, so that the 32 lanes of a warp (one point per lane) read consecutive
// addresses:
//   vec16 == 0:  word w of point `lane` in block b  ->  codes_il[(b*nw + w)*32 + lane]
//   vec16 == 1:  (nw multiple of 4) words are grouped by four so that a lane fetches 16 bytes:
//                codes_il[((b*(nw/4) + w/4)*32 + lane)*4 + (w & 3)]
// Byte s & 3 of word s >> 2 is the code of subspace s; bytes of padding subspaces and of padding
// points are 0.
#include "common.cuh"

namespace ivfpq {

namespace {

__global__ void __launch_bounds__(256) relayout_kernel(const uint8_t* __restrict__ codes,
                                                       const int64_t* __restrict__ list_off,
                                                       const int64_t* __restrict__ list_blk, int nsub, int nw,
                                                       int vec16, uint32_t* __restrict__ codes_il) {
    const int list = blockIdx.x;
    const int64_t p0 = list_off[list];
    const int64_t len = list_off[list + 1] - p0;
    const int64_t b0 = list_blk[list];
    const int64_t nblk = list_blk[list + 1] - b0;
    const int64_t nslots = nblk * kPointsPerBlock * nw;
    for (int64_t i = threadIdx.x; i < nslots; i += blockDim.x) {
        // enumerate destination words in storage order of the vec16 == 0 layout
        const int lane = (int)(i % kPointsPerBlock);
        const int w = (int)((i / kPointsPerBlock) % nw);
        const int64_t b = i / ((int64_t)kPointsPerBlock * nw);
        const int64_t pos = b * kPointsPerBlock + lane;
        uint32_t word = 0;
        if (pos < len) {
            const uint8_t* src = codes + (p0 + pos) * nsub;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int s = w * 4 + j;
                if (s < nsub) word |= (uint32_t)src[s] << (8 * j);
            }
        }
        int64_t dst;
        if (vec16)
            dst = (((b0 + b) * (nw >> 2) + (w >> 2)) * kPointsPerBlock + lane) * 4 + (w & 3);
        else
            dst = ((b0 + b) * nw + w) * kPointsPerBlock + lane;
        codes_il[dst] = word;
    }
}

}  // namespace

cudaError_t launch_relayout(const ivfpq_index* ix, const uint8_t* codes, uint32_t* codes_il, cudaStream_t st) {
    if (ix->nlist > 0 && ix->nblocks > 0)
        relayout_kernel<<<ix->nlist, 256, 0, st>>>(codes, ix->list_off, ix->list_blk, ix->nsub, ix->nw,
                                                   ix->vec16, codes_il);
    return cudaGetLastError();
}

}  // namespace ivfpq

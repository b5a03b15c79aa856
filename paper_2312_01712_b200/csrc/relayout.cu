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

__host__ __device__ inline int rot_lane_bytes(int w) { return w >= 16 ? w : (w == 8 ? 8 : (w > 0 ? 4 : 0)); }

// Rotated layout (see scan_rot.cu): a 32-point block is a sequence of per-group chunks; in the
// chunk of a group of width w the lane at position `lane` stores, as byte i (i < w), the code of
// subspace s0 + ((lane ^ i) & (w-1)).  Lanes are interleaved at the granularity of the vector the
// scan loads: 16 bytes (w >= 16), 8 bytes (w == 8) or 4 bytes (w <= 4).
__global__ void __launch_bounds__(256) relayout_rot_kernel(const uint8_t* __restrict__ codes,
                                                           const int64_t* __restrict__ list_off,
                                                           const int64_t* __restrict__ list_blk, int nsub,
                                                           int w0, int w1, int w2, int block_bytes,
                                                           unsigned char* __restrict__ dst) {
    const int list = blockIdx.x;
    const int64_t p0 = list_off[list];
    const int64_t len = list_off[list + 1] - p0;
    const int64_t b0 = list_blk[list];
    const int64_t nblk = list_blk[list + 1] - b0;
    const int gw[3] = {w0, w1, w2};
    for (int64_t i = threadIdx.x; i < nblk * kPointsPerBlock; i += blockDim.x) {
        const int lane = (int)(i & 31);
        const int64_t b = i >> 5;
        const int64_t pos = i;
        const uint8_t* src = codes + (p0 + pos) * nsub;
        unsigned char* blk = dst + (b0 + b) * block_bytes;
        int s0 = 0, chunk = 0;
        for (int g = 0; g < 3; ++g) {
            const int w = gw[g];
            if (w == 0) break;
            const int lb = rot_lane_bytes(w);
            const int vec = lb >= 16 ? 16 : lb;  // bytes per lane per vector
            for (int i2 = 0; i2 < lb; ++i2) {
                unsigned char v = 0;
                if (i2 < w && pos < len) v = src[s0 + ((lane ^ i2) & (w - 1))];
                // vector number i2 / vec, lanes interleaved per vector
                blk[chunk + (i2 / vec) * 32 * vec + lane * vec + (i2 % vec)] = v;
            }
            s0 += w;
            chunk += 32 * lb;
        }
    }
}

// Entry-major codebook copy per group: cbt[s0*256*dsub + ((e*w + c)*dsub + j)] = cb[s0+c][e][j];
// entries e >= ksub are zero.
__global__ void __launch_bounds__(256) relayout_cbt_kernel(const float* __restrict__ cb, int nsub, int dsub,
                                                           int ksub, int w0, int w1, int w2,
                                                           float* __restrict__ cbt) {
    const int gw[3] = {w0, w1, w2};
    const int total = nsub * 256 * dsub;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        int s0 = 0, g = 0;
        while (g < 2 && i >= (s0 + gw[g]) * 256 * dsub) {
            s0 += gw[g];
            ++g;
        }
        const int w = gw[g];
        const int r = i - s0 * 256 * dsub;
        const int j = r % dsub;
        const int c = (r / dsub) % w;
        const int e = r / (dsub * w);
        cbt[i] = e < ksub ? cb[((size_t)(s0 + c) * ksub + e) * dsub + j] : 0.0f;
    }
}

// Smallest id (as an unsigned number) of every 32-point block: a candidate that ties with the
// threshold distance enters only with a smaller id than the threshold's, so a block whose smallest
// id is not below it is decided without reading its ids (Sec. 5.3's scores tie often: hit counts
// are small integers, and every point that missed everywhere has the same value).
__global__ void __launch_bounds__(256) block_min_id_kernel(const int32_t* __restrict__ ids,
                                                           const int64_t* __restrict__ list_off,
                                                           const int64_t* __restrict__ list_blk,
                                                           uint32_t* __restrict__ blk_min) {
    const int list = blockIdx.x;
    const int64_t p0 = list_off[list];
    const int64_t len = list_off[list + 1] - p0;
    const int64_t b0 = list_blk[list];
    const int64_t nblk = list_blk[list + 1] - b0;
    const int lane = threadIdx.x & 31;
    for (int64_t b = threadIdx.x >> 5; b < nblk; b += blockDim.x >> 5) {
        const int64_t pos = b * kPointsPerBlock + lane;
        uint32_t v = pos < len ? (uint32_t)ids[p0 + pos] : 0xFFFFFFFFu;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
        if (lane == 0) blk_min[b0 + b] = v;
    }
}

}  // namespace

cudaError_t launch_block_min_id(const ivfpq_index* ix, uint32_t* blk_min, cudaStream_t st) {
    if (ix->nlist > 0 && ix->nblocks > 0)
        block_min_id_kernel<<<ix->nlist, 256, 0, st>>>(ix->ids, ix->list_off, ix->list_blk, blk_min);
    return cudaGetLastError();
}

cudaError_t launch_relayout(const ivfpq_index* ix, const uint8_t* codes, uint32_t* codes_il, float* cbt,
                            cudaStream_t st) {
    if (ix->rot) {
        if (ix->nblocks > 0)
            relayout_rot_kernel<<<ix->nlist, 256, 0, st>>>(codes, ix->list_off, ix->list_blk, ix->nsub, ix->gw[0],
                                                           ix->gw[1], ix->gw[2], ix->block_bytes,
                                                           reinterpret_cast<unsigned char*>(codes_il));
        relayout_cbt_kernel<<<64, 256, 0, st>>>(ix->cb, ix->nsub, ix->dsub, ix->ksub, ix->gw[0], ix->gw[1],
                                                ix->gw[2], cbt);
    } else if (ix->nlist > 0 && ix->nblocks > 0) {
        relayout_kernel<<<ix->nlist, 256, 0, st>>>(codes, ix->list_off, ix->list_blk, ix->nsub, ix->nw,
                                                   ix->vec16, codes_il);
    }
    return cudaGetLastError();
}

}  // namespace ivfpq

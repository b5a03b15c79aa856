// Dynamic threshold front-end (paper Sec. 4.1 "Determining Proper Threshold"; Algorithm 2:
// thres = poly_regressor(density_map(x, y))).  Every 2-d subspace carries a grid x grid map of
// cell densities; the threshold of a query in a subspace is a polynomial of the density of the cell
// that the query's own projection (before the centroid is subtracted) falls into.  The output is
// the [nq][nsub] radius array that ivfpq_search_sparse takes in mode 1.
//
// (For subspaces of other widths: thresholds_knn_kernel below.)
//
// One thread per (query, subspace): one 8-byte load of the projection, one gather from the density
// map (L2-resident: nsub x grid^2 x 4 bytes), a Horner evaluation.  Memory-trivial: the whole batch
// reads nq x d x 4 bytes and writes nq x nsub x 4 bytes.
#include "common.cuh"

namespace ivfpq {

namespace {

__device__ __forceinline__ int border_clamped_cell(float v, int grid) {
    const float f = floorf(v);
    int c = 0;                                   // NaN and everything below the grid: first cell
    if (f >= (float)grid) c = grid - 1;
    else if (f > 0.0f) c = (int)f;
    return min(c, grid - 1);
}

__global__ void __launch_bounds__(256) thresholds_kernel(const float* __restrict__ queries, int64_t nq, int nsub, int grid,
                                                         int degree, const float* __restrict__ density,
                                                         const float* __restrict__ origin, const float* __restrict__ inv_cell,
                                                         const float* __restrict__ coef, float* __restrict__ radius) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nq * nsub) return;
    const int s = (int)(i % nsub);
    const float2 xy = *reinterpret_cast<const float2*>(queries + 2 * i);   // row q, columns 2 s and 2 s + 1
    const float2 o = *reinterpret_cast<const float2*>(origin + 2 * s);
    const float2 w = *reinterpret_cast<const float2*>(inv_cell + 2 * s);
    const int col = border_clamped_cell(__fmul_rn(__fsub_rn(xy.x, o.x), w.x), grid);
    const int row = border_clamped_cell(__fmul_rn(__fsub_rn(xy.y, o.y), w.y), grid);
    const float dens = __ldg(density + ((size_t)s * grid + row) * grid + col);
    const float* cf = coef + (size_t)s * (degree + 1);
    float acc = __ldg(cf + degree);
    for (int k = degree - 1; k >= 0; --k) acc = __fmaf_rn(acc, dens, __ldg(cf + k));
    radius[i] = acc > 0.0f ? acc : 0.0f;
}

// Thresholds for subspaces of any width: the density around the query's residual projection
// (against its nearest cluster) is measured by the distance to its kth-nearest codebook entry, and
// the per-subspace polynomial is evaluated on that distance (the density map of Sec. 4.1 is a 2-d
// grid and has no counterpart for wider subspaces).  One warp per (query, subspace): lane l holds the
// entries l, l + 32, ...; squared distances by the table arithmetic (fma chain, ascending
// dimension); the kth smallest by a radix selection over the bits of the non-negative floats.
template <int DSUB_T>
__global__ void __launch_bounds__(256) thresholds_knn_kernel(const float* __restrict__ queries, int64_t nq, int d, int nsub,
                                                             int dsub_rt, int ksub, const float* __restrict__ cent,
                                                             const float* __restrict__ cb, const int32_t* __restrict__ probe0,
                                                             int nlist, int kth, int degree, const float* __restrict__ coef,
                                                             float* __restrict__ radius, int* __restrict__ status) {
    const int dsub = DSUB_T > 0 ? DSUB_T : dsub_rt;
    const int lane = threadIdx.x & 31;
    const int64_t w = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (w >= nq * nsub) return;   // whole warps leave together
    const int64_t q = w / nsub;
    const int s = (int)(w % nsub);
    int c = probe0[q];
    if (c < 0 || c >= nlist) {
        if (lane == 0) atomicOr(status, kFlagBadList);
        c = 0;
    }
    const float* qp = queries + q * d + (int64_t)s * dsub;
    const float* cp = cent + (int64_t)c * d + (int64_t)s * dsub;
    uint32_t bits[8];
#pragma unroll
    for (int m = 0; m < 8; ++m) {
        const int e = lane + 32 * m;
        bits[m] = 0xFFFFFFFFu;   // beyond the codebook: after every real value
        if (e < ksub) {
            const float* ent = cb + ((size_t)s * ksub + e) * dsub;
            float a = 0.0f;
            for (int j = 0; j < dsub; ++j) {
                const float r = __fsub_rn(__ldg(qp + j), __ldg(cp + j));
                const float t = __fsub_rn(r, __ldg(ent + j));
                a = __fmaf_rn(t, t, a);
            }
            bits[m] = __float_as_uint(a);
        }
    }
    uint32_t prefix = 0;
    int need = kth;   // rank wanted among the values that share the prefix
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t mask = bit == 31 ? 0u : (0xFFFFFFFFu << (bit + 1));
        int zeros = 0;
#pragma unroll
        for (int m = 0; m < 8; ++m) zeros += ((bits[m] & mask) == prefix && ((bits[m] >> bit) & 1u) == 0u) ? 1 : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zeros += __shfl_xor_sync(0xFFFFFFFFu, zeros, o);
        if (need > zeros) {
            need -= zeros;
            prefix |= 1u << bit;
        }
    }
    if (lane == 0) {
        const float v = __fsqrt_rn(__uint_as_float(prefix));
        const float* cf = coef + (size_t)s * (degree + 1);
        float acc = __ldg(cf + degree);
        for (int k = degree - 1; k >= 0; --k) acc = __fmaf_rn(acc, v, __ldg(cf + k));
        radius[q * nsub + s] = acc > 0.0f ? acc : 0.0f;
    }
}

}  // namespace

cudaError_t launch_thresholds_knn(const ivfpq_index* ix, const float* queries, int64_t nq, const int32_t* probe0, int kth,
                                  int degree, const float* coef, float* radius, int* status, cudaStream_t st) {
    const int64_t warps = nq * ix->nsub;
    const unsigned blocks = (unsigned)((warps + 7) / 8);
#define IVFPQ_KNN_ARGS queries, nq, ix->d, ix->nsub, ix->dsub, ix->ksub, ix->cent, ix->cb, probe0, ix->nlist, kth, degree, coef, radius, status
    if (ix->dsub == 8) thresholds_knn_kernel<8><<<blocks, 256, 0, st>>>(IVFPQ_KNN_ARGS);
    else if (ix->dsub == 4) thresholds_knn_kernel<4><<<blocks, 256, 0, st>>>(IVFPQ_KNN_ARGS);
    else if (ix->dsub == 2) thresholds_knn_kernel<2><<<blocks, 256, 0, st>>>(IVFPQ_KNN_ARGS);
    else thresholds_knn_kernel<0><<<blocks, 256, 0, st>>>(IVFPQ_KNN_ARGS);
#undef IVFPQ_KNN_ARGS
    return cudaGetLastError();
}

cudaError_t launch_thresholds(const float* queries, int64_t nq, int nsub, const ivfpq_threshold_model_t* m,
                              float* radius, cudaStream_t st) {
    const int64_t total = nq * nsub;
    const int64_t blocks = (total + 255) / 256;
    thresholds_kernel<<<(unsigned)blocks, 256, 0, st>>>(queries, nq, nsub, m->grid, m->degree, m->density, m->origin,
                                                         m->inv_cell, m->coef, radius);
    return cudaGetLastError();
}

}  // namespace ivfpq

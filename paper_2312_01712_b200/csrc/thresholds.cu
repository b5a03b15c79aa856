// Dynamic threshold front-end (paper Sec. 4.1 "Determining Proper Threshold"; Algorithm 2:
// thres = poly_regressor(density_map(x, y))).  Every 2-d subspace carries a grid x grid map of
// cell densities; the threshold of a query in a subspace is a polynomial of the density of the cell
// that the query's own projection (before the centroid is subtracted) falls into.  The output is
// the [nq][nsub] radius array that ivfpq_search_sparse takes in mode 1.
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

}  // namespace

cudaError_t launch_thresholds(const float* queries, int64_t nq, int nsub, const ivfpq_threshold_model_t* m,
                              float* radius, cudaStream_t st) {
    const int64_t total = nq * nsub;
    const int64_t blocks = (total + 255) / 256;
    thresholds_kernel<<<(unsigned)blocks, 256, 0, st>>>(queries, nq, nsub, m->grid, m->degree, m->density, m->origin,
                                                         m->inv_cell, m->coef, radius);
    return cudaGetLastError();
}

}  // namespace ivfpq

// Filtering stage (paper Sec. 2.1 "Online Search", step A): squared L2 distance from every
// query to every IVF centroid, then the nprobe closest clusters per query.
//
// The distance is evaluated in the direct form sum_j (q_j - c_j)^2 with one fused multiply-add
// per dimension, j ascending, fp32: the selection must reproduce the defining arithmetic bit for
// bit, and the GEMM form |c|^2 - 2 q.c + |q|^2 that the paper uses on tensor cores (Sec. 4.3,
// last paragraph) rounds differently near the nprobe-th distance.
#include "common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

constexpr int TQ = 64;   // queries per CTA tile
constexpr int TC = 64;   // centroids per CTA tile
constexpr int TK = 16;   // dimensions per shared-memory stage

// out[(q - q0) * nlist + c] = sum_j fma(q_j - c_j, q_j - c_j, acc), for q in [q0, q0 + nqc)
__global__ void __launch_bounds__(256) coarse_dist_kernel(const float* __restrict__ queries, int64_t q0,
                                                          int nqc, const float* __restrict__ cent,
                                                          int nlist, int d, float* __restrict__ out) {
    __shared__ __align__(16) float qs[TK][TQ + 4];
    __shared__ __align__(16) float cs[TK][TC + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15;   // centroid group
    const int ty = tid >> 4;   // query group
    const int cbase = blockIdx.x * TC;
    const int qbase = blockIdx.y * TQ;

    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0f;

    for (int k0 = 0; k0 < d; k0 += TK) {
        __syncthreads();
#pragma unroll
        for (int i = 0; i < (TQ * TK) / 256; ++i) {
            int idx = tid + i * 256;
            int row = idx / TK, kk = idx % TK;
            int j = k0 + kk;
            int q = qbase + row;
            int c = cbase + row;
            qs[kk][row] = (q < nqc && j < d) ? queries[(q0 + q) * (int64_t)d + j] : 0.0f;
            cs[kk][row] = (c < nlist && j < d) ? cent[(int64_t)c * d + j] : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            const float4 qv = *reinterpret_cast<const float4*>(&qs[kk][ty * 4]);
            const float4 cv = *reinterpret_cast<const float4*>(&cs[kk][tx * 4]);
            const float qa[4] = {qv.x, qv.y, qv.z, qv.w};
            const float ca[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    float t = __fsub_rn(qa[a], ca[b]);
                    acc[a][b] = __fmaf_rn(t, t, acc[a][b]);
                }
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        int q = qbase + ty * 4 + a;
        if (q >= nqc) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int c = cbase + tx * 4 + b;
            if (c < nlist) out[(int64_t)q * nlist + c] = acc[a][b];
        }
    }
}

// One CTA per query: the nprobe smallest (distance, cluster id) pairs, ascending.
__global__ void __launch_bounds__(256) select_probes_kernel(const float* __restrict__ dist, int nlist,
                                                            int nprobe, int32_t* __restrict__ probe_ids,
                                                            float* __restrict__ probe_d, int64_t q0,
                                                            int* __restrict__ status) {
    __shared__ unsigned long long buf[kTopkCap];
    __shared__ int cnt;
    __shared__ unsigned long long tau;
    __shared__ int hist[kTopkHistInts];
    TopkState t{buf, &cnt, &tau, hist};
    topk_init(t);
    const float* row = dist + (int64_t)blockIdx.x * nlist;
    for (int base = 0; base < nlist; base += blockDim.x) {
        int c = base + threadIdx.x;
        if (c < nlist) {
            unsigned long long key = make_key(row[c], (uint32_t)c);
            if (key < tau) {
                if (!topk_push(t, key)) atomicOr(status, kFlagOverflow);
            }
        }
        topk_round_end<256>(t, nprobe, 256);
    }
    topk_finalize<256>(t, nprobe);
    const int64_t q = q0 + blockIdx.x;
    for (int i = threadIdx.x; i < nprobe; i += blockDim.x) {
        unsigned long long key = i < cnt ? buf[i] : kKeyPad;
        probe_ids[q * nprobe + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
        probe_d[q * nprobe + i] = __uint_as_float((uint32_t)(key >> 32));
    }
}

}  // namespace

cudaError_t launch_coarse(const ivfpq_index* ix, const float* queries, int64_t nq, int32_t nprobe,
                          float* coarse_tile, int64_t qchunk, int32_t* probe_ids, float* probe_d,
                          int* status, cudaStream_t st, int64_t* launches) {
    for (int64_t q0 = 0; q0 < nq; q0 += qchunk) {
        const int nqc = (int)((nq - q0 < qchunk) ? (nq - q0) : qchunk);
        dim3 grid((ix->nlist + TC - 1) / TC, (nqc + TQ - 1) / TQ);
        coarse_dist_kernel<<<grid, 256, 0, st>>>(queries, q0, nqc, ix->cent, ix->nlist, ix->d, coarse_tile);
        select_probes_kernel<<<nqc, 256, 0, st>>>(coarse_tile, ix->nlist, nprobe, probe_ids, probe_d, q0, status);
        *launches += 2;
    }
    return cudaGetLastError();
}

}  // namespace ivfpq

// Filtering stage (paper Sec. 2.1 "Online Search", step A): squared L2 distance from every
// query to every IVF centroid, then the nprobe closest clusters per query.
//
// The distance is evaluated in the direct form sum_j (q_j - c_j)^2 with one fused multiply-add
// per dimension, j ascending, fp32: the selection must reproduce the defining arithmetic bit for
// bit, and the GEMM form |c|^2 - 2 q.c + |q|^2 that the paper uses on tensor cores (Sec. 5.3,
// last paragraph) rounds differently near the nprobe-th distance.
#include <mutex>

#include "common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

constexpr int TQ = 64;   // queries per CTA tile
constexpr int TC = 64;   // centroids per CTA tile
constexpr int TK = 16;   // dimensions per shared-memory stage

// out[(q - q0) * nlist + c] = sum_j fma(q_j - c_j, q_j - c_j, acc), for q in [q0, q0 + nqc).
// IP (paper Sec. 4.2 "Inner Product Similarity Support": filtering by inner product): the tile holds
// -(sum_j fma(q_j, c_j, acc)), so that "smallest first" selects the largest inner products.
template <bool IP>
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
                    if (IP) {
                        acc[a][b] = __fmaf_rn(qa[a], ca[b], acc[a][b]);
                    } else {
                        float t = __fsub_rn(qa[a], ca[b]);
                        acc[a][b] = __fmaf_rn(t, t, acc[a][b]);
                    }
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
            if (c < nlist) out[(int64_t)q * nlist + c] = IP ? -acc[a][b] : acc[a][b];
        }
    }
}

// One CTA per query: the nprobe smallest (distance, cluster id) pairs, ascending.  SIGNED: the
// values may be negative (negated inner products) and the keys use the order-preserving bit map.
template <bool SIGNED>
__global__ void __launch_bounds__(256) select_probes_kernel(const float* __restrict__ dist, int nlist,
                                                            int nprobe, int32_t* __restrict__ probe_ids,
                                                            float* __restrict__ probe_d, int64_t q0,
                                                            int* __restrict__ status) {
    __shared__ unsigned long long buf[kTopkCap];
    __shared__ int cnt;
    __shared__ unsigned long long tau;
    __shared__ int hist[kTopkHistInts];
    TopkState t{buf, &cnt, &tau, hist, SIGNED ? kKeyPadSigned : kKeyPad};
    topk_init(t);
    const float* row = dist + (int64_t)blockIdx.x * nlist;
    for (int base = 0; base < nlist; base += blockDim.x) {
        int c = base + threadIdx.x;
        if (c < nlist) {
            unsigned long long key = SIGNED ? ((unsigned long long)ordered_bits(row[c]) << 32) | (uint32_t)c
                                            : make_key(row[c], (uint32_t)c);
            if (key < tau) {
                if (!topk_push(t, key)) atomicOr(status, kFlagOverflow);
            }
        }
        topk_round_end<256>(t, nprobe, 256);
    }
    topk_finalize<256>(t, nprobe);
    const int64_t q = q0 + blockIdx.x;
    for (int i = threadIdx.x; i < nprobe; i += blockDim.x) {
        unsigned long long key = i < cnt ? buf[i] : t.pad;
        probe_ids[q * nprobe + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
        probe_d[q * nprobe + i] = SIGNED ? from_ordered_bits((uint32_t)(key >> 32)) : __uint_as_float((uint32_t)(key >> 32));
    }
}

}  // namespace

namespace {
__global__ void negate_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = -in[i];
}
}  // namespace

// out[i] = -in[i]: the filtering stage of the inner-product path keeps -(q.c); callers see q.c.
cudaError_t launch_negate(const float* in, float* out, int64_t n, cudaStream_t st) {
    negate_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(in, out, n);
    return cudaGetLastError();
}

cudaError_t launch_coarse(const ivfpq_index* ix, const float* queries, int64_t nq, int32_t nprobe,
                          float* coarse_tile, int64_t qchunk, int32_t* probe_ids, float* probe_d,
                          int* status, cudaStream_t st, int64_t* launches) {
    // tensor-core proposal + exact decision when the shape allows it (16-byte aligned rows)
    const bool ip = ix->metric == IVFPQ_METRIC_IP;
    const bool mma_shape = ix->cnorm != nullptr && (reinterpret_cast<uintptr_t>(queries) & 15) == 0 &&
                           (reinterpret_cast<uintptr_t>(ix->cent) & 15) == 0;
    const int64_t qchunk_row = qchunk;   // queries whose full rows fit the scratch region (the plain kernels need those)
    const size_t region = coarse_region_bytes(ix, qchunk);   // bytes of scratch the caller provides
    bool mma = mma_shape, fused = false;
    // L2: the proposal works on centred operands; the centred queries of a chunk take d floats each at
    // the front of the same region (no centring when not even one query fits that way)
    const size_t qc_bytes = (mma && ix->cent_c) ? (size_t)ix->d * 4 : 0;
    bool centred = qc_bytes != 0;
    if (mma) {
        if (coarse_mma_fused(ix->nlist, nprobe) && !ix->test_fault) {
            // the fused path needs another amount of scratch per query than a full row: its own chunking of the same region
            int64_t fit = (int64_t)((region > 256 ? region - 256 : 0) / (coarse_mma_fused_bytes_per_query(ix->nlist, nprobe) + qc_bytes));   // 256: alignment of the second part
            if (fit >= 1) {
                if (fit >= 128) fit -= fit % 128;   // whole query tiles of the tensor-core kernel
                qchunk = fit < nq ? fit : nq;   // more queries per chunk than full rows would allow, or fewer
                fused = true;
            }
        }
        if (!fused && centred) {
            // (full rows and centred queries of `qchunk` queries fit by the region's definition)
        }
    }
    for (int64_t q0 = 0; q0 < nq; q0 += qchunk) {
        int nqc = (int)((nq - q0 < qchunk) ? (nq - q0) : qchunk);
        if (mma) {
            // [centred queries of the chunk][tile rows, or the fused path's scratch]: both 256-byte aligned
            float* q_centred = centred ? coarse_tile : nullptr;
            float* tile = centred ? reinterpret_cast<float*>(reinterpret_cast<char*>(coarse_tile) + align_up((size_t)qchunk * qc_bytes, 256)) : coarse_tile;
            const cudaError_t e = launch_coarse_mma(ix, queries, q0, nqc, nprobe, fused, q_centred, tile, probe_ids, probe_d, status, st, launches);
            if (e == cudaSuccess) continue;
            if (e != cudaErrorNotSupported) return e;
            mma = false;   // the tensor maps could not be built: the plain kernels, in chunks of full rows
            qchunk = qchunk_row;
            nqc = (int)((nq - q0 < qchunk) ? (nq - q0) : qchunk);
        }
        dim3 grid((ix->nlist + TC - 1) / TC, (nqc + TQ - 1) / TQ);
        if (ip) {
            coarse_dist_kernel<true><<<grid, 256, 0, st>>>(queries, q0, nqc, ix->cent, ix->nlist, ix->d, coarse_tile);
            select_probes_kernel<true><<<nqc, 256, 0, st>>>(coarse_tile, ix->nlist, nprobe, probe_ids, probe_d, q0, status);
        } else {
            coarse_dist_kernel<false><<<grid, 256, 0, st>>>(queries, q0, nqc, ix->cent, ix->nlist, ix->d, coarse_tile);
            select_probes_kernel<false><<<nqc, 256, 0, st>>>(coarse_tile, ix->nlist, nprobe, probe_ids, probe_d, q0, status);
        }
        *launches += 2;
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Filtering stage without any caller-provided or allocated scratch (ivfpq_probe_static).
//
// The [queries][nlist] distance tile that coarse_dist_kernel writes and select_probes_kernel reads
// lives in a fixed array inside the library image.  Every GPU that loads the library carries these
// bytes until the process exits; all calls on a device share them.
// ---------------------------------------------------------------------------------------------
namespace {

// first 256 bytes: device status word (cleared by every call); the rest: the distance tile
static __device__ __align__(256) unsigned char g_static_scratch[IVFPQ_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can
// use: the device address has to be asked for, once per device, with that device current.
int static_scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= kMaxDevices) return IVFPQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[device]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return IVFPQ_ERR_CUDA;
        g_static_ptr[device] = p;
    }
    *out = static_cast<unsigned char*>(g_static_ptr[device]);
    return IVFPQ_OK;
}

}  // namespace

}  // namespace ivfpq

extern "C" int ivfpq_probe_static(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                                  int32_t* probe_ids, float* probe_d, void* stream) {
    if (!index || !queries || !probe_ids || !probe_d) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (nq <= 0 || nprobe <= 0) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (nprobe > index->nlist || nprobe > IVFPQ_MAX_NPROBE || nq > (int64_t)1 << 24) return IVFPQ_ERR_UNSUPPORTED;
    if (index->metric != IVFPQ_METRIC_L2) return IVFPQ_ERR_UNSUPPORTED;
    if (index->nlist > IVFPQ_STATIC_MAX_NLIST) return IVFPQ_ERR_STATIC_LIMIT;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (dev != index->device) return IVFPQ_ERR_INVALID_ARGUMENT;  // the index lives on another GPU
    unsigned char* scratch = nullptr;
    const int rc = ivfpq::static_scratch_address(dev, &scratch);
    if (rc != IVFPQ_OK) return rc;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    // the status word must start at zero; the tile is fully rewritten before it is read
    if (cudaMemsetAsync(scratch, 0, 256, st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    // status word, then the filtering stage's region for chunks of qchunk queries (coarse_region_bytes)
    int64_t qchunk = ((int64_t)IVFPQ_STATIC_SCRATCH_BYTES - 512) / ((int64_t)index->nlist * 4 + (int64_t)index->d * 4);
    if (qchunk > nq) qchunk = nq;
    int64_t launches = 0;
    if (ivfpq::launch_coarse(index, queries, nq, nprobe, reinterpret_cast<float*>(scratch + 256), qchunk,
                             probe_ids, probe_d, reinterpret_cast<int*>(scratch), st, &launches) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    return IVFPQ_OK;
}

extern "C" int ivfpq_static_status(void* stream) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return IVFPQ_ERR_CUDA;
    unsigned char* scratch = nullptr;
    const int rc = ivfpq::static_scratch_address(dev, &scratch);
    if (rc != IVFPQ_OK) return rc;
    int flags = 0;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&flags, scratch, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    return flags != 0 ? IVFPQ_ERR_DEVICE_FLAG : IVFPQ_OK;
}

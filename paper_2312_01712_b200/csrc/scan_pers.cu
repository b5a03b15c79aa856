// Persistent variant of the fused selective-LUT / list-scan / top-k kernel for the 16 x 8
// product quantizer (16 subspaces of 8 dimensions, 256 entries), the shape of the SIFT-like
// workloads.  Same computation as scan.cu / scan_rot.cu (paper Sec. 2.1 steps B-D with the
// selection of Sec. 3.1 / Algorithm 2 and the miss constant of Sec. 4.3) and the same
// conflict-free rotated table layout as scan_rot.cu, organised for one resident CTA per SM:
//
//   * the whole codebook (128 KB) lives in the CTA's registers for the lifetime of the kernel:
//     thread t owns column c = t & 15 (one subspace) and the entries u, u + NT/16, ... with
//     u = t / 16, so building a table reads nothing but the probed centroid (512 B);
//   * the CTA loops over (query, probe-slice) work items; per probed cluster it builds the table
//     from registers, then all warps stream the cluster's code blocks (next block prefetched);
//   * candidates go to the CTA's streaming top-k; a warp checks a soft fill limit before every
//     block and the CTA compacts only when that limit was hit, so a cluster costs two barriers.
#include "common.cuh"
#include "scan_common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

constexpr int kW = 16;           // group width = number of subspaces
constexpr int kDsub = 8;
constexpr int kSoftLimit = 1536; // compaction is requested once this many candidates are buffered

__host__ __device__ inline size_t pers_smem_bytes(int nprobe, bool dbg) {
    size_t b = (size_t)kTopkCap * 8;   // candidate keys
    b += 256 * 32 * 4;                 // table: 256 entries x 32 columns
    b += IVFPQ_MAX_NSUB * 4;           // squared thresholds
    b += 32 + kTopkHistInts * 4;       // counters, selection histogram
    if (dbg) b += IVFPQ_MAX_NSUB * 8 * 4 + (size_t)(nprobe + 1) * 8;
    return b;
}

template <int NT, bool DBG>
__global__ void __launch_bounds__(NT, 1) scan_pers16x8_kernel(const ScanParams p, const int64_t nitems) {
    constexpr int EP = NT / kW;     // entries per pass
    constexpr int NE = 256 / EP;    // entries per thread
    constexpr int kWarps = NT / 32;
    static_assert(kSoftLimit + NT <= kTopkCap && IVFPQ_MAX_K < kSoftLimit, "candidate buffer limits");
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(smem);
    float* lut = reinterpret_cast<float*>(smem + (size_t)kTopkCap * 8);
    float* r2 = lut + 256 * 32;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(r2 + IVFPQ_MAX_NSUB);
    int* cnt_p = reinterpret_cast<int*>(tau_p + 1);
    int* hist_p = reinterpret_cast<int*>(tau_p + 4);
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(hist_p + kTopkHistInts);           // DBG only
    long long* vprefix = reinterpret_cast<long long*>(hitmask + IVFPQ_MAX_NSUB * 8);   // DBG only

    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int c = tid & (kW - 1);
    const int u = tid / kW;
    const int usub = lane / kW;
    const int ksub = p.ksub;
    const int d = kW * kDsub;
    TopkState t{kbuf, cnt_p, tau_p, hist_p};

    // codebook slice of this thread: entries u + EP*m of subspace c
    float cbr[NE][kDsub];
#pragma unroll
    for (int m = 0; m < NE; ++m) {
        const int e = u + EP * m;
        const float4* src = reinterpret_cast<const float4*>(p.cbt + ((size_t)e * kW + c) * kDsub);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        cbr[m][0] = a.x; cbr[m][1] = a.y; cbr[m][2] = a.z; cbr[m][3] = a.w;
        cbr[m][4] = b.x; cbr[m][5] = b.y; cbr[m][6] = b.z; cbr[m][7] = b.w;
    }

    for (int64_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int64_t q = item / p.nsplit;
        const int split = (int)(item % p.nsplit);
        __syncthreads();  // the previous item's results have been read out of the candidate buffer
        if (tid < kW) {
            float v = 0.0f;
            if (!p.dense) {
                const float* rad = p.radius_mode == 1 ? p.radius + q * kW : p.radius;
                const float r = __fmul_rn(rad[tid], p.scale);
                v = __fmul_rn(r, r);
            }
            r2[tid] = v;
        }
        if (DBG && tid == 0) {
            long long run = 0;
            for (int i = 0; i < p.nprobe; ++i) {
                vprefix[i] = run;
                const int cl = p.probe_ids[q * p.nprobe + i];
                if (cl >= 0 && cl < p.nlist) run += p.list_off[cl + 1] - p.list_off[cl];
            }
            vprefix[p.nprobe] = run;
            if (p.visit_count) p.visit_count[q] = run;
        }
        topk_init(t);  // contains a barrier
        float P = 0.0f;
        if (!p.dense) {
            if (p.miss_penalty >= 0.0f) {
                P = p.miss_penalty;
            } else {
#pragma unroll
                for (int s = 0; s < kW; ++s) P = __fadd_rn(P, r2[s]);
            }
        }
        const float thr = r2[c];
        float qv[kDsub];
        {
            const float4* src = reinterpret_cast<const float4*>(p.queries + q * d + c * kDsub);
            const float4 a = __ldg(src), b = __ldg(src + 1);
            qv[0] = a.x; qv[1] = a.y; qv[2] = a.z; qv[3] = a.w;
            qv[4] = b.x; qv[5] = b.y; qv[6] = b.z; qv[7] = b.w;
        }

        for (int pi = split; pi < p.nprobe; pi += p.nsplit) {
            const int cl = p.probe_ids[q * p.nprobe + pi];
            if (cl < 0 || cl >= p.nlist) {  // uniform over the CTA
                if (tid == 0) atomicOr(p.status, kFlagBadList);
                continue;
            }
            // residual of this thread's subspace (paper step B), kept in registers
            float r[kDsub];
            {
                const float4* src = reinterpret_cast<const float4*>(p.cent + (int64_t)cl * d + c * kDsub);
                const float4 a = __ldg(src), b = __ldg(src + 1);
                r[0] = __fsub_rn(qv[0], a.x); r[1] = __fsub_rn(qv[1], a.y);
                r[2] = __fsub_rn(qv[2], a.z); r[3] = __fsub_rn(qv[3], a.w);
                r[4] = __fsub_rn(qv[4], b.x); r[5] = __fsub_rn(qv[5], b.y);
                r[6] = __fsub_rn(qv[6], b.z); r[7] = __fsub_rn(qv[7], b.w);
            }
            if (DBG) {
                __syncthreads();
                for (int i = tid; i < IVFPQ_MAX_NSUB * 8; i += NT) hitmask[i] = 0;
                __syncthreads();
            }
            // ---- selective table from the register-resident codebook (steps C + selection) ----
#pragma unroll
            for (int m = 0; m < NE; ++m) {
                const int e = u + EP * m;
                float d2 = 0.0f;
#pragma unroll
                for (int j = 0; j < kDsub; ++j) {
                    const float tt = __fsub_rn(r[j], cbr[m][j]);
                    d2 = __fmaf_rn(tt, tt, d2);
                }
                const bool hit = e < ksub && (p.dense || d2 <= thr);
                const float val = hit ? d2 : P;
                float* row = lut + e * 32 + c;
                row[(usub & 1) * kW] = val;          // the two half-warps write different columns
                row[((usub + 1) & 1) * kW] = val;
                if (DBG && hit) atomicOr(&hitmask[c * 8 + (e >> 5)], 1u << (e & 31));
            }
            __syncthreads();
            if (DBG && p.masks)
                for (int i = tid; i < kW * 8; i += NT) p.masks[(q * p.nprobe + pi) * kW * 8 + i] = hitmask[i];

            // ---- scan the cluster (step D) ----
            const int64_t p0 = p.list_off[cl];
            const int64_t len = p.list_off[cl + 1] - p0;
            const int64_t b0 = p.list_blk[cl];
            const int64_t nblk = p.list_blk[cl + 1] - b0;
            const bool list_ok = (nblk == (len + kPointsPerBlock - 1) / kPointsPerBlock) && len >= 0;
            if (!list_ok && tid == 0) atomicOr(p.status, kFlagBadList);
            const uint4* cp = reinterpret_cast<const uint4*>(p.codes_il) + b0 * 32 + lane;
            int64_t blk = list_ok ? warp : nblk;
            uint4 next = make_uint4(0, 0, 0, 0);
            if (blk < nblk) next = __ldg(cp + blk * 32);
            while (true) {
                const unsigned long long tau = *tau_p;
                const uint32_t tau_hi = (uint32_t)(tau >> 32);
                while (blk < nblk) {
                    if (*reinterpret_cast<volatile int*>(cnt_p) >= kSoftLimit) break;
                    const uint4 cur = next;
                    if (blk + kWarps < nblk) next = __ldg(cp + (blk + kWarps) * 32);
                    const uint32_t wv[4] = {cur.x, cur.y, cur.z, cur.w};
                    float acc0 = 0.0f, acc1 = 0.0f;
                    unsigned long long hs = 0;
#pragma unroll
                    for (int i = 0; i < kW; ++i) {
                        const uint32_t code = (wv[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                        const float v = lut[code * 32 + (lane ^ i)];
                        if (i & 1) acc1 += v; else acc0 += v;
                        if (DBG) {
                            const int s = (lane ^ i) & (kW - 1);
                            hs |= (unsigned long long)((hitmask[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
                        }
                    }
                    const float acc = acc0 + acc1;
                    const int64_t pos = blk * kPointsPerBlock + lane;
                    if (pos < len) {
                        if (DBG) {
                            const int64_t vi = vprefix[pi] + pos;
                            if (vi < p.visit_stride) {
                                if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                                if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = acc;
                                if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[p0 + pos];
                            }
                        }
                        if (__float_as_uint(acc) <= tau_hi) {
                            const unsigned long long key = make_key(acc, (uint32_t)p.ids[p0 + pos]);
                            if (key < tau) {
                                if (!topk_push(t, key)) atomicOr(p.status, kFlagOverflow);
                            }
                        }
                    }
                    blk += kWarps;
                }
                // also the barrier that protects the table from the next cluster's build
                if (!__syncthreads_or(blk < nblk)) break;
                topk_select<NT>(t, p.k);
            }
        }

        topk_finalize<NT>(t, p.k);
        const int n = *cnt_p;
        if (p.nsplit == 1) {
            for (int i = tid; i < p.k; i += NT) {
                const unsigned long long key = i < n ? kbuf[i] : kKeyPad;
                p.out_dist[q * p.k + i] = __uint_as_float((uint32_t)(key >> 32));
                p.out_ids[q * p.k + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
            }
        } else {
            unsigned long long* dst = p.partial + (q * p.nsplit + split) * p.k;
            for (int i = tid; i < p.k; i += NT) dst[i] = i < n ? kbuf[i] : kKeyPad;
        }
    }
}

}  // namespace

cudaError_t launch_scan_pers(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                             cudaStream_t st) {
    constexpr int NT = 512;
    const size_t smem = pers_smem_bytes(nprobe, debug);
    int64_t grid = ix->sm_count;
    if (grid > nitems) grid = nitems;
    cudaError_t e;
    if (debug) {
        auto kern = scan_pers16x8_kernel<NT, true>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)grid, NT, smem, st>>>(sp, nitems);
    } else {
        auto kern = scan_pers16x8_kernel<NT, false>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)grid, NT, smem, st>>>(sp, nitems);
    }
    return cudaGetLastError();
}

}  // namespace ivfpq

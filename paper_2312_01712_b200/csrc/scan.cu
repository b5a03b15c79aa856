// Selective L2-LUT construction fused with the list scan and the per-query top-k, plus the
// merge of partial results.
//
// One CTA serves one query (or one slice of a query's probe list).  For every probed cluster it
//   1. forms the residual query - centroid (paper Sec. 2.1 "Online Search", step B);
//   2. builds the look-up table in shared memory: thread e computes, per subspace, the squared
//      distance between the residual projection and codebook entry e (step C) and keeps it only
//      when it is within the squared threshold of that subspace (the selection of Sec. 4.1 /
//      Algorithm 2, whose ray test decides exactly "distance <= thres * thres_scale");
//      an unselected slot holds the miss constant P, so that the scan needs no branch for the
//      large constant that points with an unselected entry receive (Sec. 5.3);
//   3. streams the cluster's codes (32-point interleaved blocks, one point per lane) and sums
//      one table value per subspace (step D);
//   4. feeds (distance, id) into a CTA-wide streaming top-k.
// The table is never written to global memory.
#include <math.h>

#include "common.cuh"
#include "scan_common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

constexpr int kBlocksPerWarpRound = 4;                                            // 32-point blocks per warp per round
constexpr int kRoundPoints = kScanThreads * kBlocksPerWarpRound;                  // candidates per round, CTA-wide
static_assert(IVFPQ_MAX_K + kRoundPoints <= kTopkCap, "candidate buffer too small for a round");

__host__ __device__ inline size_t scan_smem_bytes(int nw, int d, int nprobe, bool dbg) {
    size_t b = (size_t)kTopkCap * 8;              // candidate keys
    b += (size_t)nw * 4 * 256 * 4;                // table, padded subspaces included
    b += align_up((size_t)d * 4, 16);             // residual
    b += IVFPQ_MAX_NSUB * 4;                      // squared thresholds
    b += 32 + kTopkHistInts * 4;                  // counters, selection histogram
    if (dbg) b += IVFPQ_MAX_NSUB * 8 * 4 + (size_t)(nprobe + 1) * 8;
    return b;
}

// Adds the four table values selected by the code bytes of one word (subspaces s0..s0+3).
template <bool DBG>
__device__ __forceinline__ void accum_word(uint32_t wv, int s0, const float* lut, const uint32_t* hitmask,
                                           int nsub, float& acc, unsigned long long& hs) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int s = s0 + b;
        const uint32_t code = (wv >> (8 * b)) & 0xFFu;
        acc += lut[s * 256 + code];
        if (DBG && s < nsub)
            hs |= (unsigned long long)((hitmask[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
    }
}

template <int NW_T, int DSUB_T, bool VEC16, bool DBG>
__global__ void __launch_bounds__(kScanThreads) scan_kernel(const ScanParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int nw = NW_T ? NW_T : p.nw;
    const int dsub = DSUB_T ? DSUB_T : p.dsub;
    const int nsub = p.nsub;
    const int ksub = p.ksub;
    const int d = p.d;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;

    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(smem);
    float* lut = reinterpret_cast<float*>(smem + (size_t)kTopkCap * 8);
    float* res = lut + (size_t)nw * 4 * 256;
    float* r2 = res + align_up((size_t)d * 4, 16) / 4;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(r2 + IVFPQ_MAX_NSUB);
    int* cnt_p = reinterpret_cast<int*>(tau_p + 1);
    int* hist_p = reinterpret_cast<int*>(tau_p + 4);
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(hist_p + kTopkHistInts);  // DBG only
    long long* vprefix = reinterpret_cast<long long*>(hitmask + IVFPQ_MAX_NSUB * 8);  // DBG only

    const int64_t q = blockIdx.x / p.nsplit;
    const int split = blockIdx.x % p.nsplit;
    TopkState t{kbuf, cnt_p, tau_p, hist_p};

    // squared thresholds of this query, one per subspace; the miss constant
    if (tid < nsub) {
        float v = 0.0f;
        if (!p.dense) {
            const float* rad = p.radius_mode == 1 ? p.radius + q * nsub : p.radius;
            float r = __fmul_rn(rad[tid], p.scale);
            v = __fmul_rn(r, r);
        }
        r2[tid] = v;
    }
    if (DBG && tid == 0) {
        long long run = 0;
        for (int i = 0; i < p.nprobe; ++i) {
            vprefix[i] = run;
            int c = p.probe_ids[q * p.nprobe + i];
            if (c >= 0 && c < p.nlist) run += p.list_off[c + 1] - p.list_off[c];
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
            for (int s = 0; s < nsub; ++s) P = __fadd_rn(P, r2[s]);
        }
    }

    for (int pi = split; pi < p.nprobe; pi += p.nsplit) {
        const int c = p.probe_ids[q * p.nprobe + pi];
        if (c < 0 || c >= p.nlist) {  // uniform over the CTA
            if (tid == 0) atomicOr(p.status, kFlagBadList);
            continue;
        }
        __syncthreads();  // the previous cluster's scan no longer reads the table
        for (int j = tid; j < d; j += kScanThreads)
            res[j] = __fsub_rn(p.queries[q * d + j], p.cent[(int64_t)c * d + j]);
        for (int i = nsub * 256 + tid; i < nw * 4 * 256; i += kScanThreads) lut[i] = 0.0f;
        __syncthreads();

        // ---- selective table: thread e owns entry e of every subspace ----
        for (int s = 0; s < nsub; ++s) {
            float d2 = 0.0f;
            if (tid < ksub) {
                const float* ent = p.cb + ((int64_t)s * ksub + tid) * dsub;
                const float* rs = res + s * dsub;
                if (DSUB_T != 0 && DSUB_T % 4 == 0) {
#pragma unroll
                    for (int j4 = 0; j4 < (DSUB_T ? DSUB_T : 4) / 4; ++j4) {
                        const float4 ev = __ldg(reinterpret_cast<const float4*>(ent) + j4);
                        float tt;
                        tt = __fsub_rn(rs[4 * j4 + 0], ev.x); d2 = __fmaf_rn(tt, tt, d2);
                        tt = __fsub_rn(rs[4 * j4 + 1], ev.y); d2 = __fmaf_rn(tt, tt, d2);
                        tt = __fsub_rn(rs[4 * j4 + 2], ev.z); d2 = __fmaf_rn(tt, tt, d2);
                        tt = __fsub_rn(rs[4 * j4 + 3], ev.w); d2 = __fmaf_rn(tt, tt, d2);
                    }
                } else if (DSUB_T == 2) {
                    const float2 ev = __ldg(reinterpret_cast<const float2*>(ent));
                    float tt;
                    tt = __fsub_rn(rs[0], ev.x); d2 = __fmaf_rn(tt, tt, d2);
                    tt = __fsub_rn(rs[1], ev.y); d2 = __fmaf_rn(tt, tt, d2);
                } else {
                    for (int j = 0; j < dsub; ++j) {
                        float tt = __fsub_rn(rs[j], __ldg(ent + j));
                        d2 = __fmaf_rn(tt, tt, d2);
                    }
                }
            }
            const bool hit = tid < ksub && (p.dense || d2 <= r2[s]);
            lut[s * 256 + tid] = table_value(p.score, hit, d2, r2[s], P);
            if (DBG) {
                unsigned m = __ballot_sync(0xFFFFFFFFu, hit);
                if (lane == 0) {
                    hitmask[s * 8 + warp] = m;
                    if (p.masks) p.masks[((q * p.nprobe + pi) * nsub + s) * 8 + warp] = m;
                }
            }
        }
        __syncthreads();

        // ---- scan the cluster ----
        const int64_t p0 = p.list_off[c];
        const int64_t len = p.list_off[c + 1] - p0;
        const int64_t b0 = p.list_blk[c];
        const int64_t nblk = p.list_blk[c + 1] - b0;
        if (nblk != (len + kPointsPerBlock - 1) / kPointsPerBlock || len < 0) {
            if (tid == 0) atomicOr(p.status, kFlagBadList);
            continue;
        }
        for (int64_t bb = 0; bb < nblk; bb += (kScanThreads / 32) * kBlocksPerWarpRound) {
            const unsigned long long tau = *tau_p;
            const uint32_t tau_hi = (uint32_t)(tau >> 32);
#pragma unroll 1
            for (int r = 0; r < kBlocksPerWarpRound; ++r) {
                const int64_t blk = bb + r * (kScanThreads / 32) + warp;
                if (blk >= nblk) break;
                float acc = 0.0f;
                unsigned long long hs = 0;
                if constexpr (VEC16) {
                    const int G = nw >> 2;
                    const uint4* cp = reinterpret_cast<const uint4*>(p.codes_il) + (b0 + blk) * G * 32 + lane;
                    if constexpr (NW_T != 0) {
#pragma unroll
                        for (int g = 0; g < NW_T / 4; ++g) {
                            const uint4 v = __ldg(cp + g * 32);
                            accum_word<DBG>(v.x, g * 16 + 0, lut, hitmask, nsub, acc, hs);
                            accum_word<DBG>(v.y, g * 16 + 4, lut, hitmask, nsub, acc, hs);
                            accum_word<DBG>(v.z, g * 16 + 8, lut, hitmask, nsub, acc, hs);
                            accum_word<DBG>(v.w, g * 16 + 12, lut, hitmask, nsub, acc, hs);
                        }
                    } else {
                        for (int g = 0; g < G; ++g) {
                            const uint4 v = __ldg(cp + g * 32);
                            accum_word<DBG>(v.x, g * 16 + 0, lut, hitmask, nsub, acc, hs);
                            accum_word<DBG>(v.y, g * 16 + 4, lut, hitmask, nsub, acc, hs);
                            accum_word<DBG>(v.z, g * 16 + 8, lut, hitmask, nsub, acc, hs);
                            accum_word<DBG>(v.w, g * 16 + 12, lut, hitmask, nsub, acc, hs);
                        }
                    }
                } else {
                    const uint32_t* cp = p.codes_il + (b0 + blk) * nw * 32 + lane;
                    if constexpr (NW_T != 0) {
#pragma unroll
                        for (int w = 0; w < NW_T; ++w)
                            accum_word<DBG>(__ldg(cp + w * 32), w * 4, lut, hitmask, nsub, acc, hs);
                    } else {
                        for (int w = 0; w < nw; ++w)
                            accum_word<DBG>(__ldg(cp + w * 32), w * 4, lut, hitmask, nsub, acc, hs);
                    }
                }
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
            }
            topk_round_end<kScanThreads>(t, p.k, kRoundPoints);
        }
    }

    topk_finalize<kScanThreads>(t, p.k);
    const int n = *cnt_p;
    if (p.nsplit == 1) {
        for (int i = tid; i < p.k; i += kScanThreads) {
            const unsigned long long key = i < n ? kbuf[i] : kKeyPad;
            p.out_dist[q * p.k + i] = __uint_as_float((uint32_t)(key >> 32));
            p.out_ids[q * p.k + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
        }
    } else {
        unsigned long long* dst = p.partial + (q * p.nsplit + split) * p.k;
        for (int i = tid; i < p.k; i += kScanThreads) dst[i] = i < n ? kbuf[i] : kKeyPad;
    }
}

// Inner-product similarity (paper Sec. 4.2 "Inner Product Similarity Support") for any code shape.
// Internally a point is ranked by the cost -(similarity), so that the streaming top-k, which keeps
// the smallest keys, applies unchanged; keys use the order-preserving bit map because costs can be
// negative.  One table per query serves all its probed clusters: slot (s, e) holds -(q_s.e) when
// entry e is selected (|q_s - e|^2 <= R_s^2 + |e|^2) and the miss constant P otherwise; a point's
// cost is -(q.c) from the filtering stage plus one slot per subspace.
template <bool DBG>
__global__ void __launch_bounds__(kScanThreads) scan_ip_kernel(const ScanParams p) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int nw = p.nw, dsub = p.dsub, nsub = p.nsub, ksub = p.ksub, d = p.d;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;

    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(smem);
    float* lut = reinterpret_cast<float*>(smem + (size_t)kTopkCap * 8);
    float* qv = lut + (size_t)nw * 4 * 256;
    float* r2 = qv + align_up((size_t)d * 4, 16) / 4;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(r2 + IVFPQ_MAX_NSUB);
    int* cnt_p = reinterpret_cast<int*>(tau_p + 1);
    int* hist_p = reinterpret_cast<int*>(tau_p + 4);
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(hist_p + kTopkHistInts);  // DBG only
    long long* vprefix = reinterpret_cast<long long*>(hitmask + IVFPQ_MAX_NSUB * 8);  // DBG only

    const int64_t q = blockIdx.x / p.nsplit;
    const int split = blockIdx.x % p.nsplit;
    TopkState t{kbuf, cnt_p, tau_p, hist_p, kKeyPadSigned};

    if (tid < nsub) {
        float v = 0.0f;
        if (!p.dense) {
            const float* rad = p.radius_mode == 1 ? p.radius + q * nsub : p.radius;
            float r = __fmul_rn(rad[tid], p.scale);
            v = __fmul_rn(r, r);
        }
        r2[tid] = v;
    }
    for (int j = tid; j < d; j += kScanThreads) qv[j] = p.queries[q * d + j];
    for (int i = nsub * 256 + tid; i < nw * 4 * 256; i += kScanThreads) lut[i] = 0.0f;   // padded subspaces add nothing
    if (DBG && tid == 0) {
        long long run = 0;
        for (int i = 0; i < p.nprobe; ++i) {
            vprefix[i] = run;
            int c = p.probe_ids[q * p.nprobe + i];
            if (c >= 0 && c < p.nlist) run += p.list_off[c + 1] - p.list_off[c];
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
            for (int s = 0; s < nsub; ++s) P = __fadd_rn(P, r2[s]);
        }
    }

    // ---- the query's table: thread e owns entry e of every subspace ----
    for (int s = 0; s < nsub; ++s) {
        float d2 = 0.0f, en2 = 0.0f, ip = 0.0f;
        if (tid < ksub) {
            const float* ent = p.cb + ((int64_t)s * ksub + tid) * dsub;
            const float* qs = qv + s * dsub;
            for (int j = 0; j < dsub; ++j) {
                const float ev = __ldg(ent + j);
                const float tt = __fsub_rn(qs[j], ev);
                d2 = __fmaf_rn(tt, tt, d2);
                en2 = __fmaf_rn(ev, ev, en2);
                ip = __fmaf_rn(qs[j], ev, ip);
            }
        }
        const bool hit = tid < ksub && (p.dense || d2 <= __fadd_rn(r2[s], en2));
        lut[s * 256 + tid] = hit ? -ip : P;
        if (DBG) {
            unsigned m = __ballot_sync(0xFFFFFFFFu, hit);
            if (lane == 0) hitmask[s * 8 + warp] = m;
        }
    }
    __syncthreads();

    for (int pi = split; pi < p.nprobe; pi += p.nsplit) {
        const int c = p.probe_ids[q * p.nprobe + pi];
        if (c < 0 || c >= p.nlist) {  // uniform over the CTA
            if (tid == 0) atomicOr(p.status, kFlagBadList);
            continue;
        }
        if (DBG && p.masks)
            for (int i = tid; i < nsub * 8; i += kScanThreads) p.masks[(q * p.nprobe + pi) * nsub * 8 + i] = hitmask[i];
        const float base = p.probe_d[q * p.nprobe + pi];   // -(q.c)
        const int64_t p0 = p.list_off[c];
        const int64_t len = p.list_off[c + 1] - p0;
        const int64_t b0 = p.list_blk[c];
        const int64_t nblk = p.list_blk[c + 1] - b0;
        if (nblk != (len + kPointsPerBlock - 1) / kPointsPerBlock || len < 0) {
            if (tid == 0) atomicOr(p.status, kFlagBadList);
            continue;
        }
        for (int64_t bb = 0; bb < nblk; bb += (kScanThreads / 32) * kBlocksPerWarpRound) {
            const unsigned long long tau = *tau_p;
            const uint32_t tau_hi = (uint32_t)(tau >> 32);
#pragma unroll 1
            for (int r = 0; r < kBlocksPerWarpRound; ++r) {
                const int64_t blk = bb + r * (kScanThreads / 32) + warp;
                if (blk >= nblk) break;
                float acc = base;
                unsigned long long hs = 0;
                if (p.vec16) {
                    const int G = nw >> 2;
                    const uint4* cp = reinterpret_cast<const uint4*>(p.codes_il) + (b0 + blk) * G * 32 + lane;
                    for (int g = 0; g < G; ++g) {
                        const uint4 v = __ldg(cp + g * 32);
                        accum_word<DBG>(v.x, g * 16 + 0, lut, hitmask, nsub, acc, hs);
                        accum_word<DBG>(v.y, g * 16 + 4, lut, hitmask, nsub, acc, hs);
                        accum_word<DBG>(v.z, g * 16 + 8, lut, hitmask, nsub, acc, hs);
                        accum_word<DBG>(v.w, g * 16 + 12, lut, hitmask, nsub, acc, hs);
                    }
                } else {
                    const uint32_t* cp = p.codes_il + (b0 + blk) * nw * 32 + lane;
                    for (int w = 0; w < nw; ++w) accum_word<DBG>(__ldg(cp + w * 32), w * 4, lut, hitmask, nsub, acc, hs);
                }
                const int64_t pos = blk * kPointsPerBlock + lane;
                if (pos < len) {
                    if (DBG) {
                        const int64_t vi = vprefix[pi] + pos;
                        if (vi < p.visit_stride) {
                            if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                            if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = -acc;
                            if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[p0 + pos];
                        }
                    }
                    const uint32_t ab = ordered_bits(acc);
                    if (ab <= tau_hi) {
                        const unsigned long long key = ((unsigned long long)ab << 32) | (uint32_t)p.ids[p0 + pos];
                        if (key < tau) {
                            if (!topk_push(t, key)) atomicOr(p.status, kFlagOverflow);
                        }
                    }
                }
            }
            topk_round_end<kScanThreads>(t, p.k, kRoundPoints);
        }
    }

    topk_finalize<kScanThreads>(t, p.k);
    const int n = *cnt_p;
    if (p.nsplit == 1) {
        for (int i = tid; i < p.k; i += kScanThreads) {
            const unsigned long long key = i < n ? kbuf[i] : kKeyPadSigned;
            p.out_dist[q * p.k + i] = -from_ordered_bits((uint32_t)(key >> 32));
            p.out_ids[q * p.k + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
        }
    } else {
        unsigned long long* dst = p.partial + (q * p.nsplit + split) * p.k;
        for (int i = tid; i < p.k; i += kScanThreads) dst[i] = i < n ? kbuf[i] : kKeyPadSigned;
    }
}

// Merge of the per-slice sorted candidate lists of one query (paper Sec. 2.1, last paragraph:
// the top-k over everything that was visited).  SIGNED: keys of the inner-product path (negated
// similarities under the order-preserving bit map), decoded back to similarities.
template <bool SIGNED>
__global__ void __launch_bounds__(kScanThreads) merge_kernel(const unsigned long long* __restrict__ partial,
                                                             int nsplit, int k, float* __restrict__ out_dist,
                                                             int32_t* __restrict__ out_ids, int* __restrict__ status) {
    __shared__ unsigned long long buf[kTopkCap];
    __shared__ int cnt;
    __shared__ unsigned long long tau;
    __shared__ int hist[kTopkHistInts];
    TopkState t{buf, &cnt, &tau, hist, SIGNED ? kKeyPadSigned : kKeyPad};
    topk_init(t);
    const int64_t q = blockIdx.x;
    const unsigned long long* src = partial + q * nsplit * (int64_t)k;
    const int total = nsplit * k;
    for (int base = 0; base < total; base += kScanThreads) {
        const int i = base + threadIdx.x;
        if (i < total) {
            const unsigned long long key = src[i];
            if (key < tau) {  // the pad key equals the initial threshold and is never pushed
                if (!topk_push(t, key)) atomicOr(status, kFlagOverflow);
            }
        }
        topk_round_end<kScanThreads>(t, k, kScanThreads);
    }
    topk_finalize<kScanThreads>(t, k);
    for (int i = threadIdx.x; i < k; i += kScanThreads) {
        const unsigned long long key = i < cnt ? buf[i] : t.pad;
        out_dist[q * k + i] = SIGNED ? -from_ordered_bits((uint32_t)(key >> 32)) : __uint_as_float((uint32_t)(key >> 32));
        out_ids[q * k + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
    }
}

template <bool DBG>
cudaError_t launch_ip(const ScanParams& sp, int64_t grid, size_t smem, cudaStream_t st) {
    auto kern = scan_ip_kernel<DBG>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)grid, kScanThreads, smem, st>>>(sp);
    return cudaGetLastError();
}

template <int NW_T, int DSUB_T, bool VEC16, bool DBG>
cudaError_t launch_one(const ScanParams& sp, int64_t grid, size_t smem, cudaStream_t st) {
    auto kern = scan_kernel<NW_T, DSUB_T, VEC16, DBG>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)grid, kScanThreads, smem, st>>>(sp);
    return cudaGetLastError();
}

template <bool DBG>
cudaError_t dispatch(const ivfpq_index* ix, const ScanParams& sp, int64_t grid, size_t smem, cudaStream_t st) {
    if (ix->nw == 4 && ix->dsub == 8 && ix->vec16) return launch_one<4, 8, true, DBG>(sp, grid, smem, st);
    if (ix->nw == 12 && ix->dsub == 2 && ix->vec16) return launch_one<12, 2, true, DBG>(sp, grid, smem, st);
    if (ix->nw == 13 && ix->dsub == 4 && !ix->vec16) return launch_one<13, 4, false, DBG>(sp, grid, smem, st);
    if (ix->vec16) return launch_one<0, 0, true, DBG>(sp, grid, smem, st);
    return launch_one<0, 0, false, DBG>(sp, grid, smem, st);
}

}  // namespace

// Which list scan serves a sparsity-aware search of the 16 x 8 shape: the code stream (work
// proportional to the list lengths) unless the caller asked for the walk through the entry ->
// points map (work proportional to the selected entries; measured slower on this hardware at every
// radius tried, see the option's description).
static bool use_entry_map(const ivfpq_index* ix, const SearchArgs& a) {
    return !a.dense && ix->map_pos && ix->sparse_scan == IVFPQ_SPARSE_SCAN_MAP;
}

cudaError_t launch_scan(const SearchArgs& a, const WorkspaceLayout& wl, char* ws, cudaStream_t st,
                        int64_t* launches) {
    const ivfpq_index* ix = a.ix;
    ScanParams sp{};
    sp.cent = ix->cent;
    sp.cb = ix->cb;
    sp.cbt = ix->cbt;
    sp.ids = ix->ids;
    sp.blk_min = ix->blk_min;
    sp.codes_il = ix->codes_il;
    sp.list_off = ix->list_off;
    sp.list_blk = ix->list_blk;
    sp.chunk_first = ix->chunk_first;
    sp.map_off = ix->map_off;
    sp.map_pos = ix->map_pos;
    sp.map_group = ix->map_group;
    sp.d = ix->d;
    sp.nlist = ix->nlist;
    sp.nsub = ix->nsub;
    sp.dsub = ix->dsub;
    sp.ksub = ix->ksub;
    sp.nw = ix->nw;
    sp.vec16 = ix->vec16;
    sp.queries = a.queries;
    sp.probe_ids = reinterpret_cast<const int32_t*>(ws + wl.probe_ids_off);
    sp.probe_d = reinterpret_cast<const float*>(ws + wl.probe_d_off);
    sp.nprobe = a.nprobe;
    sp.radius = a.radius;
    sp.radius_mode = a.radius_mode;
    sp.scale = a.scale;
    sp.miss_penalty = a.miss_penalty;
    sp.score = a.dense ? IVFPQ_SCORE_DISTANCE : a.score;
    sp.dense = a.dense ? 1 : 0;
    sp.k = a.k;
    sp.nsplit = a.debug ? 1 : wl.nsplit;
    sp.out_dist = a.out_dist;
    sp.out_ids = a.out_ids;
    sp.partial = reinterpret_cast<unsigned long long*>(ws + wl.partial_off);
    sp.status = reinterpret_cast<int*>(ws + wl.status_off);
    sp.work = sp.status + 1;
    sp.masks = a.masks;
    sp.visit_count = a.visit_count;
    sp.visit_stride = a.visit_stride;
    sp.visit_hits = reinterpret_cast<unsigned long long*>(a.visit_hits);
    sp.visit_dist = a.visit_dist;
    sp.visit_ids = a.visit_ids;

    const size_t smem = scan_smem_bytes(ix->nw, ix->d, a.nprobe, a.debug);
    const int64_t grid = a.nq * sp.nsplit;
    cudaError_t e;
    const bool ip = ix->metric == IVFPQ_METRIC_IP;
    if (ip && ix->rot)
        e = launch_scan_rot(ix, sp, grid, a.debug, a.nprobe, st);
    else if (ip)
        e = a.debug ? launch_ip<true>(sp, grid, smem, st) : launch_ip<false>(sp, grid, smem, st);
    else if (pers_shape(ix) && use_entry_map(ix, a))
        e = launch_scan16x8_map(ix, sp, grid, a.debug, a.nprobe, st);
    else if (pers_shape(ix))
        e = launch_scan16x8(ix, sp, grid, a.debug, a.nprobe, st);
    else if (ix->rot)
        e = launch_scan_rot(ix, sp, grid, a.debug, a.nprobe, st);
    else
        e = a.debug ? dispatch<true>(ix, sp, grid, smem, st) : dispatch<false>(ix, sp, grid, smem, st);
    if (e != cudaSuccess) return e;
    *launches += 1;
    if (sp.nsplit > 1) {
        if (ip)
            merge_kernel<true><<<(unsigned)a.nq, kScanThreads, 0, st>>>(sp.partial, sp.nsplit, a.k, a.out_dist, a.out_ids, sp.status);
        else
            merge_kernel<false><<<(unsigned)a.nq, kScanThreads, 0, st>>>(sp.partial, sp.nsplit, a.k, a.out_dist, a.out_ids, sp.status);
        *launches += 1;
        e = cudaGetLastError();
    }
    return e;
}

}  // namespace ivfpq

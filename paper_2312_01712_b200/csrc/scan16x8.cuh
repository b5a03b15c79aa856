// Supporting pieces of the persistent kernel of the 16 x 8 product quantizer (scan16x8.cu): list
// metadata staging, the per-query thresholds, the candidate buffer protocol (position keys,
// compaction, ranked output) and the small PTX helpers.
#pragma once

#include "common.cuh"
#include "scan_common.cuh"
#include "topk.cuh"

namespace ivfpq {
namespace pq16x8 {

constexpr int kW = 16;        // subspaces
constexpr int kDsub = 8;      // dimensions per subspace
constexpr int kD = kW * kDsub;
constexpr int kMetaCap = 128; // clusters whose metadata is staged at a time

struct ProbeMeta {
    long long b0;   // first 32-point code block of the list
    int p0;         // first point of the list (index into ids; ntotal < 2^31)
    int len;        // points in the list (0 when the cluster id or its tables were invalid)
    int cl;         // cluster id, clamped into range
    int pad;
};

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// Asks for the 128-byte lines of the warp's addresses to be brought into L2 (no register, no wait).
__device__ __forceinline__ void prefetch_l2(const void* gptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(gptr)); }

// Squared threshold of subspace `s` for query q (Algorithm 2: thres * thres_scale, squared); 0 for
// the dense search, where it is not used.
__device__ __forceinline__ float squared_threshold(const ScanParams& p, int64_t q, int s) {
    if (p.dense) return 0.0f;
    const float* rad = p.radius_mode == 1 ? p.radius + q * kW : p.radius;
    const float r = __fmul_rn(rad[s], p.scale);
    return __fmul_rn(r, r);
}

// The miss constant P: the caller's value, or the sum of the squared thresholds (ascending s).
__device__ __forceinline__ float miss_constant(const ScanParams& p, const float* r2) {
    if (p.dense) return 0.0f;
    if (p.miss_penalty >= 0.0f) return p.miss_penalty;
    float P = 0.0f;
#pragma unroll
    for (int s = 0; s < kW; ++s) P = __fadd_rn(P, r2[s]);
    return P;
}

// Metadata of probe `pi` of query q, with every table entry checked before use: an out-of-range
// cluster id or inconsistent list tables raise the status flag and leave an empty list.
__device__ __forceinline__ ProbeMeta load_probe_meta(const ScanParams& p, int64_t q, int pi) {
    ProbeMeta m;
    m.b0 = 0;
    m.p0 = 0;
    m.len = 0;
    m.pad = 0;
    int cl = p.probe_ids[q * p.nprobe + pi];
    if (cl < 0 || cl >= p.nlist) {
        atomicOr(p.status, kFlagBadList);
        cl = 0;
    } else {
        const long long p0 = p.list_off[cl], p1 = p.list_off[cl + 1];
        const long long b0 = p.list_blk[cl], b1 = p.list_blk[cl + 1];
        const long long len = p1 - p0;
        if (len < 0 || p1 > 0x7FFFFFFFll || b1 - b0 != (len + kPointsPerBlock - 1) / kPointsPerBlock) {
            atomicOr(p.status, kFlagBadList);
        } else {
            m.len = (int)len;
            m.b0 = b0;
            m.p0 = (int)p0;
        }
    }
    m.cl = cl;
    return m;
}

// Visiting-order prefix sums of the probed list lengths (stage dumps only; one thread).
__device__ inline void fill_visit_prefix(const ScanParams& p, int64_t q, long long* vprefix) {
    long long run = 0;
    for (int i = 0; i < p.nprobe; ++i) {
        vprefix[i] = run;
        const int cl = p.probe_ids[q * p.nprobe + i];
        if (cl >= 0 && cl < p.nlist) run += p.list_off[cl + 1] - p.list_off[cl];
    }
    vprefix[p.nprobe] = run;
    if (p.visit_count) p.visit_count[q] = run;
}

// ---- candidate buffer protocol ------------------------------------------------------------------
// Candidates are pushed as (distance bits, position of the point in the id array).  The keys pushed
// since the last compaction are translated to (distance, id) - equal distances are ordered by id -
// right before the buffer is compacted; the first *ntrans keys already hold ids.  All threads of
// the CTA call these after a barrier that follows the last push.
// `keep_max`: the compaction refines its cut until at most that many keys survive (when it can).
template <int NT, int CAP>
__device__ __forceinline__ void compact_candidates(const TopkState& t, int* ntrans, int* qs, int k,
                                                   const int32_t* __restrict__ ids, int keep_max) {
    const int n = min(*t.cnt, CAP);
    for (int i = *ntrans + threadIdx.x; i < n; i += NT) {
        const unsigned long long key = t.buf[i];
        const uint32_t id = (uint32_t)__ldg(ids + (uint32_t)(key & 0xFFFFFFFFull));
        t.buf[i] = (key & 0xFFFFFFFF00000000ull) | id;
    }
    topk_quick_compact<NT, CtaGroup, CAP, true>(t, k, qs, keep_max);   // starts and ends with a barrier
    if (threadIdx.x == 0) *ntrans = *t.cnt;            // read again only after later barriers
}

// The exact k smallest (distance, id), ascending, of one query (paper Sec. 2.1, last paragraph):
// to the output arrays, or, when the query's probes are split over several CTAs, to this slice's
// partial list.  Unfilled slots are (+inf, -1).
template <int NT, int CAP>
__device__ __forceinline__ void emit_topk(const ScanParams& p, const TopkState& t, int* ntrans, int* qs, int64_t q,
                                          int split) {
    compact_candidates<NT, CAP>(t, ntrans, qs, p.k, p.ids, p.k + 64);   // leaves k or a few more keys
    __syncthreads();
    const int n = min(*t.cnt, CAP);
    const int tid = threadIdx.x;
    if (p.nsplit == 1) {
        float* od = p.out_dist + q * p.k;
        int32_t* oi = p.out_ids + q * p.k;
        topk_emit_ranked<NT, CtaGroup>(t, n, p.k, [&](int rank, unsigned long long key) {
            od[rank] = __uint_as_float((uint32_t)(key >> 32));
            oi[rank] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
        });
        for (int i = n + tid; i < p.k; i += NT) {
            od[i] = __uint_as_float((uint32_t)(kKeyPad >> 32));
            oi[i] = -1;
        }
    } else {
        unsigned long long* dst = p.partial + (q * p.nsplit + split) * p.k;
        topk_emit_ranked<NT, CtaGroup>(t, n, p.k, [&](int rank, unsigned long long key) { dst[rank] = key; });
        for (int i = n + tid; i < p.k; i += NT) dst[i] = kKeyPad;
    }
}

}  // namespace pq16x8
}  // namespace ivfpq

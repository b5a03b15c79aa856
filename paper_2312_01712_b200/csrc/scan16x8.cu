// Persistent fused selective-LUT / list-scan / top-k kernel for the 16 x 8 product quantizer (16
// subspaces of 8 dimensions, 256 entries), the shape of the SIFT-like workloads.  Same computation
// as scan.cu (paper Sec. 2.1 steps B-D with the selection of Sec. 4.1 / Algorithm 2 and the miss
// constant of Sec. 5.3).  One CTA per SM loops over (query, probe slice) items.
//
//   * Two instances, chosen when the index is loaded.  16 warps (128 registers per thread): the
//     whole 128 KB codebook lives in registers - thread t owns subspace c = t & 15 and the entries
//     u, u + 32, ... with u = t / 16 - which makes the table build cheapest: for short lists,
//     where the build weighs as much as the scan.  32 warps (64 registers): two entries of a
//     thread in registers, two in shared memory (two 16-byte loads per entry, conflict-free);
//     eight warps per scheduler hide the latency of code blocks that stream from HBM: for long
//     lists.  Either way building a table reads nothing from global memory but the probed centroid
//     (512 B, copied one or two pairs of clusters ahead with cp.async).
//   * Table layout: 256 rows (entries) of 256 bytes; a row holds two tables side by side, 32
//     columns each; column x holds the value of subspace x & 15 (two copies).  Lane l looks up, at
//     step i, column l ^ i: the 32 lanes of a warp touch 32 different banks whatever the codes
//     are.  The code bytes are stored in that visiting order when the index is loaded.  The table
//     regions sit at shared-window addresses 0x10000 (and 0x20000), so one byte-permute forms the address (byte 0:
//     the lane's column offset for that step, byte 1: the code, bytes 2-3: zero) and the table base
//     is the immediate of the load: three instructions per look-up.
//   * Clusters are taken two at a time and their two lists are dealt to the warps as one sequence
//     of blocks, so that the barrier at the end of a phase waits for block counts that differ by
//     one per pair of lists.  16 warps: four tables (a second 64 KB region); in one phase a warp
//     builds its share of the next pair's tables and then scans this pair's lists - one barrier
//     per pair.  32 warps (no room for four tables beside the shared codebook half): a phase that
//     builds the pair's two tables, a phase that scans its lists.
//   * The score (distance / hit count / reward-penalty) is a template parameter: testing it for
//     every table entry cost the distance search 9 %.
//   * Code blocks: two per warp in registers, requested before the table build, refilled in
//     two-block rounds without register copies; the 32-warp instance also asks for the lines
//     further ahead to be brought into L2 (prefetch.global.L2, three blocks ahead and the first
//     blocks of the next list), which keeps enough bytes in flight without spending registers.
//   * Candidates go to the CTA's candidate buffer as (distance, position in the id array); only
//     lanes that push look at its fill level; ids are read when the buffer is compacted (one
//     histogram pass, topk.cuh); the final k are ranked by counting and written straight to the
//     output.
#include <type_traits>

#include "scan16x8.cuh"

namespace ivfpq {

namespace {

using namespace pq16x8;

// NT = threads per CTA: 1024 (entries u, u + 64 of a thread in registers, u + 128, u + 192 in shared
// memory) or 512 (all eight entries of a thread in registers, no shared codebook).
template <int NT>
struct Shape {
    static constexpr int kWarps = NT / 32;
    static constexpr int kEP = NT / kW;                   // entries per pass
    static constexpr int kNE = 256 / kEP;                 // entries per thread
    static constexpr int kRegEntries = NT == 1024 ? 2 : kNE;
    static_assert(NT == 512 || NT == 1024, "thread counts this kernel is written for");
};
constexpr int kRowBytes = 256;    // one table row (two tables side by side)
constexpr uint32_t kLutWin = 0x10000;   // shared-window address of the table region (64 KB)
constexpr uint32_t kCbWin = 0x20000;    // shared-window address of the shared half of the codebook (64 KB)
constexpr int kCap = 4096;        // candidate buffer slots
constexpr int kSoftLimit = 2048;  // compaction is requested once this many candidates are buffered
constexpr int kPfDist = 3;         // blocks (per warp) that the L2 prefetch runs ahead of the scan
static_assert(kSoftLimit + 2 * 1024 <= kCap && IVFPQ_MAX_K < kSoftLimit, "candidate buffer limits");


// Auxiliary shared memory in front of the table region, in bytes.
__host__ __device__ inline int scan16x8_aux_bytes(int nprobe, bool dbg) {
    int b = kCap * 8;                         // candidate keys
    b += kMetaCap * (int)sizeof(ProbeMeta);
    b += kD * 4 + 4 * kD * 4 + 64;            // query, four centroids, squared thresholds
    b += 32 + kQuickWords * 4;                // threshold, counters, compaction histogram
    if (dbg) b += 4 * kW * 8 * 4 + (nprobe + 1) * 8;
    return (b + 255) & ~255;
}

// One table look-up.  `word` holds four code bytes, `pack` the lane's column offsets (lane ^ i) * 4
// of the same four steps; T = byte of both that belongs to this step.  The permute builds
// {0, 0, code, column offset} (the zero bytes are the replicated sign of the column offset, which is
// below 128); the table base is the immediate.
template <int T, int TABLE>
__device__ __forceinline__ float lut_gather(uint32_t word, uint32_t pack) {
    uint32_t addr;
    float v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(addr) : "r"(word), "r"(pack), "n"(((12 + T) << 12) | ((12 + T) << 8) | (T << 4) | (4 + T)));
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"((int)kLutWin + (TABLE >> 1) * 0x10000 + (TABLE & 1) * 128) : "memory");
    return v;
}

// Sum of the 16 table values of the lane's point.  Byte i of `cur` = code of subspace (lane ^ i) & 15.
// AB > 0: early abandon.  Every table value is >= 0 (squared distances, the miss constant, counts), so
// the running sum only grows (fp32 addition of non-negative terms is monotone, and the final value
// adds the same two partial sums): once every lane of the warp is at or above `tau_cut`, no point of
// the block can pass the candidate test and the remaining look-ups are skipped; the value returned is
// then some number at or above the cut.  AB = 1 tests after the second code word, AB = 2 after the
// first and the second (the sparsity-aware search, where a miss alone can put a point out of reach).
template <int TABLE, int AB>
__device__ __forceinline__ float gather16(const uint4 cur, const uint32_t (&pk)[4], const uint32_t tau_cut) {
    float a0 = lut_gather<0, TABLE>(cur.x, pk[0]);
    float a1 = lut_gather<1, TABLE>(cur.x, pk[0]);
    a0 += lut_gather<2, TABLE>(cur.x, pk[0]);
    a1 += lut_gather<3, TABLE>(cur.x, pk[0]);
    if (AB >= 2) {
        const float part = a0 + a1;
        if (__all_sync(0xFFFFFFFFu, __float_as_uint(part) >= tau_cut)) return part;
    }
    a0 += lut_gather<0, TABLE>(cur.y, pk[1]);
    a1 += lut_gather<1, TABLE>(cur.y, pk[1]);
    a0 += lut_gather<2, TABLE>(cur.y, pk[1]);
    a1 += lut_gather<3, TABLE>(cur.y, pk[1]);
    if (AB >= 1) {
        const float part = a0 + a1;
        if (__all_sync(0xFFFFFFFFu, __float_as_uint(part) >= tau_cut)) return part;
    }
    a0 += lut_gather<0, TABLE>(cur.z, pk[2]);
    a1 += lut_gather<1, TABLE>(cur.z, pk[2]);
    a0 += lut_gather<2, TABLE>(cur.z, pk[2]);
    a1 += lut_gather<3, TABLE>(cur.z, pk[2]);
    a0 += lut_gather<0, TABLE>(cur.w, pk[3]);
    a1 += lut_gather<1, TABLE>(cur.w, pk[3]);
    a0 += lut_gather<2, TABLE>(cur.w, pk[3]);
    a1 += lut_gather<3, TABLE>(cur.w, pk[3]);
    return a0 + a1;
}

template <int NT, bool DBG, int SCORE_T, int AB>
__global__ void __launch_bounds__(NT, 1) scan16x8_kernel(const ScanParams p, const int64_t nitems) {
    constexpr int kNT = NT;
    constexpr int kWarps = Shape<NT>::kWarps;
    constexpr int kEP = Shape<NT>::kEP;
    constexpr int kNE = Shape<NT>::kNE;
    constexpr int kRegEntries = Shape<NT>::kRegEntries;
    constexpr int kPf = NT == 1024 ? kPfDist : 0;   // the 16-warp instance serves short, L2-resident lists
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int c = tid & (kW - 1);   // subspace of this thread in the table build
    const int u = tid / kW;         // first entry of this thread (0..63)
    const int half = lane >> 4;
    const int ksub = p.ksub;

    // ---- shared-memory carve-up: auxiliary data below the table region ----
    const uint32_t win = (uint32_t)__cvta_generic_to_shared(smem);
    if (win + (uint32_t)scan16x8_aux_bytes(p.nprobe, DBG) > kLutWin) {  // uniform: layout does not fit this window offset
        if (tid == 0) atomicOr(p.status, kFlagLayout);
        return;
    }
    unsigned char* const lut_gen = smem + (kLutWin - win);   // table region as a generic pointer
    float* const cb_s = reinterpret_cast<float*>(smem + (kCbWin - win));
    unsigned char* a = smem;
    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(a);
    a += (size_t)kCap * 8;
    ProbeMeta* meta = reinterpret_cast<ProbeMeta*>(a);
    a += kMetaCap * sizeof(ProbeMeta);
    float* qs = reinterpret_cast<float*>(a);
    float* cent_s = qs + kD;          // [4][128]
    float* r2 = cent_s + 4 * kD;      // [16]
    a += kD * 4 + 4 * kD * 4 + 64;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(a);
    int* cnt_p = reinterpret_cast<int*>(a + 8);
    int* ntrans_p = cnt_p + 1;
    int* next_p = cnt_p + 2;   // the item this CTA takes next
    a += 32;
    int* hist_p = reinterpret_cast<int*>(a);
    a += kQuickWords * 4;
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(a);                        // DBG only: [4][16][8]
    long long* vprefix = reinterpret_cast<long long*>(a + 4 * kW * 8 * 4);     // DBG only
    TopkState t{kbuf, cnt_p, tau_p, hist_p};

    // ---- codebook: the first kRegEntries entries of a thread in registers, the others (32 warps
    //      only: entries 128..255) in shared memory as [entry - 128][half of the 8 dimensions]
    //      [subspace][4 floats] ----
    float cbr[kRegEntries][kDsub];
#pragma unroll
    for (int m = 0; m < kNE; ++m) {
        const int e = u + kEP * m;
        const float4* src = reinterpret_cast<const float4*>(p.cbt + ((size_t)e * kW + c) * kDsub);
        const float4 v0 = __ldg(src), v1 = __ldg(src + 1);
        if (m < kRegEntries) {
            float* dst = cbr[m < kRegEntries ? m : 0];
            dst[0] = v0.x; dst[1] = v0.y; dst[2] = v0.z; dst[3] = v0.w;
            dst[4] = v1.x; dst[5] = v1.y; dst[6] = v1.z; dst[7] = v1.w;
        } else {
            float4* dst = reinterpret_cast<float4*>(cb_s + (size_t)(e - kRegEntries * kEP) * (2 * kW * 4));
            dst[c] = v0;
            dst[kW + c] = v1;
        }
    }
    // row u, columns c and c + 16; the two half-warps (rows u, u + 1) write the copies in opposite
    // order so that a warp's 32 stores hit 32 banks
    const int st_a = u * kRowBytes + (c + (half ? 16 : 0)) * 4;
    const int st_b = u * kRowBytes + (c + (half ? 0 : 16)) * 4;
    // column offsets (lane ^ i) * 4 of the 16 steps, four per register
    uint32_t pk[4];
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
        uint32_t v = 0;
#pragma unroll
        for (int tt = 0; tt < 4; ++tt) v |= (uint32_t)(((lane ^ (4 * k4 + tt)) * 4) & 0xFF) << (8 * tt);
        pk[k4] = v;
    }

    // This thread's share of a table (steps B, C + selection): residual of subspace c from the
    // staged centroid, squared distance to its four entries, kept when within the threshold.
    auto build = [&](unsigned char* lutb, const float* cs, float thr, float P, uint32_t* hm) {
        float r[kDsub];
        {
            const float4 qa = *reinterpret_cast<const float4*>(qs + c * kDsub);
            const float4 qb = *reinterpret_cast<const float4*>(qs + c * kDsub + 4);
            const float4 ca = *reinterpret_cast<const float4*>(cs + c * kDsub);
            const float4 cb = *reinterpret_cast<const float4*>(cs + c * kDsub + 4);
            r[0] = __fsub_rn(qa.x, ca.x); r[1] = __fsub_rn(qa.y, ca.y);
            r[2] = __fsub_rn(qa.z, ca.z); r[3] = __fsub_rn(qa.w, ca.w);
            r[4] = __fsub_rn(qb.x, cb.x); r[5] = __fsub_rn(qb.y, cb.y);
            r[6] = __fsub_rn(qb.z, cb.z); r[7] = __fsub_rn(qb.w, cb.w);
        }
#pragma unroll
        for (int m = 0; m < kNE; ++m) {
            float e8[kDsub];
            if (m < kRegEntries) {
#pragma unroll
                for (int j = 0; j < kDsub; ++j) e8[j] = cbr[m < kRegEntries ? m : 0][j];
            } else {
                const float4* src = reinterpret_cast<const float4*>(cb_s + (size_t)(u + kEP * (m - kRegEntries)) * (2 * kW * 4));
                const float4 v0 = src[c], v1 = src[kW + c];
                e8[0] = v0.x; e8[1] = v0.y; e8[2] = v0.z; e8[3] = v0.w;
                e8[4] = v1.x; e8[5] = v1.y; e8[6] = v1.z; e8[7] = v1.w;
            }
            float d2 = 0.0f;
#pragma unroll
            for (int j = 0; j < kDsub; ++j) {
                const float tt = __fsub_rn(r[j], e8[j]);
                d2 = __fmaf_rn(tt, tt, d2);
            }
            const int e = u + kEP * m;
            const bool hit = e < ksub && (p.dense || d2 <= thr);
            const float val = table_value<SCORE_T>(p.score, hit, d2, thr, P);
            unsigned char* row = lutb + m * (kEP * kRowBytes);
            *reinterpret_cast<float*>(row + st_a) = val;
            *reinterpret_cast<float*>(row + st_b) = val;
            if (DBG && hit) atomicOr(&hm[c * 8 + (e >> 5)], 1u << (e & 31));
        }
    };
    // copies centroid `cl` (128 floats) into cs[0..128): one float4 per thread of one warp
    auto fetch_cent = [&](int cl, float* cs, int l) { cp_async16(cs + 4 * l, p.cent + (int64_t)cl * kD + 4 * l); };

    topk_quick_init<kNT>(hist_p);  // contains a barrier: the shared half of the codebook is complete too

    // Items beyond the first come from a global counter (lists differ in length: a fixed stride
    // leaves the CTAs finishing at different times); the draw is made at the start of an item and read
    // at its end.
    for (int64_t item = blockIdx.x; item < nitems; item = *next_p) {
        const int64_t q = item / p.nsplit;
        const int split = (int)(item % p.nsplit);
        const int np_item = (p.nprobe - split + p.nsplit - 1) / p.nsplit;  // probes split, split + nsplit, ...
        __syncthreads();  // the previous item's results have been read out of the candidate buffer
        if (tid < kW) {
            r2[tid] = squared_threshold(p, q, tid);
        } else if (tid >= 32 && tid < 64) {
            reinterpret_cast<float4*>(qs)[tid - 32] = __ldg(reinterpret_cast<const float4*>(p.queries + q * kD) + (tid - 32));
        } else if (tid == 64) {
            *cnt_p = 0;
            *ntrans_p = 0;
            *tau_p = kKeyPad;
        } else if (tid == 65) {
            *next_p = (int)gridDim.x + atomicAdd(p.work, 1);
        }
        if (DBG && tid == 96) fill_visit_prefix(p, q, vprefix);
        float P = 0.0f, thr = 0.0f;

        for (int t0 = 0; t0 < np_item; t0 += kMetaCap) {
            const int nt = min(kMetaCap, np_item - t0);
            // ---- stage the metadata of the tile's clusters (the previous tile ended with a barrier) ----
            if (tid >= 128 && tid < 128 + nt) meta[tid - 128] = load_probe_meta(p, q, split + (t0 + tid - 128) * p.nsplit);
            if (DBG)
                for (int i = tid; i < 4 * kW * 8; i += kNT) hitmask[i] = 0;
            __syncthreads();
            if (t0 == 0) {
                P = miss_constant(p, r2);
                thr = r2[c];
            }

            // The clusters are taken two at a time, their lists as one sequence of blocks dealt
            // round-robin to the warps: the warps' block counts differ by one per pair of lists, not
            // per list (the barrier that ends a phase waits for the slowest warp).
            //   16 warps (kAhead): four tables (two 64 KB regions).  In one phase a warp builds its share
            //   of the NEXT pair's tables and then scans its blocks of this pair: one barrier per pair,
            //   and warps that build overlap with warps that scan.
            //   32 warps: two tables.  Phase A builds the pair's tables, phase B scans its lists.
            // Cluster j of the tile uses centroid slot and hit-mask buffer j & 3 (kAhead) or j & 1.
            constexpr bool kAhead = kNT == 512;
            constexpr int kSlots = kAhead ? 4 : 2;
            auto table_of = [&](int jj) {   // table of cluster jj as a generic pointer
                return lut_gen + (kAhead ? ((jj >> 1) & 1) * 0x10000 : 0) + (jj & 1) * 128;
            };
            auto build_cluster = [&](int jj) {
                build(table_of(jj), cent_s + (jj & (kSlots - 1)) * kD, thr, P, hitmask + (jj & (kSlots - 1)) * kW * 8);
            };
            // ---- prologue: centroids of the tile's first clusters (and, kAhead, the first pair's tables) ----
            if (tid < 32 * kSlots && (tid >> 5) < nt) fetch_cent(meta[tid >> 5].cl, cent_s + (tid >> 5) * kD, lane);
            cp_async_wait_all();
            __syncthreads();
            if (kAhead) {
                build_cluster(0);
                if (nt > 1) build_cluster(1);
                __syncthreads();
            }

            for (int j = 0; j < nt; j += 2) {
                const bool two = j + 1 < nt;
                if (!kAhead) {
                    if (DBG && j > 0) {
                        for (int i = tid; i < 2 * kW * 8; i += kNT) hitmask[i] = 0;
                        __syncthreads();
                    }
                    // ---- phase A: the tables of clusters j and j + 1 ----
                    build_cluster(j);
                    if (two) build_cluster(j + 1);
                    __syncthreads();
                }
                if (DBG) {
                    // the masks of this pair are complete (previous barrier)
                    if (p.masks)
                        for (int i = tid; i < (two ? 2 : 1) * kW * 8; i += kNT) {
                            const int jj = j + i / (kW * 8);
                            p.masks[(q * p.nprobe + split + (t0 + jj) * p.nsplit) * kW * 8 + i % (kW * 8)] =
                                hitmask[(jj & (kSlots - 1)) * kW * 8 + i % (kW * 8)];
                        }
                    if (kAhead) {   // clear the buffers of the next pair before its tables are built
                        for (int i = tid; i < 2 * kW * 8; i += kNT) hitmask[((j + 2) & 3) * kW * 8 + i] = 0;
                        __syncthreads();
                    }
                }
                // ---- scan the lists of clusters j and j + 1 (step D) ----
                // Scan state of the list the warp is in: it owns blocks first, first + kWarps, ...:
                // `rem` of them are left, `ptr` is this lane's 16 bytes of the next one, `pos` the
                // position of the lane's point in the list; two blocks are always in registers.
                constexpr int kStep = kWarps * 32;   // uint4 elements between two blocks of a warp
                int li = 0, first = warp, pi = 0, rem = 0, pos = 0;
                ProbeMeta m = meta[j];
                const uint4* ptr = nullptr;
                const uint32_t* hm = hitmask;
                uint4 n0 = make_uint4(0, 0, 0, 0), n1 = make_uint4(0, 0, 0, 0);
                auto enter = [&](int l) {
                    m = meta[j + l];
                    pi = split + (t0 + j + l) * p.nsplit;
                    hm = hitmask + ((j + l) & (kSlots - 1)) * kW * 8;
                    const int nblk = (m.len + kPointsPerBlock - 1) / kPointsPerBlock;
                    rem = nblk > first ? (nblk - first + kWarps - 1) / kWarps : 0;
                    ptr = reinterpret_cast<const uint4*>(p.codes_il) + m.b0 * 32 + lane + first * 32;
                    pos = first * kPointsPerBlock + lane;
                    if (rem > 0) n0 = __ldg(ptr);
                    if (rem > 1) n1 = __ldg(ptr + kStep);
                    // where the round-robin continues in the next list: the second list of the pair
                    // goes on from this one's end, the next pair starts over
                    const int next_first = l == 0 ? first + rem * kWarps - nblk : warp;
                    if (kPf > 0 && j + l + 1 < nt) {   // the warp's first blocks of the next list: into L2 meanwhile
                        const ProbeMeta m1 = meta[j + l + 1];
                        const int nblk1 = (m1.len + kPointsPerBlock - 1) / kPointsPerBlock;
                        const uint4* cp1 = reinterpret_cast<const uint4*>(p.codes_il) + m1.b0 * 32 + lane;
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (next_first + i * kWarps < nblk1) prefetch_l2(cp1 + (int64_t)(next_first + i * kWarps) * 32);
                    }
                    first = next_first;
                };
                enter(0);   // the first two blocks are requested now and needed after the table build
                if (kAhead) {
                    // centroids of the pair after the next into the slots that the previous phase's
                    // builds have read; this thread's share of the next pair's tables
                    if (tid < 64 && j + 4 + (tid >> 5) < nt)
                        fetch_cent(meta[j + 4 + (tid >> 5)].cl, cent_s + ((j + 4 + (tid >> 5)) & 3) * kD, lane);
                    if (j + 2 < nt) build_cluster(j + 2);
                    if (j + 3 < nt) build_cluster(j + 3);
                } else {
                    // centroids of the next pair into the slots that phase A has read
                    if (tid < 64 && j + 2 + (tid >> 5) < nt)
                        fetch_cent(meta[j + 2 + (tid >> 5)].cl, cent_s + (tid >> 5) * kD, lane);
                }
                while (true) {
                    const unsigned long long tau = *tau_p;
                    const uint32_t tau_hi = (uint32_t)(tau >> 32), tau_lo = (uint32_t)tau;
                    // one compare in the common case: distances below tau_cut are candidates; a tie with the
                    // threshold distance (only possible when the threshold carries an id) is then decided by id
                    const uint32_t tau_cut = tau_hi + (tau_lo != 0 ? 1u : 0u);
                    bool stop = false;   // a candidate of this lane landed at or beyond the soft limit
                    bool halt = false;   // ... of this warp, as seen at the end of a round
                    auto scan_blocks = [&](auto table_tag) {
                        constexpr int TABLE = decltype(table_tag)::value;
                        // one block: 16 look-ups per lane, stage dumps, candidate test
                        auto consider = [&](const uint4 cur, const float acc, const int bpos) {
                            if (bpos < m.len) {
                                if (DBG) {
                                    unsigned long long hs = 0;
                                    const uint32_t wv[4] = {cur.x, cur.y, cur.z, cur.w};
#pragma unroll
                                    for (int i = 0; i < kW; ++i) {
                                        const uint32_t code = (wv[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                                        const int s = (lane ^ i) & (kW - 1);
                                        hs |= (unsigned long long)((hm[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
                                    }
                                    const int64_t vi = vprefix[pi] + bpos;
                                    if (vi < p.visit_stride) {
                                        if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                                        if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = acc;
                                        if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[m.p0 + bpos];
                                    }
                                }
                                // key < threshold, key = (distance, id).  The id is read only for a tie with
                                // the threshold distance (many points can share a distance: every point
                                // that missed in all subspaces has 16 P), and only in a block whose
                                // smallest id is below the threshold's
                                const uint32_t ab = __float_as_uint(acc);
                                if (ab < tau_cut && (ab != tau_hi || (__ldg(p.blk_min + m.b0 + (bpos >> 5)) < tau_lo &&
                                                                      (uint32_t)__ldg(p.ids + m.p0 + bpos) < tau_lo))) {
                                    const int slot = atomicAdd(cnt_p, 1);
                                    if (slot < kCap) kbuf[slot] = make_key(acc, (uint32_t)(m.p0 + bpos));
                                    else atomicOr(p.status, kFlagOverflow);
                                    stop |= slot >= kSoftLimit;
                                }
                            }
                        };
                        // the look-ups of one block
                        auto g16 = [&](const uint4 v) -> float { return gather16<TABLE, AB>(v, pk, tau_cut); };
                        // Two blocks per round; each code register is refilled right after its block
                        // has been consumed (no copies).  The fill level of the candidate buffer is
                        // only looked at by lanes that push: a warp leaves the loop at the end of a
                        // round in which one of its candidates landed beyond the soft limit, which
                        // bounds the overshoot by 64 candidates per warp.
                        while (rem >= 2 && !halt) {
                            if constexpr (kNT == 512) {
                                // L2-resident lists, four warps per scheduler: the look-ups of both blocks
                                // first (32 independent loads, four running sums), then the two tests
                                const float acc0 = g16(n0);
                                const float acc1 = g16(n1);
                                if (DBG) {   // the stage dumps read the codes: keep them until then
                                    consider(n0, acc0, pos);
                                    consider(n1, acc1, pos + kWarps * kPointsPerBlock);
                                }
                                const uint4 z = make_uint4(0, 0, 0, 0);
                                if (rem > 2) n0 = __ldg(ptr + 2 * kStep);
                                if (rem > 3) n1 = __ldg(ptr + 3 * kStep);
                                if (!DBG) {
                                    consider(z, acc0, pos);
                                    consider(z, acc1, pos + kWarps * kPointsPerBlock);
                                }
                            } else {
                                // lists streamed from HBM: each code register is refilled as soon as its
                                // block has been consumed
                                consider(n0, g16(n0), pos);
                                if (rem > 2) n0 = __ldg(ptr + 2 * kStep);
                                consider(n1, g16(n1), pos + kWarps * kPointsPerBlock);
                                if (rem > 3) n1 = __ldg(ptr + 3 * kStep);
                            }
                            if (kPf > 0) {
                                if (rem > kPf + 1) prefetch_l2(ptr + (kPf + 1) * kStep);
                                if (rem > kPf + 2) prefetch_l2(ptr + (kPf + 2) * kStep);
                            }
                            ptr += 2 * kStep;
                            pos += 2 * kWarps * kPointsPerBlock;
                            rem -= 2;
                            halt = __any_sync(0xFFFFFFFFu, stop);
                        }
                        if (rem == 1 && !halt) {
                            consider(n0, g16(n0), pos);
                            rem = 0;
                            halt = __any_sync(0xFFFFFFFFu, stop);
                        }
                    };
                    while (true) {
                        const int table = (kAhead ? ((j >> 1) & 1) * 2 : 0) + li;
                        if (table == 0) scan_blocks(std::integral_constant<int, 0>{});
                        else if (table == 1) scan_blocks(std::integral_constant<int, 1>{});
                        else if (kAhead && table == 2) scan_blocks(std::integral_constant<int, 2>{});
                        else if (kAhead) scan_blocks(std::integral_constant<int, 3>{});
                        if (halt || li == 1 || !two) break;
                        li = 1;
                        enter(1);
                    }
                    cp_async_wait_all();
                    // the barrier that ends the pair (tables free, next centroids staged); a set flag
                    // means that some warp saw the soft limit or has blocks left: the buffer is
                    // compacted and the scan resumes where it stopped
                    if (!__syncthreads_or(rem > 0 || halt || (li == 0 && two))) break;
                    compact_candidates<kNT, kCap>(t, ntrans_p, hist_p, p.k, p.ids, kSoftLimit / 2);   // between lists any cut that frees half the buffer will do
                }
            }
        }

        emit_topk<kNT, kCap>(p, t, ntrans_p, hist_p, q, split);
    }
}

template <int NT, bool DBG, int SCORE_T, int AB>
cudaError_t launch_inst(const ScanParams& sp, int64_t grid, int64_t nitems, cudaStream_t st) {
    // covers, for any window offset, the auxiliary area, the table region and a second 64 KB region:
    // the shared half of the codebook (32 warps) or the second pair of tables (16 warps)
    const size_t smem = (size_t)kCbWin + 65536;
    auto kern = scan16x8_kernel<NT, DBG, SCORE_T, AB>;
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)grid, NT, smem, st>>>(sp, nitems);
    return cudaGetLastError();
}

// Instances: stage dumps (score read at run time, every point evaluated in full), one per score
// otherwise.  Early abandon only in the 32-warp instance, whose long lists stream from HBM with the
// issue slots nearly full: there it takes the 100 M-point workload's list scan from 17.6 to 15.4 ms
// (dense search, test after two code words) and to 14.3 ms (sparsity-aware, test after one and
// two).  The 16-warp instance issues the 32 look-ups of two blocks back to back; the branches cost
// it more than the skipped look-ups save (1 M points, 16 probes: 2.48 -> 2.53 -> 2.61 ms).
template <int NT>
cudaError_t launch_nt(const ScanParams& sp, int64_t grid, int64_t nitems, bool debug, cudaStream_t st) {
    constexpr int kAbDense = NT == 1024 ? 1 : 0, kAbSparse = NT == 1024 ? 2 : 0;
    if (debug) return launch_inst<NT, true, -1, 0>(sp, grid, nitems, st);
    // (at the radii where the hit count ranks best nearly every point misses nearly everywhere: the
    // threshold stays above the misses of half the subspaces, no block is abandoned: no votes)
    if (sp.score == IVFPQ_SCORE_HIT_COUNT) return launch_inst<NT, false, IVFPQ_SCORE_HIT_COUNT, 0>(sp, grid, nitems, st);
    if (sp.score == IVFPQ_SCORE_REWARD_PENALTY) return launch_inst<NT, false, IVFPQ_SCORE_REWARD_PENALTY, kAbSparse>(sp, grid, nitems, st);
    if (sp.dense) return launch_inst<NT, false, IVFPQ_SCORE_DISTANCE, kAbDense>(sp, grid, nitems, st);
    return launch_inst<NT, false, IVFPQ_SCORE_DISTANCE, kAbSparse>(sp, grid, nitems, st);
}

}  // namespace

cudaError_t launch_scan16x8(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                             cudaStream_t st) {
    (void)nprobe;
    int64_t grid = ix->sm_count;
    if (grid > nitems) grid = nitems;
    return ix->pers_warps == 16 ? launch_nt<512>(sp, grid, nitems, debug, st) : launch_nt<1024>(sp, grid, nitems, debug, st);
}

}  // namespace ivfpq

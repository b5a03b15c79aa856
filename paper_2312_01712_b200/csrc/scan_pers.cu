// Persistent variant of the fused selective-LUT / list-scan / top-k kernel for the 16 x 8
// product quantizer (16 subspaces of 8 dimensions, 256 entries), the shape of the SIFT-like
// workloads.  Same computation as scan.cu (paper Sec. 2.1 steps B-D with the selection of
// Sec. 3.1 / Algorithm 2 and the miss constant of Sec. 4.3), organised for one resident CTA of
// 16 warps per SM:
//
//   * the whole codebook (128 KB) lives in the CTA's registers for the lifetime of the kernel:
//     thread t owns subspace c = t & 15 and the entries u, u + 32, ... with u = t / 16, so
//     building a table reads nothing but the probed centroid (512 B);
//   * the table of a (query, cluster) pair is 256 rows (entries) of 256 bytes in shared memory;
//     column x of a row holds the value of subspace x & 15, for x = 0..47.  Lane l of a warp (one
//     point per lane) looks up, at step i, column l + i: the 32 lanes touch 32 consecutive
//     columns = 32 different banks whatever the codes are, and over i = 0..15 a lane meets every
//     subspace once.  The code bytes are stored in that visiting order when the index is loaded;
//   * the table base is aligned to 64 KB in the shared window, so one byte-permute instruction
//     forms the whole address (byte 0: lane * 4, byte 1: the code, bytes 2-3: the base) and the
//     step offset 4 * i is the immediate of the load: three instructions per look-up;
//   * two tables are kept: while the warps scan the list of cluster j they have already built
//     their share of the table of cluster j + 1, and one barrier per cluster separates the
//     phases.  Warps drift apart inside a phase pair, so table arithmetic and table gathers of
//     different warps overlap on the SM;
//   * list metadata of the item's clusters is staged in shared memory once per item; the first
//     code blocks of a list are requested before the table build and arrive during it;
//   * candidates go to the CTA's candidate buffer as (distance, position in the id array): the
//     id itself is read only when the buffer is compacted, for all new candidates at once, so
//     the scan loop never waits for that load.  Only lanes that push look at the fill level; the
//     CTA compacts when a candidate landed beyond a soft limit, with one histogram pass over the
//     distances (topk.cuh); the final k are ranked by counting and written straight to the output.
#include "scan16x8.cuh"

namespace ivfpq {

namespace {

using namespace pq16x8;

constexpr int kNT = 512;          // threads per CTA
constexpr int kWarps = kNT / 32;
constexpr int kEP = kNT / kW;     // entries per pass (32)
constexpr int kNE = 256 / kEP;    // entries per thread (8)
constexpr int kRowBytes = 256;    // one table row
constexpr int kLutBytes = 256 * kRowBytes;  // one table: 64 KB
constexpr int kCap = 4096;        // candidate buffer slots
constexpr int kSoftLimit = 2048;  // compaction is requested once a candidate lands beyond this many
static_assert(kSoftLimit + 2 * kNT <= kCap && IVFPQ_MAX_K < kSoftLimit, "candidate buffer limits");


// Auxiliary shared memory (everything except the two tables), in bytes.
__host__ __device__ inline int pers_aux_bytes(int nprobe, bool dbg) {
    int b = kCap * 8;                     // candidate keys
    b += kMetaCap * (int)sizeof(ProbeMeta);
    b += kW * kDsub * 4;                  // query
    b += 64 * 4;                          // squared thresholds (padded)
    b += 32 + kQuickWords * 4;    // threshold, counters, compaction histogram
    if (dbg) b += 2 * kW * 8 * 4 + (nprobe + 1) * 8;
    return (b + 255) & ~255;
}

// Dynamic shared memory to request.  The kernel aligns the tables to 64 KB inside the shared
// window; the bytes in front of them hold the auxiliary data when they suffice, otherwise the
// auxiliary data follows the tables.  Either way this size is enough for any window offset.
inline size_t pers_smem_bytes(int nprobe, bool dbg) {
    const size_t aux = (size_t)pers_aux_bytes(nprobe, dbg);
    const size_t a = 65536 + 2 * (size_t)kLutBytes;
    const size_t b = 2 * (size_t)kLutBytes + 2 * aux;
    return a > b ? a : b;
}

// One table look-up: address = {bytes 3,2 of bsel, code byte BYTE of word, byte 0 of bsel} + IMM.
template <int BYTE, int IMM>
__device__ __forceinline__ float lut_gather(uint32_t word, uint32_t bsel) {
    uint32_t addr;
    float v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(addr) : "r"(word), "r"(bsel), "n"(0x7604 | (BYTE << 4)));
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(IMM) : "memory");
    return v;
}

// Sum of the 16 table values of the lane's point.  `cur` holds the lane's code bytes in visiting
// order (byte i = code of subspace (lane + i) & 15).
__device__ __forceinline__ float gather16(const uint4 cur, uint32_t bsel) {
    float a0 = lut_gather<0, 0>(cur.x, bsel);
    float a1 = lut_gather<1, 4>(cur.x, bsel);
    a0 += lut_gather<2, 8>(cur.x, bsel);
    a1 += lut_gather<3, 12>(cur.x, bsel);
    a0 += lut_gather<0, 16>(cur.y, bsel);
    a1 += lut_gather<1, 20>(cur.y, bsel);
    a0 += lut_gather<2, 24>(cur.y, bsel);
    a1 += lut_gather<3, 28>(cur.y, bsel);
    a0 += lut_gather<0, 32>(cur.z, bsel);
    a1 += lut_gather<1, 36>(cur.z, bsel);
    a0 += lut_gather<2, 40>(cur.z, bsel);
    a1 += lut_gather<3, 44>(cur.z, bsel);
    a0 += lut_gather<0, 48>(cur.w, bsel);
    a1 += lut_gather<1, 52>(cur.w, bsel);
    a0 += lut_gather<2, 56>(cur.w, bsel);
    a1 += lut_gather<3, 60>(cur.w, bsel);
    return a0 + a1;
}

template <bool DBG>
__global__ void __launch_bounds__(kNT, 1) scan_pers16x8_kernel(const ScanParams p, const int64_t nitems) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int c = tid & (kW - 1);   // subspace of this thread in the table build
    const int u = tid / kW;         // first entry of this thread
    const int half = lane >> 4;
    const int ksub = p.ksub;
    constexpr int d = kD;

    // ---- shared-memory carve-up ----
    const uint32_t win = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t pad = (0u - win) & 0xFFFFu;
    const uint32_t lut_win = win + pad;                 // shared-window address of table 0, 64 KB aligned
    unsigned char* const lut_gen = smem + pad;          // the same location as a generic pointer
    const int aux_bytes = pers_aux_bytes(p.nprobe, DBG);
    unsigned char* const aux = (pad >= (uint32_t)aux_bytes) ? smem : smem + pad + 2 * kLutBytes;
    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(aux);
    ProbeMeta* meta = reinterpret_cast<ProbeMeta*>(aux + (size_t)kCap * 8);
    float* qs = reinterpret_cast<float*>(meta + kMetaCap);
    float* r2 = qs + d;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(r2 + 64);
    int* cnt_p = reinterpret_cast<int*>(tau_p + 1);
    int* ntrans_p = cnt_p + 1;                                                   // keys that already hold ids
    int* hist_p = reinterpret_cast<int*>(tau_p + 4);                             // [kQuickWords]
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(hist_p + kQuickWords);     // DBG only: [2][16][8]
    long long* vprefix = reinterpret_cast<long long*>(hitmask + 2 * kW * 8);     // DBG only
    TopkState t{kbuf, cnt_p, tau_p, hist_p};

    // ---- codebook slice of this thread: entries u + 32 m of subspace c ----
    float cbr[kNE][kDsub];
#pragma unroll
    for (int m = 0; m < kNE; ++m) {
        const int e = u + kEP * m;
        const float4* src = reinterpret_cast<const float4*>(p.cbt + ((size_t)e * kW + c) * kDsub);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        cbr[m][0] = a.x; cbr[m][1] = a.y; cbr[m][2] = a.z; cbr[m][3] = a.w;
        cbr[m][4] = b.x; cbr[m][5] = b.y; cbr[m][6] = b.z; cbr[m][7] = b.w;
    }
    // table-store offsets of this thread inside a table: row u, columns c, c + 16, c + 32; the
    // two half-warps write the first two copies in opposite order (different banks)
    const int st_a = u * kRowBytes + (c + (half ? 16 : 0)) * 4;
    const int st_b = u * kRowBytes + (c + (half ? 0 : 16)) * 4;
    const int st_c = u * kRowBytes + (c + 32) * 4;

    // Builds this thread's share of a table.  `r` is the residual of subspace c (paper step B).
    auto build = [&](unsigned char* lutb, const float (&r)[kDsub], float thr, float P, uint32_t* hm) {
#pragma unroll
        for (int m = 0; m < kNE; ++m) {
            float d2 = 0.0f;
#pragma unroll
            for (int j = 0; j < kDsub; ++j) {
                const float tt = __fsub_rn(r[j], cbr[m][j]);
                d2 = __fmaf_rn(tt, tt, d2);
            }
            const int e = u + kEP * m;
            const bool hit = e < ksub && (p.dense || d2 <= thr);
            const float val = hit ? d2 : P;
            unsigned char* row = lutb + m * (kEP * kRowBytes);
            *reinterpret_cast<float*>(row + st_a) = val;
            *reinterpret_cast<float*>(row + st_b) = val;
            *reinterpret_cast<float*>(row + st_c) = val;
            if (DBG && hit) atomicOr(&hm[c * 8 + (e >> 5)], 1u << (e & 31));
        }
    };
    auto load_cent = [&](int cl, float (&cv)[kDsub]) {
        const float4* src = reinterpret_cast<const float4*>(p.cent + (int64_t)cl * d + c * kDsub);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        cv[0] = a.x; cv[1] = a.y; cv[2] = a.z; cv[3] = a.w;
        cv[4] = b.x; cv[5] = b.y; cv[6] = b.z; cv[7] = b.w;
    };
    auto residual = [&](const float (&cv)[kDsub], float (&r)[kDsub]) {
        const float4 a = *reinterpret_cast<const float4*>(qs + c * kDsub);
        const float4 b = *reinterpret_cast<const float4*>(qs + c * kDsub + 4);
        r[0] = __fsub_rn(a.x, cv[0]); r[1] = __fsub_rn(a.y, cv[1]);
        r[2] = __fsub_rn(a.z, cv[2]); r[3] = __fsub_rn(a.w, cv[3]);
        r[4] = __fsub_rn(b.x, cv[4]); r[5] = __fsub_rn(b.y, cv[5]);
        r[6] = __fsub_rn(b.z, cv[6]); r[7] = __fsub_rn(b.w, cv[7]);
    };

    topk_quick_init<kNT>(hist_p);

    for (int64_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int64_t q = item / p.nsplit;
        const int split = (int)(item % p.nsplit);
        const int np_item = (p.nprobe - split + p.nsplit - 1) / p.nsplit;  // probes split, split + nsplit, ...
        __syncthreads();  // the previous item's results have been read out of the candidate buffer
        if (tid < kW) {
            r2[tid] = squared_threshold(p, q, tid);
        } else if (tid >= 32 && tid < 64) {
            reinterpret_cast<float4*>(qs)[tid - 32] = __ldg(reinterpret_cast<const float4*>(p.queries + q * d) + (tid - 32));
        }
        if (DBG && tid == 64) fill_visit_prefix(p, q, vprefix);
        if (tid == 0) *ntrans_p = 0;
        topk_init(t);  // contains a barrier
        const float P = miss_constant(p, r2);
        const float thr = r2[c];

        for (int t0 = 0; t0 < np_item; t0 += kMetaCap) {
            const int nt = min(kMetaCap, np_item - t0);
            // ---- stage the metadata of the tile's clusters (the previous tile ended with a barrier) ----
            if (tid < nt) meta[tid] = load_probe_meta(p, q, split + (t0 + tid) * p.nsplit);
            if (DBG)
                for (int i = tid; i < 2 * kW * 8; i += kNT) hitmask[i] = 0;
            __syncthreads();

            // ---- prologue: table of the tile's first cluster, centroid of the second ----
            float cnext[kDsub];
            {
                float cv[kDsub], r[kDsub];
                load_cent(meta[0].cl, cv);
                if (nt > 1) load_cent(meta[1].cl, cnext);
                residual(cv, r);
                build(lut_gen, r, thr, P, hitmask);
            }
            __syncthreads();

            for (int j = 0; j < nt; ++j) {
                const ProbeMeta m = meta[j];
                const int pi = split + (t0 + j) * p.nsplit;
                const int nblk = (m.len + kPointsPerBlock - 1) / kPointsPerBlock;
                const uint4* cp = reinterpret_cast<const uint4*>(p.codes_il) + m.b0 * 32 + lane;
                // The warp owns blocks warp, warp + 16, ...: `rem` of them are left, `ptr` is this lane's
                // 16 bytes of the next one, `pos` the position of the lane's point in the list.  The
                // first two blocks are requested now and needed after the table build.
                constexpr int kStep = kWarps * 32;   // uint4 elements between two blocks of a warp
                int rem = nblk > warp ? (nblk - warp + kWarps - 1) / kWarps : 0;
                const uint4* ptr = cp + warp * 32;
                int pos = warp * kPointsPerBlock + lane;
                uint4 n0 = make_uint4(0, 0, 0, 0), n1 = make_uint4(0, 0, 0, 0);
                if (rem > 0) n0 = __ldg(ptr);
                if (rem > 1) n1 = __ldg(ptr + kStep);

                if (DBG) {
                    // masks of cluster j are complete (previous barrier); clear the other buffer
                    if (p.masks)
                        for (int i = tid; i < kW * 8; i += kNT)
                            p.masks[(q * p.nprobe + pi) * kW * 8 + i] = hitmask[(j & 1) * kW * 8 + i];
                    for (int i = tid; i < kW * 8; i += kNT) hitmask[((j + 1) & 1) * kW * 8 + i] = 0;
                    __syncthreads();
                }
                // ---- this thread's share of the next cluster's table (steps B, C + selection) ----
                if (j + 1 < nt) {
                    float r[kDsub];
                    residual(cnext, r);
                    if (j + 2 < nt) load_cent(meta[j + 2].cl, cnext);
                    build(lut_gen + ((j + 1) & 1) * kLutBytes, r, thr, P, hitmask + ((j + 1) & 1) * kW * 8);
                }

                // ---- scan the list of cluster j (step D) ----
                const uint32_t bsel = (lut_win + (uint32_t)(j & 1) * kLutBytes) | (uint32_t)(lane * 4);
                const uint32_t* hm = hitmask + (j & 1) * kW * 8;
                while (true) {
                    const uint32_t tau_hi = (uint32_t)(*tau_p >> 32);
                    bool stop = false;   // a candidate of this lane landed at or beyond the soft limit
                    bool halt = false;   // ... of this warp, as seen at the end of a round
                    // one block: 16 look-ups per lane, stage dumps, candidate test
                    auto one = [&](const uint4 cur, const int bpos) {
                        const float acc = gather16(cur, bsel);
                        if (bpos < m.len) {
                            if (DBG) {
                                unsigned long long hs = 0;
                                const uint32_t wv[4] = {cur.x, cur.y, cur.z, cur.w};
#pragma unroll
                                for (int i = 0; i < kW; ++i) {
                                    const uint32_t code = (wv[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                                    const int s = (lane + i) & (kW - 1);
                                    hs |= (unsigned long long)((hm[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
                                }
                                const int64_t vi = vprefix[pi] + bpos;
                                if (vi < p.visit_stride) {
                                    if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                                    if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = acc;
                                    if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[m.p0 + bpos];
                                }
                            }
                            // distance-only test: a tie with the threshold distance is sorted out
                            // at the next compaction, once the id is known
                            if (__float_as_uint(acc) <= tau_hi) {
                                const int slot = atomicAdd(cnt_p, 1);
                                if (slot < kCap) kbuf[slot] = make_key(acc, (uint32_t)(m.p0 + bpos));
                                else atomicOr(p.status, kFlagOverflow);
                                stop |= slot >= kSoftLimit;
                            }
                        }
                    };
                    // Two blocks per round; each code register is refilled right after its block has
                    // been consumed (no copies).  The fill level of the candidate buffer is only
                    // looked at by lanes that push: a warp leaves the loop at the end of a round in
                    // which one of its candidates landed beyond the soft limit, which bounds the
                    // overshoot by 64 candidates per warp.
                    while (rem >= 2 && !halt) {
                        one(n0, pos);
                        if (rem > 2) n0 = __ldg(ptr + 2 * kStep);
                        one(n1, pos + kWarps * kPointsPerBlock);
                        if (rem > 3) n1 = __ldg(ptr + 3 * kStep);
                        ptr += 2 * kStep;
                        pos += 2 * kWarps * kPointsPerBlock;
                        rem -= 2;
                        halt = __any_sync(0xFFFFFFFFu, stop);
                    }
                    if (rem == 1 && !halt) {
                        one(n0, pos);
                        rem = 0;
                        halt = __any_sync(0xFFFFFFFFu, stop);
                    }
                    // the barrier that separates cluster j from cluster j + 1 (table j + 1 complete,
                    // table j free); a set flag means some warp saw the soft limit (it may have
                    // finished its blocks all the same: the buffer is compacted before the next list)
                    if (!__syncthreads_or(rem > 0 || halt)) break;
                    compact_candidates<kNT, kCap>(t, ntrans_p, hist_p, p.k, p.ids);
                }
            }
        }

        emit_topk<kNT, kCap>(p, t, ntrans_p, hist_p, q, split);
    }
}

}  // namespace

cudaError_t launch_scan_pers(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                             cudaStream_t st) {
    const size_t smem = pers_smem_bytes(nprobe, debug);
    int64_t grid = ix->sm_count;
    if (grid > nitems) grid = nitems;
    cudaError_t e;
    if (debug) {
        auto kern = scan_pers16x8_kernel<true>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)grid, kNT, smem, st>>>(sp, nitems);
    } else {
        auto kern = scan_pers16x8_kernel<false>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)grid, kNT, smem, st>>>(sp, nitems);
    }
    return cudaGetLastError();
}

}  // namespace ivfpq

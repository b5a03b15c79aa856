// Warp-specialised persistent kernel for the 16 x 8 product quantizer (16 subspaces of 8
// dimensions, 256 entries): selective L2-LUT construction, list scan and top-k of paper Sec. 2.1
// steps B-D with the selection of Sec. 3.1 / Algorithm 2 and the miss constant of Sec. 4.3.
//
// One CTA of 16 warps per SM, two roles:
//
//   * 8 builder warps hold the whole codebook (128 KB) in registers - thread t owns subspace
//     c = t & 15 and the entries u, u + 16, ... with u = t / 16 - and do nothing but turn
//     (query, cluster) pairs into look-up tables: residual = query - centroid, squared distance
//     to each entry, selected when within the subspace's threshold, else the miss constant;
//   * 8 gather warps stream the codes of the probed lists (one point per lane), sum one table
//     value per subspace and feed the candidates into the CTA's candidate buffer, which they
//     compact and finally rank among themselves.
//
// The register file is split accordingly (setmaxnreg): the CTA starts with 128 registers per
// thread, the builder threads grow to 168 and the gather threads shrink to 88 (the sum must stay
// inside what the CTA was launched with, or the growing side waits forever).  The two roles meet only through a ring of four tables in shared memory
// with a full / empty mbarrier pair per table, so table arithmetic and table gathers overlap
// freely, the builders run up to four clusters ahead (also across queries: the next query's
// tables are built while the gather warps rank the current one), and there is no CTA-wide
// barrier in the steady state.
//
// Table layout: 256 rows (entries) of 256 bytes; a row holds two tables side by side, 32 columns
// each; column x holds the value of subspace x & 15 (two copies).  Lane l looks up, at step i,
// column l ^ i: the 32 lanes of a warp touch 32 different banks whatever the codes are.  The
// code bytes are stored in that visiting order when the index is loaded.  The table region sits
// at shared-window address 0x10000, so one byte-permute forms the address (byte 0: the lane's
// column offset for that step, byte 1: the code) and the table base is the immediate of the
// load: three instructions per look-up.
//
// Every gather warp owns the code blocks b with b = (warp - slot) mod 8 of each list, which
// needs no coordination and evens out over consecutive lists; it keeps four blocks in flight
// across list boundaries.  Candidates carry the position of the point; ids are read when the
// buffer is compacted (topk.cuh).  All waits are bounded: a wait that runs out raises a status
// flag and the kernel runs on to its end without waiting again.
#include <type_traits>

#include "common.cuh"
#include "scan_common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

constexpr int kW = 16;
constexpr int kDsub = 8;
constexpr int kD = kW * kDsub;
constexpr int kBuildThreads = 256;
constexpr int kGatherWarps = 8;
constexpr int kGatherThreads = kGatherWarps * 32;
constexpr int kThreads = kBuildThreads + kGatherThreads;
constexpr int kBuildRegs = 168;
constexpr int kGatherRegs = 88;
constexpr int kNB = 4;                       // tables in the ring
constexpr int kRowBytes = 256;               // one table row (two tables side by side)
constexpr uint32_t kLutWin = 0x10000;        // shared-window address of the table region
constexpr int kLutRegion = 2 * 65536;        // two 64 KB halves, two tables each
constexpr int kEP = kBuildThreads / kW;      // entries per pass (16)
constexpr int kNE = 256 / kEP;               // entries per builder thread (16)
constexpr int kSoftLimit = 1536;             // compaction is requested once this many candidates are buffered
constexpr int kMetaCap = 128;                // clusters whose metadata is staged at a time
constexpr int kDepth = 4;                    // code blocks in flight per gather warp
constexpr unsigned kSpinLimit = 1u << 20;    // bounded wait: attempts of up to ~1 us each
static_assert(kSoftLimit + (kGatherWarps + 1) * 32 <= kTopkCap && IVFPQ_MAX_K < kSoftLimit, "candidate buffer limits");
static_assert(kBuildThreads * kBuildRegs + kGatherThreads * kGatherRegs <= (65536 / kThreads / 8 * 8) * kThreads,
              "the register split must fit the registers the CTA is launched with");
static_assert(kBuildThreads % 128 == 0 && kGatherThreads % 128 == 0, "setmaxnreg works on groups of four warps");

struct GatherMeta {
    long long b0;   // first 32-point code block of the list
    int p0;         // first point of the list (index into ids; ntotal < 2^31)
    int len;        // points in the list (0 when the cluster id or its tables were invalid)
};

struct GatherGroup {
    __device__ __forceinline__ static int tid() { return threadIdx.x - kBuildThreads; }
    __device__ __forceinline__ static void sync() { asm volatile("bar.sync 1, %0;" ::"n"(kGatherThreads) : "memory"); }
};
struct BuildGroup {
    __device__ __forceinline__ static void sync() { asm volatile("bar.sync 2, %0;" ::"n"(kBuildThreads) : "memory"); }
};

// OR of `pred` over the gather warps (named barrier 1).
__device__ __forceinline__ bool gather_or(bool pred) {
    uint32_t out;
    asm volatile(
        "{ .reg .pred p, q; setp.ne.u32 q, %1, 0; bar.red.or.pred p, 1, %2, q; selp.u32 %0, 1, 0, p; }"
        : "=r"(out)
        : "r"((uint32_t)pred), "n"(kGatherThreads)
        : "memory");
    return out != 0;
}

// ---- mbarrier helpers (shared-window addresses) ----
__device__ __forceinline__ void mbar_init(uint32_t a, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(a), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t a) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(a) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t a, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(a), "r"(parity), "r"(1000u)
        : "memory");
    return ok != 0;
}

// Auxiliary shared memory in front of the table region, in bytes.
__host__ __device__ inline int ws_aux_bytes(int nprobe, bool dbg) {
    int b = kTopkCap * 8;                         // candidate keys
    b += 2 * kNB * 8;                             // full / empty mbarriers
    b += 32;                                      // threshold, counters
    b += kQuickWords * 4;                         // compaction histogram
    b += kMetaCap * (int)sizeof(GatherMeta);      // list metadata (gather side)
    b += kMetaCap * 4;                            // cluster ids (builder side)
    b += kD * 4 + 64;                             // query, squared thresholds
    if (dbg) b += kNB * kW * 8 * 4 + (nprobe + 1) * 8;
    return (b + 255) & ~255;
}

struct Shared {
    unsigned long long* kbuf;
    uint32_t full, empty;          // shared-window addresses of the mbarrier arrays
    unsigned long long* tau;
    int* cnt;
    int* ntrans;
    int* dead;
    int* qs;
    GatherMeta* gmeta;
    int* bmeta;
    float* q;
    float* r2;
    uint32_t* hitmask;             // DBG: [kNB][16][8]
    long long* vprefix;            // DBG
    unsigned char* lut;            // generic pointer to shared-window address kLutWin
};

__device__ __forceinline__ Shared carve(unsigned char* smem, uint32_t win) {
    Shared s;
    unsigned char* a = smem;
    s.kbuf = reinterpret_cast<unsigned long long*>(a);
    a += (size_t)kTopkCap * 8;
    s.full = win + (uint32_t)(a - smem);
    s.empty = s.full + kNB * 8;
    a += 2 * kNB * 8;
    s.tau = reinterpret_cast<unsigned long long*>(a);
    s.cnt = reinterpret_cast<int*>(a + 8);
    s.ntrans = s.cnt + 1;
    s.dead = s.cnt + 2;
    a += 32;
    s.qs = reinterpret_cast<int*>(a);
    a += kQuickWords * 4;
    s.gmeta = reinterpret_cast<GatherMeta*>(a);
    a += kMetaCap * sizeof(GatherMeta);
    s.bmeta = reinterpret_cast<int*>(a);
    a += kMetaCap * 4;
    s.q = reinterpret_cast<float*>(a);
    a += kD * 4;
    s.r2 = reinterpret_cast<float*>(a);
    a += 64;
    s.hitmask = reinterpret_cast<uint32_t*>(a);
    s.vprefix = reinterpret_cast<long long*>(a + kNB * kW * 8 * 4);
    s.lut = smem + (kLutWin - win);
    return s;
}

// Bounded wait on an mbarrier phase.  After the first wait that runs out, no wait blocks again.
__device__ __forceinline__ void mbar_wait(uint32_t a, uint32_t parity, int* dead, int* status) {
    if (mbar_try(a, parity)) return;
    for (unsigned i = 0; i < kSpinLimit; ++i) {
        if (mbar_try(a, parity)) return;
        if (*reinterpret_cast<volatile int*>(dead)) return;
    }
    *reinterpret_cast<volatile int*>(dead) = 1;
    atomicOr(status, kFlagTimeout);
}

// Table t (0..3) of the ring: byte offset from the start of the table region.
__host__ __device__ constexpr int table_offset(int t) { return (t >> 1) * 65536 + (t & 1) * 128; }

// One table look-up.  `word` holds four code bytes, `pack` the lane's column offsets (lane ^ i) * 4
// of the same four steps; T = byte of both that belongs to this step.  The permute builds
// {0, 0, code, column offset}; the table base is the immediate.
template <int T, int TABLE>
__device__ __forceinline__ float lut_gather(uint32_t word, uint32_t pack) {
    uint32_t addr;
    float v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(addr) : "r"(word), "r"(pack), "n"(((12 + T) << 12) | ((12 + T) << 8) | (T << 4) | (4 + T)));
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"((int)kLutWin + table_offset(TABLE)) : "memory");
    return v;
}

// Sum of the 16 table values of the lane's point.  Byte i of `cur` = code of subspace (lane ^ i) & 15.
template <int TABLE>
__device__ __forceinline__ float gather16(const uint4 cur, const uint32_t (&pk)[4]) {
    float a0 = lut_gather<0, TABLE>(cur.x, pk[0]);
    float a1 = lut_gather<1, TABLE>(cur.x, pk[0]);
    a0 += lut_gather<2, TABLE>(cur.x, pk[0]);
    a1 += lut_gather<3, TABLE>(cur.x, pk[0]);
    a0 += lut_gather<0, TABLE>(cur.y, pk[1]);
    a1 += lut_gather<1, TABLE>(cur.y, pk[1]);
    a0 += lut_gather<2, TABLE>(cur.y, pk[1]);
    a1 += lut_gather<3, TABLE>(cur.y, pk[1]);
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

// ---------------------------------------------------------------------------------------------
// builder role
// ---------------------------------------------------------------------------------------------
template <bool DBG>
__device__ __forceinline__ void builder_role(const ScanParams& p, const int64_t nitems, const Shared& sh) {
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int c = tid & (kW - 1);
    const int u = tid / kW;
    const int half = lane >> 4;
    const int ksub = p.ksub;

    float cbr[kNE][kDsub];
#pragma unroll
    for (int m = 0; m < kNE; ++m) {
        const int e = u + kEP * m;
        const float4* src = reinterpret_cast<const float4*>(p.cbt + ((size_t)e * kW + c) * kDsub);
        const float4 a = __ldg(src), b = __ldg(src + 1);
        cbr[m][0] = a.x; cbr[m][1] = a.y; cbr[m][2] = a.z; cbr[m][3] = a.w;
        cbr[m][4] = b.x; cbr[m][5] = b.y; cbr[m][6] = b.z; cbr[m][7] = b.w;
    }
    // row u, columns c and c + 16; the two half-warps (rows u, u + 1) write the copies in opposite
    // order so that a warp's 32 stores hit 32 banks
    const int st_a = u * kRowBytes + (c + (half ? 16 : 0)) * 4;
    const int st_b = u * kRowBytes + (c + (half ? 0 : 16)) * 4;

    unsigned n = 0;  // tables built so far (position in the ring)
    for (int64_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int64_t q = item / p.nsplit;
        const int split = (int)(item % p.nsplit);
        const int np_item = (p.nprobe - split + p.nsplit - 1) / p.nsplit;
        BuildGroup::sync();  // the previous item's query, thresholds and cluster ids are no longer read
        if (tid < kW) {
            float v = 0.0f;
            if (!p.dense) {
                const float* rad = p.radius_mode == 1 ? p.radius + q * kW : p.radius;
                const float r = __fmul_rn(rad[tid], p.scale);
                v = __fmul_rn(r, r);
            }
            sh.r2[tid] = v;
        } else if (tid >= 32 && tid < 64) {
            reinterpret_cast<float4*>(sh.q)[tid - 32] = __ldg(reinterpret_cast<const float4*>(p.queries + q * kD) + (tid - 32));
        }
        float P = 0.0f, thr = 0.0f;
        for (int t0 = 0; t0 < np_item; t0 += kMetaCap) {
            const int nt = min(kMetaCap, np_item - t0);
            if (t0 > 0) BuildGroup::sync();
            if (tid < nt) {
                const int pi = split + (t0 + tid) * p.nsplit;
                int cl = p.probe_ids[q * p.nprobe + pi];
                if (cl < 0 || cl >= p.nlist) cl = 0;  // the gather side raises the flag and scans nothing
                sh.bmeta[tid] = cl;
            }
            BuildGroup::sync();
            if (t0 == 0) {
                if (!p.dense) {
                    if (p.miss_penalty >= 0.0f) {
                        P = p.miss_penalty;
                    } else {
#pragma unroll
                        for (int s = 0; s < kW; ++s) P = __fadd_rn(P, sh.r2[s]);
                    }
                }
                thr = sh.r2[c];
            }
            const float4 qa = *reinterpret_cast<const float4*>(sh.q + c * kDsub);
            const float4 qb = *reinterpret_cast<const float4*>(sh.q + c * kDsub + 4);
            float4 ca, cb;
            {
                const float4* src = reinterpret_cast<const float4*>(p.cent + (int64_t)sh.bmeta[0] * kD + c * kDsub);
                ca = __ldg(src);
                cb = __ldg(src + 1);
            }
            for (int j = 0; j < nt; ++j) {
                // residual of this thread's subspace (paper step B); centroid of the next cluster
                float r[kDsub];
                r[0] = __fsub_rn(qa.x, ca.x); r[1] = __fsub_rn(qa.y, ca.y);
                r[2] = __fsub_rn(qa.z, ca.z); r[3] = __fsub_rn(qa.w, ca.w);
                r[4] = __fsub_rn(qb.x, cb.x); r[5] = __fsub_rn(qb.y, cb.y);
                r[6] = __fsub_rn(qb.z, cb.z); r[7] = __fsub_rn(qb.w, cb.w);
                if (j + 1 < nt) {
                    const float4* src = reinterpret_cast<const float4*>(p.cent + (int64_t)sh.bmeta[j + 1] * kD + c * kDsub);
                    ca = __ldg(src);
                    cb = __ldg(src + 1);
                }
                const unsigned t = n & (kNB - 1);
                mbar_wait(sh.empty + t * 8, ((n / kNB) & 1) ^ 1, sh.dead, p.status);  // the gather warps are done with table t
                uint32_t* hm = sh.hitmask + t * kW * 8;
                if (DBG) {
                    for (int i = tid; i < kW * 8; i += kBuildThreads) hm[i] = 0;
                    BuildGroup::sync();
                }
                unsigned char* lutb = sh.lut + table_offset((int)t);
                // ---- steps C + selection: squared distance to each entry, kept when within the threshold ----
#pragma unroll
                for (int m = 0; m < kNE; ++m) {
                    float d2 = 0.0f;
#pragma unroll
                    for (int jj = 0; jj < kDsub; ++jj) {
                        const float tt = __fsub_rn(r[jj], cbr[m][jj]);
                        d2 = __fmaf_rn(tt, tt, d2);
                    }
                    const int e = u + kEP * m;
                    const bool hit = e < ksub && (p.dense || d2 <= thr);
                    const float val = hit ? d2 : P;
                    unsigned char* row = lutb + m * (kEP * kRowBytes);
                    *reinterpret_cast<float*>(row + st_a) = val;
                    *reinterpret_cast<float*>(row + st_b) = val;
                    if (DBG && hit) atomicOr(&hm[c * 8 + (e >> 5)], 1u << (e & 31));
                }
                if (DBG) {
                    BuildGroup::sync();
                    if (p.masks) {
                        const int pi = split + (t0 + j) * p.nsplit;
                        for (int i = tid; i < kW * 8; i += kBuildThreads) p.masks[(q * p.nprobe + pi) * kW * 8 + i] = hm[i];
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(sh.full + t * 8);  // release: the warp's table rows are visible to the waiters
                ++n;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// gather role
// ---------------------------------------------------------------------------------------------
struct CodeBlock {
    uint4 codes;
    int j;     // cluster of the block inside the staged tile; the tile size when there is none
    int blk;
};

// The keys pushed since the last compaction carry the position of the point in the id array;
// replace it by the id (equal distances are ordered by id).  Called by all gather threads after a
// barrier that follows the last push; the first *ntrans keys already hold ids.
__device__ __forceinline__ void translate_new_keys(const TopkState& t, const int* ntrans,
                                                   const int32_t* __restrict__ ids) {
    const int n = min(*t.cnt, kTopkCap);
    for (int i = *ntrans + GatherGroup::tid(); i < n; i += kGatherThreads) {
        const unsigned long long key = t.buf[i];
        const uint32_t id = (uint32_t)__ldg(ids + (uint32_t)(key & 0xFFFFFFFFull));
        t.buf[i] = (key & 0xFFFFFFFF00000000ull) | id;
    }
    // the compaction that follows starts with a barrier
}

__device__ __forceinline__ void compact_candidates(const TopkState& t, const Shared& sh, int k, const int32_t* ids) {
    translate_new_keys(t, sh.ntrans, ids);
    topk_quick_compact<kGatherThreads, GatherGroup>(t, k, sh.qs);
    if (GatherGroup::tid() == 0) *sh.ntrans = *sh.cnt;  // read again only after later barriers
}

template <bool DBG>
__device__ __forceinline__ void gather_role(const ScanParams& p, const int64_t nitems, const Shared& sh) {
    const int gtid = GatherGroup::tid();
    const int lane = gtid & 31;
    const int gw = gtid >> 5;
    TopkState t{sh.kbuf, sh.cnt, sh.tau, sh.qs};

    // column offsets (lane ^ i) * 4 of the 16 steps, four per register
    uint32_t pk[4];
#pragma unroll
    for (int k4 = 0; k4 < 4; ++k4) {
        uint32_t v = 0;
#pragma unroll
        for (int tt = 0; tt < 4; ++tt) v |= (uint32_t)(((lane ^ (4 * k4 + tt)) * 4) & 0xFF) << (8 * tt);
        pk[k4] = v;
    }

    unsigned n = 0;  // tables consumed so far (position in the ring)
    for (int64_t item = blockIdx.x; item < nitems; item += gridDim.x) {
        const int64_t q = item / p.nsplit;
        const int split = (int)(item % p.nsplit);
        const int np_item = (p.nprobe - split + p.nsplit - 1) / p.nsplit;
        GatherGroup::sync();  // the previous item's results have been written, its metadata is no longer read
        if (gtid == 0) {
            *sh.cnt = 0;
            *sh.ntrans = 0;
            *sh.tau = kKeyPad;
        }
        if (DBG && gtid == 32) {
            long long run = 0;
            for (int i = 0; i < p.nprobe; ++i) {
                sh.vprefix[i] = run;
                const int cl = p.probe_ids[q * p.nprobe + i];
                if (cl >= 0 && cl < p.nlist) run += p.list_off[cl + 1] - p.list_off[cl];
            }
            sh.vprefix[p.nprobe] = run;
            if (p.visit_count) p.visit_count[q] = run;
        }

        for (int t0 = 0; t0 < np_item; t0 += kMetaCap) {
            const int nt = min(kMetaCap, np_item - t0);
            // every warp is done with the previous tile's metadata; the warps come here one by one,
            // so this is the same meeting point as a request for compaction
            if (t0 > 0)
                while (gather_or(false)) compact_candidates(t, sh, p.k, p.ids);
            if (gtid < nt) {
                const int pi = split + (t0 + gtid) * p.nsplit;
                const int cl = p.probe_ids[q * p.nprobe + pi];
                GatherMeta m;
                m.b0 = 0;
                m.p0 = 0;
                m.len = 0;
                if (cl < 0 || cl >= p.nlist) {
                    atomicOr(p.status, kFlagBadList);
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
                sh.gmeta[gtid] = m;
            }
            GatherGroup::sync();

            // ---- this warp's blocks of the tile, in order, kDepth of them in flight ----
            int itj = -1, itblk = 0, itnblk = 0;
            const uint4* itcp = nullptr;
            auto next_block = [&]() -> CodeBlock {
                CodeBlock e;
                itblk += kGatherWarps;
                while (itj < nt && itblk >= itnblk) {
                    ++itj;
                    if (itj < nt) {
                        const GatherMeta m = sh.gmeta[itj];
                        itnblk = (m.len + kPointsPerBlock - 1) / kPointsPerBlock;
                        itcp = reinterpret_cast<const uint4*>(p.codes_il) + m.b0 * 32 + lane;
                        // the warp that starts a list rotates from list to list
                        itblk = (int)((gw + kGatherWarps - ((n + (unsigned)itj) % kGatherWarps)) % kGatherWarps);
                    }
                }
                e.j = itj < nt ? itj : nt;
                e.blk = itblk;
                e.codes = make_uint4(0, 0, 0, 0);
                if (itj < nt) e.codes = __ldg(itcp + (int64_t)itblk * 32);
                return e;
            };
            CodeBlock e[kDepth];
#pragma unroll
            for (int i = 0; i < kDepth; ++i) e[i] = next_block();

            for (int j = 0; j < nt; ++j) {
                const unsigned tb = (n + (unsigned)j) & (kNB - 1);
                const uint32_t fullb = sh.full + tb * 8;
                const uint32_t parity = (((n + (unsigned)j) / kNB) & 1);
                // wait for table j; join a compaction that other warps ask for meanwhile
                {
                    unsigned spins = 0;
                    while (!mbar_try(fullb, parity)) {
                        if (*reinterpret_cast<volatile int*>(sh.dead)) break;
                        if (*reinterpret_cast<volatile int*>(sh.cnt) >= kSoftLimit) {
                            if (gather_or(true)) compact_candidates(t, sh, p.k, p.ids);
                            continue;
                        }
                        if (++spins >= kSpinLimit) {
                            *reinterpret_cast<volatile int*>(sh.dead) = 1;
                            atomicOr(p.status, kFlagTimeout);
                            break;
                        }
                    }
                }
                const GatherMeta m = sh.gmeta[j];
                const int pi = split + (t0 + j) * p.nsplit;
                uint32_t tau_hi = (uint32_t)(*sh.tau >> 32);
                const uint32_t* hm = sh.hitmask + tb * kW * 8;

                auto scan_blocks = [&](auto table_tag) {
                    constexpr int TABLE = decltype(table_tag)::value;
                    while (e[0].j == j) {
                        if (*reinterpret_cast<volatile int*>(sh.cnt) >= kSoftLimit) {
                            if (gather_or(true)) compact_candidates(t, sh, p.k, p.ids);
                            tau_hi = (uint32_t)(*sh.tau >> 32);
                            continue;
                        }
                        const uint4 cur = e[0].codes;
                        const int blk = e[0].blk;
#pragma unroll
                        for (int i = 0; i + 1 < kDepth; ++i) e[i] = e[i + 1];
                        e[kDepth - 1] = next_block();
                        const float acc = gather16<TABLE>(cur, pk);
                        const int pos = blk * kPointsPerBlock + lane;
                        if (pos < m.len) {
                            if (DBG) {
                                unsigned long long hs = 0;
                                const uint32_t wv[4] = {cur.x, cur.y, cur.z, cur.w};
#pragma unroll
                                for (int i = 0; i < kW; ++i) {
                                    const uint32_t code = (wv[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                                    const int s = (lane ^ i) & (kW - 1);
                                    hs |= (unsigned long long)((hm[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
                                }
                                const int64_t vi = sh.vprefix[pi] + pos;
                                if (vi < p.visit_stride) {
                                    if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                                    if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = acc;
                                    if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[m.p0 + pos];
                                }
                            }
                            // distance-only test: a tie with the threshold distance is sorted out at
                            // the next compaction, once the id is known
                            if (__float_as_uint(acc) <= tau_hi) {
                                if (!topk_push(t, make_key(acc, (uint32_t)(m.p0 + pos)))) atomicOr(p.status, kFlagOverflow);
                            }
                        }
                    }
                };
                switch (tb) {
                    case 0: scan_blocks(std::integral_constant<int, 0>{}); break;
                    case 1: scan_blocks(std::integral_constant<int, 1>{}); break;
                    case 2: scan_blocks(std::integral_constant<int, 2>{}); break;
                    default: scan_blocks(std::integral_constant<int, 3>{}); break;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(sh.empty + tb * 8);  // this warp no longer reads table tb
            }
            n += (unsigned)nt;
        }

        // ---- every warp has finished the item's lists: compact while somebody still asks, then rank ----
        while (gather_or(false)) compact_candidates(t, sh, p.k, p.ids);
        compact_candidates(t, sh, p.k, p.ids);  // leaves k or a few more keys, ids in place
        GatherGroup::sync();
        const int nkeys = min(*sh.cnt, kTopkCap);
        if (p.nsplit == 1) {
            float* od = p.out_dist + q * p.k;
            int32_t* oi = p.out_ids + q * p.k;
            topk_emit_ranked<kGatherThreads, GatherGroup>(t, nkeys, p.k, [&](int rank, unsigned long long key) {
                od[rank] = __uint_as_float((uint32_t)(key >> 32));
                oi[rank] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
            });
            for (int i = nkeys + gtid; i < p.k; i += kGatherThreads) {
                od[i] = __uint_as_float((uint32_t)(kKeyPad >> 32));
                oi[i] = -1;
            }
        } else {
            unsigned long long* dst = p.partial + (q * p.nsplit + split) * p.k;
            topk_emit_ranked<kGatherThreads, GatherGroup>(t, nkeys, p.k, [&](int rank, unsigned long long key) { dst[rank] = key; });
            for (int i = nkeys + gtid; i < p.k; i += kGatherThreads) dst[i] = kKeyPad;
        }
    }
}

template <bool DBG>
__global__ void __launch_bounds__(kThreads, 1) scan_ws16x8_kernel(const ScanParams p, const int64_t nitems) {
    extern __shared__ __align__(16) unsigned char smem[];
    const uint32_t win = (uint32_t)__cvta_generic_to_shared(smem);
    if (win + (uint32_t)ws_aux_bytes(p.nprobe, DBG) > kLutWin) {  // uniform: the layout does not fit this window offset
        if (threadIdx.x == 0) atomicOr(p.status, kFlagLayout);
        return;
    }
    const Shared sh = carve(smem, win);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNB; ++i) {
            mbar_init(sh.full + i * 8, kBuildThreads / 32);
            mbar_init(sh.empty + i * 8, kGatherWarps);
        }
        *sh.dead = 0;
    }
    for (int i = threadIdx.x; i < kQuickWords; i += kThreads) sh.qs[i] = (i == kQuickBins) ? -1 : 0;
    __syncthreads();
    if (threadIdx.x < kBuildThreads) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kBuildRegs));
        builder_role<DBG>(p, nitems, sh);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kGatherRegs));
        gather_role<DBG>(p, nitems, sh);
    }
}

}  // namespace

cudaError_t launch_scan_ws(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                           cudaStream_t st) {
    (void)nprobe;
    const size_t smem = (size_t)kLutWin + kLutRegion;  // covers the table region for any window offset
    int64_t grid = ix->sm_count;
    if (grid > nitems) grid = nitems;
    cudaError_t e;
    if (debug) {
        auto kern = scan_ws16x8_kernel<true>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)grid, kThreads, smem, st>>>(sp, nitems);
    } else {
        auto kern = scan_ws16x8_kernel<false>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<(unsigned)grid, kThreads, smem, st>>>(sp, nitems);
    }
    return cudaGetLastError();
}

}  // namespace ivfpq

// Rotated-layout variant of the fused selective-LUT / list-scan / top-k kernel.
//
// Same computation as scan.cu (paper Sec. 2.1 steps B-D with the selection of Sec. 4.1 /
// Algorithm 2 and the miss constant of Sec. 5.3), different shared-memory organisation, chosen
// so that the table gathers of a warp never collide on a bank whatever the codes are:
//
//   * the subspaces are split into groups of width w (a power of two, 32 or less); a group's table
//     is stored entry-major, LUT_g[entry][32 columns], and column (copy*w + c) of every row holds
//     the value of subspace s0+c, replicated 32/w times;
//   * a lane (one point per lane) walks its w code bytes of the group in a lane-specific order:
//     at step i it looks up subspace s0 + ((lane ^ i) & (w-1)) in column lane ^ i.  At any step
//     the 32 lanes therefore touch the 32 different columns = 32 different banks;
//   * the code bytes are stored in that rotated order when the index is loaded, so byte i of the
//     lane's vector is the one it needs at step i.
// The table is built with lanes running over the columns of a row (not over entries), reading
// the codebook from an entry-major copy made at load time, so both the codebook loads and the
// table stores are contiguous / conflict-free.
#include <type_traits>

#include "common.cuh"
#include "scan_common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

// Floats of one group table: 256 entries x 32 columns; a group of width 4 or less keeps one
// compact copy (256 x w: its few look-ups may collide on a bank, but it costs 8 KB less per subspace).
__host__ __device__ constexpr int row_stride(int w) { return w <= 4 ? w : 32; }
__host__ __device__ constexpr int group_floats(int w) { return 256 * row_stride(w); }


__host__ __device__ constexpr int lane_bytes(int w) { return w >= 16 ? w : (w == 8 ? 8 : (w > 0 ? 4 : 0)); }

// Paired layout (shapes whose first two groups are 32 and 16 wide): the two tables share rows of
// 256 bytes, [32 columns of group 0 | 32 columns of group 1], at a fixed address of the CTA's
// shared window, so that a look-up address is {code, column offset} put together by one byte
// permute and the base is an immediate of the load.
constexpr int kPairRowFloats = 64;
// shared-window address of the paired tables (64 KB per cluster): behind the auxiliary data, which is
// larger for the instance that works on two clusters at a time (4096 candidate slots, two residuals)
__host__ __device__ constexpr uint32_t pair_win(int nc) { return nc == 2 ? 0xA000u : 0x5000u; }
__host__ __device__ constexpr int cand_cap(int nc) { return nc == 2 ? 2 * kTopkCap : kTopkCap; }

template <int W0, int W1, int W2>
struct Groups {
    static constexpr bool kPaired = (W0 == 32 && W1 == 16);
    static constexpr int kNsub = W0 + W1 + W2;
    static constexpr int kBlockBytes = 32 * (lane_bytes(W0) + lane_bytes(W1) + lane_bytes(W2));
    __host__ __device__ static constexpr int width(int g) { return g == 0 ? W0 : (g == 1 ? W1 : W2); }
    __host__ __device__ static constexpr int s0(int g) { return g == 0 ? 0 : (g == 1 ? W0 : W0 + W1); }
    // byte offset of group g's chunk inside a 32-point block
    // float offset of group g's table inside the table region, and the size of the region
    __host__ __device__ static constexpr int lut_off(int g) {
        if (kPaired) return g == 0 ? 0 : (g == 1 ? 32 : 256 * kPairRowFloats);
        return g == 0 ? 0 : (g == 1 ? group_floats(W0) : group_floats(W0) + group_floats(W1));
    }
    // floats between two rows of group g's table
    __host__ __device__ static constexpr int stride(int g) {
        return (kPaired && g < 2) ? kPairRowFloats : row_stride(width(g));
    }
    static constexpr int kLutFloats = group_floats(W0) + (W1 > 0 ? group_floats(W1) : 0) + (W2 > 0 ? group_floats(W2) : 0);
    __host__ __device__ static constexpr int chunk_off(int g) {
        return 32 * (g == 0 ? 0 : (g == 1 ? lane_bytes(W0) : lane_bytes(W0) + lane_bytes(W1)));
    }
};

// Bytes in front of the tables: candidate keys, residual(s), thresholds, counters, histogram.
__host__ __device__ inline size_t rot_aux_bytes(int d, int nc) {
    return (size_t)cand_cap(nc) * 8 + nc * align_up((size_t)d * 4, 16) + IVFPQ_MAX_NSUB * 4 + 32 + kTopkHistInts * 4;
}

// Dynamic shared memory of a launch.  Paired layout: everything up to the fixed table address
// (whatever the window offset of the allocation turns out to be), the tables, the debug area.
// Inner product: the lists of a tile of probed clusters are scanned as one sequence of blocks.
constexpr int kIpTile = 64;
struct IpProbe {
    long long p0, b0;   // first point and first block of the list
    int len, blk_end;   // points of the list; blocks of the tile up to and including this list
    float base;         // -(q.c)
    int pi;             // probe number, -1: invalid cluster id
};
__host__ __device__ inline size_t rot_smem_bytes(bool paired, int lut_floats, int d, int nprobe, bool dbg, int nc, bool ip = false) {
    size_t b = paired ? (size_t)pair_win(nc) : rot_aux_bytes(d, nc);
    b += (size_t)nc * lut_floats * 4;
    if (dbg) b += (size_t)nc * IVFPQ_MAX_NSUB * 8 * 4 + align_up((size_t)(nprobe + 1) * 8, 16);
    if (ip) b += (size_t)kIpTile * sizeof(IpProbe);
    return b;
}

// Table of one group for NC (query, cluster) pairs of the same query: thread t owns column
// c = t & (W-1) and the entries u, u + NT/W, ... with u = t / W.  Every codebook entry is loaded once
// and measured against the residuals of all NC clusters (the codebook comes through L2: with two
// clusters per pass its traffic per table halves).  lut_step / res_step / hm_step: distance between
// the clusters' tables, residuals and stage-dump masks.
// IP (inner-product index, paper Sec. 4.2): `res_g` is the query itself; an entry is selected when
// |q_s - e|^2 <= R_s^2 + |e|^2 and its slot then holds -(q_s.e), the miss constant otherwise.
template <int W, int DSUB, int NT, bool DBG, int SCORE_T, int NC, int RS = row_stride(W), bool IP = false>
__device__ __forceinline__ void build_group(float* __restrict__ lutg, int lut_step, const float* __restrict__ cbt_g,
                                            const float* __restrict__ res_g, int res_step, const float* __restrict__ r2_g,
                                            int ksub, bool dense, int score, float P, uint32_t* hitmask_g, int hm_step) {
    constexpr int EP = NT / W;      // entries per pass
    constexpr int NCOPY = (RS == kPairRowFloats ? 32 : RS) / W;   // copies within the group's 32 (or w) columns
    const int t = threadIdx.x;
    const int c = t & (W - 1);
    const int u = t / W;
    const int usub = (t & 31) / W;  // which of the warp's entries this lane works on
    float r[NC][DSUB];
#pragma unroll
    for (int k = 0; k < NC; ++k)
#pragma unroll
        for (int j = 0; j < DSUB; ++j) r[k][j] = res_g[k * res_step + c * DSUB + j];
    const float thr = r2_g[c];
#pragma unroll 4   // four codebook loads in flight per thread (the build waits on L2): 2 -> 4 took 4-7 % off the kernel, 8 spills
    for (int e = u; e < 256; e += EP) {
        float d2[NC];
        bool hit[NC];
#pragma unroll
        for (int k = 0; k < NC; ++k) {
            d2[k] = 0.0f;
            hit[k] = false;
        }
        if (e < ksub) {
            const float* ent = cbt_g + ((size_t)e * W + c) * DSUB;
            float ev[DSUB];
            if constexpr (DSUB % 4 == 0) {
#pragma unroll
                for (int j4 = 0; j4 < DSUB / 4; ++j4) {
                    const float4 x = __ldg(reinterpret_cast<const float4*>(ent) + j4);
                    ev[4 * j4] = x.x; ev[4 * j4 + 1] = x.y; ev[4 * j4 + 2] = x.z; ev[4 * j4 + 3] = x.w;
                }
            } else if constexpr (DSUB % 2 == 0) {
#pragma unroll
                for (int j2 = 0; j2 < DSUB / 2; ++j2) {
                    const float2 x = __ldg(reinterpret_cast<const float2*>(ent) + j2);
                    ev[2 * j2] = x.x; ev[2 * j2 + 1] = x.y;
                }
            } else {
#pragma unroll
                for (int j = 0; j < DSUB; ++j) ev[j] = __ldg(ent + j);
            }
#pragma unroll
            for (int k = 0; k < NC; ++k) {
                float en2 = 0.0f, ipv = 0.0f;
#pragma unroll
                for (int j = 0; j < DSUB; ++j) {
                    const float tt = __fsub_rn(r[k][j], ev[j]);
                    d2[k] = __fmaf_rn(tt, tt, d2[k]);
                    if (IP) {
                        en2 = __fmaf_rn(ev[j], ev[j], en2);
                        ipv = __fmaf_rn(r[k][j], ev[j], ipv);
                    }
                }
                if (IP) {
                    hit[k] = dense || d2[k] <= __fadd_rn(thr, en2);
                    d2[k] = -ipv;
                } else {
                    hit[k] = dense || d2[k] <= thr;
                }
            }
        }
#pragma unroll
        for (int k = 0; k < NC; ++k) {
            const float val = IP ? (hit[k] ? d2[k] : P) : table_value<SCORE_T>(score, hit[k], d2[k], thr, P);
            float* row = lutg + k * lut_step + e * RS + c;
#pragma unroll
            for (int it = 0; it < NCOPY; ++it) {
                const int copy = (it + usub) & (NCOPY - 1);  // lanes of a warp write different columns
                row[copy * W] = val;
            }
            if (DBG && hit[k]) atomicOr(&hitmask_g[k * hm_step + c * 8 + (e >> 5)], 1u << (e & 31));
        }
    }
}

// Sum of the table values of one group for the lane's point.  `bytes` holds the lane's code bytes
// of the group in rotated order.
template <int W, bool DBG>
__device__ __forceinline__ void gather_group(const float* __restrict__ lutg, const uint32_t* words, int lane,
                                             int s0, const uint32_t* hitmask, float& acc,
                                             unsigned long long& hs) {
#pragma unroll
    for (int i = 0; i < W; ++i) {
        const uint32_t code = (words[i >> 2] >> (8 * (i & 3))) & 0xFFu;
        acc += lutg[code * row_stride(W) + ((lane ^ i) & (row_stride(W) - 1))];
        if (DBG) {
            const int s = s0 + ((lane ^ i) & (W - 1));
            hs |= (unsigned long long)((hitmask[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
        }
    }
}

// One look-up of the paired tables.  `word` holds four code bytes, `pack` the lane's column offsets
// (lane ^ i) * 4 of the same four steps; T = the byte of both that belongs to this step, G = group.
// The permute builds {0, 0, code, column offset} (the zero bytes are the replicated sign of the
// column offset, which is below 128); the table address is the immediate.
template <int T, int BASE>
__device__ __forceinline__ float pair_gather(uint32_t word, uint32_t pack) {
    uint32_t addr;
    float v;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(addr) : "r"(word), "r"(pack), "n"(((12 + T) << 12) | ((12 + T) << 8) | (T << 4) | (4 + T)));
    asm volatile("ld.shared.f32 %0, [%1+%2];" : "=f"(v) : "r"(addr), "n"(BASE) : "memory");
    return v;
}

// Table values of NW code words (4 NW subspaces of one group, whose 32 columns start at the
// shared-window address BASE) added to two running sums.
template <int NW, int BASE>
__device__ __forceinline__ void pair_gather_words(const uint32_t* words, const uint32_t* pk, float& a0, float& a1) {
#pragma unroll
    for (int j = 0; j < NW; ++j) {
        a0 += pair_gather<0, BASE>(words[j], pk[j]);
        a1 += pair_gather<1, BASE>(words[j], pk[j]);
        a0 += pair_gather<2, BASE>(words[j], pk[j]);
        a1 += pair_gather<3, BASE>(words[j], pk[j]);
    }
}

// Stage dumps: the subspaces of a group in which the lane's point hit a selected entry.
template <int W>
__device__ __forceinline__ void hits_group(const uint32_t* words, int lane, int s0, const uint32_t* hitmask,
                                           unsigned long long& hs) {
#pragma unroll
    for (int i = 0; i < W; ++i) {
        const uint32_t code = (words[i >> 2] >> (8 * (i & 3))) & 0xFFu;
        const int s = s0 + ((lane ^ i) & (W - 1));
        hs |= (unsigned long long)((hitmask[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
    }
}

template <int W>
__device__ __forceinline__ void load_group_codes(const unsigned char* __restrict__ chunk, int lane,
                                                 uint32_t* words) {
    if constexpr (W >= 16) {
#pragma unroll
        for (int v = 0; v < W / 16; ++v) {
            const uint4 x = __ldg(reinterpret_cast<const uint4*>(chunk) + v * 32 + lane);
            words[4 * v + 0] = x.x;
            words[4 * v + 1] = x.y;
            words[4 * v + 2] = x.z;
            words[4 * v + 3] = x.w;
        }
    } else if constexpr (W == 8) {
        const uint2 x = __ldg(reinterpret_cast<const uint2*>(chunk) + lane);
        words[0] = x.x;
        words[1] = x.y;
    } else {
        words[0] = __ldg(reinterpret_cast<const uint32_t*>(chunk) + lane);
    }
}

// NC = clusters per phase: 1 (one table at a time) or 2 (1024 threads, one CTA per SM; the tables of
// two probed clusters are built in one pass over the codebook, then both lists are scanned as one
// sequence of blocks).
// IP: the inner-product index.  One table per query (built from the query, before the first
// cluster) serves all its probed clusters; a point's cost is -(q.c) from the filtering stage plus one
// slot per subspace; keys carry the cost under the order-preserving bit map (costs can be negative)
// and the reported value is the similarity, -cost.
template <int W0, int W1, int W2, int DSUB, int NT, bool DBG, int SCORE_T, int NC, bool IP = false>
__global__ void __launch_bounds__(NT, NT == 512 ? 2 : 1) scan_rot_kernel(const ScanParams p) {
    static_assert(!IP || NC == 1, "the inner-product instance works on one cluster at a time");
    using GR = Groups<W0, W1, W2>;
    constexpr int kWarps = NT / 32;
    constexpr int kCapN = cand_cap(NC);
    constexpr uint32_t kWin = pair_win(NC);
    // bytes between the tables of two clusters (the immediate bases of the paired look-ups follow from it)
    constexpr int kSetBytes = ((GR::kLutFloats * 4 + 255) / 256) * 256;
    // A warp stops after the block in which one of its candidates landed at or beyond the soft limit
    // (at most 32 more per warp): the buffer is then reduced to the k smallest at the next barrier.
    constexpr int kSoft = kCapN - 32 * kWarps;
    static_assert(IVFPQ_MAX_K < kSoft, "candidate buffer too small for the soft limit");
    extern __shared__ __align__(16) unsigned char smem[];
    const int nsub = GR::kNsub;
    const int ksub = p.ksub;
    const int d = p.d;
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int dpad = (int)(align_up((size_t)d * 4, 16) / 4);

    // candidate keys | residual(s) | thresholds | counters | histogram | tables | debug area; in the
    // paired layout the tables start at the fixed window address kWin
    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(smem);
    float* res = reinterpret_cast<float*>(smem + (size_t)kCapN * 8);   // [NC][dpad]
    float* r2 = res + NC * dpad;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(r2 + IVFPQ_MAX_NSUB);
    int* cnt_p = reinterpret_cast<int*>(tau_p + 1);
    int* hist_p = reinterpret_cast<int*>(tau_p + 4);
    size_t lut_at = rot_aux_bytes(d, NC);
    if constexpr (GR::kPaired) {
        const uint32_t win = (uint32_t)__cvta_generic_to_shared(smem);
        if (win + lut_at > kWin) {   // uniform: the layout does not fit this window offset
            if (tid == 0) atomicOr(p.status, kFlagLayout);
            return;
        }
        lut_at = kWin - win;
    }
    float* lut = reinterpret_cast<float*>(smem + lut_at);                                           // [NC] sets of kSetBytes
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(smem + lut_at + (size_t)NC * kSetBytes);       // DBG only: [NC][64][8]
    long long* vprefix = reinterpret_cast<long long*>(hitmask + NC * IVFPQ_MAX_NSUB * 8);           // DBG only
    IpProbe* ipm = reinterpret_cast<IpProbe*>(smem + lut_at + (size_t)NC * kSetBytes +
                                              (DBG ? (size_t)NC * IVFPQ_MAX_NSUB * 8 * 4 + align_up((size_t)(p.nprobe + 1) * 8, 16) : 0));   // IP only
    constexpr int kSetFloats = kSetBytes / 4;
    // paired layout: column offsets (lane ^ i) * 4 of the 32 steps, four per register
    uint32_t pk[GR::kPaired ? 8 : 1];
    if constexpr (GR::kPaired) {
#pragma unroll
        for (int k4 = 0; k4 < 8; ++k4) {
            uint32_t v = 0;
#pragma unroll
            for (int tt = 0; tt < 4; ++tt) v |= (uint32_t)(((lane ^ (4 * k4 + tt)) * 4) & 0xFF) << (8 * tt);
            pk[k4] = v;
        }
    }

    const int64_t q = blockIdx.x / p.nsplit;
    const int split = blockIdx.x % p.nsplit;
    TopkState t{kbuf, cnt_p, tau_p, hist_p, IP ? kKeyPadSigned : kKeyPad};

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
    topk_init(t);
    float P = 0.0f;
    if (!p.dense) {
        if (p.miss_penalty >= 0.0f) {
            P = p.miss_penalty;
        } else {
            for (int s = 0; s < nsub; ++s) P = __fadd_rn(P, r2[s]);
        }
    }

    // the tables of all groups from the vector(s) in `res`
    auto build_tables = [&]() {
        build_group<W0, DSUB, NT, DBG, SCORE_T, NC, GR::stride(0), IP>(lut, kSetFloats, p.cbt, res, dpad, r2, ksub, p.dense, p.score, P,
                                                                  hitmask, IVFPQ_MAX_NSUB * 8);
        if constexpr (W1 > 0)
            build_group<W1, DSUB, NT, DBG, SCORE_T, NC, GR::stride(1), IP>(lut + GR::lut_off(1), kSetFloats,
                                                                      p.cbt + (size_t)GR::s0(1) * 256 * DSUB, res + GR::s0(1) * DSUB, dpad,
                                                                      r2 + GR::s0(1), ksub, p.dense, p.score, P,
                                                                      hitmask + GR::s0(1) * 8, IVFPQ_MAX_NSUB * 8);
        if constexpr (W2 > 0)
            build_group<W2, DSUB, NT, DBG, SCORE_T, NC, row_stride(W2), IP>(lut + GR::lut_off(2), kSetFloats, p.cbt + (size_t)GR::s0(2) * 256 * DSUB,
                                                       res + GR::s0(2) * DSUB, dpad, r2 + GR::s0(2), ksub, p.dense, p.score, P,
                                                       hitmask + GR::s0(2) * 8, IVFPQ_MAX_NSUB * 8);
    };
    if (IP) {
        for (int j = tid; j < d; j += NT) res[j] = p.queries[q * d + j];
        if (DBG)
            for (int i = tid; i < NC * IVFPQ_MAX_NSUB * 8; i += NT) hitmask[i] = 0;
        __syncthreads();
        build_tables();
        __syncthreads();
    }

    // One block of 32 points of the list that starts at block B0 / point P0 and holds LEN points, against the
    // tables of cluster slot K (a compile-time constant: the table bases are immediates); PI = its probe
    // number (stage dumps), BASE = -(q.c) (inner product).  Returns whether the warp has to stop.
    auto scan_block = [&](auto slot_tag, int64_t blk, int64_t B0, int64_t LEN, int64_t P0, int PI, float BASE,
                  unsigned long long tau, uint32_t tau_hi) -> bool {
        constexpr int K = decltype(slot_tag)::value;
        bool stop = false;
        const unsigned char* bp = reinterpret_cast<const unsigned char*>(p.codes_il) + (B0 + blk) * GR::kBlockBytes;
        const float* lutk = lut + K * kSetFloats;
        const uint32_t* hm = hitmask + K * IVFPQ_MAX_NSUB * 8;
        uint32_t w0[W0 >= 4 ? W0 / 4 : 1];
        uint32_t w1[W1 >= 4 ? W1 / 4 : 1];
        uint32_t w2[W2 >= 4 ? W2 / 4 : 1];
        (void)lutk; (void)w1; (void)w2;   // unused in the instances without those groups
        load_group_codes<W0>(bp, lane, w0);
        if constexpr (W1 > 0) load_group_codes<W1>(bp + GR::chunk_off(1), lane, w1);
        if constexpr (W2 > 0) load_group_codes<W2>(bp + GR::chunk_off(2), lane, w2);
        float acc = 0.0f;
        unsigned long long hs = 0;
        if constexpr (GR::kPaired) {
            float a0 = 0.0f, a1 = 0.0f;
            pair_gather_words<W0 / 4, (int)kWin + K * kSetBytes>(w0, pk, a0, a1);
            pair_gather_words<W1 / 4, (int)kWin + K * kSetBytes + 128>(w1, pk, a0, a1);
            acc = a0 + a1;
            if (DBG) {
                hits_group<W0>(w0, lane, 0, hm, hs);
                hits_group<W1>(w1, lane, GR::s0(1), hm, hs);
            }
        } else {
            gather_group<W0, DBG>(lutk, w0, lane, 0, hm, acc, hs);
            if constexpr (W1 > 0) gather_group<W1, DBG>(lutk + GR::lut_off(1), w1, lane, GR::s0(1), hm, acc, hs);
        }
        if constexpr (W2 > 0) gather_group<W2, DBG>(lutk + GR::lut_off(2), w2, lane, GR::s0(2), hm, acc, hs);
        if (IP) acc += BASE;
        const int64_t pos = blk * kPointsPerBlock + lane;
        if (pos < LEN) {
            if (DBG) {
                const int64_t vi = vprefix[PI] + pos;
                if (vi < p.visit_stride) {
                    if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                    if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = IP ? -acc : acc;
                    if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[P0 + pos];
                }
            }
            const uint32_t ab = IP ? ordered_bits(acc) : __float_as_uint(acc);
            if (ab <= tau_hi) {
                const unsigned long long key = ((unsigned long long)ab << 32) | (uint32_t)p.ids[P0 + pos];
                if (key < tau) {
                    const int slot = atomicAdd(cnt_p, 1);
                    if (slot < kCapN) kbuf[slot] = key;
                    else atomicOr(p.status, kFlagOverflow);
                    stop = slot >= kSoft;
                }
            }
        }
        return __any_sync(0xFFFFFFFFu, stop);
    };

    // ---- inner product: the table is the same for every cluster, so nothing separates the lists: a
    //      tile of up to kIpTile probed clusters is staged (one thread per cluster: the chain of
    //      dependent loads from the probe list to the list tables is paid once per tile, not once per
    //      cluster) and its lists are scanned as one sequence of blocks, with a barrier only when the
    //      candidate buffer has to be reduced ----
    if constexpr (IP) {
        const int np_item = (p.nprobe - split + p.nsplit - 1) / p.nsplit;   // probes split, split + nsplit, ...
        for (int t0 = 0; t0 < np_item; t0 += kIpTile) {
            const int nt = min(kIpTile, np_item - t0);
            __syncthreads();   // the previous tile's entries are no longer read
            if (tid < nt) {
                IpProbe m;
                m.pi = split + (t0 + tid) * p.nsplit;
                m.p0 = m.b0 = 0;
                m.len = m.blk_end = 0;
                m.base = 0.0f;
                const int c = p.probe_ids[q * p.nprobe + m.pi];
                if (c < 0 || c >= p.nlist) {
                    atomicOr(p.status, kFlagBadList);
                    m.pi = -1;
                } else {
                    m.p0 = p.list_off[c];
                    const int64_t len = p.list_off[c + 1] - m.p0;
                    m.b0 = p.list_blk[c];
                    const int64_t nblk = p.list_blk[c + 1] - m.b0;
                    if (nblk != (len + kPointsPerBlock - 1) / kPointsPerBlock || len < 0) {
                        atomicOr(p.status, kFlagBadList);
                    } else {
                        m.len = (int)len;
                        m.blk_end = (int)nblk;
                    }
                    m.base = p.probe_d[q * p.nprobe + m.pi];
                }
                ipm[tid] = m;
            }
            __syncthreads();
            if (tid == 0) {
                int run = 0;
                for (int i = 0; i < nt; ++i) {
                    run += ipm[i].blk_end;
                    ipm[i].blk_end = run;
                }
            }
            __syncthreads();
            if (DBG && p.masks) {
                for (int i = tid; i < nt * nsub * 8; i += NT) {
                    const IpProbe& m = ipm[i / (nsub * 8)];
                    if (m.pi >= 0) p.masks[(q * p.nprobe + m.pi) * nsub * 8 + i % (nsub * 8)] = hitmask[i % (nsub * 8)];
                }
            }
            const int total = ipm[nt - 1].blk_end;
            int gb = warp, ci = 0;
            while (true) {
                const unsigned long long tau = *tau_p;
                const uint32_t tau_hi = (uint32_t)(tau >> 32);
                bool halt = false;
#pragma unroll 1
                for (; gb < total && !halt; gb += kWarps) {
                    while (gb >= ipm[ci].blk_end) ++ci;   // gb only grows: the cursor follows it
                    const IpProbe m = ipm[ci];
                    const int first = ci > 0 ? ipm[ci - 1].blk_end : 0;
                    halt = scan_block(std::integral_constant<int, 0>{}, gb - first, m.b0, m.len, m.p0, m.pi, m.base, tau, tau_hi);
                }
                if (!__syncthreads_or(gb < total || halt)) break;
                topk_select<NT, CtaGroup, kCapN>(t, p.k);
            }
        }
    }

    if constexpr (!IP)
    for (int pi0 = split; pi0 < p.nprobe; pi0 += p.nsplit * NC) {
        // ---- the clusters of this phase; an invalid id leaves an empty list behind ----
        int cl[NC];
        int64_t p0[NC], len[NC], b0[NC], nblk[NC];
#pragma unroll
        for (int k = 0; k < NC; ++k) {
            const int pi = pi0 + k * p.nsplit;
            cl[k] = -1;
            p0[k] = len[k] = b0[k] = nblk[k] = 0;
            if (pi < p.nprobe) {
                const int c = p.probe_ids[q * p.nprobe + pi];
                if (c < 0 || c >= p.nlist) {
                    if (tid == 0) atomicOr(p.status, kFlagBadList);
                } else {
                    cl[k] = c;
                    p0[k] = p.list_off[c];
                    len[k] = p.list_off[c + 1] - p0[k];
                    b0[k] = p.list_blk[c];
                    nblk[k] = p.list_blk[c + 1] - b0[k];
                    if (nblk[k] != (len[k] + kPointsPerBlock - 1) / kPointsPerBlock || len[k] < 0) {
                        if (tid == 0) atomicOr(p.status, kFlagBadList);
                        len[k] = nblk[k] = 0;
                    }
                }
            }
        }
        // (the barrier that ended the previous phase's scan makes the tables and `res` free)
        if (!IP) {
#pragma unroll
            for (int k = 0; k < NC; ++k) {
                const int c = cl[k] >= 0 ? cl[k] : 0;   // a table is built for every slot; an empty slot is never scanned
                for (int j = tid; j < d; j += NT) res[k * dpad + j] = __fsub_rn(p.queries[q * d + j], p.cent[(int64_t)c * d + j]);
            }
            if (DBG)
                for (int i = tid; i < NC * IVFPQ_MAX_NSUB * 8; i += NT) hitmask[i] = 0;
            __syncthreads();
        }

        // ---- selective tables, one per group and cluster (inner product: built once, above) ----
        if (!IP) build_tables();
        __syncthreads();
        if (DBG && p.masks) {
#pragma unroll
            for (int k = 0; k < NC; ++k) {
                const int pi = pi0 + k * p.nsplit;
                if (pi < p.nprobe && cl[k] >= 0)
                    for (int i = tid; i < nsub * 8; i += NT)
                        p.masks[(q * p.nprobe + pi) * nsub * 8 + i] = hitmask[k * IVFPQ_MAX_NSUB * 8 + i];
            }
        }

        // ---- scan the lists of this phase as one sequence of blocks: the warp takes blocks warp,
        //      warp + kWarps, ...; block numbers at or beyond nblk[0] belong to the second list ----
        const int64_t nblk_all = NC == 2 ? nblk[0] + nblk[NC - 1] : nblk[0];
        const float base = (IP && pi0 < p.nprobe) ? p.probe_d[q * p.nprobe + pi0] : 0.0f;   // inner product: -(q.c) of the cluster
        int64_t gb = warp;
        while (true) {
            const unsigned long long tau = *tau_p;
            const uint32_t tau_hi = (uint32_t)(tau >> 32);
            bool halt = false;
#pragma unroll 1
            for (; gb < nblk_all && !halt; gb += kWarps) {
                if (NC == 1 || gb < nblk[0])
                    halt = scan_block(std::integral_constant<int, 0>{}, gb, b0[0], len[0], p0[0], pi0, base, tau, tau_hi);
                else
                    halt = scan_block(std::integral_constant<int, NC - 1>{}, gb - nblk[0], b0[NC - 1], len[NC - 1], p0[NC - 1],
                                      pi0 + (NC - 1) * p.nsplit, 0.0f, tau, tau_hi);
            }
            // The barrier that ends the phase (tables free for the next one).  A set flag means that a
            // warp met the soft limit (it may have finished its blocks all the same): the buffer is
            // reduced to the k smallest keys and the scan resumes where it stopped.
            if (!__syncthreads_or(gb < nblk_all || halt)) break;
            topk_select<NT, CtaGroup, kCapN>(t, p.k);
        }
    }

    // the k smallest keys, ascending
    topk_select<NT, CtaGroup, kCapN>(t, p.k);
    __syncthreads();
    {
        const int nk = min(*cnt_p, kCapN);
        int n2 = 2;
        while (n2 < nk) n2 <<= 1;
        for (int i = nk + tid; i < n2; i += NT) kbuf[i] = ~0ull;
        bitonic_sort(kbuf, n2);
    }
    const int n = min(*cnt_p, p.k);
    if (p.nsplit == 1) {
        for (int i = tid; i < p.k; i += NT) {
            const unsigned long long key = i < n ? kbuf[i] : t.pad;
            p.out_dist[q * p.k + i] = IP ? -from_ordered_bits((uint32_t)(key >> 32)) : __uint_as_float((uint32_t)(key >> 32));
            p.out_ids[q * p.k + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
        }
    } else {
        unsigned long long* dst = p.partial + (q * p.nsplit + split) * p.k;
        for (int i = tid; i < p.k; i += NT) dst[i] = i < n ? kbuf[i] : t.pad;
    }
}

template <int W0, int W1, int W2, int DSUB, int NT, bool DBG, int SCORE_T, int NC, bool IP = false>
cudaError_t launch_rot_inst(const ScanParams& sp, int64_t grid, int nprobe, cudaStream_t st) {
    const size_t smem = rot_smem_bytes(Groups<W0, W1, W2>::kPaired, (((Groups<W0, W1, W2>::kLutFloats * 4 + 255) / 256) * 256) / 4, sp.d,
                                       nprobe, DBG, NC, IP);
    auto kern = scan_rot_kernel<W0, W1, W2, DSUB, NT, DBG, SCORE_T, NC, IP>;
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)grid, NT, smem, st>>>(sp);
    return cudaGetLastError();
}

// Instances: stage dumps (score read at run time), one per score otherwise.
template <int W0, int W1, int W2, int DSUB, int NT, int NC>
cudaError_t launch_rot(const ScanParams& sp, int64_t grid, bool debug, int nprobe, cudaStream_t st) {
    if (debug) return launch_rot_inst<W0, W1, W2, DSUB, NT, true, -1, NC>(sp, grid, nprobe, st);
    if (sp.score == IVFPQ_SCORE_HIT_COUNT)
        return launch_rot_inst<W0, W1, W2, DSUB, NT, false, IVFPQ_SCORE_HIT_COUNT, NC>(sp, grid, nprobe, st);
    if (sp.score == IVFPQ_SCORE_REWARD_PENALTY)
        return launch_rot_inst<W0, W1, W2, DSUB, NT, false, IVFPQ_SCORE_REWARD_PENALTY, NC>(sp, grid, nprobe, st);
    return launch_rot_inst<W0, W1, W2, DSUB, NT, false, IVFPQ_SCORE_DISTANCE, NC>(sp, grid, nprobe, st);
}

// Inner product: distances only (one production instance, one with stage dumps).
template <int W0, int W1, int W2, int DSUB, int NT>
cudaError_t launch_rot_ip(const ScanParams& sp, int64_t grid, bool debug, int nprobe, cudaStream_t st) {
    if (debug) return launch_rot_inst<W0, W1, W2, DSUB, NT, true, IVFPQ_SCORE_DISTANCE, 1, true>(sp, grid, nprobe, st);
    return launch_rot_inst<W0, W1, W2, DSUB, NT, false, IVFPQ_SCORE_DISTANCE, 1, true>(sp, grid, nprobe, st);
}

}  // namespace

// Decomposition of nsub into at most three power-of-two group widths (largest first), or false.
bool rot_group_widths(int nsub, int w[3]) {
    w[0] = w[1] = w[2] = 0;
    int rest = nsub, n = 0;
    for (int cand = 32; cand >= 1 && rest > 0; cand >>= 1) {
        while (rest >= cand) {
            if (n == 3) return false;
            w[n++] = cand;
            rest -= cand;
        }
    }
    return rest == 0;
}

int rot_block_bytes(const int w[3]) { return 32 * (lane_bytes(w[0]) + lane_bytes(w[1]) + lane_bytes(w[2])); }

bool rot_supported(int nsub, int dsub) {
    return (nsub == 16 && dsub == 8) || (nsub == 48 && dsub == 2) || (nsub == 50 && dsub == 4) ||
           (nsub == 8 && dsub == 4) || (nsub == 12 && dsub == 2);
}

cudaError_t launch_scan_rot(const ivfpq_index* ix, const ScanParams& sp, int64_t grid, bool debug, int nprobe,
                            cudaStream_t st) {
    // The wide shapes run 512 threads per CTA at 64 registers, two CTAs per SM (32 warps): the table
    // build waits on codebook loads from L2 and needs the warps to hide them.  The other arrangement
    // (IVFPQ_ROT_KERNEL=pair when the index is loaded: 1024 threads, one CTA per SM, the tables of two
    // probed clusters per pass over the codebook) halves the codebook traffic but measured slower
    // (48 x 2: 4.0 -> 5.2 ms, 50 x 4: 12.1 -> 13.8 ms): one CTA's 32 warps meet at every barrier,
    // where two independent CTAs of 16 warps overlap.
    if (ix->metric == IVFPQ_METRIC_IP) {
        if (ix->nsub == 16 && ix->dsub == 8) return launch_rot_ip<16, 0, 0, 8, 512>(sp, grid, debug, nprobe, st);
        if (ix->nsub == 48 && ix->dsub == 2) return launch_rot_ip<32, 16, 0, 2, 512>(sp, grid, debug, nprobe, st);
        if (ix->nsub == 50 && ix->dsub == 4) return launch_rot_ip<32, 16, 2, 4, 512>(sp, grid, debug, nprobe, st);
        if (ix->nsub == 8 && ix->dsub == 4) return launch_rot_ip<8, 0, 0, 4, 256>(sp, grid, debug, nprobe, st);
        if (ix->nsub == 12 && ix->dsub == 2) return launch_rot_ip<8, 4, 0, 2, 256>(sp, grid, debug, nprobe, st);
        return cudaErrorNotSupported;
    }
    const bool pair = ix->rot_pair != 0;
    if (ix->nsub == 48 && ix->dsub == 2)
        return pair ? launch_rot<32, 16, 0, 2, 1024, 2>(sp, grid, debug, nprobe, st) : launch_rot<32, 16, 0, 2, 512, 1>(sp, grid, debug, nprobe, st);
    if (ix->nsub == 50 && ix->dsub == 4)
        return pair ? launch_rot<32, 16, 2, 4, 1024, 2>(sp, grid, debug, nprobe, st) : launch_rot<32, 16, 2, 4, 512, 1>(sp, grid, debug, nprobe, st);
    if (ix->nsub == 8 && ix->dsub == 4) return launch_rot<8, 0, 0, 4, 256, 1>(sp, grid, debug, nprobe, st);
    if (ix->nsub == 12 && ix->dsub == 2) return launch_rot<8, 4, 0, 2, 256, 1>(sp, grid, debug, nprobe, st);
    return cudaErrorNotSupported;
}

}  // namespace ivfpq

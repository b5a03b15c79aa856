// Filtering stage on the 5th-generation tensor cores (paper Sec. 2.1 "Online Search", step A; the
// GEMM form |c|^2 - 2 q.c + |q|^2 of Sec. 5.3, last paragraph).
//
// The tensor cores only *propose*: the nprobe closest clusters are decided by the defining fp32
// arithmetic (sum over dimensions of fma(t, t, acc), t = q_j - c_j, j ascending), because the probe
// lists must not depend on how a GEMM rounds.  Under L2 they work on centred operands (queries and
// centroids minus the centroids' mean: the distance is the same, the norms - and with them the error
// bound of the TF32 products - are smaller); the exact decision keeps the original vectors.
//
//   1. coarse_mma_kernel: approx[q][c] = |c|^2 - 2 q.c for a tile of queries against all centroids.
//      TMA (cp.async.bulk.tensor, 128-byte swizzle) stages fp32 tiles of queries and centroids in
//      shared memory as they are in global memory (both are K-major: the dimension runs fastest);
//      one elected thread issues tcgen05.mma kind::tf32 (128 x 128 x 8 per instruction) into a
//      double-buffered fp32 accumulator in tensor memory; four warps read the accumulator back
//      with tcgen05.ld and write the approximate distances.
//   2. probe_rerank_kernel (one CTA per query): the nprobe-th smallest approximate distance plus
//      twice a rigorous error bound of the TF32 products gives a cut that no true member of the
//      answer can exceed; every centroid under the cut is re-evaluated with the defining
//      arithmetic and the nprobe smallest (distance, cluster id) are returned.  When the cut lets
//      too many centroids through, the CTA evaluates all of them exactly instead.
//      Rows of at most 1024 clusters with few probes take probe_rerank_warp_kernel: the same
//      decision with one warp per query and no block barrier.
//
//   Many clusters, few probes (nlist >= 8192, nprobe <= 64): the [queries][nlist] tile is never
//   written.  A first pass runs the same kernel over the first quarter (few probes: eighth) of the centroids only (at
//   most 4096; a random sample of the clusters: k-means was seeded with random points); probe_bound_kernel takes each
//   query's nprobe-th smallest value of that sample, which is an upper bound of the nprobe-th
//   smallest over all clusters, and adds twice the error bound; the main pass compares every
//   accumulator value with that cut in the epilogue and appends only the survivors (value,
//   cluster) to a short per-query list (a few times nprobe entries), from which
//   probe_rerank_kernel proceeds as it does from a full row.  A list that overflows falls back to
//   the exact evaluation of all clusters for that query.
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the status flag, the roles
// leave their loops, the tensor memory is released and the kernel returns.
#include <cuda.h>

#include "common.cuh"
#include "topk.cuh"

namespace ivfpq {

namespace {

constexpr int kTileM = 128;          // queries per CTA tile (= TMEM lanes)
constexpr int kTileN = 128;          // centroids per MMA tile (= TMEM columns per accumulator)
constexpr int kKBlock = 32;          // fp32 elements per 128-byte swizzle row
constexpr int kTileBytes = kTileM * kKBlock * 4;   // one [128 rows][128 bytes] tile: 16 KB
constexpr int kStages = 8;           // centroid tiles in flight, at most (as many as the shared memory holds beside the query tiles)
constexpr int kMaxKBlocks = 8;       // dimension <= 256
constexpr int kEpiWarps = 8;         // two per tensor-memory lane quarter, 64 columns of the tile each
constexpr int kMmaThreads = 64 + 32 * kEpiWarps;   // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr int kTmemCols = 256;       // two accumulators of 128 columns
constexpr unsigned kSpinLimit = 1u << 22;       // polls of one bounded wait
constexpr unsigned kSpinLimitTest = 1u << 16;   // ... while the test-only fault option is on (about a millisecond)
constexpr int kCandCap = kTopkCap;   // centroids that may pass the cut before the exact fallback
constexpr int kWarpRowMax = 1024;     // clusters whose row one warp keeps in registers (probe_rerank_warp_kernel)
constexpr int kWarpCand = 128;        // clusters under the cut that the warp kernel ranks itself
constexpr int kWarpLowBit = 8;        // the warp kernel's bound is within 2^8 units in the last place of the order statistic
constexpr int kWarpKernelThreads = 128;
constexpr int kStageRow = 36;         // floats per staged slice row: 32 dimensions + padding
__host__ __device__ inline size_t warp_rerank_smem_per_warp(int d) {
    return align_up((size_t)d * 4, 16) + (size_t)kWarpCand * 8 + (size_t)kWarpCand * 4 + (size_t)32 * kStageRow * 4;
}

// ---- PTX wrappers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false (and the abort word set) when it ran out or somebody else gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_word, int* status,
                                          unsigned limit) {
    for (unsigned i = 0; i < limit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_word) return false;
    }
    *abort_word = 1;
    atomicOr(status, kFlagTimeout);
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 128 x 8, TF32 inputs, fp32 accumulation.
__device__ __forceinline__ void tc_mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %4, 0;\n"
        "  tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p; }"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u)
        : "memory");
}
// 32 lanes x 32 consecutive columns of 32-bit accumulators: thread = lane, v[i] = column i.
__device__ __forceinline__ void tc_load_32x32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major [rows][128 bytes] tile with 128-byte swizzle: rows
// are 128 bytes apart, groups of 8 rows 1024 bytes apart; `k_bytes` selects the 32-byte slice of the
// row that one TF32 instruction (K = 8) consumes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t tile_addr, int k_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)(((tile_addr + (uint32_t)k_bytes) >> 4) & 0x3FFFu);   // start address
    d |= (uint64_t)1 << 16;                                              // leading byte offset (16 B; unused here)
    d |= (uint64_t)(1024 >> 4) << 32;                                    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                                              // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                                              // 128-byte swizzle
    return d;
}
// Instruction descriptor: fp32 accumulator, TF32 A and B, both K-major, N = 128, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(kTileN >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);

struct MmaShared {
    unsigned long long q_full;
    unsigned long long full[kStages];
    unsigned long long empty[kStages];
    unsigned long long acc_full[2];
    unsigned long long acc_empty[2];
    uint32_t tmem_base;
    int abort_word;
    float cn[2][kTileN];   // squared norms of the centroids of the tile in work and of the next one
    int epi_stop[2];       // what the epilogue warps agree on after their barrier: somebody gave up
};

// out[(q - q0) * nlist + c] = cnorm[c] - 2 q.c (TF32 products), q in [q0, q0 + nqc), all c.
// grid.x: query tiles of 128, grid.y: centroid-tile groups.
__global__ void __launch_bounds__(kMmaThreads, 1)
coarse_mma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_c,
                  const float* __restrict__ cnorm, int nqc, int nlist, int kblocks, float* __restrict__ out,
                  int* __restrict__ status, int skip_last_load, int ntile_run, int out_stride,
                  const float* __restrict__ cutp, int* __restrict__ ccount, uint2* __restrict__ cand, int ccap, int nstages,
                  int ip) {
    // ip: inner-product filtering (Sec. 4.2): the values are -2 q.c, the norm term is left out.
    // ntile_run: centroid tiles to process (the first ones); out_stride: floats per row of `out`.
    // cutp != null: nothing is written to `out`; values at or under the row's cut are appended to
    // cand[q][ccount[q]++] (up to ccap entries are stored, the count keeps running).
    // Test-only: with skip_last_load the producer of the first CTA leaves out its very last centroid tile
    // (nothing is handed to the copy engine, nothing is left in flight), so the wait for that tile runs
    // out: the way the bounded waits give up is then observable without any fault.
    const unsigned limit = skip_last_load ? kSpinLimitTest : kSpinLimit;
    extern __shared__ __align__(1024) unsigned char dyn[];
    // the swizzled tiles need 1024-byte alignment in the shared window
    const uint32_t dyn_addr = smem_u32(dyn);
    const uint32_t pad = (1024u - (dyn_addr & 1023u)) & 1023u;
    unsigned char* base = dyn + pad;
    const uint32_t q_smem = dyn_addr + pad;                                   // kblocks tiles
    const uint32_t b_smem = q_smem + (uint32_t)kblocks * kTileBytes;          // kStages tiles
    MmaShared* sh = reinterpret_cast<MmaShared*>(base + (size_t)(kblocks + nstages) * kTileBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = blockIdx.x;
    const int ntile = ntile_run;
    volatile int* abort_word = &sh->abort_word;

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&sh->q_full), 1);
        for (int i = 0; i < nstages; ++i) {
            mbar_init(smem_u32(&sh->full[i]), 1);
            mbar_init(smem_u32(&sh->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&sh->acc_full[i]), 1);
            mbar_init(smem_u32(&sh->acc_empty[i]), kEpiWarps);
        }
        sh->abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {  // one warp owns the tensor-memory allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            mbar_expect_tx(smem_u32(&sh->q_full), (uint32_t)kblocks * kTileBytes);
            for (int kb = 0; kb < kblocks; ++kb)
                tma_load_2d(q_smem + kb * kTileBytes, &map_q, kb * kKBlock, qt * kTileM, smem_u32(&sh->q_full));
            unsigned it = 0;
            bool ok = true;
            for (int ct = blockIdx.y; ct < ntile && ok; ct += gridDim.y) {
                for (int kb = 0; kb < kblocks && ok; ++kb, ++it) {
                    const unsigned s = it % (unsigned)nstages;
                    ok = mbar_wait(smem_u32(&sh->empty[s]), ((it / (unsigned)nstages) & 1) ^ 1, abort_word, status, limit);
                    if (!ok) break;
                    if (skip_last_load && blockIdx.x == 0 && blockIdx.y == 0 && ct + (int)gridDim.y >= ntile && kb == kblocks - 1) break;
                    mbar_expect_tx(smem_u32(&sh->full[s]), kTileBytes);
                    tma_load_2d(b_smem + s * kTileBytes, &map_c, kb * kKBlock, ct * kTileN, smem_u32(&sh->full[s]));
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            bool ok = mbar_wait(smem_u32(&sh->q_full), 0, abort_word, status, limit);
            unsigned it = 0, t = 0;
            for (int ct = blockIdx.y; ct < ntile && ok; ct += gridDim.y, ++t) {
                const unsigned buf = t & 1;
                ok = mbar_wait(smem_u32(&sh->acc_empty[buf]), ((t >> 1) & 1) ^ 1, abort_word, status, limit);
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < kblocks && ok; ++kb, ++it) {
                    const unsigned s = it % (unsigned)nstages;
                    ok = mbar_wait(smem_u32(&sh->full[s]), (it / (unsigned)nstages) & 1, abort_word, status, limit);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < kKBlock / 8; ++k)
                        tc_mma_tf32(tmem + buf * kTileN, smem_desc_sw128(q_smem + kb * kTileBytes, k * 32),
                                    smem_desc_sw128(b_smem + s * kTileBytes, k * 32), kInstrDesc, (kb | k) != 0 ? 1u : 0u);
                    tc_commit(smem_u32(&sh->empty[s]));   // the stage is free once these MMAs have read it
                }
                if (ok) tc_commit(smem_u32(&sh->acc_full[buf]));
            }
        }
    } else {
        // ---- epilogue: warp w reads TMEM lanes 32 (w % 4) .. + 31 = query rows of the tile; the two
        //      warps of a lane quarter take 64 columns each.  The squared norms of a tile's centroids are
        //      staged in shared memory one tile ahead (every wait here is exposed: one warp per role). ----
        const int quarter = warp & 3;
        const int chalf = (warp - 2) >> 2;            // 0: columns 0..63, 1: columns 64..127
        const int et = threadIdx.x - 64;              // 0 .. 255 among the epilogue threads
        const int row = quarter * 32 + lane;
        const int q = qt * kTileM + row;
        const float cut = (cutp != nullptr && q < nqc) ? cutp[q] : 0.0f;
        const float kInf = __int_as_float(0x7F800000);
        auto epi_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory"); };
        if (et < kTileN) {
            const int c = blockIdx.y * kTileN + et;
            sh->cn[0][et] = (blockIdx.y < ntile && c < nlist) ? (ip ? 0.0f : __ldg(cnorm + c)) : kInf;
        }
        epi_sync();
        // All epilogue warps meet at a named barrier once per tile, so they must leave the loop in the
        // same iteration: whether somebody gave up is read by one thread before the barrier and by
        // everybody after it (two slots: a slot is rewritten only after the following barrier).
        unsigned t = 0;
        for (int ct = blockIdx.y; ct < ntile; ct += gridDim.y, ++t) {
            const unsigned buf = t & 1;
            float cn_next = kInf;   // this thread's share of the next tile's norms: requested now, stored after the tile
            if (et < kTileN && ct + (int)gridDim.y < ntile) {
                const int c = (ct + (int)gridDim.y) * kTileN + et;
                if (c < nlist) cn_next = ip ? 0.0f : __ldg(cnorm + c);
            }
            const bool ok = mbar_wait(smem_u32(&sh->acc_full[buf]), (t >> 1) & 1, abort_word, status, limit);
            if (ok) {
            tc_fence_after();
            const float* cns = sh->cn[buf];
            // warp-collective: |c|^2 - 2 q.c of the 32 columns of group cc (+inf beyond the last centroid)
            auto values = [&](int cc, float (&val)[32]) {
                uint32_t v[32];
                tc_load_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + buf * kTileN + cc * 32, v);
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(cns + cc * 32 + i);
                    val[i] = fmaf(-2.0f, __uint_as_float(v[i]), x.x);
                    val[i + 1] = fmaf(-2.0f, __uint_as_float(v[i + 1]), x.y);
                    val[i + 2] = fmaf(-2.0f, __uint_as_float(v[i + 2]), x.z);
                    val[i + 3] = fmaf(-2.0f, __uint_as_float(v[i + 3]), x.w);
                }
            };
            if (cutp != nullptr) {
                // Fused decision: only what may belong to the probe list leaves the kernel.  First pass
                // over the warp's two column groups: which values are at or under the row's cut; one
                // counter update per row and half tile (a global atomic per surviving value would be
                // waited for one after the other); second pass over the groups that hold survivors.
                uint32_t masks[2];
                int total = 0;
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    float val[32];
                    values(2 * chalf + g, val);
                    uint32_t pass = 0;
#pragma unroll
                    for (int i = 0; i < 32; ++i) pass |= (val[i] <= cut ? 1u : 0u) << i;   // +inf never passes a finite cut
                    if (q >= nqc) pass = 0;
                    masks[g] = pass;
                    total += __popc(pass);
                }
                int slot = total > 0 ? atomicAdd(ccount + q, total) : 0;
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    if (__any_sync(0xFFFFFFFFu, masks[g] != 0u)) {
                        float val[32];
                        values(2 * chalf + g, val);
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            if ((masks[g] >> i) & 1u) {
                                if (slot < ccap)
                                    cand[(size_t)q * ccap + slot] = make_uint2(__float_as_uint(val[i]), (uint32_t)(ct * kTileN + (2 * chalf + g) * 32 + i));
                                ++slot;
                            }
                        }
                    }
                }
            } else {
#pragma unroll 1
                for (int g = 0; g < 2; ++g) {
                    const int cc = 2 * chalf + g;
                    float val[32];
                    values(cc, val);
                    const int c0 = ct * kTileN + cc * 32;
                    if (q < nqc) {
                        float* dst = out + (size_t)q * out_stride + c0;
                        if (c0 + 32 <= nlist && (out_stride & 3) == 0) {
#pragma unroll
                            for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(val[i], val[i + 1], val[i + 2], val[i + 3]);
                        } else {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (c0 + i < nlist) dst[i] = val[i];
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->acc_empty[buf]));
            }
            if (et < kTileN) sh->cn[buf ^ 1][et] = cn_next;
            if (et == 0) sh->epi_stop[buf] = *abort_word;
            epi_sync();   // the next tile's norms are in place (its buffer was last read two barriers ago)
            if (sh->epi_stop[buf]) break;
        }
    }

    // ---- teardown: everybody is done with tensor memory before it is released ----
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// |c|^2 per centroid (fp32) and the largest of them (as ordered uint bits).
__global__ void __launch_bounds__(256) cnorm_kernel(const float* __restrict__ cent, int nlist, int d,
                                                    float* __restrict__ cnorm, unsigned* __restrict__ cmax_bits) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= nlist) return;
    float s = 0.0f;
    for (int j = 0; j < d; ++j) {
        const float x = cent[(size_t)c * d + j];
        s = fmaf(x, x, s);
    }
    cnorm[c] = s;
    atomicMax(cmax_bits, __float_as_uint(s));
}

// Centring of the proposal's operands (L2 only).  A squared distance does not change when the same
// vector is subtracted from the query and from the centroid, while the error of the TF32 products
// scales with the norms of the factors: the tensor cores therefore work on q - mu and c - mu, mu the
// mean of the centroids (any fixed vector would do; its rounding does not matter).  The exact decision
// keeps the original vectors.
__global__ void __launch_bounds__(256) centroid_mean_kernel(const float* __restrict__ cent, int nlist, int d,
                                                            float* __restrict__ mu) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    float s = 0.0f;
    for (int c = 0; c < nlist; ++c) s += cent[(size_t)c * d + j];
    mu[j] = s / (float)nlist;
}

// out[r][j] = in[r][j] - mu[j]
__global__ void __launch_bounds__(256) subtract_mean_kernel(const float* __restrict__ in, const float* __restrict__ mu,
                                                            int64_t n, int d, float* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = __fsub_rn(in[i], mu[i % d]);
}

// |approx - exact| <= eps for the tile value of one (query, centroid) pair.  qn, cmax: squared norm of
// the query and largest squared norm of a centroid AS THE TENSOR CORES SAW THEM (centred for L2).
// First term: TF32 keeps 10 mantissa bits of each factor (relative 2^-10 each, 2^-9 per product),
// summed over the dimensions by Cauchy-Schwarz and doubled by the factor -2 (inner product: the cost
// is half the tile value).  Second term, fp32 rounding.  L2, centred operands q' = fl(q - mu),
// c' = fl(c - mu): the tensor-core accumulation (d), the two squared norms (d + 1 each), the final
// additions, the exact chain on the other side ((d + 2) on |q - c|^2 <= 2 (|q'|^2 + |c'|^2)) and the
// rounding of the centring itself (2^-22 (|q'|^2 + |c'|^2)), each at most 2^-24 of that magnitude per
// operation: (4 d + 17) 2^-24 (|q'|^2 + |c'|^2), taken as 4 d + 32.  Inner product (not centred): the
// accumulation on both sides, on |q||c|.
__device__ __forceinline__ float proposal_eps(bool ip, float qn, float cmax, int d) {
    const float qc = sqrtf(qn) * sqrtf(cmax);
    return ip ? 0.625f * 0.00390625f * qc + (float)(2 * d + 8) * 5.9604645e-8f * qc
              : 1.25f * 0.00390625f * qc + (float)(4 * d + 32) * 5.9604645e-8f * (qn + cmax);
}

// One CTA per query: cut from the approximate distances, exact re-evaluation of everything under
// the cut, the nprobe smallest (distance, cluster id) ascending.
template <bool IP>
__global__ void __launch_bounds__(256) probe_rerank_kernel(const float* __restrict__ approx, const float* __restrict__ queries,
                                                          const float* __restrict__ cent, const unsigned* __restrict__ cmax_bits,
                                                          int nlist, int d, int nprobe, int64_t q0,
                                                          int32_t* __restrict__ probe_ids, float* __restrict__ probe_d,
                                                          int* __restrict__ status, const uint2* __restrict__ clist,
                                                          const int* __restrict__ ccount, int ccap, const float* __restrict__ mu) {
    // mu != null: the tile values come from centred operands; qn is then |q - mu|^2
    // clist != null: the proposals are the (value, cluster) pairs the filtering epilogue kept for this
    // query instead of a full row; a list that did not fit means: evaluate every cluster exactly.
    extern __shared__ __align__(1024) unsigned char dyn[];
    unsigned long long* buf = reinterpret_cast<unsigned long long*>(dyn);                 // [kTopkCap]
    int* cand = reinterpret_cast<int*>(dyn + (size_t)kTopkCap * 8);                       // [kCandCap]
    float* qs = reinterpret_cast<float*>(cand + kCandCap);                                // [d]
    __shared__ int cnt;
    __shared__ unsigned long long tau;
    __shared__ int hist[kQuickWords];   // also the exact selection's histogram (kTopkHistInts words)
    __shared__ float red[8];
    __shared__ int ncand;
    static_assert(kQuickWords >= kTopkHistInts, "shared histogram words");
    TopkState t{buf, &cnt, &tau, hist, IP ? kKeyPadSigned : kKeyPad};
    const int tid = threadIdx.x;
    const int64_t q = q0 + blockIdx.x;
    const float* row = approx + (size_t)blockIdx.x * nlist;
    const bool from_list = clist != nullptr;
    const uint2* cl = clist + (size_t)blockIdx.x * ccap;
    const int nlisted = from_list ? ccount[blockIdx.x] : 0;
    const int nsrc = from_list ? min(nlisted, ccap) : nlist;
    auto src_val = [&](int i) { return from_list ? __uint_as_float(cl[i].x) : row[i]; };
    auto src_id = [&](int i) { return from_list ? (int)cl[i].y : i; };

    float part = 0.0f;
    for (int j = tid; j < d; j += 256) {
        const float x = queries[q * d + j];
        qs[j] = x;
        const float xc = mu ? __fsub_rn(x, mu[j]) : x;
        part = fmaf(xc, xc, part);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
    if ((tid & 31) == 0) red[tid >> 5] = part;
    if (tid == 0) ncand = 0;
    for (int i = tid; i < kQuickWords; i += 256) hist[i] = (i == kQuickBins) ? -1 : 0;
    topk_init(t);  // contains a barrier
    float qn = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) qn += red[i];
    const float cmax = __uint_as_float(*cmax_bits);
    const float eps = proposal_eps(IP, qn, cmax, d);
    // what the two sides are ranked by: squared distance (tile value + |q|^2, clamped at 0), or the cost -q.c
    auto approx_of = [&](float v) { return IP ? 0.5f * v : fmaxf(v + qn, 0.0f); };
    auto key_of = [&](float x, int id) {
        return IP ? ((unsigned long long)ordered_bits(x) << 32) | (uint32_t)id : make_key(x, (uint32_t)id);
    };
    auto value_of = [&](unsigned long long key) {
        return IP ? from_ordered_bits((uint32_t)(key >> 32)) : __uint_as_float((uint32_t)(key >> 32));
    };

    // exact squared distance by the defining arithmetic (rows are 16-byte aligned, d % 4 == 0)
    auto exact = [&](int c) {
        const float4* cv = reinterpret_cast<const float4*>(cent + (size_t)c * d);
        float a = 0.0f;
        // one thread per centroid (the chain's order is part of the definition); its row comes from
        // L2, so eight 16-byte loads are requested before the first is used
        constexpr int kAhead = 8;
        const int n4 = d >> 2;
        for (int j0 = 0; j0 < n4; j0 += kAhead) {
            float4 cc[kAhead];
#pragma unroll
            for (int u = 0; u < kAhead; ++u) cc[u] = __ldg(cv + min(j0 + u, n4 - 1));
#pragma unroll
            for (int u = 0; u < kAhead; ++u) {
                if (j0 + u < n4) {
                    const float4 qq = *reinterpret_cast<const float4*>(qs + 4 * (j0 + u));
                    float tt;
                    if (IP) {
                        a = __fmaf_rn(qq.x, cc[u].x, a);
                        a = __fmaf_rn(qq.y, cc[u].y, a);
                        a = __fmaf_rn(qq.z, cc[u].z, a);
                        a = __fmaf_rn(qq.w, cc[u].w, a);
                    } else {
                        tt = __fsub_rn(qq.x, cc[u].x); a = __fmaf_rn(tt, tt, a);
                        tt = __fsub_rn(qq.y, cc[u].y); a = __fmaf_rn(tt, tt, a);
                        tt = __fsub_rn(qq.z, cc[u].z); a = __fmaf_rn(tt, tt, a);
                        tt = __fsub_rn(qq.w, cc[u].w); a = __fmaf_rn(tt, tt, a);
                    }
                }
            }
        }
        return IP ? -a : a;
    };

    bool all_exact = nprobe >= nlist || (from_list && (nlisted > ccap || nlisted < nprobe));
    if (!all_exact) {
        // ---- a bound at or above the nprobe-th smallest approximate distance: stream the row
        //      through the buffer, compacting by histogram whenever it could overflow ----
        if (nsrc <= kTopkCap) {
            // the whole row fits the buffer: every key goes to its own slot, no counting, no barriers
            for (int c = tid; c < nsrc; c += 256) buf[c] = key_of(approx_of(src_val(c)), src_id(c));
            if (tid == 0) cnt = nsrc;
        } else {
            for (int base = 0; base < nsrc; base += 256) {
                const int c = base + tid;
                if (c < nsrc) {
                    const unsigned long long key = key_of(approx_of(src_val(c)), src_id(c));
                    if (key < tau) {
                        if (!topk_push(t, key)) atomicOr(status, kFlagOverflow);
                    }
                }
                __syncthreads();
                const int filled = cnt;
                __syncthreads();
                if (filled + 256 > kTopkCap) topk_quick_compact<256, CtaGroup, kTopkCap, IP>(t, nprobe, hist, nprobe + nprobe / 2 + 8);
            }
        }
        // (costs of both signs span most of the bit range: their boundary bin is split again)
        topk_quick_compact<256, CtaGroup, kTopkCap, IP>(t, nprobe, hist, nprobe + nprobe / 2 + 8);   // starts and ends with a barrier
        const float bound = value_of(tau);   // every kept key is below it; +inf when nothing was dropped
        const float cut = bound + 2.0f * eps;
        __syncthreads();
        // ---- everything under the cut ----
        for (int c = tid; c < nsrc; c += 256) {
            if (approx_of(src_val(c)) <= cut) {
                const int pos = atomicAdd(&ncand, 1);
                if (pos < kCandCap) cand[pos] = src_id(c);
            }
        }
        __syncthreads();
        all_exact = ncand > kCandCap;   // uniform
    }
    __syncthreads();
    topk_init(t);
    if (all_exact) {
        for (int base = 0; base < nlist; base += 256) {
            const int c = base + tid;
            if (c < nlist) {
                const unsigned long long key = key_of(exact(c), c);
                if (key < tau) {
                    if (!topk_push(t, key)) atomicOr(status, kFlagOverflow);
                }
            }
            topk_round_end<256>(t, nprobe, 256);
        }
        topk_finalize<256>(t, nprobe);
        for (int i = tid; i < nprobe; i += 256) {
            const unsigned long long key = i < cnt ? buf[i] : t.pad;
            probe_ids[q * nprobe + i] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
            probe_d[q * nprobe + i] = value_of(key);
        }
    } else {
        const int n = ncand;   // nprobe <= n <= kCandCap = buffer size
        for (int i = tid; i < n; i += 256) {
            const int c = cand[i];
            buf[i] = key_of(exact(c), c);
        }
        __syncthreads();
        topk_emit_ranked<256>(t, n, nprobe, [&](int rank, unsigned long long key) {
            probe_ids[q * nprobe + rank] = (int32_t)(uint32_t)(key & 0xFFFFFFFFull);
            probe_d[q * nprobe + rank] = value_of(key);
        });
    }
}

// The same decision for short rows, one warp per query: a row of at most 1024 approximate values
// lives in the warp's registers (32 per lane, as order-preserving bits), the bound at or above the
// nprobe-th smallest comes from a bit-by-bit search with warp-wide counts (no shared histogram, no
// block barrier), the clusters under the cut are evaluated exactly, one per lane, and ranked by
// counting.  32 queries are in flight per SM instead of the 4 of the CTA kernel, whose phases leave
// most of its threads idle on such rows.  More clusters under the cut than the warp's buffer holds
// (kWarpCand) are taken in several passes.
template <bool IP>
__global__ void __launch_bounds__(kWarpKernelThreads, 8) probe_rerank_warp_kernel(
    const float* __restrict__ approx, const float* __restrict__ queries, const float* __restrict__ cent,
    const unsigned* __restrict__ cmax_bits, int nlist, int d, int nprobe, int64_t q0, int nqc,
    int32_t* __restrict__ probe_ids, float* __restrict__ probe_d, const uint2* __restrict__ clist,
    const int* __restrict__ ccount, int ccap, const float* __restrict__ mu) {
    // clist != null: the proposals are the (value, cluster) pairs the filtering epilogue kept for the
    // query (at most ccap <= kWarpRowMax); a list that did not fit, or is shorter than nprobe, means:
    // every cluster is evaluated exactly
    extern __shared__ __align__(1024) unsigned char dyn[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ql = blockIdx.x * (kWarpKernelThreads / 32) + warp;
    if (ql >= nqc) return;   // whole warps; the kernel has no block barrier
    const int64_t q = q0 + ql;
    unsigned char* mine = dyn + (size_t)warp * warp_rerank_smem_per_warp(d);
    float* qs = reinterpret_cast<float*>(mine);                                                   // [d]
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(mine + align_up((size_t)d * 4, 16));   // [kWarpCand]
    int* cand = reinterpret_cast<int*>(keys + kWarpCand);                                         // [kWarpCand]
    float* stage = reinterpret_cast<float*>(cand + kWarpCand);                                    // [32][kStageRow]
    const float* row = approx + (size_t)ql * nlist;
    const bool from_list = clist != nullptr;
    const uint2* cl = clist + (size_t)ql * ccap;
    const int nlisted = from_list ? ccount[ql] : 0;
    const int nsrc = from_list ? min(nlisted, ccap) : nlist;
    auto src_val = [&](int i) { return from_list ? __uint_as_float(cl[i].x) : row[i]; };
    auto src_id = [&](int i) { return from_list ? (int)cl[i].y : i; };

    // the row first: its 32 loads per lane are in flight while the query is staged
    float rv[kWarpRowMax / 32];
#pragma unroll
    for (int j = 0; j < kWarpRowMax / 32; ++j) rv[j] = j * 32 + lane < nsrc ? src_val(j * 32 + lane) : 0.0f;
    float part = 0.0f;
    for (int j = lane; j < d; j += 32) {
        const float x = queries[q * d + j];
        qs[j] = x;
        const float xc = mu ? __fsub_rn(x, mu[j]) : x;   // centred operands: |q - mu|^2
        part = fmaf(xc, xc, part);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
    const float qn = part;
    const float cmax = __uint_as_float(*cmax_bits);
    const float eps = proposal_eps(IP, qn, cmax, d);   // (any order of the |q|^2 sum is covered by its second term)
    __syncwarp();

    // what a cluster is proposed by, as bits whose unsigned order is the order of the values:
    // squared distance (tile value + |q|^2, clamped at 0) or the cost -q.c (half the tile value)
    uint32_t k[kWarpRowMax / 32];
#pragma unroll
    for (int j = 0; j < kWarpRowMax / 32; ++j) {
        const int c = j * 32 + lane;
        uint32_t key = 0xFFFFFFFFu;
        if (c < nsrc) key = IP ? ordered_bits(0.5f * rv[j]) : __float_as_uint(fmaxf(rv[j] + qn, 0.0f));
        k[j] = key;
    }
    // A key at or above the nprobe-th smallest: the bits that all keys share are skipped, the others
    // are fixed from the top with warp-wide counts of the keys below a trial value, down to bit
    // kWarpLowBit or until exactly nprobe keys lie below the trial value.
    uint32_t lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
    for (int j = 0; j < kWarpRowMax / 32; ++j) {
        lo = min(lo, k[j]);
        if (k[j] != 0xFFFFFFFFu) hi = max(hi, k[j]);
    }
    lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    hi = __reduce_max_sync(0xFFFFFFFFu, hi);
    const int top = 31 - __clz(lo ^ hi);                       // highest bit in which two keys differ (-1: none)
    uint32_t prefix = top >= 31 ? 0u : lo & ~((2u << max(top, 0)) - 1u) ;
    if (top < 0) prefix = lo;
    int unknown = top;                                          // bits unknown..0 of the order statistic are open
    bool exact_cut = false;
#pragma unroll 1
    for (int b = top; b >= kWarpLowBit; --b) {
        const uint32_t trial = prefix | (1u << b);
        int cnt = 0;
#pragma unroll
        for (int j = 0; j < kWarpRowMax / 32; ++j) cnt += k[j] < trial ? 1 : 0;
        cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
        unknown = b - 1;
        if (cnt == nprobe) {   // exactly the wanted keys lie below the trial value
            prefix = trial - 1u;
            exact_cut = true;
            break;
        }
        if (cnt < nprobe) prefix = trial;
    }
    const uint32_t bound_key = exact_cut ? prefix : (unknown >= 0 ? prefix | ((2u << unknown) - 1u) : prefix);
    const float bound = IP ? from_ordered_bits(bound_key) : __uint_as_float(bound_key);
    const float cut = bound + 2.0f * eps;

    // ---- the clusters under the cut, in cluster order, `kWarpCand` at a time: exact values by the
    //      defining arithmetic, then the nprobe smallest (value, cluster) so far are kept and the next
    //      clusters join them.  Nearly always one pass.  Fewer than nprobe under the cut can only mean
    //      that the cut is not a number: every cluster is then evaluated. ----
    int total = 0;
#pragma unroll
    for (int j = 0; j < kWarpRowMax / 32; ++j) {
        const float v = IP ? from_ordered_bits(k[j]) : __uint_as_float(k[j]);
        const bool pass = j * 32 + lane < nsrc && v <= cut;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, pass);
        const int pos = total + __popc(bal & ((1u << lane) - 1u));
        if (pass && pos < kWarpCand) cand[pos] = src_id(j * 32 + lane);
        total += __popc(bal);
    }
    bool all = false;
    if (total < nprobe || (from_list && nlisted > ccap)) {
        __syncwarp();
        all = true;
        total = nlist;
        for (int i = lane; i < min(nlist, kWarpCand); i += 32) cand[i] = i;
    }
    const int nslice = (d + 31) >> 5;
    const int n4 = d >> 2;
    int kept = 0, done = 0;
    int m = min(total, kWarpCand);
    while (true) {
        const int cur = kept + m;
        __syncwarp();
        // Exact values, one cluster per lane (the order of a chain is part of the definition).  The
        // centroid rows come from L2: 32 lanes reading 32 different rows would cost one tag look-up
        // per lane and load, so the warp fetches slices of 32 dimensions of 32 rows with contiguous
        // loads (8 lanes per row), passes them through shared memory (rows padded to 36 floats:
        // conflict-free 16-byte reads), and requests the next slice before it works on the current one.
        for (int base = kept; base < cur; base += 32) {
            const int i = base + lane;
            const int c = i < cur ? cand[i] : -1;
            float a = 0.0f;
            float4 nx[8];
            auto request = [&](int sl) {
    #pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int r = base + u * 4 + (lane >> 3);          // row of this lane in load u
                    const int j4 = sl * 8 + (lane & 7);                // its 16-byte piece of the slice
                    nx[u] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    if (r < cur && j4 < n4) nx[u] = __ldg(reinterpret_cast<const float4*>(cent + (size_t)cand[r] * d) + j4);
                }
            };
            request(0);
            for (int sl = 0; sl < nslice; ++sl) {
                __syncwarp();   // the previous slice has been read
    #pragma unroll
                for (int u = 0; u < 8; ++u)
                    *reinterpret_cast<float4*>(stage + (u * 4 + (lane >> 3)) * kStageRow + 4 * (lane & 7)) = nx[u];
                __syncwarp();
                if (sl + 1 < nslice) request(sl + 1);
                if (c >= 0) {
    #pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int j4 = sl * 8 + u;
                        if (j4 < n4) {
                            const float4 cc = *reinterpret_cast<const float4*>(stage + lane * kStageRow + 4 * u);
                            const float4 qq = *reinterpret_cast<const float4*>(qs + 4 * j4);
                            float tt;
                            if (IP) {
                                a = __fmaf_rn(qq.x, cc.x, a);
                                a = __fmaf_rn(qq.y, cc.y, a);
                                a = __fmaf_rn(qq.z, cc.z, a);
                                a = __fmaf_rn(qq.w, cc.w, a);
                            } else {
                                tt = __fsub_rn(qq.x, cc.x); a = __fmaf_rn(tt, tt, a);
                                tt = __fsub_rn(qq.y, cc.y); a = __fmaf_rn(tt, tt, a);
                                tt = __fsub_rn(qq.z, cc.z); a = __fmaf_rn(tt, tt, a);
                                tt = __fsub_rn(qq.w, cc.w); a = __fmaf_rn(tt, tt, a);
                            }
                        }
                    }
                }
            }
            if (c >= 0) keys[i] = IP ? ((unsigned long long)ordered_bits(-a) << 32) | (uint32_t)c : make_key(a, (uint32_t)c);
        }
        __syncwarp();
        done += m;
        // ---- ranks by counting (keys are distinct: they carry the cluster) ----
        const bool last = done >= total;
        unsigned long long* tmp = reinterpret_cast<unsigned long long*>(stage);   // free between passes
        for (int i = lane; i < cur; i += 32) {
            const unsigned long long me = keys[i];
            int rank = 0;
            for (int j = 0; j < cur; ++j) rank += keys[j] < me ? 1 : 0;
            if (rank < nprobe) {
                if (last) {
                    probe_ids[q * nprobe + rank] = (int32_t)(uint32_t)(me & 0xFFFFFFFFull);
                    probe_d[q * nprobe + rank] = IP ? from_ordered_bits((uint32_t)(me >> 32)) : __uint_as_float((uint32_t)(me >> 32));
                } else {
                    tmp[rank] = me;
                }
            }
        }
        if (last) break;
        __syncwarp();   // every rank has been counted: the nprobe smallest move to the front
        for (int i = lane; i < nprobe; i += 32) keys[i] = tmp[i];
        kept = nprobe;
        // the next clusters under the cut, from the row itself (the registers that held it are in use)
        m = min(total - done, kWarpCand - kept);
        if (all) {
            for (int i = lane; i < m; i += 32) cand[kept + i] = done + i;
        } else {
            int run = 0;
#pragma unroll 1
            for (int j = 0; j < kWarpRowMax / 32; ++j) {
                const int i = j * 32 + lane;
                bool pass = false;
                if (i < nsrc) {
                    const float v = IP ? 0.5f * src_val(i) : fmaxf(src_val(i) + qn, 0.0f);
                    pass = v <= cut;
                }
                const unsigned bal = __ballot_sync(0xFFFFFFFFu, pass);
                const int pos = run + __popc(bal & ((1u << lane) - 1u)) - done;
                if (pass && pos >= 0 && pos < m) cand[kept + pos] = src_id(i);
                run += __popc(bal);
            }
        }
        __syncwarp();
    }
}

// One CTA per query: an upper bound of the nprobe-th smallest of the query's `m` sampled values (any m
// clusters: the value is then an upper bound of the nprobe-th smallest over all clusters), plus twice
// the error bound of the approximate values, is the cut the filtering epilogue compares with.  Also
// clears the query's candidate counter.  Values are |c|^2 - 2 q.c (without |q|^2, which is constant
// per query).  m <= 16 * 256: every thread keeps its values in registers, as order-preserving bits.
// Two histogram passes of 256 bins (the value range, then the bin that holds the wanted rank) place
// the bound within 2^-16 of the range above the exact order statistic.
constexpr int kBoundPerThread = 16;
__global__ void __launch_bounds__(256) probe_bound_kernel(const float* __restrict__ sample, int m, const float* __restrict__ queries,
                                                         const unsigned* __restrict__ cmax_bits, int d, int nprobe, int64_t q0,
                                                         float* __restrict__ cutp, int* __restrict__ ccount, int ip,
                                                         const float* __restrict__ mu) {
    __shared__ int hist[256];
    __shared__ int wsum[8];
    __shared__ unsigned mm[2];
    __shared__ int found[2];
    __shared__ float red[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ql = blockIdx.x;
    const float* row = sample + (size_t)ql * m;
    uint32_t ob[kBoundPerThread];
    uint32_t lo = 0xFFFFFFFFu, hi = 0u;
#pragma unroll
    for (int j = 0; j < kBoundPerThread; ++j) {
        const int i = tid + 256 * j;
        ob[j] = i < m ? ordered_bits(row[i]) : 0xFFFFFFFFu;   // beyond the sample: after every real value
        if (i < m) {
            lo = min(lo, ob[j]);
            hi = max(hi, ob[j]);
        }
    }
    float qn = 0.0f;
    for (int j = tid; j < d; j += 256) {
        const float x = queries[(q0 + ql) * d + j];
        const float xc = mu ? __fsub_rn(x, mu[j]) : x;
        qn = fmaf(xc, xc, qn);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) qn += __shfl_xor_sync(0xFFFFFFFFu, qn, o);
    lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    hi = __reduce_max_sync(0xFFFFFFFFu, hi);
    if (tid == 0) {
        mm[0] = 0xFFFFFFFFu;
        mm[1] = 0u;
    }
    hist[tid] = 0;
    __syncthreads();
    if (lane == 0) {
        red[warp] = qn;
        atomicMin(&mm[0], lo);
        atomicMax(&mm[1], hi);
    }
    __syncthreads();
    lo = mm[0];
    hi = mm[1];
    uint32_t base = lo;        // first value of the bin range in work
    uint32_t top = hi;         // every value of interest is <= top
    int need = nprobe;         // rank wanted among the values >= base
    for (int pass = 0; pass < 2; ++pass) {
        const uint32_t range = top - base;
        int shift = 0;   // smallest shift with (range >> shift) < 256
        if (range >= 256u) shift = (32 - __clz(range)) - 8;
#pragma unroll
        for (int j = 0; j < kBoundPerThread; ++j)
            if (ob[j] >= base && ob[j] <= top) atomicAdd(&hist[(ob[j] - base) >> shift], 1);
        __syncthreads();
        const int v = hist[tid];
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += x;
        }
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < warp; ++w) before += wsum[w];
        incl += before;
        if (incl - v < need && need <= incl) {   // exactly one thread: its bin holds the wanted rank
            found[0] = tid;
            found[1] = incl - v;
        }
        hist[tid] = 0;
        __syncthreads();
        const int bin = found[0];
        need -= found[1];
        const uint32_t nbase = base + ((uint32_t)bin << shift);
        const unsigned long long ntop = (unsigned long long)nbase + ((1ull << shift) - 1ull);
        base = nbase;
        top = ntop < (unsigned long long)top ? (uint32_t)ntop : top;
        if (shift == 0) break;   // the bin is a single value (uniform)
    }
    if (tid == 0) {
        qn = 0.0f;
        for (int i = 0; i < 8; ++i) qn += red[i];
        const float kth = from_ordered_bits(top);   // at or above the nprobe-th smallest sampled value
        const float cmax = __uint_as_float(*cmax_bits);
        // error bound of the tile value: |c|^2 - 2 q.c against the squared distance, or -2 q.c against twice the cost
        const float eps = ip ? 2.0f * proposal_eps(true, qn, cmax, d) : proposal_eps(false, qn, cmax, d);
        cutp[ql] = kth + 2.0f * eps + 1e-6f * fabsf(kth);   // the last term: the two sides add |q|^2 in different places
        ccount[ql] = 0;
    }
}

// ---- host side ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
        if (qres != cudaDriverEntryPointSuccess) return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// [rows][d] fp32 row-major, boxes of 128 rows x 32 columns, 128-byte swizzle, zero fill outside.
bool make_map(CUtensorMap* map, const float* ptr, int64_t rows, int d) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * 4};
    const cuuint32_t box[2] = {(cuuint32_t)kKBlock, (cuuint32_t)kTileM};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool coarse_mma_supported(int d, int nlist) {
    return d % 4 == 0 && d >= 4 && (d + kKBlock - 1) / kKBlock <= kMaxKBlocks && nlist >= 1 && encode_tiled_fn() != nullptr;
}

// norms | their maximum | (L2) mean of the centroids | centred centroids
size_t coarse_mma_derived_bytes(int nlist, int d, bool centered) {
    size_t b = align_up((size_t)nlist * 4, 256) + 256;
    if (centered) b += align_up((size_t)d * 4, 256) + align_up((size_t)nlist * d * 4, 256);
    return b;
}

// mu = mean of the centroids, cent_c = cent - mu (derived buffer of an L2 index).
cudaError_t launch_center(const float* cent, int nlist, int d, float* mu, float* cent_c, cudaStream_t st) {
    centroid_mean_kernel<<<(d + 255) / 256, 256, 0, st>>>(cent, nlist, d, mu);
    const int64_t n = (int64_t)nlist * d;
    subtract_mean_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(cent, mu, n, d, cent_c);
    return cudaGetLastError();
}

// Fills cnorm[nlist] and the max word behind it (derived buffer of the index).
cudaError_t launch_cnorm(const float* cent, int nlist, int d, float* cnorm, cudaStream_t st) {
    unsigned* cmax = reinterpret_cast<unsigned*>(reinterpret_cast<char*>(cnorm) + align_up((size_t)nlist * 4, 256));
    cudaError_t e = cudaMemsetAsync(cmax, 0, 4, st);
    if (e != cudaSuccess) return e;
    cnorm_kernel<<<(nlist + 255) / 256, 256, 0, st>>>(cent, nlist, d, cnorm, cmax);
    return cudaGetLastError();
}

constexpr int kSampleMax = 256 * kBoundPerThread;   // clusters of the bound-giving first pass, at most
constexpr int kListCap = 1024;                      // candidate entries kept per query by the fused epilogue

// Clusters of the first pass: a quarter of them (whole tiles, at most kSampleMax), or an eighth when
// the list expected from that smaller sample (nlist * nprobe / sample) still stays within a quarter
// of the list capacity (measured on 16 384 clusters, 32 probes: filtering 0.61 -> 0.56 ms).
static int sample_clusters(int nlist, int nprobe) {
    int m = (nlist / 4) / kTileN * kTileN;
    const int h = (nlist / 8) / kTileN * kTileN;
    if (h >= 8 * kTileN && (int64_t)nlist * nprobe / h <= kListCap / 4) m = h;
    return m > kSampleMax ? kSampleMax : m;
}

// Whether the fused path (no [queries][nlist] tile) serves this shape: many clusters, and an expected
// list (nlist * nprobe / sample, before the widening by the error bound) well under its capacity.
bool coarse_mma_fused(int nlist, int nprobe) {
    if (nlist < 8192) return false;   // measured on 1024 clusters: 0.25 ms against 0.16 ms through full rows
    return (int64_t)nlist * nprobe / sample_clusters(nlist, nprobe) <= kListCap / 4;
}

// Bytes of scratch per query of the fused path: sample row, cut, counter, candidate list.
size_t coarse_mma_fused_bytes_per_query(int nlist, int nprobe) { return (size_t)sample_clusters(nlist, nprobe) * 4 + 8 + (size_t)kListCap * 8; }

// Tensor-core filtering of the queries [q0, q0 + nqc): returns cudaErrorNotSupported when the
// tensor maps cannot be built (the caller then uses the plain kernels).  `tile` is scratch of at
// least nqc * nlist floats (full-tile path) or, with `fused`, nqc * coarse_mma_fused_bytes_per_query() bytes.
cudaError_t launch_coarse_mma(const ivfpq_index* ix, const float* queries, int64_t q0, int nqc, int32_t nprobe, bool fused,
                              float* q_centered, float* tile, int32_t* probe_ids, float* probe_d, int* status, cudaStream_t st,
                              int64_t* launches) {
    // L2 with room for the centred queries (nqc x d floats): the proposal works on centred operands
    const float* mu = (ix->cent_c && q_centered) ? ix->mu : nullptr;
    alignas(64) CUtensorMap map_q, map_c;
    if (!make_map(&map_q, mu ? q_centered : queries + q0 * ix->d, nqc, ix->d)) return cudaErrorNotSupported;
    if (!make_map(&map_c, mu ? ix->cent_c : ix->cent, ix->nlist, ix->d)) return cudaErrorNotSupported;
    if (mu) {
        const int64_t n = (int64_t)nqc * ix->d;
        subtract_mean_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(queries + q0 * ix->d, mu, n, ix->d, q_centered);
        *launches += 1;
    }
    const int kblocks = (ix->d + kKBlock - 1) / kKBlock;
    const int qtiles = (nqc + kTileM - 1) / kTileM;
    const int ntile = (ix->nlist + kTileN - 1) / kTileN;
    // Into how many CTAs the centroid tiles of one query tile are split: one CTA per SM (shared memory),
    // so the grid runs in waves of sm_count CTAs; the split with the fewest (waves x tiles per CTA,
    // one more tile's worth per CTA for its start-up) wins.  (Rounding the split up to "about two
    // waves" gave 308 CTAs on 148 SMs for 22 query tiles: a third wave of 12 CTAs.)
    auto csplit_for = [&](int tiles) {
        int best = 1;
        long best_cost = -1;
        for (int cs = 1; cs <= tiles && cs <= 4 * ix->sm_count; ++cs) {
            const long waves = ((long)qtiles * cs + ix->sm_count - 1) / ix->sm_count;
            const long cost = waves * ((tiles + cs - 1) / cs + 1);
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                best = cs;
            }
        }
        return best;
    };
    int nstages = 12 - kblocks;   // 16 KB tiles: queries + stages within about 200 KB
    if (nstages > kStages) nstages = kStages;
    const size_t smem = 1024 + (size_t)(kblocks + nstages) * kTileBytes + sizeof(MmaShared);
    cudaError_t e = cudaFuncSetAttribute(coarse_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const float* cnorm = ix->cnorm;
    const unsigned* cmax = reinterpret_cast<const unsigned*>(reinterpret_cast<const char*>(cnorm) + align_up((size_t)ix->nlist * 4, 256));
    const size_t smem2 = (size_t)kTopkCap * 8 + (size_t)kCandCap * 4 + align_up((size_t)ix->d * 4, 16);
    const int ip = ix->metric == IVFPQ_METRIC_IP ? 1 : 0;
    e = ip ? cudaFuncSetAttribute(probe_rerank_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2)
           : cudaFuncSetAttribute(probe_rerank_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2);
    if (e != cudaSuccess) return e;
    auto rerank = ip ? probe_rerank_kernel<true> : probe_rerank_kernel<false>;

    if (fused) {   // the caller checked coarse_mma_fused() and sized the scratch for it
        // scratch: [nqc][sample] values | [nqc] cuts | [nqc] counters | [nqc][kListCap] (value, cluster)
        const int nsample = sample_clusters(ix->nlist, nprobe);
        float* sample = tile;
        float* cutp = sample + (size_t)nqc * nsample;
        int* ccount = reinterpret_cast<int*>(cutp + nqc);
        uint2* clist = reinterpret_cast<uint2*>(ccount + nqc);   // 8-byte aligned: 2 nqc words of cuts and counters before it
        const int stile = nsample / kTileN;
        coarse_mma_kernel<<<dim3(qtiles, csplit_for(stile)), kMmaThreads, smem, st>>>(
            map_q, map_c, cnorm, nqc, ix->nlist, kblocks, sample, status, 0, stile, nsample, nullptr, nullptr, nullptr, 0, nstages, ip);
        probe_bound_kernel<<<nqc, 256, 0, st>>>(sample, nsample, queries, cmax, ix->d, nprobe, q0, cutp, ccount, ip, mu);
        coarse_mma_kernel<<<dim3(qtiles, csplit_for(ntile)), kMmaThreads, smem, st>>>(
            map_q, map_c, cnorm, nqc, ix->nlist, kblocks, nullptr, status, 0, ntile, 0, cutp, ccount, clist, kListCap, nstages, ip);
        if (nprobe <= kWarpCand / 2 && nprobe < ix->nlist && kListCap <= kWarpRowMax) {
            constexpr int kWarpsPerCta = kWarpKernelThreads / 32;
            const size_t smem3 = (size_t)kWarpsPerCta * warp_rerank_smem_per_warp(ix->d);
            auto by_warp_kernel = ip ? probe_rerank_warp_kernel<true> : probe_rerank_warp_kernel<false>;
            by_warp_kernel<<<(nqc + kWarpsPerCta - 1) / kWarpsPerCta, kWarpKernelThreads, smem3, st>>>(
                nullptr, queries, ix->cent, cmax, ix->nlist, ix->d, nprobe, q0, nqc, probe_ids, probe_d, clist, ccount, kListCap, mu);
        } else {
            rerank<<<nqc, 256, smem2, st>>>(nullptr, queries, ix->cent, cmax, ix->nlist, ix->d, nprobe, q0, probe_ids,
                                                          probe_d, status, clist, ccount, kListCap, mu);
        }
        *launches += 4;
        return cudaGetLastError();
    }
    coarse_mma_kernel<<<dim3(qtiles, csplit_for(ntile)), kMmaThreads, smem, st>>>(map_q, map_c, cnorm, nqc, ix->nlist, kblocks, tile, status,
                                                                                 ix->test_fault, ntile, ix->nlist, nullptr, nullptr, nullptr, 0, nstages, ip);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    // short rows and few probes: one warp per query
    if (ix->nlist <= kWarpRowMax && nprobe <= kWarpCand / 2 && nprobe < ix->nlist) {
        constexpr int kWarpsPerCta = kWarpKernelThreads / 32;
        const size_t smem3 = (size_t)kWarpsPerCta * warp_rerank_smem_per_warp(ix->d);
        auto by_warp_kernel = ip ? probe_rerank_warp_kernel<true> : probe_rerank_warp_kernel<false>;
        by_warp_kernel<<<(nqc + kWarpsPerCta - 1) / kWarpsPerCta, kWarpKernelThreads, smem3, st>>>(
            tile, queries, ix->cent, cmax, ix->nlist, ix->d, nprobe, q0, nqc, probe_ids, probe_d, nullptr, nullptr, 0, mu);
    } else {
        rerank<<<nqc, 256, smem2, st>>>(tile, queries, ix->cent, cmax, ix->nlist, ix->d, nprobe, q0, probe_ids,
                                                      probe_d, status, nullptr, nullptr, 0, mu);
    }
    *launches += 2;
    return cudaGetLastError();
}

}  // namespace ivfpq

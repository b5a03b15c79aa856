// Internal declarations shared by the translation units of the IVFPQ library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ivfpq.h"

namespace ivfpq {

constexpr int kPointsPerBlock = 32;  // points per interleaved code block (one warp, one point per lane)
constexpr int kScanThreads = 256;    // threads per scan CTA (= max entries per codebook)
constexpr int kTopkCap = 2048;       // candidate buffer slots per CTA (>= IVFPQ_MAX_K + kScanThreads)
constexpr int kMapChunk = 8192;      // points per chunk of the entry -> points map (entry_map.cu)

// Device status bits (workspace status word).
constexpr int kFlagBadList = 1;   // a probed cluster id or code block was out of range and was skipped
constexpr int kFlagOverflow = 2;  // the candidate buffer would have overflowed; the candidate was dropped
constexpr int kFlagTimeout = 4;   // a bounded wait between cooperating warps ran out
constexpr int kFlagLayout = 8;    // the kernel's shared-memory layout does not fit the window offset it was given
constexpr int kFlagMap = 16;      // the entry -> points map disagrees with the codes (stage-dump instances check this)

inline __host__ __device__ size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace ivfpq

// Host-side handle.  All pointers are device pointers into caller-owned memory.
struct ivfpq_index {
    int32_t d, nlist, nsub, dsub, ksub;
    int32_t metric;           // IVFPQ_METRIC_*
    int64_t ntotal;
    const float* cent;        // [nlist][d]
    const float* cb;          // [nsub][ksub][dsub]
    const int32_t* ids;       // [ntotal] list-contiguous
    // derived tables (inside the caller's derived buffer)
    const int64_t* list_off;  // [nlist+1] point offsets (index into ids)
    const int64_t* list_blk;  // [nlist+1] offsets in 32-point code blocks
    const uint32_t* codes_il; // interleaved codes, see relayout.cu
    int32_t nw;               // 4-byte code words per point (nsub rounded up to a multiple of 4)
    int32_t vec16;            // 1: words grouped by four (16-byte lane loads), 0: single words
    int64_t nblocks;          // total 32-point blocks
    // rotated layout (scan_rot.cu): subspace groups of power-of-two width, codes stored per lane in
    // the lane's own visiting order, codebook copied entry-major per group
    int32_t pers_warps;       // 16 x 8 shape: warps per CTA of the persistent kernel (16: short lists, 32: long lists)
    int32_t rot;              // 1: rotated layout in use
    int32_t rot_pair;         // wide rotated shapes: 1 = two clusters per table-build pass (scan_rot.cu)
    int32_t gw[3];            // group widths, largest first, 0 = unused
    int32_t block_bytes;      // bytes of one 32-point code block in the rotated layout
    const float* cbt;         // [group][entry 0..255][column][dsub]
    const float* cnorm;       // [nlist] squared centroid norms + their maximum (tensor-core filtering), or null
    const float* mu;          // [d] mean of the centroids, and
    const float* cent_c;      // [nlist][d] centroids minus that mean: the tensor-core proposal of an L2 index works on these
                              // (cnorm then holds their norms); null for the inner product
    // entry -> points map (entry_map.cu; 16 x 8 shape under L2 only, null otherwise)
    const int32_t* chunk_first;  // [nlist+1] chunks before each list
    const uint32_t* map_off;     // [nchunks][nsub][256]: first position | point count << 16 of every entry
    const uint16_t* map_pos;     // [ntotal * nsub]
    int64_t nchunks;
    int32_t map_group;        // lanes that share one entry's point list in the scatter (4, 8, 16 or 32)
    int32_t sparse_scan;      // IVFPQ_OPT_SPARSE_SCAN
    int32_t test_fault;       // IVFPQ_OPT_TEST_FAULT
    int64_t max_list_len;
    const uint32_t* blk_min;     // [nblocks] smallest id (unsigned) of every 32-point block
    // host state
    int32_t device;
    int32_t sm_count;
    int32_t nsplit_opt;       // 0 = automatic
    mutable int64_t last_launches;
    int32_t timing;           // IVFPQ_OPT_TIMING
    mutable cudaEvent_t ev[3];  // start, after filtering, end (created lazily)
    mutable bool ev_ready, ev_recorded;
    // host entry point: a copy stream and events that let the transfers of one slice of the batch
    // overlap with the search of another (created on first use)
    mutable cudaStream_t copy_stream;
    mutable cudaEvent_t pipe_ev[12];
    mutable bool pipe_ready;
};

namespace ivfpq {

// Shape served by the persistent kernels (scan16x8.cu).
// Scratch of the filtering stage for chunks of `qchunk` queries: a [qchunk][nlist] tile of proposed
// values (or the fused path's smaller per-query scratch) and the centred queries of the chunk.
inline size_t coarse_region_bytes(const ivfpq_index* ix, int64_t qchunk) {
    return (size_t)qchunk * ((size_t)ix->nlist * 4 + (size_t)ix->d * 4) + 256;
}
inline bool pers_shape(const ivfpq_index* ix) { return ix->rot && ix->nsub == 16 && ix->dsub == 8; }

struct SearchArgs {
    const ivfpq_index* ix;
    const float* queries;     // dev [nq][d]
    int64_t nq;
    int32_t nprobe;
    int32_t k;
    bool dense;
    const float* radius;      // dev
    int32_t radius_mode;
    float scale;
    float miss_penalty;
    int32_t score;            // IVFPQ_SCORE_*
    float* out_dist;
    int32_t* out_ids;
    // dumps (debug build of the kernels), all optional
    bool debug;
    int32_t* probe_ids_out;
    float* probe_d_out;
    uint32_t* masks;
    int64_t* visit_count;
    int64_t visit_stride;
    uint64_t* visit_hits;
    float* visit_dist;
    int32_t* visit_ids;
};

// Workspace carve-up (all offsets 256-byte aligned).
struct WorkspaceLayout {
    size_t status_off;      // 4 x int32
    size_t probe_ids_off;   // [nq][nprobe] int32
    size_t probe_d_off;     // [nq][nprobe] fp32
    size_t coarse_off;      // [qchunk][nlist] fp32
    size_t partial_off;     // [nq][nsplit][k] uint64 keys (nsplit > 1 only)
    size_t total;
    int64_t qchunk;
    int32_t nsplit;
};

WorkspaceLayout plan_workspace(const ivfpq_index* ix, int64_t nq, int32_t nprobe, int32_t k);

// Launchers (return cudaError_t of the launch; count launches into *launches).
cudaError_t launch_block_min_id(const ivfpq_index* ix, uint32_t* blk_min, cudaStream_t st);
cudaError_t launch_relayout(const ivfpq_index* ix, const uint8_t* codes, uint32_t* codes_il, float* cbt,
                            cudaStream_t st);
bool rot_group_widths(int nsub, int w[3]);
int rot_block_bytes(const int w[3]);
bool rot_supported(int nsub, int dsub);
// Tensor-core filtering (coarse_mma.cu).
bool coarse_mma_supported(int d, int nlist);
size_t coarse_mma_derived_bytes(int nlist, int d, bool centered);
bool coarse_mma_fused(int nlist, int nprobe);
size_t coarse_mma_fused_bytes_per_query(int nlist, int nprobe);
cudaError_t launch_entry_map(const ivfpq_index* ix, const uint8_t* codes, cudaStream_t st);
cudaError_t launch_cnorm(const float* cent, int nlist, int d, float* cnorm, cudaStream_t st);
cudaError_t launch_center(const float* cent, int nlist, int d, float* mu, float* cent_c, cudaStream_t st);
cudaError_t launch_coarse_mma(const ivfpq_index* ix, const float* queries, int64_t q0, int nqc, int32_t nprobe, bool fused,
                              float* q_centered, float* tile, int32_t* probe_ids, float* probe_d, int* status, cudaStream_t st,
                              int64_t* launches);
cudaError_t launch_coarse(const ivfpq_index* ix, const float* queries, int64_t nq, int32_t nprobe,
                          float* coarse_tile, int64_t qchunk, int32_t* probe_ids, float* probe_d,
                          int* status, cudaStream_t st, int64_t* launches);
cudaError_t launch_entry_stats(const ivfpq_index* ix, const uint8_t* codes, const float* queries, int64_t nq,
                               const int64_t* nbr, int k, int32_t* usage, unsigned long long* rank_hist, int* status,
                               cudaStream_t st);
cudaError_t launch_negate(const float* in, float* out, int64_t n, cudaStream_t st);
cudaError_t launch_thresholds(const float* queries, int64_t nq, int nsub, const ivfpq_threshold_model_t* m,
                              float* radius, cudaStream_t st);
cudaError_t launch_thresholds_knn(const ivfpq_index* ix, const float* queries, int64_t nq, const int32_t* probe0, int kth,
                                  int degree, const float* coef, float* radius, int* status, cudaStream_t st);
cudaError_t launch_scan(const SearchArgs& a, const WorkspaceLayout& wl, char* ws, cudaStream_t st,
                        int64_t* launches);

}  // namespace ivfpq

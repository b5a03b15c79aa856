// Parameters shared by the list-scan kernels.
#pragma once

#include "common.cuh"

namespace ivfpq {

struct ScanParams {
    const float* cent;
    const float* cb;
    const float* cbt;
    const int32_t* ids;
    const uint32_t* blk_min;      // smallest id of every 32-point block
    const uint32_t* codes_il;
    const int64_t* list_off;
    const int64_t* list_blk;
    const int32_t* chunk_first;   // entry -> points map (entry_map.cu), null when the index has none
    const uint32_t* map_off;
    const uint16_t* map_pos;
    int map_group;
    int d, nlist, nsub, dsub, ksub, nw;
    int vec16;   // generic layout: 1 = code words grouped by four (16-byte lane loads)
    const float* queries;
    const int32_t* probe_ids;
    const float* probe_d;   // filtering value per probe; inner-product path: -(q.c), the start of every sum
    int nprobe;
    const float* radius;
    int radius_mode;
    float scale;
    float miss_penalty;
    int score;   // IVFPQ_SCORE_*; 0 for the dense search
    int dense;
    int k;
    int nsplit;
    float* out_dist;
    int32_t* out_ids;
    unsigned long long* partial;
    int* status;
    int* work;   // zeroed per launch: the persistent kernels draw their items beyond the first from it
    // stage dumps (DBG instantiations only)
    uint32_t* masks;
    int64_t* visit_count;
    int64_t visit_stride;
    unsigned long long* visit_hits;
    float* visit_dist;
    int32_t* visit_ids;
};

// What a table slot holds for an entry at squared distance d2 from the residual projection, given
// whether it was selected (`hit`: d2 <= thr, always true for the dense search).  Distances: the
// squared distance, or the miss constant P (paper Sec. 5.3).  Count scores (Sec. 5.4): 0 / 1 for
// selected / not selected; with the inner sphere of half the radius 0 / 1 / 2 for inside the inner
// sphere / between the two / outside both.  The list scan sums slots, whatever they hold.
// SCORE_T >= 0: a kernel instance compiled for that score; SCORE_T < 0: the score is read at run time
// (stage-dump instances, generic kernel).  The choice is made per launch, not per entry: with the
// score tested for every entry the table build of the 16 x 8 kernel cost 9 % of the whole search,
// that of the 50 x 4 kernel 15 %.
template <int SCORE_T = -1>
__device__ __forceinline__ float table_value(int score, bool hit, float d2, float thr, float P) {
    const int sc = SCORE_T >= 0 ? SCORE_T : score;
    if (sc == IVFPQ_SCORE_DISTANCE) return hit ? d2 : P;
    if (sc == IVFPQ_SCORE_HIT_COUNT) return hit ? 0.0f : 1.0f;
    return !hit ? 2.0f : (d2 <= __fmul_rn(0.25f, thr) ? 0.0f : 1.0f);
}

// Rotated-layout scan (scan_rot.cu); returns cudaErrorNotSupported when the index shape has no
// specialised instance.
cudaError_t launch_scan_rot(const ivfpq_index* ix, const ScanParams& sp, int64_t grid, bool debug,
                            int nprobe, cudaStream_t st);

// Sparsity-aware scan of the 16 x 8 quantizer through the entry -> points map (scan16x8_map.cu).
cudaError_t launch_scan16x8_map(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                                 cudaStream_t st);

// Persistent scan for the 16 x 8 quantizer, 16 or 32 warps per SM (scan16x8.cu).
cudaError_t launch_scan16x8(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                             cudaStream_t st);

}  // namespace ivfpq

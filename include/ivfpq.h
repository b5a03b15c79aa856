/*
 * ivfpq.h - C ABI of the B200 (sm_100a) sparsity-aware IVFPQ query library.
 *
 * The library runs the online search phase of an IVFPQ index on one GPU:
 *   (1) filtering: squared-L2 distances from each query to the IVF centroids, the nprobe
 *       closest clusters are kept (paper Sec. 2.1 "Online Search", step A);
 *   (2) L2-LUT construction for every (query, probed cluster): residual = query - centroid,
 *       squared distance from each residual projection to each codebook entry (steps B, C);
 *       in the sparsity-aware search only the entries within the threshold radius of the
 *       projection are selected (Sec. 4.1; Algorithm 2, whose ray/sphere test decides exactly
 *       "distance <= thres * thres_scale");
 *   (3) distance calculation: every point of a probed cluster accumulates the table values of
 *       its codes; a subspace whose entry was not selected contributes the large constant P
 *       instead (Sec. 2.1 step D; Sec. 5.3, paragraph after Algorithm 2); then the k
 *       smallest (distance, id) pairs per query (Sec. 2.1, last paragraph).
 *
 * Naming: nsub = number of PQ subspaces (the paper's D/M), dsub = dimensions per subspace (the
 * paper's M), ksub = entries per codebook (the paper's E, at most 256: codes are bytes),
 * nlist = IVF clusters (C), nprobe = probed clusters per query (nprobs).
 * All distances are SQUARED L2 (Eq. "metric").  All floating point is fp32.
 *
 * Inner-product similarity (metric = IVFPQ_METRIC_IP; Sec. 4.2 "Inner Product Similarity Support"):
 *   (1) filtering keeps the nprobe clusters with the LARGEST inner product q.c;
 *   (2) the table is built from the query's own projection q_s (with residual codes the similarity
 *       splits into q.c plus q_s.e per subspace, so one table serves all probed clusters); the
 *       sphere of entry e has radius sqrt(R^2 + |e|^2), R the subspace's threshold: the entry is
 *       selected when |q_s - e|^2 <= R^2 + |e|^2, and its table value is q_s.e (the paper recovers
 *       it from the hit time as (|q_s|^2 + |e|^2 - |q_s - e|^2) / 2);
 *   (3) similarity = q.c + sum of the selected table values - m * P for m unselected subspaces
 *       (miss_penalty P, default sum of (radius*scale)^2); the k LARGEST (similarity, then smaller
 *       id) per query, padded with (-inf, -1).
 *   out_dist, probe_d and the dumps then hold similarities.  Defining arithmetic: inner products
 *   and |e|^2 as one fused multiply-add per dimension, ascending; |q_s - e|^2 as for L2; the test
 *   compares with the fp32 sum R^2 + |e|^2.  The count scores, ivfpq_probe_static, the entry ->
 *   points map and the persistent 16 x 8 kernels are L2-only; an inner-product index of a shape
 *   with a conflict-free code layout is served by that layout's scan kernel, other shapes by the
 *   generic one (filtering goes through the same tensor-core proposal + exact decision as L2).
 *
 * Conventions for every entry point:
 *   - returns IVFPQ_OK (0) or a negative IVFPQ_ERR_* code; never throws, never aborts;
 *   - "dev" pointers are device memory owned by the caller (e.g. torch tensors) that must stay
 *     alive until the work enqueued on `stream` has finished; "host" pointers are host memory;
 *   - the library allocates no device memory (except where an entry point says otherwise): index
 *     arrays, derived tables, workspace, queries and outputs all belong to the caller;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream); calls are
 *     asynchronous on it unless stated otherwise;
 *   - there is no CPU fallback: without a CUDA device every compute call fails with IVFPQ_ERR_CUDA.
 */
#ifndef IVFPQ_H
#define IVFPQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IVFPQ_OK 0
#define IVFPQ_ERR_INVALID_ARGUMENT (-1) /* null pointer, non-positive size, bad offsets        */
#define IVFPQ_ERR_UNSUPPORTED (-2)      /* ksub > 256, nsub > 64, dsub > 16, k > 1024, nprobe > nlist ... */
#define IVFPQ_ERR_WORKSPACE (-3)        /* workspace or derived buffer too small / misaligned     */
#define IVFPQ_ERR_CUDA (-4)             /* a CUDA runtime call or kernel launch failed            */
#define IVFPQ_ERR_DEVICE_FLAG (-5)      /* a kernel raised its bounds / bounded-wait error flag   */
#define IVFPQ_ERR_STATIC_LIMIT (-6)     /* index too large for the scratch built into the library */

#define IVFPQ_METRIC_L2 0
#define IVFPQ_METRIC_IP 1
#define IVFPQ_MAX_K 1024
#define IVFPQ_MAX_NPROBE 1024
#define IVFPQ_MAX_NSUB 64
#define IVFPQ_MAX_DSUB 16

typedef struct ivfpq_index ivfpq_index_t; /* opaque host-side handle */

/* Description of a trained, encoded index (the conventional IVFPQ offline phase, Sec. 2.1 /
 * Algorithm 1 without the ray-tracing scene and without the entry->points map). */
typedef struct {
    int32_t d;      /* vector dimension, = nsub * dsub                                   */
    int32_t nlist;  /* IVF clusters                                                      */
    int32_t nsub;   /* PQ subspaces, 1..64                                               */
    int32_t dsub;   /* dimensions per subspace, 1..16                                    */
    int32_t ksub;   /* entries per codebook, 1..256                                      */
    int32_t metric; /* IVFPQ_METRIC_L2 (squared L2) or IVFPQ_METRIC_IP (inner product)    */
    int64_t ntotal; /* encoded points                                                    */
    const float* coarse_centroids; /* dev  [nlist][d]                                    */
    const float* codebooks;        /* dev  [nsub][ksub][dsub], trained on residuals      */
    const int64_t* list_offsets;   /* HOST [nlist+1], CSR offsets into codes/ids; copied */
    const uint8_t* codes;          /* dev  [ntotal][nsub], list-contiguous               */
    const int32_t* ids;            /* dev  [ntotal], list-contiguous, original ids >= 0  */
} ivfpq_index_desc_t;

/* Bytes of caller-owned device memory that ivfpq_index_load needs for derived tables (codes
 * re-laid-out in 32-point interleaved blocks, list tables, the smallest id of every block, for the
 * tensor-core filtering the centroids' squared norms and, under L2, a copy of the centroids with their
 * mean subtracted; for the 16 x 8 shape under L2 also the
 * inverted index from codebook entries to points of Algorithm 1, 2 bytes per code byte plus
 * 16 KB per 8192 points of a list).  0 on invalid descriptions. */
size_t ivfpq_index_derived_bytes(const ivfpq_index_desc_t* desc);

/* Validates the description, builds the derived tables in `derived_dev` (256-byte aligned, at
 * least ivfpq_index_derived_bytes) with kernels enqueued on `stream`, and returns a handle.
 * After the stream work completes the search path reads coarse_centroids, codebooks, ids and
 * derived_dev, but no longer desc->codes.  The handle itself is host memory owned by the
 * library until ivfpq_index_free. */
int ivfpq_index_load(const ivfpq_index_desc_t* desc, void* derived_dev, size_t derived_bytes,
                     void* stream, ivfpq_index_t** out);
int ivfpq_index_free(ivfpq_index_t* index);

/* Radius parameters of the sparsity-aware search.  The threshold of subspace s for query q is
 * radius[s] (mode 0) or radius[q*nsub + s] (mode 1), times `scale` (the user scaling factor,
 * thres_scale in Algorithm 2); an entry is selected when its squared distance to the residual
 * projection is <= (radius*scale)^2.  miss_penalty is the constant P added per subspace whose
 * entry was not selected; a negative value asks for the default P = sum over subspaces of
 * (radius*scale)^2 of that query, which ranks points first by number of missed subspaces.
 *
 * `score` chooses what a point is ranked by (Sec. 5.4 "Aggressive Approximation: hit count-based
 * Method"; the -H / -L / -M configurations of Sec. 6.1).  Selection, probing and the top-k rule
 * ((value, id) ascending, padded with (+inf, -1)) are the same for all three:
 *   IVFPQ_SCORE_DISTANCE        value = S + m * P as described above (miss_penalty applies).
 *   IVFPQ_SCORE_HIT_COUNT       value = number of subspaces whose entry was NOT selected
 *                               (nsub - hit count): more hits rank first.
 *   IVFPQ_SCORE_REWARD_PENALTY  every sphere has an inner sphere of half the radius; per subspace
 *                               0 when the entry is within the inner sphere (reward +1), 1 when only
 *                               within the outer one, 2 when outside both (penalty -1);
 *                               value = the sum = nsub - (rewards - penalties).  Inner test:
 *                               squared distance <= 0.25f * (radius*scale)^2.
 * The count values are small integers, exact in fp32; miss_penalty is ignored for them. */
#define IVFPQ_SCORE_DISTANCE 0
#define IVFPQ_SCORE_HIT_COUNT 1
#define IVFPQ_SCORE_REWARD_PENALTY 2
typedef struct {
    const float* radius; /* dev; mode 0: [nsub], mode 1: [nq][nsub] */
    int32_t mode;
    float scale;
    float miss_penalty;
    int32_t score;       /* IVFPQ_SCORE_*; other values: IVFPQ_ERR_INVALID_ARGUMENT */
} ivfpq_radius_t;

/* Dynamic threshold model (Sec. 4.1 "Determining Proper Threshold"): per 2-d subspace a grid x grid
 * map of cell densities (number of base projections in the cell / cell area) and a polynomial that
 * maps a density to a threshold.  All arrays are device memory owned by the caller. */
typedef struct {
    int32_t grid;          /* cells per axis, 1..4096 (the paper uses 100)                        */
    int32_t degree;        /* polynomial degree, 0..8                                              */
    const float* density;  /* dev [nsub][grid][grid]: row = cell along the second coordinate       */
    const float* origin;   /* dev [nsub][2]: lower corner of the grid, 8-byte aligned              */
    const float* inv_cell; /* dev [nsub][2]: 1 / cell size along each coordinate, 8-byte aligned   */
    const float* coef;     /* dev [nsub][degree + 1]: coefficients, ascending powers               */
} ivfpq_threshold_model_t;

/* Query-specific thresholds (Algorithm 2: thres = poly_regressor(density_map(x, y))):
 * radius_out[q][s] = max(0, polynomial_s(density_s[cell of (queries[q][2s], queries[q][2s+1])])),
 * cell = floor((coordinate - origin) * inv_cell) clamped to the grid (an undefined coordinate falls
 * into cell 0).  The projection is the query's own (the centroid is not subtracted, as in
 * Algorithm 2).  The polynomial is evaluated in fp32 by Horner's rule from the highest power, one
 * fused multiply-add per coefficient.  The result is the radius array of ivfpq_search_sparse in
 * mode 1 ([nq][nsub], before the user's scale).  Only for indexes with 2-d subspaces (dsub == 2,
 * the paper's setting), grid and degree within the limits above and nq <= 2^24:
 * IVFPQ_ERR_UNSUPPORTED otherwise; null or misaligned pointers: IVFPQ_ERR_INVALID_ARGUMENT.
 * queries dev [nq][d], 8-byte aligned; radius_out dev [nq][nsub].  Asynchronous on `stream`;
 * allocates nothing. */
int ivfpq_query_thresholds(const ivfpq_index_t* index, const float* queries, int64_t nq,
                           const ivfpq_threshold_model_t* model, float* radius_out, void* stream);

/* Query-specific thresholds for subspaces of any width.  The density map above is a 2-d grid; for
 * wider subspaces the local density around the query's projection is measured by how close its
 * kth-nearest codebook entry is (the codebook is a k-means quantizer of the residual projections,
 * so its entries crowd where the data does), and, as in Sec. 4.1, a per-subspace regression
 * polynomial turns the measurement into the threshold:
 *   radius_out[q][s] = max(0, polynomial_s(v)),  v = sqrt(kth smallest over the entries e of
 *   |r_s - e|^2),  r = query - its nearest cluster centroid (ties to the smaller cluster id).
 * Squared distances by the table arithmetic (fused multiply-add chain over ascending dimensions),
 * correctly rounded square root, Horner evaluation from the highest power with one fused
 * multiply-add per coefficient.  coef dev [nsub][degree + 1], ascending powers; with (0, 1) the
 * threshold is the kth-nearest-entry distance itself (the mean of its square over queries is what the
 * static radius calibration uses).  1 <= kth <= ksub, 0 <= degree <= 8, nq <= 2^24, L2 indexes:
 * IVFPQ_ERR_UNSUPPORTED otherwise.  The nearest clusters come from the filtering stage with one
 * probe, which needs `workspace` of ivfpq_search_workspace_bytes(index, nq, 1, 1); queries as for
 * the search calls.  Asynchronous on `stream`; allocates nothing. */
int ivfpq_query_thresholds_knn(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t kth,
                               int32_t degree, const float* coef, float* radius_out, void* workspace,
                               size_t workspace_bytes, void* stream);

/* Entry usage and locality statistics of each query's neighbours (Sec. 3.2 "Sparsity of Codebook
 * Entries Used by Top-k Neighbors", Sec. 3.3 "Spatial Locality of Codebook Entries Used by Top-k
 * Neighbors"); an analysis tool for choosing radii, not a step of the search.
 *   codes         dev [ntotal][nsub]: the list-contiguous codes the index was loaded from (the
 *                 handle keeps only a re-laid-out copy)
 *   neighbor_pos  dev [nq][k]: positions into `codes` of each query's neighbours (normally its
 *                 exact top-100), -1 = none; 1 <= k <= IVFPQ_MAX_K
 *   usage_out     dev [nq][nsub]: distinct entries of codebook s among the query's neighbours (the
 *                 paper's usage ratio is this / ksub)
 *   rank_hist     dev [nsub][ksub] unsigned 64-bit, ACCUMULATED into (zero it first): one count per
 *                 (query, neighbour, subspace) at r = the number of entries ordered before the
 *                 neighbour's own entry by (squared distance to the query's residual projection
 *                 against the centroid of the neighbour's list, entry number); the running sum
 *                 over r is the CDF of Sec. 3.3.  Distances in the search's fp32 arithmetic.
 *   flags         dev, one int32, OR-ed into (zero it first): non-zero afterwards when a position
 *                 >= ntotal or a code >= ksub was met (that neighbour or subspace was skipped).
 * Asynchronous on `stream`; allocates nothing. */
int ivfpq_entry_stats(const ivfpq_index_t* index, const uint8_t* codes, const float* queries, int64_t nq,
                      const int64_t* neighbor_pos, int32_t k, int32_t* usage_out,
                      unsigned long long* rank_hist, int32_t* flags, void* stream);

/* Workspace (dev, 256-byte aligned) needed by one search call of this shape. */
size_t ivfpq_search_workspace_bytes(const ivfpq_index_t* index, int64_t nq, int32_t nprobe, int32_t k);

/* Conventional (dense) IVFPQ search: every codebook entry is selected.
 * queries dev [nq][d], 16-byte aligned; out_dist dev [nq][k] ascending; out_ids dev [nq][k]; ties are ordered by
 * ascending id; when fewer than k points were visited the tail is (+inf, -1). */
int ivfpq_search_dense(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                       int32_t k, float* out_dist, int32_t* out_ids, void* workspace,
                       size_t workspace_bytes, void* stream);

/* Sparsity-aware search (threshold-based selective L2-LUT, Sec. 4.1 / Algorithm 2, followed
 * by the distance calculation of Sec. 5.3).  Same outputs as the dense search. */
int ivfpq_search_sparse(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                        const ivfpq_radius_t* radius, int32_t k, float* out_dist, int32_t* out_ids,
                        void* workspace, size_t workspace_bytes, void* stream);

/* End-to-end variants with HOST query and result buffers (pinned memory recommended): copy the
 * queries to the device, search, copy distances and ids back, all enqueued on `stream`.  The
 * staging areas live in the caller's workspace, whose size is given by
 * ivfpq_search_host_workspace_bytes.  `radius` (NULL = dense search) still points to a struct
 * whose `radius` array is device memory.
 * Batches of 2048 queries or more are processed in two slices: a copy stream that the
 * handle creates on first use (with a few events: host-side resources, no device memory) brings
 * the slices' queries in and takes the first slice's results out while `stream` searches the
 * second.  Everything is ordered with respect to `stream`: work enqueued on it after this call
 * sees the results in the host buffers; the device status word covers all slices.  Use pinned
 * host buffers for the copies to overlap.  Calls on one handle must not be issued from several
 * host threads at once. */
size_t ivfpq_search_host_workspace_bytes(const ivfpq_index_t* index, int64_t nq, int32_t nprobe, int32_t k);
int ivfpq_search_host(const ivfpq_index_t* index, const float* queries_host, int64_t nq, int32_t nprobe,
                      const ivfpq_radius_t* radius, int32_t k, float* out_dist_host,
                      int32_t* out_ids_host, void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream` and reports the device-side status word of the last search that used
 * `workspace`: IVFPQ_OK, IVFPQ_ERR_DEVICE_FLAG (a kernel found an out-of-range list id, code
 * block or candidate count and skipped the access) or IVFPQ_ERR_CUDA. */
int ivfpq_sync_status(const ivfpq_index_t* index, void* workspace, void* stream);

/* Tuning knobs (host-side state of the handle; not thread-safe against concurrent searches).
 *   IVFPQ_OPT_NSPLIT: number of CTAs that share one query's probe list (0 = automatic:
 *   1 for large batches, more when nq alone cannot fill the GPU).  Results do not depend on it. */
#define IVFPQ_OPT_NSPLIT 1
/*   IVFPQ_OPT_TIMING: 1 = record CUDA events around the filtering stage and around the
 *   LUT+scan(+merge) stage of every search (the events are created once, on the first timed
 *   call); 0 = off (default).  Read them with ivfpq_last_stage_ms. */
#define IVFPQ_OPT_TIMING 2
/*   IVFPQ_OPT_SPARSE_SCAN: which list scan serves ivfpq_search_sparse on an index of 16 subspaces x
 *   8 dimensions under L2, the shape for which ivfpq_index_load also builds the inverted index from
 *   codebook entries to points (Algorithm 1's Map).  IVFPQ_SPARSE_SCAN_STREAM streams the codes of
 *   every probed list as the dense search does (an unselected entry's table slot holds the
 *   constant).  IVFPQ_SPARSE_SCAN_MAP walks the map: for every selected entry the points encoded
 *   with it receive its table value; the other points are assigned the constant without any
 *   look-up (Sec. 5.3, paragraph after Algorithm 2), so the scatter work follows the number of
 *   selected entries.  IVFPQ_SPARSE_SCAN_AUTO (default) = STREAM: on B200 a table look-up costs
 *   three instructions, while the map walk pays two shared-memory atomics per (point, selected
 *   entry) pair and still has to visit every point's accumulator once; it was slower at every
 *   radius measured.  Same results either way (the sums over subspaces are taken in different
 *   orders: equal within rounding).  Other shapes have no map: MAP is refused with
 *   IVFPQ_ERR_UNSUPPORTED. */
#define IVFPQ_OPT_SPARSE_SCAN 3
#define IVFPQ_SPARSE_SCAN_AUTO 0
#define IVFPQ_SPARSE_SCAN_STREAM 1
#define IVFPQ_SPARSE_SCAN_MAP 2
/*   IVFPQ_OPT_TEST_FAULT (test-only): 1 = in every following search the tensor-core filtering kernel
 *   leaves out the last centroid tile of its first CTA and shortens its wait limits to about a
 *   millisecond, so that the bounded wait for that tile runs out.  Nothing faults and nothing is left
 *   in flight: the kernel raises its status flag, releases its tensor memory and returns; the search
 *   completes with unreliable probe lists and ivfpq_sync_status reports IVFPQ_ERR_DEVICE_FLAG.  Back
 *   to 0, the next search is normal.  IVFPQ_ERR_UNSUPPORTED for indexes that the tensor-core filtering
 *   does not serve. */
#define IVFPQ_OPT_TEST_FAULT 4
int ivfpq_index_set_option(ivfpq_index_t* index, int32_t option, int64_t value);

/* Waits for the most recent timed search on this handle to finish and writes the device time
 * in milliseconds of its filtering stage to ms[0] and of its LUT+scan+merge stage to ms[1].
 * Returns IVFPQ_ERR_INVALID_ARGUMENT when timing is off or no search has run. */
int ivfpq_last_stage_ms(const ivfpq_index_t* index, float* ms);

/* Number of kernel launches the most recent search call on this handle enqueued. */
int64_t ivfpq_last_launch_count(const ivfpq_index_t* index);

/* Filtering stage for callers that cannot provide or allocate device scratch.  (The paper has no
 * counterpart: this is the same computation as the filtering step of ivfpq_search_*, packaged for a
 * deployment constraint.)
 *
 * Who needs it: code that runs where device allocation is off the table - a serving loop that
 * handed all free device memory to its own pool at start-up, a plug-in that may not call
 * cudaMalloc because the host application forbids the implicit device-wide synchronisation it
 * causes, a caller that has no allocator to ask for a workspace buffer at all.  Such callers still
 * own their inputs and outputs; what they lack is a place for the [queries][nlist] distance tile
 * between the distance kernel and the selection kernel.  Here that tile lives in a fixed array of
 * IVFPQ_STATIC_SCRATCH_BYTES inside the library image: every GPU on which the library is loaded
 * holds those bytes until the process exits.
 *
 * Same results as ivfpq_debug_probes: probe_ids dev [nq][nprobe] ascending by (distance, cluster
 * id), probe_d dev [nq][nprobe].  The query batch is processed in chunks that fit the array.
 * The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine) and is
 * asynchronous on `stream`.  The current device must be the one the index was loaded on.
 *   - indexes with nlist > IVFPQ_STATIC_MAX_NLIST are rejected with IVFPQ_ERR_STATIC_LIMIT;
 *   - the first call on a device looks up the device address of the array (one runtime query,
 *     cached per device); make that first call outside any stream capture;
 *   - all calls on a device share the one array, which keeps whatever the previous call left in
 *     it; the call clears the status word it needs zeroed and overwrites the rest before reading
 *     it, but two calls whose kernels overlap on the GPU (different streams, different host
 *     threads) race on it: serialise them. */
#define IVFPQ_STATIC_SCRATCH_BYTES (8u << 20)
#define IVFPQ_STATIC_MAX_NLIST 16384
int ivfpq_probe_static(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                       int32_t* probe_ids, float* probe_d, void* stream);

/* Status of the most recent ivfpq_probe_static call on the current device (the paper has no
 * counterpart; it completes ivfpq_probe_static for the same callers).  That call has no workspace
 * whose status word ivfpq_sync_status could read: its kernels record a dropped candidate or a
 * bounded wait that ran out in the first word of the built-in array.  This reads that word back
 * (one small copy into a host variable, then a synchronisation of `stream`; nothing is allocated)
 * and returns IVFPQ_OK, IVFPQ_ERR_DEVICE_FLAG (the probe lists of that call are incomplete) or
 * IVFPQ_ERR_CUDA.  Call it on the stream the probe call used, before the next probe call clears
 * the word. */
int ivfpq_static_status(void* stream);

const char* ivfpq_error_string(int code);

/* ---- test-only exports (small inputs) -------------------------------------------------------
 * ivfpq_debug_probes: filtering stage alone. probe_ids dev [nq][nprobe] (ascending distance, ties
 * by ascending cluster id), probe_d dev [nq][nprobe].
 *
 * ivfpq_debug_search: the production kernels compiled with stage dumps.  radius NULL = dense.
 * Any dump pointer may be NULL.  masks dev [nq][nprobe][nsub][8] (bit e of the 256-bit row =
 * entry e selected); visit_* dev [nq][visit_stride] in visiting order (probe rank, then position
 * in the list): visit_hits bit s = subspace s selected for that point, visit_dist its
 * accumulated distance, visit_ids its id; visit_count dev [nq] int64.  Uses workspace of
 * ivfpq_search_workspace_bytes. */
int ivfpq_debug_probes(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                       int32_t* probe_ids, float* probe_d, void* workspace, size_t workspace_bytes,
                       void* stream);
int ivfpq_debug_search(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                       const ivfpq_radius_t* radius, int32_t k, float* out_dist, int32_t* out_ids,
                       int32_t* probe_ids, float* probe_d, uint32_t* masks, int64_t* visit_count,
                       int64_t visit_stride, uint64_t* visit_hits, float* visit_dist,
                       int32_t* visit_ids, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* IVFPQ_H */

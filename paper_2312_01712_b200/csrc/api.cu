// C ABI of the IVFPQ query library: argument validation, workspace carve-up, kernel sequencing.
// See include/ivfpq.h for the contract of every entry point.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"

namespace ivfpq {

namespace {

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

struct DerivedLayout {
    size_t list_off_off, list_blk_off, codes_off, cbt_off, cnorm_off, blk_min_off, chunk_first_off, map_off_off, map_pos_off, total;
    int32_t map;
    int64_t nchunks;
    int32_t mma;
    int64_t nblocks, max_len;
    int32_t nw, vec16;
    int32_t rot, gw[3], block_bytes;
};

// Validates the description and lays out the derived buffer.  Returns an IVFPQ_* code.
int plan_derived(const ivfpq_index_desc_t* d, DerivedLayout* out) {
    if (!d) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (d->d <= 0 || d->nlist <= 0 || d->nsub <= 0 || d->dsub <= 0 || d->ksub <= 0 || d->ntotal < 0)
        return IVFPQ_ERR_INVALID_ARGUMENT;
    if ((int64_t)d->nsub * d->dsub != d->d) return IVFPQ_ERR_INVALID_ARGUMENT;
    if ((d->metric != IVFPQ_METRIC_L2 && d->metric != IVFPQ_METRIC_IP) || d->ksub > 256 || d->nsub > IVFPQ_MAX_NSUB || d->dsub > IVFPQ_MAX_DSUB)
        return IVFPQ_ERR_UNSUPPORTED;
    if (d->ntotal > 0x7FFFFFFFll) return IVFPQ_ERR_UNSUPPORTED;  // ids are int32
    if (!d->list_offsets) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (d->list_offsets[0] != 0 || d->list_offsets[d->nlist] != d->ntotal) return IVFPQ_ERR_INVALID_ARGUMENT;
    int64_t nblocks = 0, max_len = 0, nchunks = 0;
    for (int c = 0; c < d->nlist; ++c) {
        const int64_t len = d->list_offsets[c + 1] - d->list_offsets[c];
        if (len < 0) return IVFPQ_ERR_INVALID_ARGUMENT;
        nblocks += (len + kPointsPerBlock - 1) / kPointsPerBlock;
        nchunks += (len + kMapChunk - 1) / kMapChunk;
        if (len > max_len) max_len = len;
    }
    out->nw = (d->nsub + 3) / 4;
    out->vec16 = (out->nw % 4 == 0) ? 1 : 0;
    out->nblocks = nblocks;
    out->max_len = max_len;
    size_t off = 0;
    out->list_off_off = off;
    off = align_up(off + sizeof(int64_t) * (size_t)(d->nlist + 1), 256);
    out->list_blk_off = off;
    off = align_up(off + sizeof(int64_t) * (size_t)(d->nlist + 1), 256);
    out->codes_off = off;
    out->rot = (rot_supported(d->nsub, d->dsub) && rot_group_widths(d->nsub, out->gw)) ? 1 : 0;
    out->block_bytes = out->rot ? rot_block_bytes(out->gw) : kPointsPerBlock * out->nw * 4;
    off = align_up(off + (size_t)nblocks * out->block_bytes, 256);
    out->cbt_off = off;
    if (out->rot) off = align_up(off + (size_t)d->nsub * 256 * d->dsub * 4, 256);
    out->cnorm_off = off;
    out->mma = coarse_mma_supported(d->d, d->nlist) ? 1 : 0;
    if (out->mma) off = align_up(off + coarse_mma_derived_bytes(d->nlist, d->d, d->metric == IVFPQ_METRIC_L2), 256);
    out->blk_min_off = off;
    off = align_up(off + (size_t)nblocks * 4, 256);
    // entry -> points map of the sparsity-aware scan: the 16 x 8 shape under L2 (element indices are 32-bit)
    out->map = (out->rot && d->metric == IVFPQ_METRIC_L2 && d->nsub == 16 && d->dsub == 8 && d->ntotal > 0 && d->ntotal * 16 < ((int64_t)1 << 32)) ? 1 : 0;
    out->nchunks = nchunks;
    out->chunk_first_off = out->map_off_off = out->map_pos_off = off;
    if (out->map) {
        out->chunk_first_off = off;
        off = align_up(off + sizeof(int32_t) * (size_t)(d->nlist + 1), 256);
        out->map_off_off = off;
        off = align_up(off + (size_t)nchunks * d->nsub * 256 * 4, 256);
        out->map_pos_off = off;
        off = align_up(off + (size_t)d->ntotal * d->nsub * 2, 256);
    }
    out->total = off > 0 ? off : 256;
    return IVFPQ_OK;
}

int check_search_shape(const ivfpq_index* ix, int64_t nq, int32_t nprobe, int32_t k) {
    if (!ix) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (nq <= 0 || nprobe <= 0 || k <= 0) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (nprobe > ix->nlist || nprobe > IVFPQ_MAX_NPROBE || k > IVFPQ_MAX_K) return IVFPQ_ERR_UNSUPPORTED;
    if (nq > (int64_t)1 << 24) return IVFPQ_ERR_UNSUPPORTED;
    return IVFPQ_OK;
}

int run_search(SearchArgs a, void* workspace, size_t workspace_bytes, void* stream, bool probes_only,
               bool keep_status = false) {
    const ivfpq_index* ix = a.ix;
    int rc = check_search_shape(ix, a.nq, a.nprobe, a.k);
    if (rc != IVFPQ_OK) return rc;
    if (!a.queries || !workspace) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (!probes_only && (!a.out_dist || !a.out_ids)) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (!a.dense) {
        if (!a.radius || (a.radius_mode != 0 && a.radius_mode != 1)) return IVFPQ_ERR_INVALID_ARGUMENT;
        if (isnan(a.scale) || isnan(a.miss_penalty)) return IVFPQ_ERR_INVALID_ARGUMENT;
        if (a.score < IVFPQ_SCORE_DISTANCE || a.score > IVFPQ_SCORE_REWARD_PENALTY) return IVFPQ_ERR_INVALID_ARGUMENT;
        if (a.score != IVFPQ_SCORE_DISTANCE && ix->metric != IVFPQ_METRIC_L2) return IVFPQ_ERR_UNSUPPORTED;
    }
    if (!aligned(a.queries, 4) || !aligned(workspace, 256)) return IVFPQ_ERR_WORKSPACE;
    if (!probes_only && !aligned(a.queries, 16)) return IVFPQ_ERR_INVALID_ARGUMENT;  // the scan kernels load rows as float4
    const WorkspaceLayout wl = plan_workspace(ix, a.nq, a.nprobe, a.k);
    if (workspace_bytes < wl.total) return IVFPQ_ERR_WORKSPACE;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    int64_t launches = 0;
    const bool timed = ix->timing != 0;
    if (timed && !ix->ev_ready) {
        for (int i = 0; i < 3; ++i)
            if (cudaEventCreate(&ix->ev[i]) != cudaSuccess) return IVFPQ_ERR_CUDA;
        ix->ev_ready = true;
    }
    // keep_status: a later slice of one batch adds its flags to those of the earlier slices
    // status block: word 0 = device flags, word 1 = work counter of the persistent scan kernels
    if (!keep_status && cudaMemsetAsync(ws + wl.status_off, 0, 16, st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (keep_status && cudaMemsetAsync(ws + wl.status_off + 4, 0, 12, st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (timed && cudaEventRecord(ix->ev[0], st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    int32_t* probe_ids = reinterpret_cast<int32_t*>(ws + wl.probe_ids_off);
    float* probe_d = reinterpret_cast<float*>(ws + wl.probe_d_off);
    if (launch_coarse(ix, a.queries, a.nq, a.nprobe, reinterpret_cast<float*>(ws + wl.coarse_off), wl.qchunk,
                      probe_ids, probe_d, reinterpret_cast<int*>(ws + wl.status_off), st, &launches) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    if (timed && cudaEventRecord(ix->ev[1], st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    const size_t pbytes = (size_t)a.nq * a.nprobe * 4;
    if (a.probe_ids_out &&
        cudaMemcpyAsync(a.probe_ids_out, probe_ids, pbytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    if (a.probe_d_out) {
        const cudaError_t e = ix->metric == IVFPQ_METRIC_IP
                                  ? launch_negate(probe_d, a.probe_d_out, (int64_t)a.nq * a.nprobe, st)
                                  : cudaMemcpyAsync(a.probe_d_out, probe_d, pbytes, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return IVFPQ_ERR_CUDA;
    }
    if (!probes_only) {
        if (launch_scan(a, wl, ws, st, &launches) != cudaSuccess) return IVFPQ_ERR_CUDA;
    }
    if (timed) {
        if (cudaEventRecord(ix->ev[2], st) != cudaSuccess) return IVFPQ_ERR_CUDA;
        ix->ev_recorded = true;
    }
    ix->last_launches = launches;
    return IVFPQ_OK;
}

}  // namespace

WorkspaceLayout plan_workspace(const ivfpq_index* ix, int64_t nq, int32_t nprobe, int32_t k) {
    WorkspaceLayout wl{};
    // query chunk of the filtering stage: keep the [qchunk][nlist] distance tile near 64 MiB, so
    // that it stays in the 126 MB L2 between the kernel that writes it and the one that selects
    // from it, with as many queries per launch as that allows (measured: 32 MiB and 96 MiB are
    // both slower on the 16 384-cluster workload)
    int64_t qchunk = ((int64_t)64 << 20) / ((int64_t)ix->nlist * 4);
    if (qchunk < 64) qchunk = 64;
    if (qchunk > nq) qchunk = nq;
    wl.qchunk = qchunk;
    int nsplit = ix->nsplit_opt;
    if (nsplit <= 0) {
        // enough CTAs for two waves of the device at 4 CTAs per SM
        const int64_t want = (int64_t)ix->sm_count * 8;
        nsplit = (int)((want + nq - 1) / nq);
        if (nsplit < 1) nsplit = 1;
    }
    if (nsplit > nprobe) nsplit = nprobe;
    if (nsplit > 64) nsplit = 64;
    wl.nsplit = nsplit;
    size_t off = 0;
    wl.status_off = off;
    off = align_up(off + 16, 256);
    wl.probe_ids_off = off;
    off = align_up(off + (size_t)nq * nprobe * 4, 256);
    wl.probe_d_off = off;
    off = align_up(off + (size_t)nq * nprobe * 4, 256);
    wl.coarse_off = off;
    off = align_up(off + coarse_region_bytes(ix, qchunk), 256);
    wl.partial_off = off;
    // sized for the largest split the option may select later, so that the option can change
    // without a new workspace query
    off = align_up(off + (size_t)nq * (size_t)(nprobe < 64 ? nprobe : 64) * k * 8, 256);
    wl.total = off;
    return wl;
}

}  // namespace ivfpq

using namespace ivfpq;

extern "C" {

size_t ivfpq_index_derived_bytes(const ivfpq_index_desc_t* desc) {
    DerivedLayout dl;
    if (plan_derived(desc, &dl) != IVFPQ_OK) return 0;
    return dl.total;
}

int ivfpq_index_load(const ivfpq_index_desc_t* desc, void* derived_dev, size_t derived_bytes, void* stream,
                     ivfpq_index_t** out) {
    if (!out) return IVFPQ_ERR_INVALID_ARGUMENT;
    *out = nullptr;
    DerivedLayout dl;
    int rc = plan_derived(desc, &dl);
    if (rc != IVFPQ_OK) return rc;
    if (!desc->coarse_centroids || !desc->codebooks || !derived_dev) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (desc->ntotal > 0 && (!desc->codes || !desc->ids)) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (!aligned(derived_dev, 256) || derived_bytes < dl.total) return IVFPQ_ERR_WORKSPACE;
    if (!aligned(desc->coarse_centroids, 16) || !aligned(desc->codebooks, 16) || !aligned(desc->ids, 4))
        return IVFPQ_ERR_INVALID_ARGUMENT;

    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return IVFPQ_ERR_CUDA;

    ivfpq_index* ix = new (std::nothrow) ivfpq_index();
    if (!ix) return IVFPQ_ERR_INVALID_ARGUMENT;
    ix->d = desc->d;
    ix->nlist = desc->nlist;
    ix->nsub = desc->nsub;
    ix->dsub = desc->dsub;
    ix->ksub = desc->ksub;
    ix->ntotal = desc->ntotal;
    ix->metric = desc->metric;
    ix->cent = desc->coarse_centroids;
    ix->cb = desc->codebooks;
    ix->ids = desc->ids;
    char* base = static_cast<char*>(derived_dev);
    ix->list_off = reinterpret_cast<const int64_t*>(base + dl.list_off_off);
    ix->list_blk = reinterpret_cast<const int64_t*>(base + dl.list_blk_off);
    ix->codes_il = reinterpret_cast<const uint32_t*>(base + dl.codes_off);
    ix->nw = dl.nw;
    ix->vec16 = dl.vec16;
    ix->nblocks = dl.nblocks;
    ix->rot = dl.rot;
    {
        // 16 x 8 shape: short lists are served best by the 16-warp instance of the persistent kernel
        // (whole codebook in registers, cheaper table build), long lists by the 32-warp instance (its
        // list scan hides more latency).  IVFPQ_SCAN_KERNEL=warps16|warps32 overrides the choice at load.
        const int64_t mean_len = desc->nlist > 0 ? desc->ntotal / desc->nlist : 0;
        ix->pers_warps = mean_len >= 2048 ? 32 : 16;
        const char* kind = getenv("IVFPQ_SCAN_KERNEL");
        if (kind && strcmp(kind, "warps16") == 0) ix->pers_warps = 16;
        if (kind && strcmp(kind, "warps32") == 0) ix->pers_warps = 32;
        const char* rk = getenv("IVFPQ_ROT_KERNEL");
        ix->rot_pair = (rk && strcmp(rk, "pair") == 0) ? 1 : 0;
    }
    for (int i = 0; i < 3; ++i) ix->gw[i] = dl.rot ? dl.gw[i] : 0;
    ix->block_bytes = dl.block_bytes;
    ix->cbt = reinterpret_cast<const float*>(base + dl.cbt_off);
    ix->cnorm = dl.mma ? reinterpret_cast<const float*>(base + dl.cnorm_off) : nullptr;
    {
        // behind the norms and their maximum: the centroids' mean and the centred centroids (L2 only)
        const bool centered = dl.mma && desc->metric == IVFPQ_METRIC_L2;
        char* at = base + dl.cnorm_off + align_up((size_t)desc->nlist * 4, 256) + 256;
        ix->mu = centered ? reinterpret_cast<const float*>(at) : nullptr;
        ix->cent_c = centered ? reinterpret_cast<const float*>(at + align_up((size_t)desc->d * 4, 256)) : nullptr;
    }
    ix->max_list_len = dl.max_len;
    ix->blk_min = reinterpret_cast<const uint32_t*>(base + dl.blk_min_off);
    ix->chunk_first = dl.map ? reinterpret_cast<const int32_t*>(base + dl.chunk_first_off) : nullptr;
    ix->map_off = dl.map ? reinterpret_cast<const uint32_t*>(base + dl.map_off_off) : nullptr;
    ix->map_pos = dl.map ? reinterpret_cast<const uint16_t*>(base + dl.map_pos_off) : nullptr;
    ix->nchunks = dl.nchunks;
    {
        // lanes per selected entry in the scatter: about the mean number of points behind one entry
        const int64_t seg = dl.nchunks > 0 ? desc->ntotal / dl.nchunks / 256 : 0;
        ix->map_group = seg < 6 ? 4 : (seg < 12 ? 8 : (seg < 24 ? 16 : 32));
    }
    ix->sparse_scan = 0;
    ix->test_fault = 0;
    ix->device = dev;
    ix->sm_count = sms;
    ix->nsplit_opt = 0;
    ix->last_launches = 0;
    ix->timing = 0;
    ix->ev_ready = false;
    ix->pipe_ready = false;
    ix->ev_recorded = false;

    // list tables: built on the host, copied synchronously (pageable source)
    const size_t n1 = (size_t)desc->nlist + 1;
    int64_t* blk = new (std::nothrow) int64_t[n1];
    int32_t* chf = new (std::nothrow) int32_t[n1];
    if (!blk || !chf) {
        delete[] blk;
        delete[] chf;
        delete ix;
        return IVFPQ_ERR_INVALID_ARGUMENT;
    }
    blk[0] = 0;
    chf[0] = 0;
    for (int c = 0; c < desc->nlist; ++c) {
        const int64_t len = desc->list_offsets[c + 1] - desc->list_offsets[c];
        blk[c + 1] = blk[c] + (len + kPointsPerBlock - 1) / kPointsPerBlock;
        chf[c + 1] = chf[c] + (int32_t)((len + kMapChunk - 1) / kMapChunk);
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(base + dl.list_off_off, desc->list_offsets, n1 * 8, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(base + dl.list_blk_off, blk, n1 * 8, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && dl.map)
        e = cudaMemcpyAsync(base + dl.chunk_first_off, chf, n1 * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);  // the host arrays may go away after return
    delete[] blk;
    delete[] chf;
    if (e == cudaSuccess)
        e = launch_relayout(ix, desc->codes, reinterpret_cast<uint32_t*>(base + dl.codes_off),
                            reinterpret_cast<float*>(base + dl.cbt_off), st);
    if (e == cudaSuccess) e = launch_block_min_id(ix, reinterpret_cast<uint32_t*>(base + dl.blk_min_off), st);
    if (e == cudaSuccess) e = launch_entry_map(ix, desc->codes, st);
    if (e == cudaSuccess && ix->cent_c)
        e = launch_center(ix->cent, ix->nlist, ix->d, const_cast<float*>(ix->mu), const_cast<float*>(ix->cent_c), st);
    if (e == cudaSuccess && ix->cnorm)
        e = launch_cnorm(ix->cent_c ? ix->cent_c : ix->cent, ix->nlist, ix->d, reinterpret_cast<float*>(base + dl.cnorm_off), st);
    if (e != cudaSuccess) {
        delete ix;
        return IVFPQ_ERR_CUDA;
    }
    *out = ix;
    return IVFPQ_OK;
}

int ivfpq_index_free(ivfpq_index_t* index) {
    if (!index) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (index->ev_ready)
        for (int i = 0; i < 3; ++i) cudaEventDestroy(index->ev[i]);
    if (index->pipe_ready) {
        for (int i = 0; i < 12; ++i) cudaEventDestroy(index->pipe_ev[i]);
        cudaStreamDestroy(index->copy_stream);
    }
    delete index;
    return IVFPQ_OK;
}

int ivfpq_query_thresholds(const ivfpq_index_t* index, const float* queries, int64_t nq,
                           const ivfpq_threshold_model_t* model, float* radius_out, void* stream) {
    if (!index || !queries || !model || !radius_out || nq <= 0) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (!model->density || !model->origin || !model->inv_cell || !model->coef) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (index->dsub != 2) return IVFPQ_ERR_UNSUPPORTED;
    if (model->grid < 1 || model->grid > 4096 || model->degree < 0 || model->degree > 8) return IVFPQ_ERR_UNSUPPORTED;
    if (nq > (int64_t)1 << 24) return IVFPQ_ERR_UNSUPPORTED;
    if (!aligned(queries, 8) || !aligned(model->origin, 8) || !aligned(model->inv_cell, 8)) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (launch_thresholds(queries, nq, index->nsub, model, radius_out, reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    return IVFPQ_OK;
}

int ivfpq_query_thresholds_knn(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t kth, int32_t degree,
                               const float* coef, float* radius_out, void* workspace, size_t workspace_bytes,
                               void* stream) {
    if (!index || !queries || !coef || !radius_out || !workspace || nq <= 0) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (index->metric != IVFPQ_METRIC_L2) return IVFPQ_ERR_UNSUPPORTED;
    if (kth < 1 || kth > index->ksub || degree < 0 || degree > 8 || nq > (int64_t)1 << 24) return IVFPQ_ERR_UNSUPPORTED;
    // the nearest cluster of every query: the filtering stage with one probe, into the workspace
    SearchArgs a{};
    a.ix = index;
    a.queries = queries;
    a.nq = nq;
    a.nprobe = 1;
    a.k = 1;
    a.dense = true;
    const int rc = run_search(a, workspace, workspace_bytes, stream, true);
    if (rc != IVFPQ_OK) return rc;
    const WorkspaceLayout wl = plan_workspace(index, nq, 1, 1);
    char* ws = static_cast<char*>(workspace);
    if (launch_thresholds_knn(index, queries, nq, reinterpret_cast<const int32_t*>(ws + wl.probe_ids_off), kth, degree, coef,
                              radius_out, reinterpret_cast<int*>(ws + wl.status_off),
                              reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    return IVFPQ_OK;
}

int ivfpq_entry_stats(const ivfpq_index_t* index, const uint8_t* codes, const float* queries, int64_t nq,
                      const int64_t* neighbor_pos, int32_t k, int32_t* usage_out,
                      unsigned long long* rank_hist, int32_t* flags, void* stream) {
    if (!index || !codes || !queries || !neighbor_pos || !usage_out || !rank_hist || !flags)
        return IVFPQ_ERR_INVALID_ARGUMENT;
    if (nq <= 0 || k <= 0) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (k > IVFPQ_MAX_K || nq > (int64_t)1 << 30) return IVFPQ_ERR_UNSUPPORTED;
    if (launch_entry_stats(index, codes, queries, nq, neighbor_pos, k, usage_out, rank_hist, flags,
                           reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    return IVFPQ_OK;
}

size_t ivfpq_search_workspace_bytes(const ivfpq_index_t* index, int64_t nq, int32_t nprobe, int32_t k) {
    if (check_search_shape(index, nq, nprobe, k) != IVFPQ_OK) return 0;
    return plan_workspace(index, nq, nprobe, k).total;
}

int ivfpq_search_dense(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe, int32_t k,
                       float* out_dist, int32_t* out_ids, void* workspace, size_t workspace_bytes, void* stream) {
    SearchArgs a{};
    a.ix = index;
    a.queries = queries;
    a.nq = nq;
    a.nprobe = nprobe;
    a.k = k;
    a.dense = true;
    a.out_dist = out_dist;
    a.out_ids = out_ids;
    return run_search(a, workspace, workspace_bytes, stream, false);
}

static void fill_radius(SearchArgs& a, const ivfpq_radius_t* radius) {
    a.dense = false;
    a.radius = radius->radius;
    a.radius_mode = radius->mode;
    a.scale = radius->scale;
    a.miss_penalty = radius->miss_penalty == 0.0f ? 0.0f : radius->miss_penalty;   // -0 counts as +0
    a.score = radius->score;
}

int ivfpq_search_sparse(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                        const ivfpq_radius_t* radius, int32_t k, float* out_dist, int32_t* out_ids,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (!radius) return IVFPQ_ERR_INVALID_ARGUMENT;
    SearchArgs a{};
    a.ix = index;
    a.queries = queries;
    a.nq = nq;
    a.nprobe = nprobe;
    a.k = k;
    fill_radius(a, radius);
    a.out_dist = out_dist;
    a.out_ids = out_ids;
    return run_search(a, workspace, workspace_bytes, stream, false);
}

size_t ivfpq_search_host_workspace_bytes(const ivfpq_index_t* index, int64_t nq, int32_t nprobe, int32_t k) {
    if (check_search_shape(index, nq, nprobe, k) != IVFPQ_OK) return 0;
    size_t core = plan_workspace(index, nq, nprobe, k).total;
    size_t off = align_up(core, 256);
    off = align_up(off + (size_t)nq * index->d * 4, 256);
    off = align_up(off + (size_t)nq * k * 4, 256);
    off = align_up(off + (size_t)nq * k * 4, 256);
    return off;
}

int ivfpq_search_host(const ivfpq_index_t* index, const float* queries_host, int64_t nq, int32_t nprobe,
                      const ivfpq_radius_t* radius, int32_t k, float* out_dist_host, int32_t* out_ids_host,
                      void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_search_shape(index, nq, nprobe, k);
    if (rc != IVFPQ_OK) return rc;
    if (!queries_host || !out_dist_host || !out_ids_host || !workspace) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (!aligned(workspace, 256)) return IVFPQ_ERR_WORKSPACE;
    if (workspace_bytes < ivfpq_search_host_workspace_bytes(index, nq, nprobe, k)) return IVFPQ_ERR_WORKSPACE;
    const size_t core = align_up(plan_workspace(index, nq, nprobe, k).total, 256);
    char* ws = static_cast<char*>(workspace);
    size_t off = core;
    float* q_dev = reinterpret_cast<float*>(ws + off);
    off = align_up(off + (size_t)nq * index->d * 4, 256);
    float* d_dev = reinterpret_cast<float*>(ws + off);
    off = align_up(off + (size_t)nq * k * 4, 256);
    int32_t* i_dev = reinterpret_cast<int32_t*>(ws + off);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    SearchArgs a{};
    a.ix = index;
    a.queries = q_dev;
    a.nq = nq;
    a.nprobe = nprobe;
    a.k = k;
    a.dense = true;
    if (radius) fill_radius(a, radius);
    a.out_dist = d_dev;
    a.out_ids = i_dev;

    // Large batches go in slices: the copy stream brings all slices' queries in and takes each
    // slice's results out while the caller's stream searches the next slice.  (With the stage
    // timing option on, the batch stays in one piece so that the stage times describe it.)
    // (measured on the 10 k-query batch: two slices +2.4 % end to end, three +1.9 %, four none)
    const int nslice = index->timing ? 1 : (nq >= 2048 ? 2 : 1);
    if (nslice > 1) {
        if (!index->pipe_ready) {
            if (cudaStreamCreateWithFlags(&index->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return IVFPQ_ERR_CUDA;
            for (int i = 0; i < 12; ++i)
                if (cudaEventCreateWithFlags(&index->pipe_ev[i], cudaEventDisableTiming) != cudaSuccess) return IVFPQ_ERR_CUDA;
            index->pipe_ready = true;
        }
        cudaStream_t cs = index->copy_stream;
        cudaEvent_t* ev = index->pipe_ev;   // [0]: start, [1 + s]: queries of slice s in, [5 + s]: slice s searched, [9]: all out
        const int64_t per = ((nq + nslice - 1) / nslice + 31) / 32 * 32;
        bool ok = cudaEventRecord(ev[0], st) == cudaSuccess && cudaStreamWaitEvent(cs, ev[0], 0) == cudaSuccess;
        for (int s = 0; ok && s < nslice; ++s) {
            const int64_t lo = s * per, n = lo < nq ? (nq - lo < per ? nq - lo : per) : 0;
            if (n <= 0) continue;
            ok = cudaMemcpyAsync(q_dev + lo * index->d, queries_host + lo * index->d, (size_t)n * index->d * 4,
                                 cudaMemcpyHostToDevice, cs) == cudaSuccess &&
                 cudaEventRecord(ev[1 + s], cs) == cudaSuccess;
        }
        if (!ok) return IVFPQ_ERR_CUDA;
        int64_t launches = 0;
        for (int s = 0; s < nslice; ++s) {
            const int64_t lo = s * per, n = lo < nq ? (nq - lo < per ? nq - lo : per) : 0;
            if (n <= 0) continue;
            if (cudaStreamWaitEvent(st, ev[1 + s], 0) != cudaSuccess) return IVFPQ_ERR_CUDA;
            SearchArgs b = a;
            b.queries = q_dev + lo * index->d;
            b.nq = n;
            b.out_dist = d_dev + lo * k;
            b.out_ids = i_dev + lo * k;
            if (!b.dense && b.radius_mode == 1) b.radius = a.radius + lo * index->nsub;
            rc = run_search(b, workspace, core, stream, false, s > 0);
            if (rc != IVFPQ_OK) return rc;
            launches += index->last_launches;
            ok = cudaEventRecord(ev[5 + s], st) == cudaSuccess && cudaStreamWaitEvent(cs, ev[5 + s], 0) == cudaSuccess &&
                 cudaMemcpyAsync(out_dist_host + lo * k, d_dev + lo * k, (size_t)n * k * 4, cudaMemcpyDeviceToHost, cs) == cudaSuccess &&
                 cudaMemcpyAsync(out_ids_host + lo * k, i_dev + lo * k, (size_t)n * k * 4, cudaMemcpyDeviceToHost, cs) == cudaSuccess;
            if (!ok) return IVFPQ_ERR_CUDA;
        }
        index->last_launches = launches;
        if (cudaEventRecord(ev[9], cs) != cudaSuccess || cudaStreamWaitEvent(st, ev[9], 0) != cudaSuccess) return IVFPQ_ERR_CUDA;
        return IVFPQ_OK;
    }

    if (cudaMemcpyAsync(q_dev, queries_host, (size_t)nq * index->d * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    rc = run_search(a, workspace, core, stream, false);
    if (rc != IVFPQ_OK) return rc;
    if (cudaMemcpyAsync(out_dist_host, d_dev, (size_t)nq * k * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    if (cudaMemcpyAsync(out_ids_host, i_dev, (size_t)nq * k * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    return IVFPQ_OK;
}

int ivfpq_sync_status(const ivfpq_index_t* index, void* workspace, void* stream) {
    if (!index || !workspace) return IVFPQ_ERR_INVALID_ARGUMENT;
    int flags[4] = {0, 0, 0, 0};
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(flags, workspace, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return IVFPQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return IVFPQ_ERR_CUDA;
    return flags[0] != 0 ? IVFPQ_ERR_DEVICE_FLAG : IVFPQ_OK;
}

int ivfpq_index_set_option(ivfpq_index_t* index, int32_t option, int64_t value) {
    if (!index) return IVFPQ_ERR_INVALID_ARGUMENT;
    switch (option) {
        case IVFPQ_OPT_NSPLIT:
            if (value < 0 || value > 64) return IVFPQ_ERR_INVALID_ARGUMENT;
            index->nsplit_opt = (int32_t)value;
            return IVFPQ_OK;
        case IVFPQ_OPT_SPARSE_SCAN:
            if (value < IVFPQ_SPARSE_SCAN_AUTO || value > IVFPQ_SPARSE_SCAN_MAP) return IVFPQ_ERR_INVALID_ARGUMENT;
            if (value == IVFPQ_SPARSE_SCAN_MAP && !index->map_pos) return IVFPQ_ERR_UNSUPPORTED;
            index->sparse_scan = (int32_t)value;
            return IVFPQ_OK;
        case IVFPQ_OPT_TEST_FAULT:
            if (value != 0 && value != 1) return IVFPQ_ERR_INVALID_ARGUMENT;
            if (value == 1 && !index->cnorm) return IVFPQ_ERR_UNSUPPORTED;   // the tensor-core filtering kernel is the one with bounded waits
            index->test_fault = (int32_t)value;
            return IVFPQ_OK;
        case IVFPQ_OPT_TIMING:
            if (value != 0 && value != 1) return IVFPQ_ERR_INVALID_ARGUMENT;
            index->timing = (int32_t)value;
            return IVFPQ_OK;
        default:
            return IVFPQ_ERR_INVALID_ARGUMENT;
    }
}

int ivfpq_last_stage_ms(const ivfpq_index_t* index, float* ms) {
    if (!index || !ms || !index->ev_ready || !index->ev_recorded) return IVFPQ_ERR_INVALID_ARGUMENT;
    if (cudaEventSynchronize(index->ev[2]) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (cudaEventElapsedTime(&ms[0], index->ev[0], index->ev[1]) != cudaSuccess) return IVFPQ_ERR_CUDA;
    if (cudaEventElapsedTime(&ms[1], index->ev[1], index->ev[2]) != cudaSuccess) return IVFPQ_ERR_CUDA;
    return IVFPQ_OK;
}

int64_t ivfpq_last_launch_count(const ivfpq_index_t* index) { return index ? index->last_launches : 0; }

const char* ivfpq_error_string(int code) {
    switch (code) {
        case IVFPQ_OK: return "ok";
        case IVFPQ_ERR_INVALID_ARGUMENT: return "invalid argument";
        case IVFPQ_ERR_UNSUPPORTED: return "unsupported shape";
        case IVFPQ_ERR_WORKSPACE: return "workspace or derived buffer too small or misaligned";
        case IVFPQ_ERR_CUDA: return "CUDA runtime error";
        case IVFPQ_ERR_DEVICE_FLAG: return "device-side status flag raised";
        case IVFPQ_ERR_STATIC_LIMIT: return "index too large for the scratch array built into the library";
        default: return "unknown error code";
    }
}

int ivfpq_debug_probes(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                       int32_t* probe_ids, float* probe_d, void* workspace, size_t workspace_bytes, void* stream) {
    if (!probe_ids || !probe_d) return IVFPQ_ERR_INVALID_ARGUMENT;
    SearchArgs a{};
    a.ix = index;
    a.queries = queries;
    a.nq = nq;
    a.nprobe = nprobe;
    a.k = 1;
    a.dense = true;
    a.probe_ids_out = probe_ids;
    a.probe_d_out = probe_d;
    return run_search(a, workspace, workspace_bytes, stream, true);
}

int ivfpq_debug_search(const ivfpq_index_t* index, const float* queries, int64_t nq, int32_t nprobe,
                       const ivfpq_radius_t* radius, int32_t k, float* out_dist, int32_t* out_ids,
                       int32_t* probe_ids, float* probe_d, uint32_t* masks, int64_t* visit_count,
                       int64_t visit_stride, uint64_t* visit_hits, float* visit_dist, int32_t* visit_ids,
                       void* workspace, size_t workspace_bytes, void* stream) {
    if (visit_stride < 0) return IVFPQ_ERR_INVALID_ARGUMENT;
    SearchArgs a{};
    a.ix = index;
    a.queries = queries;
    a.nq = nq;
    a.nprobe = nprobe;
    a.k = k;
    a.dense = true;
    if (radius) fill_radius(a, radius);
    a.out_dist = out_dist;
    a.out_ids = out_ids;
    a.debug = true;
    a.probe_ids_out = probe_ids;
    a.probe_d_out = probe_d;
    a.masks = masks;
    a.visit_count = visit_count;
    a.visit_stride = visit_stride;
    a.visit_hits = visit_hits;
    a.visit_dist = visit_dist;
    a.visit_ids = visit_ids;
    return run_search(a, workspace, workspace_bytes, stream, false);
}

}  // extern "C"

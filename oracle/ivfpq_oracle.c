/*
 * CPU oracle for the sparsity-aware IVFPQ query path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow restatement of what the path computes, written from the paper and
 * used only by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg.  It shares no code with the CUDA library and the product never calls it.
 *
 * Arithmetic: fp32, round to nearest, no contraction other than the explicit
 * fmaf() calls (compile with -ffp-contract=off and without -ffast-math).  The
 * paper does not state a precision; fp32 is this repository's reading.
 *
 * Steps (one query at a time; OpenMP only spreads independent queries):
 *   S1  filtering: squared L2 distance from the query to every IVF centroid, the
 *       nprobe closest are kept (Sec. 2.1 "Online Search", step A; Eq. "metric").
 *   S2  selective L2-LUT: for every probed cluster the residual query - centroid;
 *       in every subspace the squared distance from the residual projection to each
 *       codebook entry; an entry is selected when that distance is within the
 *       threshold radius of the subspace (Sec. 2.1 steps B, C; Sec. 4.1 "Intuition of
 *       Algorithm Enhancement" and the last sentence of "Determining Proper
 *       Threshold"; Algorithm 2, whose ray test against a sphere of radius
 *       thres*thres_scale decides exactly d <= thres*thres_scale).  The table holds
 *       the squared distance: only that makes the sum over subspaces the distance
 *       of step D.
 *   S3  distance calculation: every point of a probed cluster sums the table values
 *       of its codes over the subspaces in which its entry was selected (step D);
 *       each subspace whose entry was not selected contributes the large constant P
 *       instead of a table look-up (Sec. 5.3, paragraph after Algorithm 2).
 *   S4  the k smallest (distance, id) pairs, ascending (Sec. 2.1, last paragraph).
 * Dense search is the same with every entry selected.
 *
 * Hit-count scores (Sec. 5.4 "Aggressive Approximation: hit count-based Method"; the -L and -M
 * configurations of the evaluation plan in Sec. 6.1) replace S3's distance by a count, S1, S2's
 * selection and S4 unchanged:
 *   score 1 (hit count): a point is ranked by the number of subspaces in which its entry was
 *       selected, more hits first.  Reported value: the number of subspaces missed (nsub - hits),
 *       so that smaller is better as for distances.
 *   score 2 (reward / penalty): every sphere gets an inner sphere of half the radius; a subspace
 *       adds +1 when the entry lies within the inner sphere, -1 when it lies outside the outer
 *       one, 0 in between; more is better.  Reported value: nsub - score (0, 1 or 2 per subspace).
 *   The inner test is d2 <= 0.25f * (radius*scale)^2 on the same squared distance.
 *
 * Inner-product similarity (Sec. 4.2 "Inner Product Similarity Support"): oracle_search_ip() below.
 *   S1  filtering by inner product: the nprobe clusters with the largest q.c.
 *   S2  the sphere of entry e gets the radius sqrt(R^2 + |e|^2), R the subspace's threshold: the
 *       entry is selected when |q_s - e|^2 <= R^2 + |e|^2, and its table value is the inner product
 *       q_s.e, which the paper recovers from the hit time as (|q_s|^2 + |e|^2 - |q_s - e|^2) / 2.
 *       The projection is the query's own: with residual codes x ~ c + sum_s e_s the similarity
 *       splits into q.c (known from S1) plus q_s.e_s per subspace, so the table does not depend
 *       on the cluster.
 *   S3  similarity = q.c + sum of the table values of the selected subspaces - m * P for the m
 *       subspaces whose entry was not selected (the large constant, now a penalty).
 *   S4  the k largest (similarity, then smaller id), padded with (-inf, -1).
 *
 * Before S2, the query-specific thresholds can come from the dynamic threshold front-end (Sec. 4.1
 * "Determining Proper Threshold"; Algorithm 2, the threshold step): oracle_thresholds() below looks up the
 * density of the grid cell the query's projection falls into and evaluates the polynomial
 * regressor on it.
 *
 * Parity pins (tests/test_oracle_pins.py): radius -> inf equals dense bit for bit;
 * dense distance equals the fp64 distance to the reconstructed vector; a lossless
 * toy index reproduces brute-force exact neighbours; nesting/monotonicity in radius
 * and nprobe; a naive second implementation without any table; the ray-time
 * algebra of Algorithm 2 against the plain compare.  The paper's absolute recall
 * and throughput figures are not recoverable from its text: parity unpinned
 * against those, everything computed here is pinned by the tests above.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    float dist;
    int32_t id;
} cand_t;

static int cand_less(const void* a, const void* b) {
    const cand_t* x = (const cand_t*)a;
    const cand_t* y = (const cand_t*)b;
    if (x->dist < y->dist) return -1;
    if (x->dist > y->dist) return 1;
    if (x->id < y->id) return -1;
    if (x->id > y->id) return 1;
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* S1 for one query: dc[c] for all centroids, then the nprobe smallest by (dc, c). */
static void coarse_one(const float* q, int d, const float* cent, int nlist, int nprobe,
                       cand_t* scratch, int32_t* probe_ids, float* probe_d) {
    for (int c = 0; c < nlist; ++c) {
        float a = 0.0f;
        for (int j = 0; j < d; ++j) {
            float t = q[j] - cent[(size_t)c * d + j];
            a = fmaf(t, t, a);
        }
        scratch[c].dist = a;
        scratch[c].id = c;
    }
    qsort(scratch, (size_t)nlist, sizeof(cand_t), cand_less);
    for (int p = 0; p < nprobe; ++p) {
        probe_ids[p] = scratch[p].id;
        probe_d[p] = scratch[p].dist;
    }
}

int oracle_coarse(const float* queries, int64_t nq, int d, const float* cent, int nlist, int nprobe,
                  int32_t* probe_ids, float* probe_d) {
    if (nprobe > nlist || nprobe <= 0) return -1;
#pragma omp parallel
    {
        cand_t* scratch = (cand_t*)malloc(sizeof(cand_t) * (size_t)nlist);
#pragma omp for schedule(dynamic, 4)
        for (int64_t qi = 0; qi < nq; ++qi)
            coarse_one(queries + qi * d, d, cent, nlist, nprobe, scratch, probe_ids + qi * nprobe,
                       probe_d + qi * nprobe);
        free(scratch);
    }
    return 0;
}

/*
 * Full search.  dense != 0 ignores the radius arguments.
 *   radius       : mode 0 -> [nsub], mode 1 -> [nq][nsub]   (threshold before scaling)
 *   scale        : the user scaling factor (thres_scale of Algorithm 2)
 *   miss_penalty : P; negative -> P = sum over subspaces of the squared scaled radius
 * Optional stage dumps (NULL to skip):
 *   probe_ids/probe_d [nq][nprobe]; masks [nq][nprobe][nsub][8] (bit e of the 256-bit
 *   row = entry e selected); visit_count [nq]; and, with visit_stride slots per query in
 *   visiting order (probe rank, then position in the list): visit_hits (bit s = subspace
 *   s selected for that point), visit_dist, visit_ids.
 * score: 0 = distances (S3 as above), 1 = hit count, 2 = reward / penalty (header comment); the
 *   two count scores need a radius (not dense).
 */
int oracle_search_scored(int d, int nlist, int nsub, int dsub, int ksub, const float* cent,
                  const float* codebooks, const int64_t* list_offsets, const uint8_t* codes,
                  const int32_t* ids, const float* queries, int64_t nq, int nprobe, int dense,
                  const float* radius, int radius_mode, float scale, float miss_penalty, int score, int k,
                  float* out_dist, int32_t* out_ids, int32_t* probe_ids_out, float* probe_d_out,
                  uint32_t* masks_out, int64_t* visit_count, int64_t visit_stride,
                  uint64_t* visit_hits, float* visit_dist, int32_t* visit_ids) {
    if (d != nsub * dsub || ksub <= 0 || ksub > 256 || nsub > 64) return -2;
    if (nprobe <= 0 || nprobe > nlist || k <= 0) return -1;
    if (!dense && radius == NULL) return -1;
    if (score < 0 || score > 2 || (dense && score != 0)) return -1;
    int status = 0;

#pragma omp parallel
    {
        cand_t* scratch = (cand_t*)malloc(sizeof(cand_t) * (size_t)nlist);
        int32_t* probes = (int32_t*)malloc(sizeof(int32_t) * (size_t)nprobe);
        float* probes_d = (float*)malloc(sizeof(float) * (size_t)nprobe);
        float* lut = (float*)malloc(sizeof(float) * (size_t)nsub * ksub);
        uint8_t* hit = (uint8_t*)malloc((size_t)nsub * ksub);
        float* r2 = (float*)malloc(sizeof(float) * (size_t)nsub);
        size_t cap = 1024, n = 0;
        cand_t* vis = (cand_t*)malloc(sizeof(cand_t) * cap);

#pragma omp for schedule(dynamic, 1)
        for (int64_t qi = 0; qi < nq; ++qi) {
            const float* q = queries + qi * d;
            coarse_one(q, d, cent, nlist, nprobe, scratch, probes, probes_d);
            if (probe_ids_out) memcpy(probe_ids_out + qi * nprobe, probes, sizeof(int32_t) * nprobe);
            if (probe_d_out) memcpy(probe_d_out + qi * nprobe, probes_d, sizeof(float) * nprobe);

            /* threshold per (query, subspace), independent of the probed cluster */
            float P = 0.0f;
            if (!dense) {
                const float* rad = radius_mode == 1 ? radius + qi * nsub : radius;
                float acc = 0.0f;
                for (int s = 0; s < nsub; ++s) {
                    float r = rad[s] * scale;
                    r2[s] = r * r;
                    acc = acc + r2[s];
                }
                P = miss_penalty >= 0.0f ? miss_penalty : acc;
            }

            n = 0;
            int64_t nvis = 0;
            for (int p = 0; p < nprobe; ++p) {
                const int c = probes[p];
                /* S2: table and selection for this (query, cluster) */
                for (int s = 0; s < nsub; ++s) {
                    uint32_t mrow[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    for (int e = 0; e < ksub; ++e) {
                        const float* entry = codebooks + ((size_t)s * ksub + e) * dsub;
                        float d2 = 0.0f;
                        for (int j = 0; j < dsub; ++j) {
                            float res = q[s * dsub + j] - cent[(size_t)c * d + s * dsub + j];
                            float t = res - entry[j];
                            d2 = fmaf(t, t, d2);
                        }
                        int h = dense ? 1 : (d2 <= r2[s]);
                        /* level 2: also within the inner sphere of half the radius */
                        if (h && score == 2 && d2 <= 0.25f * r2[s]) h = 2;
                        lut[(size_t)s * ksub + e] = d2;
                        hit[(size_t)s * ksub + e] = (uint8_t)h;
                        if (h) mrow[e >> 5] |= 1u << (e & 31);
                    }
                    if (masks_out)
                        memcpy(masks_out + (((size_t)qi * nprobe + p) * nsub + s) * 8, mrow, sizeof(mrow));
                }
                /* S3: every point of the cluster */
                for (int64_t x = list_offsets[c]; x < list_offsets[c + 1]; ++x) {
                    const uint8_t* code = codes + (size_t)x * nsub;
                    float S = 0.0f;
                    int m = 0;
                    int reward = 0; /* score 2: +1 inner hit, -1 missed both spheres */
                    uint64_t hs = 0;
                    for (int s = 0; s < nsub; ++s) {
                        int e = code[s];
                        if (e < ksub && hit[(size_t)s * ksub + e]) {
                            S = S + lut[(size_t)s * ksub + e];
                            hs |= (uint64_t)1 << s;
                            if (hit[(size_t)s * ksub + e] == 2) reward += 1;
                        } else {
                            m += 1;
                            reward -= 1;
                        }
                    }
                    float dist = (m == 0) ? S : fmaf((float)m, P, S);
                    if (score == 1) dist = (float)m;
                    if (score == 2) dist = (float)(nsub - reward);
                    if (n == cap) {
                        cap *= 2;
                        vis = (cand_t*)realloc(vis, sizeof(cand_t) * cap);
                    }
                    vis[n].dist = dist;
                    vis[n].id = ids[x];
                    ++n;
                    if (nvis < visit_stride) {
                        if (visit_hits) visit_hits[qi * visit_stride + nvis] = hs;
                        if (visit_dist) visit_dist[qi * visit_stride + nvis] = dist;
                        if (visit_ids) visit_ids[qi * visit_stride + nvis] = ids[x];
                    }
                    ++nvis;
                }
            }
            if (visit_count) visit_count[qi] = nvis;

            /* S4 */
            qsort(vis, n, sizeof(cand_t), cand_less);
            for (int i = 0; i < k; ++i) {
                if ((size_t)i < n) {
                    out_dist[qi * k + i] = vis[i].dist;
                    out_ids[qi * k + i] = vis[i].id;
                } else {
                    out_dist[qi * k + i] = INFINITY;
                    out_ids[qi * k + i] = -1;
                }
            }
        }
        free(vis);
        free(r2);
        free(hit);
        free(lut);
        free(probes_d);
        free(probes);
        free(scratch);
    }
    return status;
}

int oracle_search(int d, int nlist, int nsub, int dsub, int ksub, const float* cent,
                  const float* codebooks, const int64_t* list_offsets, const uint8_t* codes,
                  const int32_t* ids, const float* queries, int64_t nq, int nprobe, int dense,
                  const float* radius, int radius_mode, float scale, float miss_penalty, int k,
                  float* out_dist, int32_t* out_ids, int32_t* probe_ids_out, float* probe_d_out,
                  uint32_t* masks_out, int64_t* visit_count, int64_t visit_stride,
                  uint64_t* visit_hits, float* visit_dist, int32_t* visit_ids) {
    return oracle_search_scored(d, nlist, nsub, dsub, ksub, cent, codebooks, list_offsets, codes, ids, queries, nq,
                                nprobe, dense, radius, radius_mode, scale, miss_penalty, 0, k, out_dist, out_ids,
                                probe_ids_out, probe_d_out, masks_out, visit_count, visit_stride, visit_hits,
                                visit_dist, visit_ids);
}

/*
 * Dynamic thresholds (Sec. 4.1 "Determining Proper Threshold": every 2-d subspace is divided into a
 * grid x grid map of cell densities; at search time the density of the cell that holds the query's
 * projection is read and a regression polynomial turns it into that query's threshold;
 * Algorithm 2: thres = poly_regressor(density_map(x, y)) with (x, y) the query's own
 * projection, taken before the centroid is subtracted).
 *   density  [nsub][grid][grid]   row = cell index along the second coordinate, column = first
 *   origin   [nsub][2]            lower corner of the grid
 *   inv_cell [nsub][2]            1 / cell size along each coordinate
 *   coef     [nsub][degree+1]     polynomial coefficients, ascending powers of the density
 *   radius   [nq][nsub]           out: max(0, polynomial(density of the cell)); projections outside the
 *                                 grid use the nearest border cell
 * fp32: cell = floor((x - origin) * inv_cell); Horner evaluation with fmaf from the highest power.
 */
int oracle_thresholds(int d, int nsub, int dsub, const float* queries, int64_t nq, int grid, int degree,
                      const float* density, const float* origin, const float* inv_cell, const float* coef,
                      float* radius) {
    if (dsub != 2 || d != nsub * dsub || grid <= 0 || degree < 0) return -2;
    for (int64_t qi = 0; qi < nq; ++qi) {
        for (int s = 0; s < nsub; ++s) {
            int cell[2];
            for (int a = 0; a < 2; ++a) {
                float t = (queries[qi * d + 2 * s + a] - origin[2 * s + a]) * inv_cell[2 * s + a];
                float f = floorf(t);
                int c = 0;
                if (f >= (float)grid) c = grid - 1;
                else if (f > 0.0f) c = (int)f;      /* NaN and negatives stay at 0 */
                if (c > grid - 1) c = grid - 1;
                cell[a] = c;
            }
            const float dens = density[((size_t)s * grid + cell[1]) * grid + cell[0]];
            const float* cf = coef + (size_t)s * (degree + 1);
            float acc = cf[degree];
            for (int i = degree - 1; i >= 0; --i) acc = fmaf(acc, dens, cf[i]);
            radius[qi * nsub + s] = acc > 0.0f ? acc : 0.0f;
        }
    }
    return 0;
}

static int float_less(const void* a, const void* b) {
    const float x = *(const float*)a, y = *(const float*)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

/*
 * Dynamic thresholds for subspaces of any width (stand-in for the density map of Sec. 4.1
 * "Determining Proper Threshold", which is a 2-d grid and exists for 2-d subspaces only).  The local
 * density around a query's projection is measured by how close its kth-nearest codebook entry is:
 * the codebook is a k-means quantizer of the residual projections, so its entries crowd where the
 * data does.  As in the paper, a per-subspace regression polynomial turns the measurement into the
 * threshold; with the coefficients (0, 1) the threshold is the kth-nearest-entry distance itself.
 *   projection  the residual against the query's nearest cluster (filtering with one probe, ties
 *               to the smaller cluster id): the frame the codebooks were trained in
 *   measurement v = sqrtf(kth smallest over the ksub entries e of |r_s - e|^2), the squared
 *               distances by the table arithmetic of S2 (fmaf chain, ascending dimension)
 *   radius[q][s] = max(0, polynomial_s(v)), Horner evaluation with fmaf from the highest power
 *   coef [nsub][degree+1], ascending powers; 1 <= kth <= ksub
 */
int oracle_thresholds_knn(int d, int nlist, int nsub, int dsub, int ksub, const float* cent, const float* codebooks,
                          const float* queries, int64_t nq, int kth, int degree, const float* coef, float* radius) {
    if (d != nsub * dsub || nlist <= 0 || ksub <= 0 || ksub > 256 || kth < 1 || kth > ksub || degree < 0) return -2;
    for (int64_t qi = 0; qi < nq; ++qi) {
        const float* q = queries + qi * d;
        int best = 0;
        float bestd = 0.0f;
        for (int c = 0; c < nlist; ++c) {
            float a = 0.0f;
            for (int j = 0; j < d; ++j) {
                const float t = q[j] - cent[(size_t)c * d + j];
                a = fmaf(t, t, a);
            }
            if (c == 0 || a < bestd) {
                bestd = a;
                best = c;
            }
        }
        for (int s = 0; s < nsub; ++s) {
            float d2[256];
            for (int e = 0; e < ksub; ++e) {
                float a = 0.0f;
                for (int j = 0; j < dsub; ++j) {
                    const float r = q[s * dsub + j] - cent[(size_t)best * d + s * dsub + j];
                    const float t = r - codebooks[((size_t)s * ksub + e) * dsub + j];
                    a = fmaf(t, t, a);
                }
                d2[e] = a;
            }
            qsort(d2, (size_t)ksub, sizeof(float), float_less);
            const float v = sqrtf(d2[kth - 1]);
            const float* cf = coef + (size_t)s * (degree + 1);
            float acc = cf[degree];
            for (int i = degree - 1; i >= 0; --i) acc = fmaf(acc, v, cf[i]);
            radius[qi * nsub + s] = acc > 0.0f ? acc : 0.0f;
        }
    }
    return 0;
}

/*
 * Entry usage and locality statistics of the neighbours of a query (Sec. 3.2 "Sparsity of Codebook
 * Entries Used by Top-k Neighbors" and Sec. 3.3 "Spatial Locality of Codebook Entries Used by Top-k
 * Neighbors").  For every query a list of neighbours is given as positions into the list-contiguous
 * codes (-1 = none), normally its exact top-100.
 *   usage[q][s]      number of distinct entries of codebook s that the neighbours of q are encoded
 *                    with (the paper's usage ratio is this over ksub)
 *   rank_hist[s][r]  += 1 for every (query, neighbour) whose entry in subspace s is the r-th closest
 *                    entry (r = 0 closest) to the residual projection of the query against the
 *                    centroid of the neighbour's list; entries are ordered by (squared distance,
 *                    entry number).  Its running sum over r is the CDF of Sec. 3.3.
 * rank_hist is accumulated into (the caller zeroes it); distances in the search's fp32 arithmetic.
 */
int oracle_entry_stats(int d, int nlist, int nsub, int dsub, int ksub, const float* cent, const float* codebooks,
                       const int64_t* list_offsets, const uint8_t* codes, const float* queries, int64_t nq,
                       const int64_t* neighbor_pos, int k, int32_t* usage, int64_t* rank_hist) {
    if (d != nsub * dsub || ksub <= 0 || ksub > 256) return -2;
    const int64_t ntotal = list_offsets[nlist];
    float* dist = (float*)malloc(sizeof(float) * (size_t)ksub);
    uint8_t* used = (uint8_t*)malloc((size_t)nsub * ksub);
    int status = 0;
    for (int64_t qi = 0; qi < nq; ++qi) {
        const float* q = queries + qi * d;
        memset(used, 0, (size_t)nsub * ksub);
        for (int j = 0; j < k; ++j) {
            const int64_t x = neighbor_pos[qi * k + j];
            if (x < 0) continue;
            if (x >= ntotal) { status = -3; continue; }
            int c = 0;                                   /* the list that holds position x */
            while (!(list_offsets[c] <= x && x < list_offsets[c + 1])) ++c;
            for (int s = 0; s < nsub; ++s) {
                const int own = codes[(size_t)x * nsub + s];
                if (own >= ksub) { status = -3; continue; }
                used[(size_t)s * ksub + own] = 1;
                for (int e = 0; e < ksub; ++e) {
                    const float* entry = codebooks + ((size_t)s * ksub + e) * dsub;
                    float d2 = 0.0f;
                    for (int t = 0; t < dsub; ++t) {
                        float res = q[s * dsub + t] - cent[(size_t)c * d + s * dsub + t];
                        float u = res - entry[t];
                        d2 = fmaf(u, u, d2);
                    }
                    dist[e] = d2;
                }
                int rank = 0;
                for (int e = 0; e < ksub; ++e)
                    if (dist[e] < dist[own] || (dist[e] == dist[own] && e < own)) ++rank;
                rank_hist[(size_t)s * ksub + rank] += 1;
            }
        }
        for (int s = 0; s < nsub; ++s) {
            int n = 0;
            for (int e = 0; e < ksub; ++e) n += used[(size_t)s * ksub + e];
            usage[qi * nsub + s] = n;
        }
    }
    free(used);
    free(dist);
    return status;
}

/* cand_less for similarities: larger first, then smaller id */
static int cand_greater(const void* a, const void* b) {
    const cand_t* x = (const cand_t*)a;
    const cand_t* y = (const cand_t*)b;
    if (x->dist > y->dist) return -1;
    if (x->dist < y->dist) return 1;
    if (x->id < y->id) return -1;
    if (x->id > y->id) return 1;
    return 0;
}

static float dot_f32(const float* a, const float* b, int n) {
    float acc = 0.0f;
    for (int j = 0; j < n; ++j) acc = fmaf(a[j], b[j], acc);
    return acc;
}

/*
 * Search under the inner-product similarity (header comment; Sec. 4.2 "Inner Product Similarity
 * Support").  Arguments as oracle_search; probe_d and visit_dist hold similarities; dense != 0
 * selects every entry.  miss_penalty < 0 asks for the default P = sum over subspaces of
 * (radius*scale)^2.
 */
int oracle_search_ip(int d, int nlist, int nsub, int dsub, int ksub, const float* cent,
                     const float* codebooks, const int64_t* list_offsets, const uint8_t* codes,
                     const int32_t* ids, const float* queries, int64_t nq, int nprobe, int dense,
                     const float* radius, int radius_mode, float scale, float miss_penalty, int k,
                     float* out_sim, int32_t* out_ids, int32_t* probe_ids_out, float* probe_ip_out,
                     uint32_t* masks_out, int64_t* visit_count, int64_t visit_stride,
                     uint64_t* visit_hits, float* visit_sim, int32_t* visit_ids) {
    if (d != nsub * dsub || ksub <= 0 || ksub > 256 || nsub > 64) return -2;
    if (nprobe <= 0 || nprobe > nlist || k <= 0) return -1;
    if (!dense && radius == NULL) return -1;

#pragma omp parallel
    {
        cand_t* scratch = (cand_t*)malloc(sizeof(cand_t) * (size_t)nlist);
        float* lut = (float*)malloc(sizeof(float) * (size_t)nsub * ksub);
        uint8_t* hit = (uint8_t*)malloc((size_t)nsub * ksub);
        float* r2 = (float*)malloc(sizeof(float) * (size_t)nsub);
        size_t cap = 1024, n = 0;
        cand_t* vis = (cand_t*)malloc(sizeof(cand_t) * cap);

#pragma omp for schedule(dynamic, 1)
        for (int64_t qi = 0; qi < nq; ++qi) {
            const float* q = queries + qi * d;
            /* S1: the nprobe largest inner products, ties to the smaller cluster id */
            for (int c = 0; c < nlist; ++c) {
                scratch[c].dist = dot_f32(q, cent + (size_t)c * d, d);
                scratch[c].id = c;
            }
            qsort(scratch, (size_t)nlist, sizeof(cand_t), cand_greater);
            if (probe_ids_out)
                for (int p = 0; p < nprobe; ++p) probe_ids_out[qi * nprobe + p] = scratch[p].id;
            if (probe_ip_out)
                for (int p = 0; p < nprobe; ++p) probe_ip_out[qi * nprobe + p] = scratch[p].dist;

            float P = 0.0f;
            if (!dense) {
                const float* rad = radius_mode == 1 ? radius + qi * nsub : radius;
                float acc = 0.0f;
                for (int s = 0; s < nsub; ++s) {
                    float r = rad[s] * scale;
                    r2[s] = r * r;
                    acc = acc + r2[s];
                }
                P = miss_penalty >= 0.0f ? miss_penalty : acc;
            }

            /* S2: one table per query */
            for (int s = 0; s < nsub; ++s) {
                uint32_t mrow[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                for (int e = 0; e < ksub; ++e) {
                    const float* entry = codebooks + ((size_t)s * ksub + e) * dsub;
                    float d2 = 0.0f;
                    for (int j = 0; j < dsub; ++j) {
                        float t = q[s * dsub + j] - entry[j];
                        d2 = fmaf(t, t, d2);
                    }
                    float en2 = dot_f32(entry, entry, dsub);
                    int h = dense ? 1 : (d2 <= r2[s] + en2);
                    lut[(size_t)s * ksub + e] = dot_f32(q + s * dsub, entry, dsub);
                    hit[(size_t)s * ksub + e] = (uint8_t)h;
                    if (h) mrow[e >> 5] |= 1u << (e & 31);
                }
                if (masks_out)
                    for (int p = 0; p < nprobe; ++p)
                        memcpy(masks_out + (((size_t)qi * nprobe + p) * nsub + s) * 8, mrow, sizeof(mrow));
            }

            n = 0;
            int64_t nvis = 0;
            for (int p = 0; p < nprobe; ++p) {
                const int c = scratch[p].id;
                const float base = scratch[p].dist; /* q.c */
                for (int64_t x = list_offsets[c]; x < list_offsets[c + 1]; ++x) {
                    const uint8_t* code = codes + (size_t)x * nsub;
                    float S = base;
                    int m = 0;
                    uint64_t hs = 0;
                    for (int s = 0; s < nsub; ++s) {
                        int e = code[s];
                        if (e < ksub && hit[(size_t)s * ksub + e]) {
                            S = S + lut[(size_t)s * ksub + e];
                            hs |= (uint64_t)1 << s;
                        } else {
                            m += 1;
                        }
                    }
                    float sim = (m == 0) ? S : fmaf(-(float)m, P, S);
                    if (n == cap) {
                        cap *= 2;
                        vis = (cand_t*)realloc(vis, sizeof(cand_t) * cap);
                    }
                    vis[n].dist = sim;
                    vis[n].id = ids[x];
                    ++n;
                    if (nvis < visit_stride) {
                        if (visit_hits) visit_hits[qi * visit_stride + nvis] = hs;
                        if (visit_sim) visit_sim[qi * visit_stride + nvis] = sim;
                        if (visit_ids) visit_ids[qi * visit_stride + nvis] = ids[x];
                    }
                    ++nvis;
                }
            }
            if (visit_count) visit_count[qi] = nvis;

            qsort(vis, n, sizeof(cand_t), cand_greater);
            for (int i = 0; i < k; ++i) {
                if ((size_t)i < n) {
                    out_sim[qi * k + i] = vis[i].dist;
                    out_ids[qi * k + i] = vis[i].id;
                } else {
                    out_sim[qi * k + i] = -INFINITY;
                    out_ids[qi * k + i] = -1;
                }
            }
        }
        free(vis);
        free(r2);
        free(hit);
        free(lut);
        free(scratch);
    }
    return 0;
}

// Sparsity-aware list scan of the 16 x 8 product quantizer through the inverted index from codebook
// entries to points (paper Sec. 5.1, Algorithm 1: `Map`; Sec. 5.3, paragraph after Algorithm 2: per
// subspace the points behind the selected entries accumulate the table value, all other points get
// the constant without a look-up).  Same results as the code-streaming kernel (scan16x8.cu); the
// work follows the number of selected entries instead of the list lengths.
//
// One persistent CTA of 16 warps per SM loops over (query, probe slice) items; the whole codebook
// lives in registers (thread = subspace c = tid & 15, entries u, u + 32, ... with u = tid / 16), as
// in the 16-warp instance of the streaming kernel.  The probed clusters of an item are taken in
// tiles: as many consecutive clusters as fit the accumulators (8192 points) and the item pool.
//   P1  selection: every thread evaluates its 8 entries per cluster with the defining arithmetic
//       (residual, fma chain, d2 <= r2); every selected entry becomes an item of a pool - the
//       selective L2-LUT in compact form - that already carries where the points behind the entry
//       are (two 16-bit offsets of the map, requested while the other entries are evaluated) and
//       the value to add (hit count + squared distance in 48-bit fixed point);
//   P2  a prefix sum over the items' point counts numbers all (point, selected entry) pairs;
//   P3  scatter: thread t takes pairs 8 t .. 8 t + 7 of each round (one binary search, then a walk),
//       loads their 16-bit positions - all loads of a round are independent and in flight together -
//       and adds the item's value to the point's accumulators with two shared-memory integer adds
//       (exact to 2^-44 of the largest threshold and independent of the order of the adds);
//   P4  sweep over the tile's points: hit count and sum give the value S + m P; points that no
//       selected entry reached cost one shared-memory load; candidates go to the CTA's
//       candidate buffer under the same protocol as in the streaming kernel (scan16x8.cuh).
// A list longer than 8192 points is processed chunk by chunk with the same items (their point
// locations are looked up again for every chunk, then P2-P4).
// Degenerate thresholds (an infinite or undefined radius, for which no fixed-point scale exists)
// and sums too small for the fixed point are evaluated point by point from the codes with the
// oracle's own operation order (slow, rare).
#include "scan16x8.cuh"

namespace ivfpq {

namespace {

using namespace pq16x8;

constexpr int kNT = 512;
constexpr int kEP = kNT / kW;       // entries per pass of the selection (32)
constexpr int kNE = 256 / kEP;      // entries per thread (8)
constexpr int kCap = 4096;          // candidate buffer slots
constexpr int kSoftLimit = 2048;    // compaction is requested once this many candidates are buffered
constexpr int kPoolCap = 4096;      // items: a single cluster can select at most 16 x 256 entries
constexpr int kAccCap = kMapChunk;  // accumulators (points of one tile)
constexpr int kTMax = 16;           // clusters per tile (one centroid-fetching warp each)
constexpr int kPairsPerThread = 8;  // pairs a thread scatters per round
constexpr int kFixBits = 48;        // fixed-point bits below the power of two above the largest threshold
static_assert(kSoftLimit + 32 * (kNT / 32) <= kCap && IVFPQ_MAX_K < kSoftLimit, "candidate buffer limits");
static_assert(kTMax <= kNT / 32 && kTMax <= 16, "tile limits (4-bit cluster slot in an item)");

struct TileUnit {
    long long b0;   // first 32-point code block of the list (stage dumps, point-by-point evaluation)
    int g0;         // global index (into the id array) of the first point of the chunk in work
    int n;          // points of that chunk
    int acc0;       // first accumulator slot
    int chunk;      // global number of that chunk
    int pi;         // probe index within the query's probe list
    int p0;         // first point of the list
};

__host__ __device__ inline int map_smem_bytes(int nprobe, bool dbg) {
    int b = kCap * 8 + kPoolCap * 16 + 2 * (kPoolCap + 8) * 4 + 2 * kAccCap * 4;
    b += kMetaCap * (int)sizeof(ProbeMeta);
    b += (kD + kTMax * kD + 16) * 4;
    b += kTMax * (int)sizeof(TileUnit) + kTMax * 4;
    b += 96 + kQuickWords * 4;
    if (dbg) b += kTMax * kW * 8 * 4 + (nprobe + 1) * 8;
    return (b + 255) & ~255;
}

// Value of one point evaluated from its codes in the oracle's order (ascending subspace; selected
// entries add their squared distance, the others count as misses; S + m P as one fused
// multiply-add).  `cw` = the point's 16 code bytes as stored (byte i = subspace (lanep ^ i) & 15).
__device__ __noinline__ float point_value(const ScanParams& p, int sc, const float* qs, const float* cs, const float* r2,
                                          float P, uint4 cw, int lanep, int* hits_out) {
    const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
    float S = 0.0f;
    int m = 0, val = 0, hits = 0;
#pragma unroll 1
    for (int s = 0; s < kW; ++s) {
        const int i = (s ^ lanep) & (kW - 1);
        const int code = (int)((w[i >> 2] >> (8 * (i & 3))) & 0xFFu);
        bool hit = false;
        float d2 = 0.0f;
        if (code < p.ksub) {
            const float* ent = p.cbt + ((size_t)code * kW + s) * kDsub;
#pragma unroll
            for (int j = 0; j < kDsub; ++j) {
                const float r = __fsub_rn(qs[s * kDsub + j], cs[s * kDsub + j]);
                const float tt = __fsub_rn(r, __ldg(ent + j));
                d2 = __fmaf_rn(tt, tt, d2);
            }
            hit = d2 <= r2[s];
        }
        hits += hit ? 1 : 0;
        if (hit) S = __fadd_rn(S, d2);
        else ++m;
        val += !hit ? 2 : (d2 <= __fmul_rn(0.25f, r2[s]) ? 0 : 1);
    }
    *hits_out = hits;
    if (sc == IVFPQ_SCORE_HIT_COUNT) return (float)m;
    if (sc == IVFPQ_SCORE_REWARD_PENALTY) return (float)val;
    return m ? __fmaf_rn((float)m, P, S) : S;
}

template <bool DBG, int SCORE_T>
__global__ void __launch_bounds__(kNT, 1) scan16x8_map_kernel(const ScanParams p, const int64_t nitems) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    const int warp = tid >> 5;
    const int c = tid & (kW - 1);   // subspace of this thread in the selection
    const int u = tid / kW;         // its first entry (0..31)
    const int ksub = p.ksub;
    const int sc = SCORE_T >= 0 ? SCORE_T : p.score;

    unsigned char* a = smem;
    unsigned long long* kbuf = reinterpret_cast<unsigned long long*>(a);
    a += (size_t)kCap * 8;
    uint4* pool = reinterpret_cast<uint4*>(a);   // x: entry | subspace << 8 | cluster slot << 12 | outer << 16, y / z: words to add, w: first position
    a += (size_t)kPoolCap * 16;
    uint32_t* ilen = reinterpret_cast<uint32_t*>(a);   // per item: points behind the entry in the chunk in work
    a += (size_t)(kPoolCap + 8) * 4;
    uint32_t* cum = reinterpret_cast<uint32_t*>(a);    // exclusive prefix of the counts of the chunk in work; [total] = all pairs
    a += (size_t)(kPoolCap + 8) * 4;
    uint32_t* accH = reinterpret_cast<uint32_t*>(a);   // hit count << 26 | high 26 bits of the fixed-point sum
    a += (size_t)kAccCap * 4;
    uint32_t* accL = reinterpret_cast<uint32_t*>(a);   // sum of the low 26 bits of the terms
    a += (size_t)kAccCap * 4;
    ProbeMeta* meta = reinterpret_cast<ProbeMeta*>(a);
    a += kMetaCap * sizeof(ProbeMeta);
    float* qs = reinterpret_cast<float*>(a);
    float* cent_s = qs + kD;           // [kTMax][128]
    float* r2 = cent_s + kTMax * kD;   // [16]
    a += (kD + kTMax * kD + 16) * 4;
    TileUnit* unit = reinterpret_cast<TileUnit*>(a);
    a += kTMax * sizeof(TileUnit);
    int* tile_items = reinterpret_cast<int*>(a);
    a += kTMax * 4;
    unsigned long long* tau_p = reinterpret_cast<unsigned long long*>(a);
    int* cnt_p = reinterpret_cast<int*>(a + 8);
    int* ntrans_p = cnt_p + 1;
    int* pool_cnt = cnt_p + 2;
    int* wsum = cnt_p + 4;   // [16] warp totals of the prefix sum
    a += 96;
    int* hist_p = reinterpret_cast<int*>(a);
    a += kQuickWords * 4;
    uint32_t* hitmask = reinterpret_cast<uint32_t*>(a);                           // DBG only: [kTMax][16][8]
    long long* vprefix = reinterpret_cast<long long*>(a + kTMax * kW * 8 * 4);    // DBG only
    TopkState t{kbuf, cnt_p, tau_p, hist_p};

    // ---- codebook: all eight entries of a thread in registers ----
    float cbr[kNE][kDsub];
#pragma unroll
    for (int m = 0; m < kNE; ++m) {
        const int e = u + kEP * m;
        const float4* src = reinterpret_cast<const float4*>(p.cbt + ((size_t)e * kW + c) * kDsub);
        const float4 v0 = __ldg(src), v1 = __ldg(src + 1);
        cbr[m][0] = v0.x; cbr[m][1] = v0.y; cbr[m][2] = v0.z; cbr[m][3] = v0.w;
        cbr[m][4] = v1.x; cbr[m][5] = v1.y; cbr[m][6] = v1.z; cbr[m][7] = v1.w;
    }
    for (int i = tid; i < kAccCap; i += kNT) {
        accH[i] = 0;
        accL[i] = 0;
    }
    topk_quick_init<kNT>(hist_p);   // contains a barrier

    // An item of the pool from its (entry, subspace, cluster slot) word and the entry's squared distance:
    // the words a point behind the entry receives, and where those points are in the chunk in work.
    auto finish_item = [&](int idx, uint32_t x, float d2, float thr_s, float up) {
        const int e = x & 255, cs_ = (x >> 8) & 15, ts = (x >> 12) & 15;
        const uint32_t outer = d2 <= __fmul_rn(0.25f, thr_s) ? 0u : 1u;   // reward/penalty: not within the inner sphere
        uint32_t wy = 1u << 26, wz = 0u;
        if (sc == IVFPQ_SCORE_DISTANCE) {
            const unsigned long long f = __float2ull_rz(__fmul_rn(d2, up));
            wy |= (uint32_t)(f >> 26);
            wz = (uint32_t)f & 0x3FFFFFFu;
        } else if (sc == IVFPQ_SCORE_REWARD_PENALTY) {
            wz = outer;
        }
        wz |= (uint32_t)ts << 28;
        const int n = unit[ts].n;
        const uint32_t ow = n > 0 ? __ldg(p.map_off + ((size_t)unit[ts].chunk * kW + cs_) * 256 + e) : 0u;
        pool[idx] = make_uint4(x, wy, wz, (uint32_t)unit[ts].g0 * (uint32_t)kW + (uint32_t)(cs_ * n) + (ow & 0xFFFFu));
        ilen[idx] = ow >> 16;
    };

    // P1 for cluster slot `ts`: this thread's eight entries of subspace c; the selected ones become
    // items.  The hit lanes only drop (entry word, d2) into the pool; the items are completed by all
    // lanes of the warp together afterwards (a warp has a hit in most passes but in few lanes).
    auto select_cluster = [&](int ts, float thr, float up) {
        const float* cs = cent_s + ts * kD;
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
        float d2v[kNE];
        uint32_t bal[kNE];
        int total = 0;
#pragma unroll
        for (int m = 0; m < kNE; ++m) {
            float d2 = 0.0f;
#pragma unroll
            for (int j = 0; j < kDsub; ++j) {
                const float tt = __fsub_rn(r[j], cbr[m][j]);
                d2 = __fmaf_rn(tt, tt, d2);
            }
            d2v[m] = d2;
            const bool hit = (u + kEP * m) < ksub && d2 <= thr;
            bal[m] = __ballot_sync(0xFFFFFFFFu, hit);
            total += __popc(bal[m]);
        }
        if (total == 0) return;   // warp-uniform
        int base = 0;
        if (lane == 0) {
            base = atomicAdd(pool_cnt, total);
            atomicAdd(&tile_items[ts], total);
        }
        base = __shfl_sync(0xFFFFFFFFu, base, 0);
        const uint32_t lt = (1u << lane) - 1u;
        int idx0 = base;
#pragma unroll
        for (int m = 0; m < kNE; ++m) {
            if ((bal[m] >> lane) & 1u) {
                const int e = u + kEP * m;
                const int idx = idx0 + __popc(bal[m] & lt);
                if (idx < kPoolCap)
                    *reinterpret_cast<uint2*>(&pool[idx]) =
                        make_uint2((uint32_t)e | ((uint32_t)c << 8) | ((uint32_t)ts << 12), __float_as_uint(d2v[m]));
                if (DBG) atomicOr(&hitmask[(ts * kW + c) * 8 + (e >> 5)], 1u << (e & 31));
            }
            idx0 += __popc(bal[m]);
        }
        __syncwarp();
        for (int i = base + lane; i < min(base + total, kPoolCap); i += 32) {
            const uint2 st = *reinterpret_cast<const uint2*>(&pool[i]);
            finish_item(i, st.x, __uint_as_float(st.y), r2[(st.x >> 8) & 15], up);
        }
    };

    int est = 512;   // expected items per cluster: sizes the next tile (adapts to what the tiles show)

    for (int64_t item = blockIdx.x; item < nitems; item += gridDim.x) {
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
        }
        if (DBG && tid == 96) fill_visit_prefix(p, q, vprefix);
        float P = 0.0f, thr = 0.0f, up = 0.0f, down = 0.0f, down26 = 0.0f;
        bool degenerate = false;

        for (int t0 = 0; t0 < np_item; t0 += kMetaCap) {
            const int nt = min(kMetaCap, np_item - t0);
            if (tid >= 128 && tid < 128 + nt) meta[tid - 128] = load_probe_meta(p, q, split + (t0 + tid - 128) * p.nsplit);
            __syncthreads();
            if (t0 == 0) {
                P = miss_constant(p, r2);
                thr = r2[c];
                // fixed-point scale: terms are below 2^ex, kept to 2^(ex - 48)
                float r2max = 0.0f;
                bool fin = true;
#pragma unroll
                for (int s = 0; s < kW; ++s) {
                    fin = fin && (r2[s] < __int_as_float(0x7F800000));   // false for +inf and for NaN
                    r2max = fmaxf(r2max, r2[s]);
                }
                degenerate = !fin;
                int ex = 0;
                if (fin) (void)frexpf(r2max, &ex);
                ex = max(ex, -78);
                up = ldexpf(1.0f, kFixBits - ex);
                down = ldexpf(1.0f, ex - kFixBits);
                down26 = ldexpf(1.0f, ex - kFixBits + 26);
            }
            // value of a point that no selected entry reached
            const float allmiss = sc == IVFPQ_SCORE_HIT_COUNT ? (float)kW
                                  : (sc == IVFPQ_SCORE_REWARD_PENALTY ? (float)(2 * kW) : __fmaf_rn((float)kW, P, 0.0f));

            int j = 0;
            while (j < nt) {
                // ---- tile: clusters j .. j + T - 1 of this window (every thread computes the same) ----
                int T = 0, pts = 0;
                bool multi = false;
                const int tmax = max(1, min(kTMax, kPoolCap / est));
                while (j + T < nt && T < tmax) {
                    const int len = meta[j + T].len;
                    if (len > kMapChunk) {
                        if (T == 0) {
                            T = 1;
                            multi = true;
                        }
                        break;
                    }
                    if (pts + len > kAccCap) break;
                    pts += len;
                    ++T;
                }
                if (tid < T) {
                    const ProbeMeta m = meta[j + tid];
                    TileUnit un;
                    un.b0 = m.b0;
                    un.g0 = un.p0 = m.p0;
                    un.n = min(m.len, kMapChunk);
                    int a0 = 0;
                    for (int i = 0; i < tid; ++i) a0 += meta[j + i].len;
                    un.acc0 = a0;
                    un.chunk = p.chunk_first[m.cl];
                    un.pi = split + (t0 + j + tid) * p.nsplit;
                    unit[tid] = un;
                    tile_items[tid] = 0;
                }
                if (tid == 32) *pool_cnt = 0;
                if (warp < T) cp_async16(cent_s + warp * kD + 4 * lane, p.cent + (int64_t)meta[j + warp].cl * kD + 4 * lane);
                if (DBG)
                    for (int i = tid; i < T * kW * 8; i += kNT) hitmask[i] = 0;
                cp_async_wait_all();
                __syncthreads();

                const int list_len = meta[j].len;
                const int nch = multi ? (list_len + kMapChunk - 1) / kMapChunk : 1;
                // ---- P1: selection ----
                int total = 0;
                if (!degenerate || DBG) {
                    for (int ts = 0; ts < T; ++ts) select_cluster(ts, thr, up);
                    __syncthreads();
                    total = *pool_cnt;
                    if (total > kPoolCap) {
                        // the pool overflowed: keep the longest prefix of clusters that fits (a single
                        // cluster always does) and select again
                        int Tn = 1, sum = tile_items[0];
                        while (Tn < T && sum + tile_items[Tn] <= kPoolCap) sum += tile_items[Tn++];
                        __syncthreads();   // everybody has read the counts
                        if (tid < Tn) tile_items[tid] = 0;
                        if (tid == 32) *pool_cnt = 0;
                        __syncthreads();
                        T = Tn;
                        for (int ts = 0; ts < T; ++ts) select_cluster(ts, thr, up);
                        __syncthreads();
                        total = *pool_cnt;
                    }
                    int mx = 0;
                    for (int ts = 0; ts < T; ++ts) mx = max(mx, tile_items[ts]);
                    est = max(64, mx + (mx >> 2) + 32);
                    if (DBG && p.masks)
                        for (int i = tid; i < T * kW * 8; i += kNT)
                            p.masks[((size_t)q * p.nprobe + unit[i / (kW * 8)].pi) * kW * 8 + i % (kW * 8)] = hitmask[i];
                }
                if (degenerate) total = 0;

                for (int ch = 0; ch < nch; ++ch) {
                    if (ch > 0) {   // next chunk of a long list (the previous sweep ended with a barrier)
                        if (tid == 0) {
                            unit[0].g0 += kMapChunk;
                            unit[0].n = min(kMapChunk, list_len - ch * kMapChunk);
                            unit[0].chunk += 1;
                        }
                        __syncthreads();
                        // the items stay; where their points are changes with the chunk
                        for (int i = tid; i < total; i += kNT) {
                            const uint32_t x = pool[i].x;
                            const int n = unit[0].n;
                            const uint32_t ow = __ldg(p.map_off + ((size_t)unit[0].chunk * kW + ((x >> 8) & 15)) * 256 + (x & 255));
                            pool[i].w = (uint32_t)unit[0].g0 * (uint32_t)kW + (uint32_t)(((x >> 8) & 15) * n) + (ow & 0xFFFFu);
                            ilen[i] = ow >> 16;
                        }
                        __syncthreads();
                    }
                    if (total > 0) {
                        // ---- P2: exclusive prefix sum of the point counts of this chunk's items ----
                        {
                            const int i0 = tid * 8;
                            uint32_t v[8], sum = 0;
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj) {
                                uint32_t x = 0;
                                if (i0 + jj < total) x = ilen[i0 + jj];
                                v[jj] = sum;
                                sum += x;
                            }
                            uint32_t incl = sum;
#pragma unroll
                            for (int o = 1; o < 32; o <<= 1) {
                                const uint32_t x = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                                if (lane >= o) incl += x;
                            }
                            if (lane == 31) wsum[warp] = (int)incl;
                            __syncthreads();
                            uint32_t wbase = 0, tot = 0;
#pragma unroll
                            for (int w = 0; w < kNT / 32; ++w) {
                                const uint32_t x = (uint32_t)wsum[w];
                                if (w < warp) wbase += x;
                                tot += x;
                            }
                            const uint32_t excl = wbase + incl - sum;
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj)
                                if (i0 + jj < total) cum[i0 + jj] = excl + v[jj];
                            if (tid == 0) cum[total] = tot;
                            __syncthreads();
                        }
                        // ---- P3: scatter the items' values to the points behind their entries ----
                        const uint32_t tot = cum[total];
                        for (uint32_t pbase = 0; pbase < tot; pbase += kNT * kPairsPerThread) {
                            const uint32_t pfirst = pbase + tid * kPairsPerThread;
                            if (pfirst < tot) {
                                int lo = 0, hi = total;   // cum[lo] <= pfirst < cum[hi]
                                while (hi - lo > 1) {
                                    const int mid = (lo + hi) >> 1;
                                    if (cum[mid] <= pfirst) lo = mid;
                                    else hi = mid;
                                }
                                int i = lo;
                                uint32_t c0 = cum[i], next = cum[i + 1], start = pool[i].w;
                                int pos[kPairsPerThread], it[kPairsPerThread];
#pragma unroll
                                for (int jj = 0; jj < kPairsPerThread; ++jj) {
                                    const uint32_t pp = pfirst + jj;
                                    it[jj] = -1;
                                    if (pp < tot) {
                                        while (pp >= next) {
                                            ++i;
                                            c0 = next;
                                            next = cum[i + 1];
                                        }
                                        if (it[jj > 0 ? jj - 1 : 0] != i) start = pool[i].w;
                                        pos[jj] = (int)__ldg(p.map_pos + start + (pp - c0));
                                        it[jj] = i;
                                    }
                                }
#pragma unroll
                                for (int jj = 0; jj < kPairsPerThread; ++jj) {
                                    if (it[jj] >= 0) {
                                        const uint4 w = pool[it[jj]];
                                        const int slot = unit[w.z >> 28].acc0 + pos[jj];
                                        atomicAdd(&accH[slot], w.y);
                                        const uint32_t lz = w.z & 0x3FFFFFFu;
                                        if (lz != 0u) atomicAdd(&accL[slot], lz);
                                    }
                                }
                            }
                        }
                        __syncthreads();
                    }

                    // ---- P4: sweep the tile's points ----
                    int ut = 0, pos = tid;
                    while (true) {
                        const unsigned long long tau = *tau_p;
                        const uint32_t tau_hi = (uint32_t)(tau >> 32), tau_lo = (uint32_t)tau;
                        const uint32_t tau_cut = tau_hi + (tau_lo != 0 ? 1u : 0u);
                        bool stop = false, halt = false;
                        while (ut < T) {
                            const TileUnit un = unit[ut];
                            while (pos - lane < un.n) {
                                if (pos < un.n) {
                                    const uint32_t h = accH[un.acc0 + pos];
                                    float dist = allmiss;
                                    int cnt = (int)(h >> 26);
                                    bool slow = degenerate;
                                    if (h != 0u) {
                                        const uint32_t l = accL[un.acc0 + pos];
                                        accH[un.acc0 + pos] = 0u;
                                        if (sc != IVFPQ_SCORE_HIT_COUNT) accL[un.acc0 + pos] = 0u;
                                        const int m = kW - cnt;
                                        if (sc == IVFPQ_SCORE_HIT_COUNT) {
                                            dist = (float)m;
                                        } else if (sc == IVFPQ_SCORE_REWARD_PENALTY) {
                                            dist = (float)(2 * m + (int)l);
                                        } else {
                                            // high and low words converted separately (three roundings of 2^-24: far
                                            // inside the tolerance, and no 64-bit conversion in the loop)
                                            const uint32_t hs = h & 0x3FFFFFFu;
                                            const float S = __fmaf_rn((float)hs, down26, __fmul_rn((float)l, down));
                                            dist = m ? __fmaf_rn((float)m, P, S) : S;
                                            slow = slow || (hs == 0u && l < (1u << 20));   // too few significant bits: evaluate from the codes
                                        }
                                    }
                                    const int lp = un.g0 - un.p0 + pos;   // position in the list
                                    unsigned long long hs = 0;
                                    if (DBG || slow) {
                                        const uint4 cw = __ldg(reinterpret_cast<const uint4*>(p.codes_il) + (un.b0 + (lp >> 5)) * 32 + (lp & 31));
                                        if (slow) {
                                            int hits;
                                            dist = point_value(p, sc, qs, cent_s + ut * kD, r2, P, cw, lp & 31, &hits);
                                            if (degenerate) cnt = hits;
                                        }
                                        if (DBG) {
                                            const uint32_t wv[4] = {cw.x, cw.y, cw.z, cw.w};
                                            const uint32_t* hm = hitmask + ut * kW * 8;
#pragma unroll
                                            for (int i = 0; i < kW; ++i) {
                                                const uint32_t code = (wv[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                                                const int s = ((lp & 31) ^ i) & (kW - 1);
                                                hs |= (unsigned long long)((hm[s * 8 + (code >> 5)] >> (code & 31)) & 1u) << s;
                                            }
                                            if (__popcll(hs) != cnt) atomicOr(p.status, kFlagMap);   // map and codes disagree
                                            const int64_t vi = vprefix[un.pi] + lp;
                                            if (vi < p.visit_stride) {
                                                if (p.visit_hits) p.visit_hits[q * p.visit_stride + vi] = hs;
                                                if (p.visit_dist) p.visit_dist[q * p.visit_stride + vi] = dist;
                                                if (p.visit_ids) p.visit_ids[q * p.visit_stride + vi] = p.ids[un.g0 + pos];
                                            }
                                        }
                                    }
                                    const uint32_t ab = __float_as_uint(dist);
                                    if (ab < tau_cut && (ab != tau_hi || (uint32_t)__ldg(p.ids + un.g0 + pos) < tau_lo)) {
                                        const int slot = atomicAdd(cnt_p, 1);
                                        if (slot < kCap) kbuf[slot] = make_key(dist, (uint32_t)(un.g0 + pos));
                                        else atomicOr(p.status, kFlagOverflow);
                                        stop |= slot >= kSoftLimit;
                                    }
                                }
                                pos += kNT;
                                halt = __any_sync(0xFFFFFFFFu, stop);
                                if (halt) break;
                            }
                            if (halt) break;
                            ++ut;
                            pos = tid;
                        }
                        // the barrier that ends the sweep (accumulators clean, pool and units free); a set flag
                        // means that some warp met the soft limit: the buffer is compacted and the sweep resumes
                        if (!__syncthreads_or(halt || ut < T)) break;
                        compact_candidates<kNT, kCap>(t, ntrans_p, hist_p, p.k, p.ids, kSoftLimit / 2);
                    }
                }
                j += T;
            }
        }

        emit_topk<kNT, kCap>(p, t, ntrans_p, hist_p, q, split);
    }
}

template <bool DBG, int SCORE_T>
cudaError_t launch_map_inst(const ScanParams& sp, int64_t grid, int64_t nitems, int nprobe, cudaStream_t st) {
    const size_t smem = (size_t)map_smem_bytes(nprobe, DBG);
    auto kern = scan16x8_map_kernel<DBG, SCORE_T>;
    const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)grid, kNT, smem, st>>>(sp, nitems);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_scan16x8_map(const ivfpq_index* ix, const ScanParams& sp, int64_t nitems, bool debug, int nprobe,
                                 cudaStream_t st) {
    int64_t grid = ix->sm_count;
    if (grid > nitems) grid = nitems;
    if (debug) return launch_map_inst<true, -1>(sp, grid, nitems, nprobe, st);
    if (sp.score == IVFPQ_SCORE_HIT_COUNT) return launch_map_inst<false, IVFPQ_SCORE_HIT_COUNT>(sp, grid, nitems, nprobe, st);
    if (sp.score == IVFPQ_SCORE_REWARD_PENALTY) return launch_map_inst<false, IVFPQ_SCORE_REWARD_PENALTY>(sp, grid, nitems, nprobe, st);
    return launch_map_inst<false, IVFPQ_SCORE_DISTANCE>(sp, grid, nitems, nprobe, st);
}

}  // namespace ivfpq

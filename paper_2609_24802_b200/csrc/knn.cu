// Generated exact kNN relation consumed by a neighbour sum (paper Section 4.9, generated kNN).
//
// The paper's kernel scans every source for every query and skips the sort of a tile that cannot
// improve the retained keys.  Here the cell directory of the radius relation orders the search
// instead, which keeps the result exact (keys are compared, never approximated) and removes the
// quadratic scan on inputs of roughly even density:
//
//   knn_cells_kernel  one warp per cell.  The points are binned with a cell edge a little above a
//                     search radius h chosen so that a ball of radius h holds about 2k points on
//                     average.  Every point closer than h to a query of the cell lies in the
//                     27-cell stencil, so a query that finds k keys <= h^2 there is finished: no
//                     point outside the stencil can have a smaller key.  The stencil is staged in
//                     shared memory (candidates farther than h from the bounding box of the
//                     cell's points are dropped), one candidate per lane is tested against eight
//                     queries, accepted keys are compacted into per-query lists by ballots, and a
//                     list that fills up is cut back to its k smallest keys, which also tightens
//                     that query's acceptance threshold.
//   knn_rings_kernel  one warp per query that found fewer than k keys within h (sparse regions,
//                     tiny inputs): it walks cubic shells of cells outwards and stops when the
//                     k-th key is no larger than the squared distance to the unexplored region, or
//                     when the whole grid has been visited.
//
// Keys are (fp32 squared distance by direct differences in a fixed operation order, source index);
// the k smallest are selected by rank counting, which also leaves them in key order.
#include "radius_shared.cuh"

namespace tiga {

constexpr int KNN_STAGE_CAP = 384;                 // staged candidates per chunk
constexpr int KNN_QCAP = 96;                       // list entries per query (cells kernel)
constexpr int KNN_QSTRIDE = KNN_QCAP + 1;
constexpr int KNN_RING_CAP = 128;                  // list entries of the rings kernel
constexpr int KNN_STAGE_BYTES = (KNN_STAGE_CAP + STAGE_PAD) * 16;
constexpr int KNN_LIST_BYTES = (QB * KNN_QSTRIDE * 8 + 15) / 16 * 16;
constexpr int KNN_TMP_BYTES = TIGA_KNN_MAX_K * 8;
constexpr int KNN_MISC_BYTES = QB * 16 + QB * 4 * 2;
constexpr int KNN_PER_WARP = KNN_STAGE_BYTES + KNN_LIST_BYTES + KNN_TMP_BYTES + KNN_MISC_BYTES;
constexpr int KNN_RING_BLOCKS = 148 * 4;

struct KnnParams {
    RadiusParams rp;        // points, features, plan
    int k;
    float h2;               // square of the search radius: the cells kernel accepts keys <= h2
    float prune2;           // staging drops candidates farther than this (squared) from the cell's points
    float hmin;             // smallest cell edge, shortened by 2^-10 (guarantee of the rings kernel)
    float* out;
    int32_t* nbr;
    float* nbr_d2;
    int32_t* queue;         // queries the cells kernel could not finish
    int32_t* queue_n;
};

// the key's squared distance: operation order fixed, nothing contracted
static __device__ __forceinline__ float key_d2(const float qx, const float qy, const float qz,
                                               const float cx, const float cy, const float cz) {
    const float dx = __fsub_rn(qx, cx), dy = __fsub_rn(qy, cy), dz = __fsub_rn(qz, cz);
    return __fadd_rn(__fadd_rn(__fmul_rn(dx, dx), __fmul_rn(dy, dy)), __fmul_rn(dz, dz));
}

static __device__ __forceinline__ bool key_less(const float2 a, const float2 b) {
    return a.y < b.y || (a.y == b.y && __float_as_int(a.x) < __float_as_int(b.x));
}

// Keeps the min(n, k) smallest keys of lq[0, n) and leaves them sorted in lq[0, min(n, k)).
// Rank counting: keys are distinct (indices are), so the ranks are a permutation.  U entries per lane.
template <int U>
static __device__ __forceinline__ int select_k_u(float2* lq, float2* tmp, const int n, const int k, const int lane) {
    float2 e[U];
    int rank[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int t = lane + 32 * u;
        e[u] = t < n ? lq[t] : make_float2(__int_as_float(0x7fffffff), __int_as_float(0x7f800000));
        rank[u] = 0;
    }
    for (int t = 0; t < n; ++t) {
        const float2 b = lq[t];
#pragma unroll
        for (int u = 0; u < U; ++u) rank[u] += key_less(b, e[u]) ? 1 : 0;
    }
    __syncwarp();
#pragma unroll
    for (int u = 0; u < U; ++u)
        if (lane + 32 * u < n && rank[u] < k) tmp[rank[u]] = e[u];
    __syncwarp();
    const int m = n < k ? n : k;
    if (lane < m) lq[lane] = tmp[lane];
    __syncwarp();
    return m;
}

static __device__ __noinline__ int select_k(float2* lq, float2* tmp, const int n, const int k, const int lane) {
    if (n <= 32) return select_k_u<1>(lq, tmp, n, k, lane);
    if (n <= 64) return select_k_u<2>(lq, tmp, n, k, lane);
    if (n <= 96) return select_k_u<3>(lq, tmp, n, k, lane);
    return select_k_u<5>(lq, tmp, n, k, lane);
}

// Writes the row of query i from its m <= k selected keys (sorted): indices, distances, neighbour sum.
static __device__ __forceinline__ void emit_row(const KnnParams& P, const int i, const float2* top, const int m, const int lane) {
    const int k = P.k, F = P.rp.F;
    if (lane < k) {
        const bool v = lane < m;
        if (P.nbr) P.nbr[(size_t)i * k + lane] = v ? __float_as_int(top[lane].x) : -1;
        if (P.nbr_d2) P.nbr_d2[(size_t)i * k + lane] = v ? top[lane].y : __int_as_float(0x7f800000);
    }
    const float* feat = P.rp.feat;
    if (F >= 8) {
        for (int f = lane; f < F; f += 32) {
            float acc = 0.f;
            for (int t = 0; t < m; ++t) acc += __ldg(feat + (size_t)__float_as_int(top[t].x) * F + f);
            P.out[(size_t)i * F + f] = acc;
        }
    } else {
        const size_t row = lane < m ? (size_t)__float_as_int(top[lane].x) * F : 0;
        for (int f = 0; f < F; ++f) {
            float v = lane < m ? __ldg(feat + row + f) : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) P.out[(size_t)i * F + f] = v;
        }
    }
}

// ------------------------------------------------------------------------------ cells kernel
__global__ void __launch_bounds__(TRAV_THREADS) knn_cells_kernel(const __grid_constant__ KnnParams P) {
    const RadiusParams& p = P.rp;
    constexpr unsigned FULL = 0xffffffffu;
    extern __shared__ __align__(16) unsigned char s_raw[];

    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int cellid = blockIdx.x * TRAV_WARPS + wib;
    if (cellid >= p.ncells) return;
    const int qs0 = p.cell_start[cellid], qe0 = p.cell_start[cellid + 1];
    if (qs0 == qe0) return;

    unsigned char* base = s_raw + (size_t)wib * KNN_PER_WARP;
    float4* stage = reinterpret_cast<float4*>(base);                                      // x, y, z, point id
    float2* list = reinterpret_cast<float2*>(base + KNN_STAGE_BYTES);                     // (point id, d2) per query
    float2* tmp = reinterpret_cast<float2*>(base + KNN_STAGE_BYTES + KNN_LIST_BYTES);
    float4* s_q = reinterpret_cast<float4*>(base + KNN_STAGE_BYTES + KNN_LIST_BYTES + KNN_TMP_BYTES);
    int* s_n = reinterpret_cast<int*>(s_q + QB);
    float* s_tau = reinterpret_cast<float*>(s_n + QB);
    const unsigned lt_mask = (1u << lane) - 1u;
    const int k = P.k;

    // ---- the stencil as nine runs of the cell-ordered points: the x neighbours are contiguous
    int r_cs = 0, r_len = 0;
    {
        const int c0 = cellid % p.nc[0], c1 = (cellid / p.nc[0]) % p.nc[1], c2 = cellid / (p.nc[0] * p.nc[1]);
        const int y = c1 + lane % 3 - 1, z = c2 + lane / 3 - 1;
        if (lane < 9 && y >= 0 && y < p.nc[1] && z >= 0 && z < p.nc[2]) {
            const int x0 = c0 > 0 ? c0 - 1 : 0, x1 = c0 + 1 < p.nc[0] ? c0 + 1 : p.nc[0] - 1;
            const int id0 = (z * p.nc[1] + y) * p.nc[0] + x0;
            r_cs = p.cell_start[id0];
            r_len = p.cell_start[id0 + (x1 - x0 + 1)] - r_cs;
        }
    }
    int r_incl = r_len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(FULL, r_incl, o);
        if (lane >= o) r_incl += v;
    }
    const int total = __shfl_sync(FULL, r_incl, 31);

    // ---- bounding box of the cell's points, one register per lane (lane d: low, lane 3 + d: high)
    float bb;
    {
        float blo[3] = {FAR_AWAY, FAR_AWAY, FAR_AWAY}, bhi[3] = {-FAR_AWAY, -FAR_AWAY, -FAR_AWAY};
        for (int q = qs0 + lane; q < qe0; q += 32) {
            const float4 pq = p.spos[q];
            blo[0] = fminf(blo[0], pq.x); bhi[0] = fmaxf(bhi[0], pq.x);
            blo[1] = fminf(blo[1], pq.y); bhi[1] = fmaxf(bhi[1], pq.y);
            blo[2] = fminf(blo[2], pq.z); bhi[2] = fmaxf(bhi[2], pq.z);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int d = 0; d < 3; ++d) {
                blo[d] = fminf(blo[d], __shfl_xor_sync(FULL, blo[d], o));
                bhi[d] = fmaxf(bhi[d], __shfl_xor_sync(FULL, bhi[d], o));
            }
        bb = lane == 0 ? blo[0] : lane == 1 ? blo[1] : lane == 2 ? blo[2] : lane == 3 ? bhi[0] : lane == 4 ? bhi[1] : bhi[2];
    }

    // ---- stages kept candidates starting at flattened stencil position v0 until the stage is
    //      full or the stencil ends; returns the next position, the kept count in ns
    auto stage_from = [&](int v0, int& ns) -> int {
        int nst = 0;
        for (; v0 < total && nst <= KNN_STAGE_CAP - 32; v0 += 32) {
            const int v = v0 + lane;
            int r = 0;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) {                 // nine runs: a four-step search
                const int probe = __shfl_sync(FULL, r_incl, r + o - 1);
                if (probe <= v) r += o;
            }
            r = r > 8 ? 8 : r;
            const int src = __shfl_sync(FULL, r_cs, r) + (v - (__shfl_sync(FULL, r_incl, r) - __shfl_sync(FULL, r_len, r)));
            const float lx = __shfl_sync(FULL, bb, 0), ly = __shfl_sync(FULL, bb, 1), lz = __shfl_sync(FULL, bb, 2);
            const float hx = __shfl_sync(FULL, bb, 3), hy = __shfl_sync(FULL, bb, 4), hz = __shfl_sync(FULL, bb, 5);
            bool keep = false;
            float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
            if (v < total) {
                c4 = __ldg(p.spos + src);
                const float ex = fmaxf(fmaxf(lx - c4.x, c4.x - hx), 0.f);
                const float ey = fmaxf(fmaxf(ly - c4.y, c4.y - hy), 0.f);
                const float ez = fmaxf(fmaxf(lz - c4.z, c4.z - hz), 0.f);
                keep = fmaf(ez, ez, fmaf(ey, ey, ex * ex)) <= P.prune2;
            }
            const unsigned m = __ballot_sync(FULL, keep);
            if (keep) stage[nst + __popc(m & lt_mask)] = c4;
            nst += __popc(m);
        }
        if (lane < STAGE_PAD) stage[nst + lane] = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-1));
        __syncwarp();
        ns = nst;
        return v0;
    };

    const bool single = total <= KNN_STAGE_CAP - 32;          // the whole stencil fits: stage it once
    int ns = 0;
    if (single) stage_from(0, ns);

    for (int qb0 = qs0; qb0 < qe0; qb0 += QB) {
        const int nq = (qe0 - qb0 < QB) ? qe0 - qb0 : QB;
        __syncwarp();
        if (lane < QB) {
            // absent queries sit far away with a negative threshold: they accept nothing
            const float4 pq = lane < nq ? p.spos[qb0 + lane] : make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-2));
            s_q[lane] = pq;
            s_n[lane] = 0;
            s_tau[lane] = lane < nq ? P.h2 : -1.f;
        }
        __syncwarp();
        int qcnt[QB];
        float tq[QB];
#pragma unroll
        for (int q = 0; q < QB; ++q) { qcnt[q] = 0; tq[q] = s_tau[q]; }

        // all queries of the batch against the ns staged candidates
        auto scan = [&](const int ns_) {
            for (int cbase = 0; cbase < ns_; cbase += 32) {
                const float4 pj = stage[cbase + lane];
                int mx = 0;
#pragma unroll
                for (int q = 0; q < QB; ++q) {
                    const float4 qv = s_q[q];
                    const float d2 = key_d2(qv.x, qv.y, qv.z, pj.x, pj.y, pj.z);
                    const bool ok = d2 <= tq[q] && __float_as_int(pj.w) != __float_as_int(qv.w);
                    const unsigned m = __ballot_sync(FULL, ok);
                    if (ok) list[q * KNN_QSTRIDE + qcnt[q] + __popc(m & lt_mask)] = make_float2(pj.w, d2);
                    qcnt[q] += __popc(m);
                    mx = qcnt[q] > mx ? qcnt[q] : mx;
                }
                if (mx > KNN_QCAP - 32) {
                    // a list may overflow on the next trip: cut every long list back to its k smallest
                    // keys; the k-th becomes that query's threshold (later equal keys are resolved by index)
                    __syncwarp();
                    if (lane == 0) {
#pragma unroll
                        for (int q = 0; q < QB; ++q) s_n[q] = qcnt[q];
                    }
                    __syncwarp();
                    for (int q = 0; q < nq; ++q) {
                        const int n = s_n[q];
                        if (n > k) {
                            const int m = select_k(list + q * KNN_QSTRIDE, tmp, n, k, lane);
                            if (lane == 0) { s_n[q] = m; s_tau[q] = list[q * KNN_QSTRIDE + k - 1].y; }
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < QB; ++q) { qcnt[q] = s_n[q]; tq[q] = s_tau[q]; }
                }
            }
        };

        if (single) {
            scan(ns);
        } else {
            for (int v = 0; v < total;) {
                int ns2;
                v = stage_from(v, ns2);
                scan(ns2);
                __syncwarp();
            }
        }

        // ---- finish the batch: k keys within h settle a query, otherwise it is handed on
        __syncwarp();
        if (lane == 0) {
#pragma unroll
            for (int q = 0; q < QB; ++q) s_n[q] = qcnt[q];
        }
        __syncwarp();
        for (int q = 0; q < nq; ++q) {
            const int n = s_n[q];
            const int i = __float_as_int(s_q[q].w);
            if (n < k) {
                if (lane == 0) P.queue[atomicAdd(P.queue_n, 1)] = i;
            } else {
                const int m = select_k(list + q * KNN_QSTRIDE, tmp, n, k, lane);
                emit_row(P, i, list + q * KNN_QSTRIDE, m, lane);
            }
        }
    }
}

// ------------------------------------------------------------------------------ rings kernel
__global__ void __launch_bounds__(TRAV_THREADS) knn_rings_kernel(const __grid_constant__ KnnParams P) {
    const RadiusParams& p = P.rp;
    constexpr unsigned FULL = 0xffffffffu;
    __shared__ float2 s_list[TRAV_WARPS][KNN_RING_CAP + 32];
    __shared__ float2 s_tmp[TRAV_WARPS][TIGA_KNN_MAX_K];

    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    float2* list = s_list[wib];
    float2* tmp = s_tmp[wib];
    const unsigned lt_mask = (1u << lane) - 1u;
    const int k = P.k;
    const int nqueue = *P.queue_n;
    const int nwarps = gridDim.x * TRAV_WARPS;
    const int nx = p.nc[0], ny = p.nc[1], nz = p.nc[2];
    const int smax = max(nx, max(ny, nz));

    for (int t = blockIdx.x * TRAV_WARPS + wib; t < nqueue; t += nwarps) {
        const int i = P.queue[t];
        const float qx = p.pos[3 * (size_t)i], qy = p.pos[3 * (size_t)i + 1], qz = p.pos[3 * (size_t)i + 2];
        const int cid = p.cell[i];
        const int cx = cid % nx, cy = (cid / nx) % ny, cz = cid / (nx * ny);
        int cnt = 0;
        float tau = 3.0e38f;
        __syncwarp();

        // one contiguous run of cell-ordered points [a, b) against the query
        auto run = [&](const int a, const int b) {
            for (int v0 = a; v0 < b; v0 += 32) {
                const int v = v0 + lane;
                bool ok = false;
                float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
                float d2 = 0.f;
                if (v < b) {
                    c4 = __ldg(p.spos + v);
                    d2 = key_d2(qx, qy, qz, c4.x, c4.y, c4.z);
                    ok = d2 <= tau && __float_as_int(c4.w) != i;
                }
                const unsigned m = __ballot_sync(FULL, ok);
                if (ok) list[cnt + __popc(m & lt_mask)] = make_float2(c4.w, d2);
                cnt += __popc(m);
                if (cnt > KNN_RING_CAP - 32) {
                    __syncwarp();
                    cnt = select_k(list, tmp, cnt, k, lane);
                    if (cnt == k) tau = list[k - 1].y;
                }
            }
        };

        for (int s = 0; s <= smax; ++s) {
            const int z0 = max(cz - s, 0), z1 = min(cz + s, nz - 1);
            const int y0 = max(cy - s, 0), y1 = min(cy + s, ny - 1);
            const int x0 = max(cx - s, 0), x1 = min(cx + s, nx - 1);
            for (int z = z0; z <= z1; ++z)
                for (int y = y0; y <= y1; ++y) {
                    const int row = (z * ny + y) * nx;
                    if (z - cz == s || cz - z == s || y - cy == s || cy - y == s) {
                        run(p.cell_start[row + x0], p.cell_start[row + x1 + 1]);      // a face row of the shell: whole x range
                    } else {
                        if (cx - s >= 0) run(p.cell_start[row + cx - s], p.cell_start[row + cx - s + 1]);
                        if (s > 0 && cx + s < nx) run(p.cell_start[row + cx + s], p.cell_start[row + cx + s + 1]);
                    }
                }
            // every point whose cell differs by more than s from the query's in some dimension is
            // farther than s cell edges away: k keys within that distance cannot be improved
            __syncwarp();
            if (cnt >= k) {
                cnt = select_k(list, tmp, cnt, k, lane);          // sorted: the k-th key is the largest kept
                tau = list[k - 1].y;
                const float g = (float)s * P.hmin;
                if (tau <= g * g) break;
            }
            if (cx - s <= 0 && cy - s <= 0 && cz - s <= 0 && cx + s >= nx - 1 && cy + s >= ny - 1 && cz + s >= nz - 1) break;
        }
        __syncwarp();
        cnt = select_k(list, tmp, cnt, k, lane);
        emit_row(P, i, list, cnt, lane);
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------ host side
// search radius: a ball of radius h holds about 2k points at the input's mean density
static float knn_search_radius(long long n, int k, const tiga_box* box) {
    double vol = 1.0, lmax = 0.0;
    for (int d = 0; d < 3; ++d) {
        vol *= (double)box->len[d];
        lmax = (double)box->len[d] > lmax ? (double)box->len[d] : lmax;
    }
    if (n < 2) return (float)lmax;
    const double h = cbrt(2.0 * (double)k * vol / ((double)n * 4.18879020478639));
    return (float)(h < lmax ? h : lmax);
}

static tiga_status knn_check(long long n, int k, const tiga_box* box) {
    if (!box || n < 0 || k < 1) return TIGA_ERR_INVALID_ARG;
    if (k > TIGA_KNN_MAX_K) return TIGA_ERR_UNSUPPORTED;
    for (int d = 0; d < 3; ++d) {
        if (!(box->len[d] > 0.f) || !isfinite(box->len[d])) return TIGA_ERR_INVALID_ARG;
        if (box->periodic[d]) return TIGA_ERR_UNSUPPORTED;
    }
    return TIGA_OK;
}

static size_t knn_carve(KnnParams* P, void* ws, int32_t** fill, RadiusLayout* lay) {
    *lay = carve_radius(&P->rp, ws, fill);
    Carver cv(ws);
    cv.off = lay->bytes;
    P->queue = cv.take<int32_t>((size_t)P->rp.n + 1);
    P->queue_n = cv.take<int32_t>(64);
    return cv.off;
}

}  // namespace tiga

using namespace tiga;

extern "C" size_t tiga_knn_workspace_bytes(int64_t n, int32_t k, const tiga_box* box) {
    if (knn_check(n, k, box) != TIGA_OK) return 0;
    KnnParams P{};
    if (fill_params(&P.rp, n, knn_search_radius(n, k, box), box) != TIGA_OK) return 0;
    int32_t* fill;
    RadiusLayout lay;
    return knn_carve(&P, nullptr, &fill, &lay) + 256;
}

extern "C" tiga_status tiga_apply_knn(const float* pos, const float* feat, int64_t n, int32_t F, int32_t k,
                                      const tiga_box* box, float* out, int32_t* nbr, float* nbr_d2,
                                      void* ws, size_t ws_bytes, void* stream) {
    tiga_status st = knn_check(n, k, box);
    if (st != TIGA_OK) return st;
    if (F < 1) return TIGA_ERR_INVALID_ARG;
    KnnParams P{};
    const float h = knn_search_radius(n, k, box);
    st = fill_params(&P.rp, n, h, box);
    if (st != TIGA_OK) return st;
    if (n == 0) return TIGA_OK;
    if (!pos || !feat || !out || !aligned16(pos)) return TIGA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_knn_workspace_bytes(n, k, box)) return TIGA_ERR_WORKSPACE;
    int32_t* fill;
    RadiusLayout lay;
    knn_carve(&P, ws, &fill, &lay);
    P.rp.pos = pos; P.rp.feat = feat; P.rp.F = F;
    P.k = k;
    P.h2 = h * h;
    P.prune2 = P.rp.r2_hi * 1.0001f;
    float hmin = P.rp.hcell[0];
    for (int d = 1; d < 3; ++d) hmin = P.rp.hcell[d] < hmin ? P.rp.hcell[d] : hmin;
    P.hmin = hmin * (1.f - 1.f / 1024.f);
    P.out = out; P.nbr = nbr; P.nbr_d2 = nbr_d2;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    TIGA_CUDA_TRY(cudaMemsetAsync(P.queue_n, 0, sizeof(int32_t), s));
    st = run_binning(P.rp, fill, lay.nblocks, s);
    if (st != TIGA_OK) return st;
    const unsigned blocks = (unsigned)((P.rp.ncells + TRAV_WARPS - 1) / TRAV_WARPS);
    constexpr int smem = KNN_PER_WARP * TRAV_WARPS;
    TIGA_CUDA_TRY(cudaFuncSetAttribute(knn_cells_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    knn_cells_kernel<<<blocks, TRAV_THREADS, smem, s>>>(P);
    knn_rings_kernel<<<KNN_RING_BLOCKS, TRAV_THREADS, 0, s>>>(P);
    return launch_status();
}

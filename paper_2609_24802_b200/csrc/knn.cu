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
//                     cell's points are dropped), one candidate per lane is tested against four
//                     queries, accepted keys are compacted into per-query lists by ballots, and a
//                     list that fills up is cut back to its k smallest keys, which also tightens
//                     that query's acceptance threshold.
//   knn_rings_kernel  one warp per query that found fewer than k keys within h (sparse regions,
//                     tiny inputs): it walks cubic shells of cells outwards and stops when the
//                     k-th key is no larger than the squared distance to the unexplored region, or
//                     when the whole grid has been visited.
//
// Keys are (fp32 squared distance by direct differences in a fixed operation order, source index),
// held as one 64-bit integer (distance bits above the index: squared distances are never negative,
// so their bit patterns order like the values).  The k smallest of a list are selected by sorting
// 32 keys at a time across the warp with a bitonic network of shuffles and merging the sorted
// groups, which also leaves the selected keys in order, one per lane.
#include "radius_shared.cuh"
#include <type_traits>

namespace tiga {

constexpr int KQB = 4;                             // queries per batch (cells kernel)
constexpr int KNN_STAGE_CAP = 192;                 // staged candidates per chunk
constexpr int KNN_QCAP = 96;                       // list entries per query (cells kernel)
constexpr int KNN_QSTRIDE = KNN_QCAP + 1;
constexpr int KNN_RING_CAP = 128;                  // list entries of the rings kernel
constexpr int KNN_STAGE_BYTES = (KNN_STAGE_CAP + STAGE_PAD) * 16;
constexpr int KNN_LIST_BYTES = (KQB * KNN_QSTRIDE * 8 + 15) / 16 * 16;
constexpr int KNN_MISC_BYTES = KQB * 16 + KQB * 4 * 2;
constexpr int KNN_PER_WARP = KNN_STAGE_BYTES + KNN_LIST_BYTES + KNN_MISC_BYTES;
static_assert(KNN_PER_WARP % 16 == 0 && KNN_LIST_BYTES % 16 == 0, "the stage and the queries are accessed as 16-byte vectors");
constexpr int KNN_RING_BLOCKS = 148 * 4;
constexpr double KNN_BALL_FACTOR = 2.0;            // expected points within the search radius, in units of k

typedef unsigned long long knn_key;                // (bits of d2) << 32 | source index
constexpr knn_key KNN_NO_KEY = ~0ull;

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

static __device__ __forceinline__ int key_index(const knn_key v) { return (int)(unsigned)(v & 0xffffffffull); }
static __device__ __forceinline__ float key_dist(const knn_key v) { return __uint_as_float((unsigned)(v >> 32)); }

// sorts 32 keys, one per lane, ascending by lane (bitonic network)
static __device__ __forceinline__ knn_key sort32(knn_key v, const int lane) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const knn_key o = __shfl_xor_sync(0xffffffffu, v, stride);
            const bool take_min = ((lane & stride) == 0) == ((lane & size) == 0);
            v = ((v < o) == take_min) ? v : o;
        }
    }
    return v;
}

// a, b sorted ascending by lane: returns the 32 smallest of both, sorted
static __device__ __forceinline__ knn_key merge_low32(const knn_key a, const knn_key b, const int lane) {
    const knn_key br = __shfl_sync(0xffffffffu, b, 31 - lane);
    knn_key c = a < br ? a : br;                              // the 32 smallest as a bitonic sequence
#pragma unroll
    for (int stride = 16; stride > 0; stride >>= 1) {
        const knn_key o = __shfl_xor_sync(0xffffffffu, c, stride);
        c = ((c < o) == ((lane & stride) == 0)) ? c : o;
    }
    return c;
}

// two independent groups of 32 keys sorted side by side (the shuffles of one hide behind the other's)
static __device__ __forceinline__ void sort32x2(knn_key& a, knn_key& b, const int lane) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            const knn_key oa = __shfl_xor_sync(0xffffffffu, a, stride);
            const knn_key ob = __shfl_xor_sync(0xffffffffu, b, stride);
            const bool take_min = ((lane & stride) == 0) == ((lane & size) == 0);
            a = ((a < oa) == take_min) ? a : oa;
            b = ((b < ob) == take_min) ? b : ob;
        }
    }
}

// The 32 smallest keys of lq[0, n), sorted, lane t holding the t-th (KNN_NO_KEY beyond n).
// List entries are (index, d2) pairs, which read as one little-endian 64-bit key.
static __device__ __noinline__ knn_key select_sorted(const float2* lq, const int n, const int lane) {
    const knn_key* l64 = reinterpret_cast<const knn_key*>(lq);
    if (n <= 32) return sort32(lane < n ? l64[lane] : KNN_NO_KEY, lane);
    knn_key best = l64[lane];
    knn_key v = 32 + lane < n ? l64[32 + lane] : KNN_NO_KEY;
    sort32x2(best, v, lane);
    best = merge_low32(best, v, lane);
    for (int base = 64; base < n; base += 32) {
        v = sort32(base + lane < n ? l64[base + lane] : KNN_NO_KEY, lane);
        best = merge_low32(best, v, lane);
    }
    return best;
}

// Writes the row of query i from its m <= k selected keys (lane t holds the t-th): indices,
// distances, neighbour sum.
static __device__ __forceinline__ void emit_row(const KnnParams& P, const int i, const knn_key top, const int m, const int lane) {
    const int k = P.k, F = P.rp.F;
    const bool v = lane < m;
    const int id = v ? key_index(top) : -1;
    if (lane < k) {
        if (P.nbr) P.nbr[(size_t)i * k + lane] = id;
        if (P.nbr_d2) P.nbr_d2[(size_t)i * k + lane] = v ? key_dist(top) : __int_as_float(0x7f800000);
    }
    const float* feat = P.rp.feat;
    if (F >= 8) {
        for (int f0 = 0; f0 < F; f0 += 32) {
            const int f = f0 + lane;
            float acc = 0.f;
            for (int t = 0; t < m; ++t) {
                const int idt = __shfl_sync(0xffffffffu, id, t);
                if (f < F) acc += __ldg(feat + (size_t)checked(idt, P.rp.n, CHECK_POINT) * F + f);
            }
            if (f < F) P.out[(size_t)i * F + f] = acc;
        }
    } else {
        const size_t row = v ? (size_t)checked(id, P.rp.n, CHECK_POINT) * F : 0;
        for (int f = 0; f < F; ++f) {
            float x = v ? __ldg(feat + row + f) : 0.f;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
            if (lane == 0) P.out[(size_t)i * F + f] = x;
        }
    }
}

// ------------------------------------------------------------------------------ cells kernel
// queries [qs0, qe0) of one cell (the whole cell, or a slice of a dense one)
__device__ __forceinline__ void knn_cell_slice(const KnnParams& P, const int cellid, const int qs0, const int qe0, unsigned char* s_raw) {
    const RadiusParams& p = P.rp;
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;

    unsigned char* base = s_raw + (size_t)wib * KNN_PER_WARP;
    float4* stage = reinterpret_cast<float4*>(base);                                      // x, y, z, point id
    float2* list = reinterpret_cast<float2*>(base + KNN_STAGE_BYTES);                     // (point id, d2) per query
    float4* s_q = reinterpret_cast<float4*>(base + KNN_STAGE_BYTES + KNN_LIST_BYTES);
    int* s_n = reinterpret_cast<int*>(s_q + KQB);
    float* s_tau = reinterpret_cast<float*>(s_n + KQB);
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
                c4 = __ldg(p.spos + checked(src, p.n, CHECK_SLOT));
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

    int ns = 0;
    const bool single = stage_from(0, ns) >= total;           // the whole (pruned) stencil fits: staged once

    for (int qb0 = qs0; qb0 < qe0; qb0 += KQB) {
        const int nq = (qe0 - qb0 < KQB) ? qe0 - qb0 : KQB;
        __syncwarp();
        if (lane < KQB) {
            // absent queries sit far away with a negative threshold: they accept nothing
            const float4 pq = lane < nq ? p.spos[qb0 + lane] : make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-2));
            s_q[lane] = pq;
            s_n[lane] = 0;
            s_tau[lane] = lane < nq ? P.h2 : -1.f;
        }
        __syncwarp();
        int qcnt[KQB];
        float tq[KQB];
#pragma unroll
        for (int q = 0; q < KQB; ++q) { qcnt[q] = 0; tq[q] = s_tau[q]; }

        // all queries of the batch against the ns staged candidates
        auto scan = [&](const int ns_, auto width) {
            constexpr int NQ = decltype(width)::value;             // queries tested per trip (a short batch tests four)
            for (int cbase = 0; cbase < ns_; cbase += 32) {
                const float4 pj = stage[cbase + lane];
                int mx = 0;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
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
                        for (int q = 0; q < KQB; ++q) s_n[q] = qcnt[q];
                    }
                    __syncwarp();
                    for (int q = 0; q < nq; ++q) {
                        const int n = s_n[q];
                        if (n > k) {
                            float2* lq = list + q * KNN_QSTRIDE;
                            const knn_key top = select_sorted(lq, n, lane);
                            __syncwarp();
                            if (lane < k) reinterpret_cast<knn_key*>(lq)[lane] = top;
                            if (lane == k - 1) { s_n[q] = k; s_tau[q] = key_dist(top); }
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < KQB; ++q) { qcnt[q] = s_n[q]; tq[q] = s_tau[q]; }
                }
            }
        };

        if (single) {
            if (nq <= KQB / 2) scan(ns, std::integral_constant<int, KQB / 2>{});
            else scan(ns, std::integral_constant<int, KQB>{});
        } else {
            for (int v = 0; v < total;) {
                int ns2;
                v = stage_from(v, ns2);
                scan(ns2, std::integral_constant<int, KQB>{});
                __syncwarp();
            }
        }

        // ---- finish the batch: k keys within h settle a query, otherwise it is handed on
        __syncwarp();
        if (lane == 0) {
#pragma unroll
            for (int q = 0; q < KQB; ++q) s_n[q] = qcnt[q];
        }
        __syncwarp();
        for (int q = 0; q < nq; ++q) {
            const int n = s_n[q];
            const int i = __float_as_int(s_q[q].w);
            if (n < k) {
                if (lane == 0) P.queue[atomicAdd(P.queue_n, 1)] = i;
            } else {
                emit_row(P, i, select_sorted(list + q * KNN_QSTRIDE, n, lane), k, lane);
            }
        }
    }
}

// CTAs [0, cell_blocks): one warp per cell; of a cell with more than QDENSE points it takes the first
// QSLICE queries.  The CTAs behind them walk the queue of the remaining slices.
__global__ void __launch_bounds__(TRAV_THREADS) knn_cells_kernel(const __grid_constant__ KnnParams P) {
    const RadiusParams& p = P.rp;
    extern __shared__ __align__(16) unsigned char s_raw[];
    if ((int)blockIdx.x < p.cell_blocks) {
        const int w = blockIdx.x * TRAV_WARPS + (threadIdx.x >> 5);
        if (w >= p.ncells) return;
        const int qs0 = p.cell_start[w], qe0 = p.cell_start[w + 1];
        if (qs0 == qe0) return;
        knn_cell_slice(P, w, qs0, qe0 - qs0 > QDENSE ? qs0 + QSLICE : qe0, s_raw);
    } else {
        const int n = *p.q_count;
        const int w = (blockIdx.x - p.cell_blocks) * TRAV_WARPS + (threadIdx.x >> 5);
        for (int it = w; it < n; it += (gridDim.x - p.cell_blocks) * TRAV_WARPS) {
            const int2 item = p.q_items[it];
            const int qs0 = p.cell_start[item.x] + item.y, end = p.cell_start[item.x + 1];
            knn_cell_slice(P, item.x, qs0, slice_end(qs0, end), s_raw);
            __syncwarp();
        }
    }
}

// ------------------------------------------------------------------------------ rings kernel
__global__ void __launch_bounds__(TRAV_THREADS) knn_rings_kernel(const __grid_constant__ KnnParams P) {
    const RadiusParams& p = P.rp;
    constexpr unsigned FULL = 0xffffffffu;
    __shared__ float2 s_list[TRAV_WARPS][KNN_RING_CAP + 32];

    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    float2* list = s_list[wib];
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

        // cuts the list back to its (at most k) smallest keys, sorted; k keys set the threshold
        auto cut = [&]() {
            const knn_key top = select_sorted(list, cnt, lane);
            __syncwarp();
            cnt = cnt < k ? cnt : k;
            if (lane < cnt) reinterpret_cast<knn_key*>(list)[lane] = top;
            if (cnt == k) tau = key_dist(__shfl_sync(FULL, top, k - 1));
            __syncwarp();
        };

        for (int s = 0; s <= smax; ++s) {
            const int z0 = max(cz - s, 0), z1 = min(cz + s, nz - 1);
            const int y0 = max(cy - s, 0), y1 = min(cy + s, ny - 1);
            const int x0 = max(cx - s, 0), x1 = min(cx + s, nx - 1);
            const int wy = y1 - y0 + 1, nrow = (z1 - z0 + 1) * wy;
            // the (y, z) rows of the shell, sixteen at a time: every lane resolves one contiguous run of
            // cell-ordered points (a face row is one run over the whole x range, an inner row has its two
            // end cells), then the runs are walked as one flat sequence so that all loads are independent
            for (int rbase = 0; rbase < nrow; rbase += 16) {
                const int rr = rbase + (lane >> 1), side = lane & 1;
                int ra = 0, rlen = 0;
                if (rr < nrow) {
                    const int z = z0 + rr / wy, y = y0 + rr % wy;
                    const int row = (z * ny + y) * nx;
                    const bool face = z - cz == s || cz - z == s || y - cy == s || cy - y == s;
                    int xa = -1, xb = -1;                                  // cells [xa, xb]
                    if (face) { if (side == 0) { xa = x0; xb = x1; } }
                    else if (side == 0) { if (cx - s >= 0) xa = xb = cx - s; }
                    else if (s > 0 && cx + s < nx) xa = xb = cx + s;
                    if (xa >= 0) {
                        ra = p.cell_start[row + xa];
                        rlen = p.cell_start[row + xb + 1] - ra;
                    }
                }
                int rincl = rlen;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t2 = __shfl_up_sync(FULL, rincl, o);
                    if (lane >= o) rincl += t2;
                }
                const int total = __shfl_sync(FULL, rincl, 31);
                for (int v0 = 0; v0 < total; v0 += 32) {
                    const int v = v0 + lane;
                    int r = 0;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const int probe = __shfl_sync(FULL, rincl, r + o - 1);
                        if (probe <= v) r += o;
                    }
                    r = r > 31 ? 31 : r;
                    const int src = __shfl_sync(FULL, ra, r) + (v - (__shfl_sync(FULL, rincl, r) - __shfl_sync(FULL, rlen, r)));
                    bool ok = false;
                    float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    float d2 = 0.f;
                    if (v < total) {
                        c4 = __ldg(p.spos + checked(src, p.n, CHECK_SLOT));
                        d2 = key_d2(qx, qy, qz, c4.x, c4.y, c4.z);
                        ok = d2 <= tau && __float_as_int(c4.w) != i;
                    }
                    const unsigned m = __ballot_sync(FULL, ok);
                    if (ok) list[cnt + __popc(m & lt_mask)] = make_float2(c4.w, d2);
                    cnt += __popc(m);
                    if (cnt > KNN_RING_CAP - 32) {
                        __syncwarp();
                        cut();
                    }
                }
            }
            // every point whose cell differs by more than s from the query's in some dimension is
            // farther than s cell edges away: k keys within that distance cannot be improved
            __syncwarp();
            if (cnt >= k) {
                cut();                                            // sorted: the k-th key is the largest kept
                const float g = (float)s * P.hmin;
                if (tau <= g * g) break;
            }
            if (cx - s <= 0 && cy - s <= 0 && cz - s <= 0 && cx + s >= nx - 1 && cy + s >= ny - 1 && cz + s >= nz - 1) break;
        }
        __syncwarp();
        emit_row(P, i, select_sorted(list, cnt, lane), cnt < k ? cnt : k, lane);
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
    const double h = cbrt(KNN_BALL_FACTOR * (double)k * vol / ((double)n * 4.18879020478639));
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
    P.rp.cell_blocks = (int)blocks;
    knn_cells_kernel<<<counted(blocks + queue_blocks(P.rp.n)), TRAV_THREADS, smem, s>>>(P);
    knn_rings_kernel<<<counted(KNN_RING_BLOCKS), TRAV_THREADS, 0, s>>>(P);
    return launch_status();
}

namespace tiga { unsigned check_status_knn(bool reset) { return read_check_status(reset); } }

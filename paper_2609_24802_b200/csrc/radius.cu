// Generated radius relation for sm_100a (paper Section 4.9, Appendix A): the relation
//   N(i) = { j != i : |p_j - p_i| <= r }
// is produced on the fly through a cell directory and consumed directly by the message
// function and a sum reducer.  Neither the accepted edges nor the per-edge messages are
// ever written to memory.  Reverse mode keeps the membership frozen (Section 5).
//
// Passes:
//   1. binning: cell id per point + per-cell counts, exclusive scan (reduce-then-scan, no
//      inter-CTA waiting), scatter into cell order, per-cell rank sort by point id (which
//      makes the scatter stable and therefore unique), sorted copy of the positions;
//   2. traversal: one warp per query cell stages the 27 neighbouring cells (wrapped or
//      clipped, contiguous ranges of the cell-ordered points) in shared memory, tests one
//      staged candidate per lane against a batch of four or eight queries, compacts accepted
//      (source, weight) pairs into one list per query and consumes the lists with groups of
//      lanes across the feature axis, so every gathered feature row is one coalesced
//      128-bit-per-lane request.  (Lennard-Jones: radius_lj.cu; edge network: radius_mlp.cu.)
//
// Exact membership: the fp32 squared distance is only a filter.  A pair whose fp32 value
// falls within a few ulps of r^2 is re-decided in fp64 with the defining formula
// (displacement, minimum image by rint, left-to-right sum, inclusive compare), so the
// neighbour set equals the double-precision one.  Candidates are staged in their original
// coordinates; a cell whose stencil wraps around a periodic face moves the points next to the
// upper face down by the box length, which is exact in fp32, so every displacement is one
// rounded subtraction of two stored coordinates, for wrapped pairs as for interior ones.
#include "radius_shared.cuh"
#include <type_traits>

namespace tiga {

constexpr int RAD_THREADS = 256;
constexpr int SCAN_BLOCK = 2048;   // elements per CTA in the scan passes
constexpr int SCAN_SMALL_CHUNKS = 4;   // up to this many chunks are scanned by one CTA in one launch

// ------------------------------------------------------------------------------ binning
__global__ void bin_count_kernel(const RadiusParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n) return;
    int c[3];
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        const float t = __fmul_rn(p.pos[3 * (size_t)i + d], p.invh[d]);   // one rounded product
        int k = (int)floorf(t);
        k = k > p.nc[d] - 1 ? p.nc[d] - 1 : k;
        k = k < 0 ? 0 : k;
        c[d] = k;
    }
    const int id = (c[2] * p.nc[1] + c[1]) * p.nc[0] + c[0];
    p.cell[i] = id;
    if (p.u_cell) p.u_cell[i] = id;
    atomicAdd(p.cnt + id, 1);
}

__device__ __forceinline__ int block_exclusive_scan(int v, int* s_warp, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = lane < (int)(blockDim.x >> 5) ? s_warp[lane] : 0;
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        s_warp[lane] = winc - w;              // exclusive prefix of the warp totals
        if (lane == 31) s_warp[32] = winc;    // block total
    }
    __syncthreads();
    const int r = s_warp[warp] + inc - v;
    *total = s_warp[32];
    __syncthreads();
    return r;
}

// pass A: per-CTA totals of SCAN_BLOCK counts
__global__ void scan_reduce_kernel(const RadiusParams p) {
    __shared__ int s_warp[33];
    const int base = blockIdx.x * SCAN_BLOCK;
    int v = 0;
    for (int k = threadIdx.x; k < SCAN_BLOCK; k += blockDim.x)
        if (base + k < p.ncells) v += p.cnt[base + k];
    int total;
    block_exclusive_scan(v, s_warp, &total);
    if (threadIdx.x == 0) p.blocksum[blockIdx.x] = total;
}

// pass B: one CTA turns the totals into exclusive offsets (sequential over chunks)
__global__ void scan_blocksums_kernel(const RadiusParams p, int nblocks) {
    __shared__ int s_warp[33];
    __shared__ int s_carry;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < nblocks; base += blockDim.x) {
        const int k = base + threadIdx.x;
        const int v = k < nblocks ? p.blocksum[k] : 0;
        int total;
        const int ex = block_exclusive_scan(v, s_warp, &total);
        const int carry = s_carry;
        if (k < nblocks) p.blocksum[k] = carry + ex;
        __syncthreads();
        if (threadIdx.x == 0) s_carry = carry + total;
        __syncthreads();
    }
}

// exclusive scan of one chunk of SCAN_BLOCK counts plus the chunk's offset -> cell_start; returns the chunk's total
static __device__ int scan_chunk(const RadiusParams& p, const int chunk, const int offset, int* s_warp) {
    constexpr int PER = SCAN_BLOCK / RAD_THREADS;
    const int base = chunk * SCAN_BLOCK + threadIdx.x * PER;
    int v[PER];
    int sum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        v[k] = (base + k < p.ncells) ? p.cnt[base + k] : 0;
        sum += v[k];
    }
    int total;
    int ex = block_exclusive_scan(sum, s_warp, &total) + offset;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        if (base + k < p.ncells) {
            p.cell_start[base + k] = ex;
            if (p.u_cell_start) p.u_cell_start[base + k] = ex;
            queue_extra_slices(p, base + k, v[k]);          // a dense cell is cut into slices for the traversals
        }
        ex += v[k];
    }
    return total;
}

static __device__ void scan_finish(const RadiusParams& p) {
    p.cell_start[p.ncells] = p.n;
    if (p.u_cell_start) p.u_cell_start[p.ncells] = p.n;
}

// pass C: exclusive scan inside every CTA's chunk plus its offset -> cell_start
__global__ void scan_apply_kernel(const RadiusParams p) {
    __shared__ int s_warp[33];
    scan_chunk(p, blockIdx.x, p.blocksum[blockIdx.x], s_warp);
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == blockDim.x - 1) scan_finish(p);
}

// Few cells (a handful of chunks): one CTA walks the chunks and carries the offset along, which replaces the
// three scan launches of small inputs by one.
__global__ void scan_small_kernel(const RadiusParams p, const int nblocks) {
    __shared__ int s_warp[33];
    int offset = 0;
    for (int chunk = 0; chunk < nblocks; ++chunk) offset += scan_chunk(p, chunk, offset, s_warp);
    if (threadIdx.x == 0) scan_finish(p);
}

__global__ void bin_scatter_kernel(const RadiusParams p, int32_t* fill) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n) return;
    const int c = p.cell[i];
    const int slot = p.cell_start[c] + atomicAdd(fill + c, 1);
    p.order_tmp[slot] = i;
}

// One thread per scattered slot: the rank of its point among the point ids of its cell gives
// the stable order (cell, then index) and the place of the sorted copy of the position.
// Neighbouring threads belong to the same cell and read the same few slots.
static __device__ void sort_dense_cells(const RadiusParams& p, int first, int stride);

// CTAs [0, point_blocks) rank the points of ordinary cells; the CTAs behind them order the queued dense cells.
__global__ void __launch_bounds__(256) bin_sort_kernel(const RadiusParams p, const int point_blocks) {
    if ((int)blockIdx.x >= point_blocks) {
        sort_dense_cells(p, blockIdx.x - point_blocks, gridDim.x - point_blocks);
        return;
    }
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= p.n) return;
    const int id = p.order_tmp[t];
    const int c = p.cell[id];
    const int s = p.cell_start[c], e = p.cell_start[c + 1];
    if (e - s > SORT_DENSE) return;        // sort_dense_cells orders this cell
    int rank = 0;
    for (int u = s; u < e; ++u) rank += (p.order_tmp[u] < id) ? 1 : 0;
    p.order[s + rank] = id;
    if (p.u_order) p.u_order[s + rank] = id;
    p.spos[s + rank] = make_float4(p.pos[3 * (size_t)id], p.pos[3 * (size_t)id + 1], p.pos[3 * (size_t)id + 2], __int_as_float(id));
}

// Cells with more than SORT_DENSE points (rank counting is quadratic in the occupancy): one CTA per
// queued cell sorts the cell's slots by point id with a bitonic network whose comparisons all point
// the same way (first step of a merge mirrors, the others are half-cleaners), so slots behind the
// segment act as +infinity without being stored; up to SORT_SMEM ids are sorted in shared memory,
// longer segments in place in global memory.
constexpr int SORT_SMEM = 2048;       // 8 KB: the ranking CTAs of the same launch keep their occupancy
static __device__ void sort_ids_ascending(int32_t* a, int m) {
    int P = 1;
    while (P < m) P <<= 1;
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < (P >> 1); t += blockDim.x) {
                const int lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int hi = (j == (k >> 1)) ? (lo ^ (k - 1)) : (lo + j);       // mirror within the block of k, then strides
                if (hi < m) {
                    const int32_t x = a[lo], y = a[hi];
                    if (x > y) { a[lo] = y; a[hi] = x; }
                }
            }
            __syncthreads();
        }
    }
}

static __device__ void sort_dense_cells(const RadiusParams& p, const int first, const int stride) {
    __shared__ int32_t s_ids[SORT_SMEM];
    const int items = *p.b_count;
    for (int it = first; it < items; it += stride) {
        const int c = p.b_items[it];
        const int s = p.cell_start[c], m = p.cell_start[c + 1] - s;
        int32_t* a = p.order_tmp + s;
        if (m <= SORT_SMEM) {
            for (int k = threadIdx.x; k < m; k += blockDim.x) s_ids[k] = a[k];
            __syncthreads();
            a = s_ids;
        }
        sort_ids_ascending(a, m);
        for (int k = threadIdx.x; k < m; k += blockDim.x) {
            const int id = a[k];
            p.order[s + k] = id;
            if (p.u_order) p.u_order[s + k] = id;
            p.spos[s + k] = make_float4(p.pos[3 * (size_t)id], p.pos[3 * (size_t)id + 1], p.pos[3 * (size_t)id + 2], __int_as_float(id));
        }
        __syncthreads();
    }
}

// every coordinate finite and inside [0, len]: any violation raises the flag
__global__ void validate_points_kernel(const float* __restrict__ pos, long long n3, float lx, float ly, float lz, int* flag) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    bool bad = false;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n3; t += stride) {
        const float v = pos[t];
        const int d = (int)(t % 3);
        const float len = d == 0 ? lx : (d == 1 ? ly : lz);
        bad = bad || !(v >= 0.f && v <= len);          // also catches NaN
    }
    if (bad) atomicOr(flag, 1);
}

// ------------------------------------------------------------------------------ traversal

// One warp per query cell.
//   staging : the candidates of the 27-cell stencil (contiguous ranges of the cell-sorted
//             positions) are copied once into shared memory in the frame of the query cell:
//             original coordinates, except that in a dimension whose stencil wraps around a
//             periodic face the points next to the upper face move down by the box length
//             (exact).  The fp32 displacement of a pair is then accurate to half an ulp of the
//             displacement itself on both sides of a face, whatever the size of the cell.
//   phase A : every lane keeps one staged candidate in registers and tests it against the
//             queries of the cell, four (forward) or eight (backward) queries per batch (their
//             coordinates are broadcast from shared memory).  Accepted pairs are compacted with a warp ballot into one
//             contiguous list per query: (source, weight) for the forward messages,
//             (staged slot, d^2 or weight) where the displacement is needed again.
//   phase B : MODE 0 (Gaussian / distance forward) and MODE 2 (Gaussian backward): LF lanes
//             span one feature row with 128-bit accesses and 32 / LF queries advance together,
//             four gathered rows in flight per lane.  (The Lennard-Jones message has its own
//             kernel in radius_lj.cu, which visits every unordered pair once.)
// Lists hold QCAP entries per query and the stage STAGE_CAP candidates; when either fills up
// the warp drains / processes and goes on, so any density works.  A cell with more than QDENSE
// points is cut into slices of QSLICE queries: its warp takes the first, the others wait in a queue (filled
// by the binning) that the CTAs appended behind the cells' CTAs walk, so a dense cell spreads over many warps.

template <int MODE> struct TravSmem {
    // queries per batch: the forward runs fastest with short batches and seven CTAs per SM, the
    // backward (more registers per pair) with long batches
    static constexpr int TQB = MODE == 0 ? 4 : QB;
    // sized for the workload's density (about 216 candidates before pruning, 32 neighbours);
    // denser inputs only mean more chunks and drains
    static constexpr int STAGE_CAP = 256;                          // candidates staged per chunk
    static constexpr int QCAP = 80;                                // list entries per query
    static constexpr int QSTRIDE = QCAP + 5;                       // room for four padding entries; odd, so the lists of different queries fall in different banks
    static constexpr int STAGE_BYTES = (STAGE_CAP + STAGE_PAD) * 16;
    static constexpr int LIST_BYTES = (TQB * QSTRIDE * 8 + 15) / 16 * 16;
    static constexpr int MISC_BYTES = TQB * 16 + 3 * TQB * 4 + TQB * 4 * 2 + 32;   // queries, their coordinates by component, counts, totals, the cell's frame
    static constexpr int PER_WARP = STAGE_BYTES + LIST_BYTES + MISC_BYTES;
    static_assert(PER_WARP % 16 == 0 && LIST_BYTES % 16 == 0, "the stage and the queries are accessed as 16-byte vectors");
};

// MODE 0: Gaussian (DIST = false) or distance-weighted (DIST = true) forward;
// 2: Gaussian backward.  MI: some periodic dimension has a single cell (explicit minimum image).
// VEC: 0 = scalar feature accesses (F % 4 != 0, forward only); 1 = 128-bit accesses, F % 4 == 0;
// 2 = additionally F == 4 LF exactly, so the row stride is a compile-time constant.
template <int MODE, int LF, bool DIST, bool MI, int VEC>
__device__ __forceinline__ void traverse_slice(const RadiusParams& p, const int cellid, const int qs0, const int qe0, unsigned char* s_raw) {
    using SM = TravSmem<MODE>;
    constexpr int STAGE_CAP = SM::STAGE_CAP, QCAP = SM::QCAP, QSTRIDE = SM::QSTRIDE, TQB = SM::TQB;
    constexpr unsigned FULL = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;

    unsigned char* base = s_raw + (size_t)wib * SM::PER_WARP;
    float4* stage = reinterpret_cast<float4*>(base);
    float2* list = reinterpret_cast<float2*>(base + SM::STAGE_BYTES);
    float4* s_q = reinterpret_cast<float4*>(base + SM::STAGE_BYTES + SM::LIST_BYTES);   // local x, y, z, point id
    float* s_qc = reinterpret_cast<float*>(s_q + TQB);                                  // x[TQB], y[TQB], z[TQB]: read two queries at a time
    int* s_n = reinterpret_cast<int*>(s_qc + 3 * TQB);                                  // list lengths of the drain in progress
    int* s_tot = s_n + TQB;                                                              // neighbours found so far in this chunk
    float* s_frame = reinterpret_cast<float*>(s_tot + TQB);                              // thresholds [3], shifts [3]

    const int c[3] = {cellid % p.nc[0], (cellid / p.nc[0]) % p.nc[1], cellid / (p.nc[0] * p.nc[1])};
    const int F = VEC == 2 ? 4 * LF : p.F;
    const float neg_c2 = !DIST ? -1.4426950408889634f / (2.f * p.p0 * p.p0) : 0.f;   // exp(-d2/(2 s^2)) = 2^(d2 * neg_c2)
    const int fl = lane % LF, grp = lane / LF;
    // a periodic dimension with three cells or fewer has no consistent shifted frame: explicit minimum image
    const bool mi0 = MI && p.periodic[0] && p.nc[0] <= 3, mi1 = MI && p.periodic[1] && p.nc[1] <= 3, mi2 = MI && p.periodic[2] && p.nc[2] <= 3;
    constexpr int QP = 32 / LF;
    const bool fvalid = VEC == 2 ? true : fl * 4 < F;
    const unsigned lt_mask = (1u << lane) - 1u;

    // displacement query - candidate of two points in the cell's frame
    auto delta = [&](const float4& q, const float4& c4, float& dx, float& dy, float& dz) {
        dx = (MI && mi0) ? mi_delta(q.x, c4.x, p.len[0], 0.5f * p.len[0]) : q.x - c4.x;
        dy = (MI && mi1) ? mi_delta(q.y, c4.y, p.len[1], 0.5f * p.len[1]) : q.y - c4.y;
        dz = (MI && mi2) ? mi_delta(q.z, c4.z, p.len[2], 0.5f * p.len[2]) : q.z - c4.z;
    };
    // frame of this cell: in a dimension whose stencil wraps around a face, every coordinate above the
    // threshold moves down by the box length (the wrapped cell at the top when the cell touches the lower
    // face; the cell and its lower neighbour when it touches the upper face).  Both shifts are exact.
    bool face = false;
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        float thr = FAR_AWAY;
        if (p.periodic[d] && p.nc[d] >= 4) {
            if (c[d] == 0) { thr = 2.5f * p.hcell[d]; face = true; }
            else if (c[d] == p.nc[d] - 1) { thr = 1.5f * p.hcell[d]; face = true; }
        }
        if (lane == d) { s_frame[d] = thr; s_frame[3 + d] = p.len[d]; }
    }
    __syncwarp();
    auto to_frame = [&](float4 v) -> float4 {
        if (face) {
            if (v.x > s_frame[0]) v.x -= s_frame[3];
            if (v.y > s_frame[1]) v.y -= s_frame[4];
            if (v.z > s_frame[2]) v.z -= s_frame[5];
        }
        return v;
    };

    // ---- all queries of the cell against the ns candidates currently staged
    auto process_chunk = [&](const int ns, const bool first_chunk) {
        if (lane < STAGE_PAD) stage[ns + lane] = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-1));
        for (int qb0 = qs0; qb0 < qe0; qb0 += TQB) {
            const int nq = (qe0 - qb0 < TQB) ? qe0 - qb0 : TQB;
            __syncwarp();
            if (lane < TQB) {
                // absent queries of a short batch sit far away: whatever is computed for them is never used
                float4 lq4 = make_float4(FAR_AWAY, FAR_AWAY, FAR_AWAY, __int_as_float(-2));
                if (lane < nq) {
                    const float4 pq = p.spos[qb0 + lane];
                    lq4 = to_frame(pq);
                    if (MODE == 2) {
                        // the backward reads the query's own feature and cotangent rows at the start of
                        // its pass: ask for them now, they arrive during phase A
                        const size_t rowq = (size_t)__float_as_int(pq.w) * F;
                        for (int off = 0; off < F; off += 32) {
                            asm volatile("prefetch.global.L1 [%0];" ::"l"(p.feat + rowq + off));
                            asm volatile("prefetch.global.L1 [%0];" ::"l"(p.gy + rowq + off));
                        }
                    }
                }
                s_q[lane] = lq4;
                s_qc[lane] = lq4.x; s_qc[TQB + lane] = lq4.y; s_qc[2 * TQB + lane] = lq4.z;
                s_tot[lane] = 0;
            }
            __syncwarp();
            int qcnt[TQB];                         // list lengths (warp uniform, kept in registers)
#pragma unroll
            for (int q = 0; q < TQB; ++q) qcnt[q] = 0;
            bool first = first_chunk;

            auto drain = [&]() {
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                    for (int q = 0; q < TQB; ++q) { s_n[q] = qcnt[q]; s_tot[q] += qcnt[q]; }
                }
                __syncwarp();
                // four entries of weight zero behind every list (source 0 / slot 0 exist): the loops below
                // read whole steps without looking at the list length
                if (lane < TQB * 4) list[(lane >> 2) * QSTRIDE + s_n[lane >> 2] + (lane & 3)] = make_float2(__int_as_float(0), 0.f);
                __syncwarp();
                {
                    for (int pass = 0; pass * QP < nq; ++pass) {
                        const int qq = pass * QP + grp;
                        const bool valid = qq < nq && fvalid;
                        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        float px = 0.f, py = 0.f, pz = 0.f;
                        int oqq = 0;
                        if (valid) {
                            const float4 qv = s_q[qq];
                            oqq = checked(__float_as_int(qv.w), p.n, CHECK_POINT);
                            const int n = s_n[qq];
                            const float2* lq = list + qq * QSTRIDE;
                            if (MODE == 0) {
                                for (int t = 0; t < n; t += 4) {
                                    float2 e[4];
                                    float4 x[4];
#pragma unroll
                                    for (int u = 0; u < 4; ++u) {      // four gathered rows in flight
                                        e[u] = lq[t + u];
                                        const float* xr = p.feat + (size_t)checked(__float_as_int(e[u].x), p.n, CHECK_POINT) * F + fl * 4;
                                        if (VEC) x[u] = __ldg(reinterpret_cast<const float4*>(xr));
                                        else x[u] = make_float4(__ldg(xr), fl * 4 + 1 < F ? __ldg(xr + 1) : 0.f,
                                                                fl * 4 + 2 < F ? __ldg(xr + 2) : 0.f, fl * 4 + 3 < F ? __ldg(xr + 3) : 0.f);
                                    }
#pragma unroll
                                    for (int u = 0; u < 4; ++u) {
                                        acc.x = fmaf(e[u].y, x[u].x, acc.x); acc.y = fmaf(e[u].y, x[u].y, acc.y);
                                        acc.z = fmaf(e[u].y, x[u].z, acc.z); acc.w = fmaf(e[u].y, x[u].w, acc.w);
                                    }
                                }
                            } else {
                                const float4 xk = __ldg(reinterpret_cast<const float4*>(p.feat + (size_t)oqq * F) + fl);
                                const float4 gk = __ldg(reinterpret_cast<const float4*>(p.gy + (size_t)oqq * F) + fl);
                                constexpr int BU = 4;      // pairs in flight per lane
                                for (int t = 0; t < n; t += BU) {
                                    float4 e[BU], xj[BU], gj[BU];
                                    float g[BU];
#pragma unroll
                                    for (int u = 0; u < BU; ++u) {
                                        const float2 en2 = lq[t + u];
                                        g[u] = en2.y;
                                        const float4 pj = stage[__float_as_int(en2.x)];
                                        float dx, dy, dz;
                                        delta(qv, pj, dx, dy, dz);
                                        e[u] = make_float4(dx, dy, dz, 0.f);
                                        const size_t row = (size_t)checked(__float_as_int(pj.w), p.n, CHECK_POINT) * F;
                                        xj[u] = __ldg(reinterpret_cast<const float4*>(p.feat + row) + fl);
                                        gj[u] = __ldg(reinterpret_cast<const float4*>(p.gy + row) + fl);
                                    }
#pragma unroll
                                    for (int u = 0; u < BU; ++u) {
                                        acc.x = fmaf(g[u], gj[u].x, acc.x); acc.y = fmaf(g[u], gj[u].y, acc.y);
                                        acc.z = fmaf(g[u], gj[u].z, acc.z); acc.w = fmaf(g[u], gj[u].w, acc.w);
                                        float part = gk.x * xj[u].x;
                                        part = fmaf(gk.y, xj[u].y, part); part = fmaf(gk.z, xj[u].z, part); part = fmaf(gk.w, xj[u].w, part);
                                        part = fmaf(gj[u].x, xk.x, part); part = fmaf(gj[u].y, xk.y, part);
                                        part = fmaf(gj[u].z, xk.z, part); part = fmaf(gj[u].w, xk.w, part);
                                        const float gpart = g[u] * part;
                                        px = fmaf(gpart, e[u].x, px); py = fmaf(gpart, e[u].y, py); pz = fmaf(gpart, e[u].z, pz);
                                    }
                                }
                            }
                            float* orow = (MODE == 0 ? p.out : p.gfeat);
                            if (orow && VEC) {
                                float4* o = reinterpret_cast<float4*>(orow + (size_t)oqq * F) + fl;
                                if (!first) { const float4 old = *o; acc.x += old.x; acc.y += old.y; acc.z += old.z; acc.w += old.w; }
                                *o = acc;
                            } else if (orow) {
                                float* o = orow + (size_t)oqq * F + fl * 4;
                                const float a4[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                                for (int c4 = 0; c4 < 4; ++c4)
                                    if (fl * 4 + c4 < F) o[c4] = first ? a4[c4] : o[c4] + a4[c4];
                            }
                        }
                        if (MODE == 2) {
#pragma unroll
                            for (int o = LF / 2; o > 0; o >>= 1) {
                                px += __shfl_xor_sync(FULL, px, o);
                                py += __shfl_xor_sync(FULL, py, o);
                                pz += __shfl_xor_sync(FULL, pz, o);
                            }
                            if (p.gpos && qq < nq && fl == 0) {
                                const float sc = -1.f / (p.p0 * p.p0);
                                float* o = p.gpos + 3 * (size_t)oqq;
                                if (first) { o[0] = sc * px; o[1] = sc * py; o[2] = sc * pz; }
                                else { o[0] += sc * px; o[1] += sc * py; o[2] += sc * pz; }
                            }
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < TQB; ++q) qcnt[q] = 0;
                first = false;
                __syncwarp();
            };

            // ---- phase A: one staged candidate per lane against the queries of the batch
            auto phase_a = [&](const int cbase, auto full_batch) -> bool {
                constexpr bool FULLB = decltype(full_batch)::value;     // all TQB queries present: no trip tests
                const float4 pj = stage[cbase + lane];
                const int idj = __float_as_int(pj.w);
                float d2q[TQB];
                float nearest = FAR_AWAY;       // smallest |d2 - r^2| seen by this lane
                if constexpr (!MI && MODE == 0) {
                    // squared distances of two queries per packed instruction (same operations and roundings
                    // as the scalar form: a product, then two fused multiply-adds)
                    const f32x2 px = pack2(pj.x, pj.x), py = pack2(pj.y, pj.y), pz = pack2(pj.z, pj.z);
                    const f32x2* qx2 = reinterpret_cast<const f32x2*>(s_qc);
#pragma unroll
                    for (int h = 0; h < TQB / 2; ++h) {
                        if (!FULLB && 2 * h >= nq) break;
                        const f32x2 dx = sub2(qx2[h], px), dy = sub2(qx2[TQB / 2 + h], py), dz = sub2(qx2[TQB + h], pz);
                        unpack2(fma2(dz, dz, fma2(dy, dy, mul2(dx, dx))), d2q[2 * h], d2q[2 * h + 1]);
                    }
#pragma unroll
                    for (int q = 0; q < TQB; ++q) {
                        if (!FULLB && q >= nq) break;
                        if (idj == __float_as_int(s_q[q].w)) d2q[q] = FAR_AWAY;            // self (by index)
                        nearest = fminf(nearest, fabsf(d2q[q] - p.r2_mid));
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < TQB; ++q) {
                        if (!FULLB && q >= nq) break;
                        const float4 qv = s_q[q];
                        float dx, dy, dz;
                        delta(qv, pj, dx, dy, dz);
                        float d2 = fmaf(dz, dz, fmaf(dy, dy, dx * dx));
                        if (idj == __float_as_int(qv.w) || (MI && idj < 0)) d2 = FAR_AWAY; // self (by index); folded sentinels
                        nearest = fminf(nearest, fabsf(d2 - p.r2_mid));
                        d2q[q] = d2;
                    }
                }
                if (__any_sync(FULL, nearest <= p.r2_band)) {
                    // some pair lies within the fp32 error band of the cutoff: decide it in fp64 and
                    // move it clear of the band (the change of d2 is below the fp32 error itself)
#pragma unroll
                    for (int q = 0; q < TQB; ++q) {
                        if (!FULLB && q >= nq) break;
                        if (fabsf(d2q[q] - p.r2_mid) <= p.r2_band)
                            d2q[q] = exact_pair(p, __float_as_int(s_q[q].w), idj) ? fminf(d2q[q], p.r2_lo) : FAR_AWAY;
                    }
                }
                int mx = 0;
#pragma unroll
                for (int q = 0; q < TQB; ++q) {
                    if (!FULLB && q >= nq) break;
                    const bool ok = d2q[q] <= p.r2_lo;
                    const unsigned m = __ballot_sync(FULL, ok);
                    float val;
                    val = DIST ? sqrtf(d2q[q]) : fast_exp2(d2q[q] * neg_c2);
                    float2* dst = list + q * QSTRIDE + qcnt[q] + __popc(m & lt_mask);
                    if (ok) *dst = make_float2(MODE == 0 ? pj.w : __int_as_float(cbase + lane), val);
                    qcnt[q] += __popc(m);
                    mx = qcnt[q] > mx ? qcnt[q] : mx;
                }
                return mx > QCAP - 32;
            };
            // one drain site: it runs when a list may overflow on the next trip and once at the end
            // (on the first chunk the final drain also writes the zero vector of a query without neighbours)
            bool need = false;
            for (int cbase = 0;; cbase += 32) {
                const bool done = cbase >= ns;
                if (done || need) drain();
                if (done) break;
                need = (nq == TQB) ? phase_a(cbase, std::true_type{}) : phase_a(cbase, std::false_type{});
            }
            if (p.count && lane < nq) {
                const int oq = __float_as_int(s_q[lane].w);
                p.count[oq] = first_chunk ? s_tot[lane] : p.count[oq] + s_tot[lane];
            }
        }
        __syncwarp();
    };

    // ---- the 27-cell stencil as candidate ranges: lane r < 27 resolves neighbour offset r
    int r_cs = 0, r_ce = 0;
    {
        const int off[3] = {lane % 3 - 1, (lane / 3) % 3 - 1, lane / 9 - 1};
        bool ok = lane < 27;
        int q[3] = {0, 0, 0};
        bool merged = false;
#pragma unroll
        for (int d = 0; d < 3; ++d) {
            if (p.nc[d] == 1) { ok = ok && off[d] == 0; continue; }
            if (d == 0 && c[0] >= 1 && c[0] <= p.nc[0] - 2) {
                // away from the x faces the three x-adjacent cells are one contiguous range
                merged = true; ok = ok && off[0] == 0; q[0] = c[0] - 1;
                continue;
            }
            int v = c[d] + off[d];
            if (v < 0) { if (p.periodic[d]) v += p.nc[d]; else ok = false; }
            else if (v >= p.nc[d]) { if (p.periodic[d]) v -= p.nc[d]; else ok = false; }
            q[d] = v;
        }
        if (ok) {
            const int id = (q[2] * p.nc[1] + q[1]) * p.nc[0] + q[0];
            r_cs = p.cell_start[id];
            r_ce = p.cell_start[id + (merged ? 3 : 1)];
        }
    }
    // flat copy: staged slot v belongs to the range whose inclusive prefix of lengths first exceeds v
    const int r_len = r_ce - r_cs;
    int r_incl = r_len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, r_incl, o);
        if (lane >= o) r_incl += t;
    }
    const int total = __shfl_sync(FULL, r_incl, 31);

    // bounding box of the cell's own points (in the cell's frame): a candidate farther than the
    // cutoff from this box cannot be a neighbour of any of them and is not staged at all, which
    // removes about 40 % of the stencil's candidates before any pair is tested
    float blo[3] = {FAR_AWAY, FAR_AWAY, FAR_AWAY}, bhi[3] = {-FAR_AWAY, -FAR_AWAY, -FAR_AWAY};
    for (int q = qs0 + lane; q < qe0; q += 32) {
        const float4 pq = to_frame(p.spos[q]);
        const float l[3] = {pq.x, pq.y, pq.z};
#pragma unroll
        for (int d = 0; d < 3; ++d) { blo[d] = fminf(blo[d], l[d]); bhi[d] = fmaxf(bhi[d], l[d]); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int d = 0; d < 3; ++d) {
            blo[d] = fminf(blo[d], __shfl_xor_sync(FULL, blo[d], o));
            bhi[d] = fmaxf(bhi[d], __shfl_xor_sync(FULL, bhi[d], o));
        }
    // the box lives in one register per lane (lane d: low bound of dimension d, lane 3 + d: high bound) and is
    // broadcast where it is used, so that it costs the pair loops below one register instead of six
    float bb = lane == 0 ? blo[0] : lane == 1 ? blo[1] : lane == 2 ? blo[2] : lane == 3 ? bhi[0] : lane == 4 ? bhi[1] : bhi[2];
    if (mi0 && (lane == 0 || lane == 3)) bb = lane == 0 ? -FAR_AWAY : FAR_AWAY;   // a dimension folded by the explicit
    if (mi1 && (lane == 1 || lane == 4)) bb = lane == 1 ? -FAR_AWAY : FAR_AWAY;   // minimum image is not pruned
    if (mi2 && (lane == 2 || lane == 5)) bb = lane == 2 ? -FAR_AWAY : FAR_AWAY;
    // The stage fills with candidates that survive the pruning and is processed when the next step's
    // candidates might not fit, so the chunks are as full as the pruning allows (one chunk for all but dense cells).
    bool first_chunk = true;
    int nst = 0;                                                             // candidates staged (warp uniform)
    constexpr int SU = 4;                                                    // staging groups in flight
    for (int k0 = 0;; k0 += 32 * SU) {
        const bool done = k0 >= total;
        const int step = done ? 0 : (total - k0 < 32 * SU ? total - k0 : 32 * SU);
        if ((done && (nst > 0 || first_chunk)) || nst + step > STAGE_CAP) {     // the one place a chunk is processed
            __syncwarp();
            process_chunk(nst, first_chunk);
            first_chunk = false;
            nst = 0;
        }
        if (done) break;
        float4 c4[SU];
#pragma unroll
        for (int u = 0; u < SU; ++u) {                                       // all loads of the step first
            const int v = k0 + 32 * u + lane;
            int r = 0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const int probe = __shfl_sync(FULL, r_incl, r + o - 1);
                if (probe <= v) r += o;
            }
            r = r > 31 ? 31 : r;
            const int src = __shfl_sync(FULL, r_cs, r) + (v - (__shfl_sync(FULL, r_incl, r) - __shfl_sync(FULL, r_len, r)));
            c4[u] = v < total ? __ldg(p.spos + checked(src, p.n, CHECK_SLOT)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const float lx = __shfl_sync(FULL, bb, 0), ly = __shfl_sync(FULL, bb, 1), lz = __shfl_sync(FULL, bb, 2);
        const float hx = __shfl_sync(FULL, bb, 3), hy = __shfl_sync(FULL, bb, 4), hz = __shfl_sync(FULL, bb, 5);
#pragma unroll
        for (int u = 0; u < SU; ++u) {
            if (32 * u >= step) break;
            const float4 val = to_frame(c4[u]);
            const float ex = fmaxf(fmaxf(lx - val.x, val.x - hx), 0.f);
            const float ey = fmaxf(fmaxf(ly - val.y, val.y - hy), 0.f);
            const float ez = fmaxf(fmaxf(lz - val.z, val.z - hz), 0.f);
            const bool keep = k0 + 32 * u + lane < total && fmaf(ez, ez, fmaf(ey, ey, ex * ex)) <= p.r2_hi * 1.0001f;
            const unsigned m = __ballot_sync(FULL, keep);
            if (keep) stage[nst + __popc(m & lt_mask)] = val;
            nst += __popc(m);
        }
    }
}

// CTAs [0, cell_blocks): warp w takes cell w (of a cell with more than QDENSE points its first QSLICE
// queries).  The CTAs behind them walk the queue of the remaining slices.
template <int MODE, int LF, bool DIST, bool MI, int VEC = 1>
__global__ void __launch_bounds__(TRAV_THREADS, (MODE == 0 ? 7 : 0)) radius_traverse_kernel(const __grid_constant__ RadiusParams p) {
    extern __shared__ __align__(16) unsigned char s_raw[];
    if ((int)blockIdx.x < p.cell_blocks) {
        const int w = blockIdx.x * TRAV_WARPS + (threadIdx.x >> 5);
        if (w >= p.ncells) return;
        const int qs0 = p.cell_start[w], qe0 = p.cell_start[w + 1];
        if (qs0 == qe0) return;
        traverse_slice<MODE, LF, DIST, MI, VEC>(p, w, qs0, qe0 - qs0 > QDENSE ? qs0 + QSLICE : qe0, s_raw);
    } else {
        const int n = *p.q_count;
        const int w = (blockIdx.x - p.cell_blocks) * TRAV_WARPS + (threadIdx.x >> 5);
        for (int it = w; it < n; it += (gridDim.x - p.cell_blocks) * TRAV_WARPS) {
            const int2 item = p.q_items[it];
            const int qs0 = p.cell_start[item.x] + item.y, end = p.cell_start[item.x + 1];
            traverse_slice<MODE, LF, DIST, MI, VEC>(p, item.x, qs0, slice_end(qs0, end), s_raw);
            __syncwarp();
        }
    }
}

// ------------------------------------------------------------------------------ host side
static long long icbrt_floor(long long v) {
    long long c = 0;
    while ((c + 1) * (c + 1) * (c + 1) <= v) ++c;
    return c;
}

static tiga_status make_grid(long long n, float r, const tiga_box* box, int nc[3], float invh[3]) {
    if (!box || n < 0) return TIGA_ERR_INVALID_ARG;
    if (!(r > 0.f) || !isfinite(r)) return TIGA_ERR_INVALID_ARG;
    long long cap = icbrt_floor(8 * (n > 0 ? n : 1));
    cap = cap > 1024 ? 1024 : (cap < 1 ? 1 : cap);
    for (int d = 0; d < 3; ++d) {
        const float L = box->len[d];
        if (!(L > 0.f) || !isfinite(L)) return TIGA_ERR_INVALID_ARG;
        if (box->periodic[d] && !((double)r < 0.5 * (double)L)) return TIGA_ERR_INVALID_ARG;
        const double q = floor((double)L / ((double)r * (1.0 + 1.0 / 1024.0)));
        long long k = q < 1.0 ? 1 : (q > (double)cap ? cap : (long long)q);
        if (box->periodic[d] && k < 3) k = 1;
        nc[d] = (int)k;
        invh[d] = (float)((double)k / (double)L);
    }
    return TIGA_OK;
}

// bytes of the queue of extra slices: at most n / QSLICE of them exist
static size_t queue_items(size_t n) { return n / QSLICE + 2; }

RadiusLayout carve_radius(RadiusParams* p, void* ws, int32_t** fill) {
    Carver cv(ws);
    const size_t n = (size_t)p->n, nc = (size_t)p->ncells;
    const int nblocks = (int)((nc + SCAN_BLOCK - 1) / SCAN_BLOCK);
    p->cnt = cv.take<int32_t>(2 * nc + 2 + 16);     // counts, then the scatter cursors, then the length of the slice queue
    p->q_count = p->cnt + 2 * nc + 2;
    p->b_count = p->q_count + 1;
    *fill = p->cnt + nc;
    p->cell = cv.take<int32_t>(n);
    p->cell_start = cv.take<int32_t>(nc + 1);
    p->order_tmp = cv.take<int32_t>(n);
    p->order = cv.take<int32_t>(n);
    p->spos = cv.take<float4>(n);
    p->blocksum = cv.take<int32_t>((size_t)nblocks + 1);
    p->q_items = cv.take<int2>(queue_items(n));
    p->b_items = cv.take<int32_t>(n / SORT_DENSE + 2);
    return RadiusLayout{cv.off, nblocks};
}

tiga_status fill_params(RadiusParams* p, long long n, float r, const tiga_box* box) {
    int nc[3];
    float invh[3];
    tiga_status st = make_grid(n, r, box, nc, invh);
    if (st != TIGA_OK) return st;
    if (n > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    p->n = (int)n;
    p->r = r;
    bool single_periodic = false;      // some periodic dimension uses the explicit minimum image (two roundings more)
    for (int d = 0; d < 3; ++d) {
        p->nc[d] = nc[d]; p->invh[d] = invh[d];
        p->len[d] = box->len[d]; p->inv_len[d] = 1.f / box->len[d];
        p->hcell[d] = box->len[d] / (float)nc[d];
        p->periodic[d] = box->periodic[d] ? 1 : 0;
        if (p->periodic[d] && nc[d] <= 3) single_periodic = true;
    }
    p->ncells = nc[0] * nc[1] * nc[2];
    const float r2 = r * r;
    const float beta = (single_periodic ? 96.f : 32.f) * 5.9604645e-8f;
    p->r2_lo = r2 * (1.f - beta);
    p->r2_hi = r2 * (1.f + beta);
    p->r2_mid = r2;
    p->r2_band = r2 * beta * 1.25f;      // a little wider than [r2_lo, r2_hi]: nothing near the cutoff escapes the exact test
    p->r2_exact = (double)r * (double)r;
    return TIGA_OK;
}

tiga_status run_binning(RadiusParams& p, int32_t* fill, int nblocks, cudaStream_t s) {
    if (p.n == 0) return TIGA_OK;
    TIGA_CUDA_TRY(cudaMemsetAsync(p.cnt, 0, (2 * (size_t)p.ncells + 2 + 16) * sizeof(int32_t), s));
    const unsigned pb = (unsigned)((p.n + 255) / 256);
    bin_count_kernel<<<counted(pb), 256, 0, s>>>(p);
    if (nblocks <= SCAN_SMALL_CHUNKS) {
        scan_small_kernel<<<counted(1), RAD_THREADS, 0, s>>>(p, nblocks);
    } else {
        scan_reduce_kernel<<<counted(nblocks), RAD_THREADS, 0, s>>>(p);
        scan_blocksums_kernel<<<counted(1), 1024, 0, s>>>(p, nblocks);
        scan_apply_kernel<<<counted(nblocks), RAD_THREADS, 0, s>>>(p);
    }
    bin_scatter_kernel<<<counted(pb), 256, 0, s>>>(p, fill);
    const long long dense_cells = (long long)p.n / SORT_DENSE + 1;          // at most this many cells can be dense
    bin_sort_kernel<<<counted(pb + (unsigned)(dense_cells < 148 ? dense_cells : 148)), 256, 0, s>>>(p, (int)pb);
    return launch_status();
}

static int feature_lanes(int F) {
    int lf = 1;
    while (lf * 4 < F) lf <<= 1;
    return lf;
}

template <int MODE, int LF, bool DIST, bool MI>
static tiga_status launch_traverse_t(const RadiusParams& p, cudaStream_t s) {
    const unsigned blocks = (unsigned)((p.ncells + TRAV_WARPS - 1) / TRAV_WARPS);
    constexpr int smem = TravSmem<MODE>::PER_WARP * TRAV_WARPS;
    if (MODE == 0 && (p.F & 3)) {
        // scalar feature accesses (only the forward supports widths that are not multiples of 4)
        auto sk = radius_traverse_kernel<MODE == 0 ? 0 : MODE, LF, DIST, MI, MODE != 0 ? 1 : 0>;
        if (smem > 48 * 1024) TIGA_CUDA_TRY(cudaFuncSetAttribute(sk, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        return cells_then_queue(p, s, [&](const RadiusParams& q, unsigned grid) { sk<<<counted(grid), TRAV_THREADS, smem, s>>>(q); });
    }
    auto kern = p.F == 4 * LF ? radius_traverse_kernel<MODE, LF, DIST, MI, 2> : radius_traverse_kernel<MODE, LF, DIST, MI, 1>;
    if (smem > 48 * 1024) TIGA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    return cells_then_queue(p, s, [&](const RadiusParams& q, unsigned grid) { kern<<<counted(grid), TRAV_THREADS, smem, s>>>(q); });
}

template <int MODE, bool DIST, bool MI>
static tiga_status launch_traverse_lf(const RadiusParams& p, cudaStream_t s) {
    switch (feature_lanes(p.F)) {
        case 1: return launch_traverse_t<MODE, 1, DIST, MI>(p, s);
        case 2: return launch_traverse_t<MODE, 2, DIST, MI>(p, s);
        case 4: return launch_traverse_t<MODE, 4, DIST, MI>(p, s);
        case 8: return launch_traverse_t<MODE, 8, DIST, MI>(p, s);
        case 16: return launch_traverse_t<MODE, 16, DIST, MI>(p, s);
        default: return launch_traverse_t<MODE, 32, DIST, MI>(p, s);
    }
}

template <int MODE, bool DIST>
static tiga_status launch_traverse(const RadiusParams& p, cudaStream_t s) {
    bool mi = false;
    for (int d = 0; d < 3; ++d) mi = mi || (p.periodic[d] && p.nc[d] <= 3);
    return mi ? launch_traverse_lf<MODE, DIST, true>(p, s) : launch_traverse_lf<MODE, DIST, false>(p, s);
}

}  // namespace tiga

using namespace tiga;

extern "C" tiga_status tiga_radius_grid(int64_t n, float r, const tiga_box* box, int32_t ncell[3], float invh[3]) {
    int nc[3];
    float ih[3];
    tiga_status st = make_grid(n, r, box, nc, ih);
    if (st != TIGA_OK) return st;
    for (int d = 0; d < 3; ++d) {
        if (ncell) ncell[d] = nc[d];
        if (invh) invh[d] = ih[d];
    }
    return TIGA_OK;
}

extern "C" tiga_status tiga_validate_points(const float* pos, int64_t n, const tiga_box* box, int level,
                                            void* ws, size_t ws_bytes, void* stream) {
    if (!box || n < 0) return TIGA_ERR_INVALID_ARG;
    for (int d = 0; d < 3; ++d)
        if (!(box->len[d] > 0.f) || !isfinite(box->len[d])) return TIGA_ERR_INVALID_ARG;
    if (n > 0 && (!pos || !aligned16(pos))) return TIGA_ERR_INVALID_ARG;
    if (level == 0 || n == 0) return TIGA_OK;
    if (!ws || ws_bytes < 16) return TIGA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int* flag = static_cast<int*>(ws);
    TIGA_CUDA_TRY(cudaMemsetAsync(flag, 0, sizeof(int), s));
    long long blocks = (3 * n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    validate_points_kernel<<<counted((unsigned)blocks), 256, 0, s>>>(pos, 3 * n, box->len[0], box->len[1], box->len[2], flag);
    if (launch_status() != TIGA_OK) return TIGA_ERR_CUDA;
    int h = 0;
    TIGA_CUDA_TRY(cudaMemcpyAsync(&h, flag, sizeof(int), cudaMemcpyDeviceToHost, s));
    TIGA_CUDA_TRY(cudaStreamSynchronize(s));
    return h ? TIGA_ERR_INVALID_POINTS : TIGA_OK;
}

extern "C" size_t tiga_radius_workspace_bytes(int64_t n, int32_t F, float r, const tiga_box* box, int backward) {
    (void)F; (void)backward;
    RadiusParams p{};
    if (fill_params(&p, n, r, box) != TIGA_OK) return 0;
    int32_t* fill;
    return carve_radius(&p, nullptr, &fill).bytes + 256;
}

extern "C" tiga_status tiga_radius_bin(const float* pos, int64_t n, float r, const tiga_box* box,
                                       int32_t* cell, int32_t* cell_start, int32_t* order,
                                       void* ws, size_t ws_bytes, void* stream) {
    RadiusParams p{};
    tiga_status st = fill_params(&p, n, r, box);
    if (st != TIGA_OK) return st;
    if (n > 0 && (!pos || !aligned16(pos))) return TIGA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_radius_workspace_bytes(n, 0, r, box, 0)) return TIGA_ERR_WORKSPACE;
    int32_t* fill;
    const RadiusLayout lay = carve_radius(&p, ws, &fill);
    p.pos = pos; p.u_cell = cell; p.u_cell_start = cell_start; p.u_order = order;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n == 0) {
        if (cell_start) TIGA_CUDA_TRY(cudaMemsetAsync(cell_start, 0, ((size_t)p.ncells + 1) * sizeof(int32_t), s));
        return TIGA_OK;
    }
    return run_binning(p, fill, lay.nblocks, s);
}

static tiga_status radius_common(RadiusParams* p, const float* pos, const float* feat, int64_t n, int32_t F,
                                 float r, const tiga_box* box, const tiga_msg* msg_p, void* ws, size_t ws_bytes,
                                 int32_t** fill, RadiusLayout* lay, int forward_only_widths) {
    if (!msg_p) return TIGA_ERR_INVALID_ARG;
    const tiga_msg msg = *msg_p;
    tiga_status st = fill_params(p, n, r, box);
    if (st != TIGA_OK) return st;
    if (msg.kind == TIGA_MSG_LJ) {
        if (!(msg.p1 > 0.f)) return TIGA_ERR_INVALID_ARG;
        F = 4;
    } else if (msg.kind == TIGA_MSG_GAUSS || msg.kind == TIGA_MSG_DIST) {
        if (F <= 0) return TIGA_ERR_INVALID_ARG;
        if (F > 128) return TIGA_ERR_UNSUPPORTED;
        if ((F % 4) && forward_only_widths == 0) return TIGA_ERR_UNSUPPORTED;
        if (msg.kind == TIGA_MSG_GAUSS && !(msg.p0 > 0.f)) return TIGA_ERR_INVALID_ARG;
        if (n > 0 && (!feat || !aligned16(feat))) return TIGA_ERR_INVALID_ARG;
    } else {
        return TIGA_ERR_UNSUPPORTED;
    }
    if (n > 0 && (!pos || !aligned16(pos))) return TIGA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_radius_workspace_bytes(n, F, r, box, 0)) return TIGA_ERR_WORKSPACE;
    *lay = carve_radius(p, ws, fill);
    p->pos = pos; p->feat = feat; p->F = F; p->p0 = msg.p0; p->p1 = msg.p1;
    return TIGA_OK;
}

extern "C" tiga_status tiga_apply_radius(const float* pos, const float* feat, int64_t n, int32_t F,
                                         float r, const tiga_box* box, const tiga_msg* msg,
                                         float* out, int32_t* count, void* ws, size_t ws_bytes, void* stream) {
    RadiusParams p{};
    int32_t* fill;
    RadiusLayout lay;
    tiga_status st = radius_common(&p, pos, feat, n, F, r, box, msg, ws, ws_bytes, &fill, &lay, 1);
    if (st != TIGA_OK) return st;
    if (n == 0) return TIGA_OK;
    if (!out || !aligned16(out)) return TIGA_ERR_INVALID_ARG;
    p.out = out; p.count = count;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = run_binning(p, fill, lay.nblocks, s);
    if (st != TIGA_OK) return st;
    if (msg->kind == TIGA_MSG_LJ) return launch_lj_pairs(p, s);
    if (msg->kind == TIGA_MSG_DIST) return launch_traverse<0, true>(p, s);
    return launch_traverse<0, false>(p, s);
}

extern "C" tiga_status tiga_apply_radius_backward(const float* pos, const float* feat, int64_t n, int32_t F,
                                                  float r, const tiga_box* box, const tiga_msg* msg,
                                                  const float* grad_out, float* grad_feat, float* grad_pos,
                                                  void* ws, size_t ws_bytes, int reuse_plan, void* stream) {
    if (!msg) return TIGA_ERR_INVALID_ARG;
    if (msg->kind != TIGA_MSG_GAUSS) return TIGA_ERR_UNSUPPORTED;
    RadiusParams p{};
    int32_t* fill;
    RadiusLayout lay;
    tiga_status st = radius_common(&p, pos, feat, n, F, r, box, msg, ws, ws_bytes, &fill, &lay, 0);
    if (st != TIGA_OK) return st;
    if (n == 0 || (!grad_feat && !grad_pos)) return TIGA_OK;
    if (!grad_out || !aligned16(grad_out)) return TIGA_ERR_INVALID_ARG;
    if ((grad_feat && !aligned16(grad_feat)) || (grad_pos && !aligned16(grad_pos))) return TIGA_ERR_INVALID_ARG;
    p.gy = grad_out; p.gfeat = grad_feat; p.gpos = grad_pos;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!reuse_plan) {
        st = run_binning(p, fill, lay.nblocks, s);
        if (st != TIGA_OK) return st;
    }
    return launch_traverse<2, false>(p, s);
}

namespace tiga { unsigned check_status_radius(bool reset) { return read_check_status(reset); } }

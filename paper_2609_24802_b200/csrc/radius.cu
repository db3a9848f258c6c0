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
//   2. traversal: one warp per query cell walks the 27 neighbouring cells (wrapped or
//      clipped).  Lanes test candidates; accepted (source, weight) pairs are compacted
//      through shared memory and consumed with lanes across the feature axis, so every
//      gathered feature row is one coalesced request.
//
// Exact membership: the fp32 squared distance is only a filter.  A pair whose fp32 value
// falls within a few ulps of r^2 is re-decided in fp64 with the defining formula
// (displacement, minimum image by rint, left-to-right sum, inclusive compare), so the
// neighbour set equals the double-precision one.  Periodic images are formed by
// subtracting the box length from whichever of the two coordinates lies next to the upper
// face, which is exact in fp32, so wrapped pairs are as accurate as interior ones.
#include "common.cuh"
#include <math.h>

namespace tiga {

constexpr int RAD_THREADS = 256;
constexpr int RAD_WARPS = RAD_THREADS / 32;
constexpr int LIST_CAP = 64;
constexpr int SCAN_BLOCK = 2048;   // elements per CTA in the scan passes

struct RadiusParams {
    const float* pos;
    const float* feat;
    const float* gy;
    float* out;
    int32_t* count;
    float* gfeat;
    float* gpos;
    int n;
    int F;
    float r;
    float r2_lo, r2_hi;       // fp32 filter band around r^2
    double r2_exact;          // (double)r * (double)r
    float len[3];
    float inv_len[3];
    int periodic[3];
    int nc[3];
    float invh[3];
    int ncells;
    float p0, p1;             // message parameters
    // plan (workspace)
    int32_t* cell;
    int32_t* cnt;
    int32_t* cell_start;
    int32_t* order_tmp;
    int32_t* order;
    float4* spos;             // positions in cell order, .w = original point id (bit pattern)
    int32_t* blocksum;
    // optional user copies of the plan
    int32_t* u_cell;
    int32_t* u_cell_start;
    int32_t* u_order;
};

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

// pass C: exclusive scan inside every CTA's chunk plus its offset -> cell_start
__global__ void scan_apply_kernel(const RadiusParams p) {
    __shared__ int s_warp[33];
    constexpr int PER = SCAN_BLOCK / RAD_THREADS;
    const int base = blockIdx.x * SCAN_BLOCK + threadIdx.x * PER;
    int v[PER];
    int sum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        v[k] = (base + k < p.ncells) ? p.cnt[base + k] : 0;
        sum += v[k];
    }
    int total;
    int ex = block_exclusive_scan(sum, s_warp, &total) + p.blocksum[blockIdx.x];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        if (base + k < p.ncells) {
            p.cell_start[base + k] = ex;
            if (p.u_cell_start) p.u_cell_start[base + k] = ex;
        }
        ex += v[k];
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == blockDim.x - 1) {
        p.cell_start[p.ncells] = p.n;
        if (p.u_cell_start) p.u_cell_start[p.ncells] = p.n;
    }
}

__global__ void bin_scatter_kernel(const RadiusParams p, int32_t* fill) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.n) return;
    const int c = p.cell[i];
    const int slot = p.cell_start[c] + atomicAdd(fill + c, 1);
    p.order_tmp[slot] = i;
}

// One warp per cell: rank of every member among the members' point ids -> stable order,
// and the sorted copy of the positions.
__global__ void bin_sort_kernel(const RadiusParams p) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= p.ncells) return;
    const int s = p.cell_start[warp], e = p.cell_start[warp + 1];
    for (int t = s + lane; t < e; t += 32) {
        const int id = p.order_tmp[t];
        int rank = 0;
        for (int u = s; u < e; ++u) rank += (p.order_tmp[u] < id) ? 1 : 0;
        p.order[s + rank] = id;
        if (p.u_order) p.u_order[s + rank] = id;
        p.spos[s + rank] = make_float4(p.pos[3 * (size_t)id], p.pos[3 * (size_t)id + 1], p.pos[3 * (size_t)id + 2], __int_as_float(id));
    }
}

// ------------------------------------------------------------------------------ traversal
// The defining predicate in double precision (same operations as the plain definition).
__device__ __noinline__ bool exact_within(const RadiusParams& p, const float4& a, const float4& b) {
    const float pa[3] = {a.x, a.y, a.z}, pb[3] = {b.x, b.y, b.z};
    double d2 = 0.0;
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        double t = __dsub_rn((double)pa[d], (double)pb[d]);
        if (p.periodic[d]) {
            const double L = (double)p.len[d];
            t = __dsub_rn(t, __dmul_rn(L, rint(__ddiv_rn(t, L))));
        }
        const double sq = __dmul_rn(t, t);
        d2 = (d == 0) ? sq : __dadd_rn(d2, sq);
    }
    return d2 <= p.r2_exact;
}

struct CellWalk {
    int cs, ce;          // candidate slots [cs, ce)
    float qs[3];         // subtract from the query coordinate (box length where the neighbour cell wrapped upwards)
    float js[3];         // subtract from the candidate coordinate (where it wrapped downwards)
};

// neighbour cell `k` (0..26) of cell (cx,cy,cz); returns false when it does not exist
__device__ __forceinline__ bool neighbour_cell(const RadiusParams& p, const int c[3], int k, CellWalk* w) {
    const int off[3] = {k % 3 - 1, (k / 3) % 3 - 1, k / 9 - 1};
    int q[3];
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        w->qs[d] = 0.f; w->js[d] = 0.f;
        if (p.nc[d] == 1) {
            if (off[d] != 0) return false;
            q[d] = 0;
            continue;
        }
        int v = c[d] + off[d];
        if (v < 0) {
            if (!p.periodic[d]) return false;
            v += p.nc[d]; w->js[d] = p.len[d];
        } else if (v >= p.nc[d]) {
            if (!p.periodic[d]) return false;
            v -= p.nc[d]; w->qs[d] = p.len[d];
        }
        q[d] = v;
    }
    const int id = (q[2] * p.nc[1] + q[1]) * p.nc[0] + q[0];
    w->cs = p.cell_start[id];
    w->ce = p.cell_start[id + 1];
    return true;
}

// fp32 displacement p_q - p_j (minimum image) and squared distance
__device__ __forceinline__ float displacement(const RadiusParams& p, const float qsh[3], const float4& pj,
                                              const CellWalk& w, float D[3]) {
    const float pjv[3] = {pj.x, pj.y, pj.z};
#pragma unroll
    for (int d = 0; d < 3; ++d) {
        float t = qsh[d] - (pjv[d] - w.js[d]);
        if (p.periodic[d] && p.nc[d] == 1) t -= p.len[d] * rintf(t * p.inv_len[d]);
        D[d] = t;
    }
    return fmaf(D[2], D[2], fmaf(D[1], D[1], D[0] * D[0]));
}

// MODE 0: GAUSS/DIST forward   1: LJ forward   2: GAUSS backward
template <int MODE>
__global__ void __launch_bounds__(RAD_THREADS) radius_kernel(const RadiusParams p, int kind) {
    __shared__ int s_id[RAD_WARPS][LIST_CAP];
    __shared__ float s_g[RAD_WARPS][LIST_CAP];
    __shared__ float s_d[MODE == 2 ? RAD_WARPS : 1][3][LIST_CAP];

    const int lane = threadIdx.x & 31;
    const int wib = threadIdx.x >> 5;
    const int cellid = blockIdx.x * RAD_WARPS + wib;
    if (cellid >= p.ncells) return;
    const int qs = p.cell_start[cellid], qe = p.cell_start[cellid + 1];
    if (qs == qe) return;
    const int c[3] = {cellid % p.nc[0], (cellid / p.nc[0]) % p.nc[1], cellid / (p.nc[0] * p.nc[1])};
    const int F = p.F;
    const float inv2s2 = (MODE != 1 && kind == TIGA_MSG_GAUSS) ? 1.f / (2.f * p.p0 * p.p0) : 0.f;
    const float inv_s2 = (MODE == 2) ? 1.f / (p.p0 * p.p0) : 0.f;

    for (int q = qs; q < qe; ++q) {
        const float4 pq = p.spos[q];
        const int oq = __float_as_int(pq.w);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};     // MODE 0: features lane+32k; MODE 1: Fx,Fy,Fz,e; MODE 2: grad_feat
        float gp[3] = {0.f, 0.f, 0.f};           // MODE 2: per-lane share of grad_pos
        float xk[4] = {0.f, 0.f, 0.f, 0.f}, gk[4] = {0.f, 0.f, 0.f, 0.f};
        if (MODE == 2) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (lane + 32 * k < F) {
                    xk[k] = p.feat[(size_t)oq * F + lane + 32 * k];
                    gk[k] = p.gy[(size_t)oq * F + lane + 32 * k];
                }
        }
        int nacc = 0;      // neighbours found (warp uniform)
        int fill = 0;      // entries waiting in the list (warp uniform)

        auto consume = [&]() {
            __syncwarp();
            if (MODE == 0) {
                for (int t = 0; t < fill; ++t) {
                    const size_t row = (size_t)s_id[wib][t] * F;
                    const float g = s_g[wib][t];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (lane + 32 * k < F) acc[k] = fmaf(g, __ldg(p.feat + row + lane + 32 * k), acc[k]);
                }
            } else if (MODE == 2) {
                for (int t = 0; t < fill; ++t) {
                    const size_t row = (size_t)s_id[wib][t] * F;
                    const float g = s_g[wib][t];
                    float part = 0.f;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (lane + 32 * k < F) {
                            const float xj = __ldg(p.feat + row + lane + 32 * k);
                            const float gj = __ldg(p.gy + row + lane + 32 * k);
                            acc[k] = fmaf(g, gj, acc[k]);
                            part = fmaf(gk[k], xj, part);
                            part = fmaf(gj, xk[k], part);
                        }
                    const float gpart = g * part;
#pragma unroll
                    for (int d = 0; d < 3; ++d) gp[d] = fmaf(gpart, s_d[MODE == 2 ? wib : 0][d][t], gp[d]);
                }
            }
            fill = 0;
            __syncwarp();
        };

        for (int k27 = 0; k27 < 27; ++k27) {
            CellWalk w;
            if (!neighbour_cell(p, c, k27, &w)) continue;
            const float qsh[3] = {pq.x - w.qs[0], pq.y - w.qs[1], pq.z - w.qs[2]};
            for (int base = w.cs; base < w.ce; base += 32) {
                const int j = base + lane;
                bool ok = false;
                float D[3] = {0.f, 0.f, 0.f};
                float d2 = 0.f;
                float4 pj = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j < w.ce && j != q) {
                    pj = p.spos[j];
                    d2 = displacement(p, qsh, pj, w, D);
                    if (d2 <= p.r2_hi) {
                        ok = true;
                        if (d2 > p.r2_lo) ok = exact_within(p, pq, pj);
                    }
                }
                if (MODE == 1) {
                    if (ok) {
                        const float inv = 1.f / d2;
                        const float qq = p.p1 * p.p1 * inv;
                        const float q3 = qq * qq * qq;
                        const float fs = 24.f * p.p0 * (2.f * q3 * q3 - q3) * inv;
                        acc[0] = fmaf(fs, D[0], acc[0]);
                        acc[1] = fmaf(fs, D[1], acc[1]);
                        acc[2] = fmaf(fs, D[2], acc[2]);
                        acc[3] += 2.f * p.p0 * (q3 * q3 - q3);
                    }
                    nacc += __popc(__ballot_sync(0xffffffffu, ok));
                } else {
                    const unsigned m = __ballot_sync(0xffffffffu, ok);
                    if (ok) {
                        const int slot = fill + __popc(m & ((1u << lane) - 1u));
                        s_id[wib][slot] = __float_as_int(pj.w);
                        s_g[wib][slot] = (kind == TIGA_MSG_GAUSS) ? __expf(-d2 * inv2s2) : sqrtf(d2);
                        if (MODE == 2) {
                            s_d[MODE == 2 ? wib : 0][0][slot] = D[0];
                            s_d[MODE == 2 ? wib : 0][1][slot] = D[1];
                            s_d[MODE == 2 ? wib : 0][2][slot] = D[2];
                        }
                    }
                    const int add = __popc(m);
                    fill += add;
                    nacc += add;
                    if (fill > LIST_CAP - 32) consume();
                }
            }
        }
        if (MODE != 1 && fill > 0) consume();

        if (MODE == 0) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (lane + 32 * k < F) p.out[(size_t)oq * F + lane + 32 * k] = acc[k];
        } else if (MODE == 1) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], o);
            if (lane == 0) reinterpret_cast<float4*>(p.out)[oq] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        } else {
            if (p.gfeat) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (lane + 32 * k < F) p.gfeat[(size_t)oq * F + lane + 32 * k] = acc[k];
            }
            if (p.gpos) {
#pragma unroll
                for (int d = 0; d < 3; ++d) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) gp[d] += __shfl_xor_sync(0xffffffffu, gp[d], o);
                }
                if (lane < 3) p.gpos[3 * (size_t)oq + lane] = -inv_s2 * (lane == 0 ? gp[0] : (lane == 1 ? gp[1] : gp[2]));
            }
        }
        if (p.count && lane == 0) p.count[oq] = nacc;
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

struct RadiusLayout {
    size_t bytes;
    int nblocks;
};

static RadiusLayout carve_radius(RadiusParams* p, void* ws, int32_t** fill) {
    Carver cv(ws);
    const size_t n = (size_t)p->n, nc = (size_t)p->ncells;
    const int nblocks = (int)((nc + SCAN_BLOCK - 1) / SCAN_BLOCK);
    p->cnt = cv.take<int32_t>(2 * nc + 2);          // counts, then the scatter cursors
    *fill = p->cnt + nc;
    p->cell = cv.take<int32_t>(n);
    p->cell_start = cv.take<int32_t>(nc + 1);
    p->order_tmp = cv.take<int32_t>(n);
    p->order = cv.take<int32_t>(n);
    p->spos = cv.take<float4>(n);
    p->blocksum = cv.take<int32_t>((size_t)nblocks + 1);
    return RadiusLayout{cv.off, nblocks};
}

static tiga_status fill_params(RadiusParams* p, long long n, float r, const tiga_box* box) {
    int nc[3];
    float invh[3];
    tiga_status st = make_grid(n, r, box, nc, invh);
    if (st != TIGA_OK) return st;
    if (n > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    p->n = (int)n;
    p->r = r;
    bool single_periodic = false;
    for (int d = 0; d < 3; ++d) {
        p->nc[d] = nc[d]; p->invh[d] = invh[d];
        p->len[d] = box->len[d]; p->inv_len[d] = 1.f / box->len[d];
        p->periodic[d] = box->periodic[d] ? 1 : 0;
        if (p->periodic[d] && nc[d] == 1) single_periodic = true;
    }
    p->ncells = nc[0] * nc[1] * nc[2];
    const float r2 = r * r;
    const float beta = (single_periodic ? 64.f : 16.f) * 5.9604645e-8f;
    p->r2_lo = r2 * (1.f - beta);
    p->r2_hi = r2 * (1.f + beta);
    p->r2_exact = (double)r * (double)r;
    return TIGA_OK;
}

static tiga_status run_binning(RadiusParams& p, int32_t* fill, int nblocks, cudaStream_t s) {
    if (p.n == 0) return TIGA_OK;
    TIGA_CUDA_TRY(cudaMemsetAsync(p.cnt, 0, (2 * (size_t)p.ncells + 2) * sizeof(int32_t), s));
    const unsigned pb = (unsigned)((p.n + 255) / 256);
    bin_count_kernel<<<pb, 256, 0, s>>>(p);
    scan_reduce_kernel<<<nblocks, RAD_THREADS, 0, s>>>(p);
    scan_blocksums_kernel<<<1, 1024, 0, s>>>(p, nblocks);
    scan_apply_kernel<<<nblocks, RAD_THREADS, 0, s>>>(p);
    bin_scatter_kernel<<<pb, 256, 0, s>>>(p, fill);
    bin_sort_kernel<<<(unsigned)(((size_t)p.ncells * 32 + 255) / 256), 256, 0, s>>>(p);
    return launch_status();
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
                                 int32_t** fill, RadiusLayout* lay) {
    if (!msg_p) return TIGA_ERR_INVALID_ARG;
    const tiga_msg msg = *msg_p;
    tiga_status st = fill_params(p, n, r, box);
    if (st != TIGA_OK) return st;
    if (msg.kind == TIGA_MSG_LJ) {
        if (!(msg.p1 > 0.f)) return TIGA_ERR_INVALID_ARG;
        F = 4;
    } else if (msg.kind == TIGA_MSG_GAUSS || msg.kind == TIGA_MSG_DIST) {
        if (F <= 0) return TIGA_ERR_INVALID_ARG;
        if (F % 4 || F > 128) return TIGA_ERR_UNSUPPORTED;
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
    tiga_status st = radius_common(&p, pos, feat, n, F, r, box, msg, ws, ws_bytes, &fill, &lay);
    if (st != TIGA_OK) return st;
    if (n == 0) return TIGA_OK;
    if (!out || !aligned16(out)) return TIGA_ERR_INVALID_ARG;
    p.out = out; p.count = count;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    st = run_binning(p, fill, lay.nblocks, s);
    if (st != TIGA_OK) return st;
    const unsigned blocks = (unsigned)((p.ncells + RAD_WARPS - 1) / RAD_WARPS);
    if (msg->kind == TIGA_MSG_LJ) radius_kernel<1><<<blocks, RAD_THREADS, 0, s>>>(p, msg->kind);
    else radius_kernel<0><<<blocks, RAD_THREADS, 0, s>>>(p, msg->kind);
    return launch_status();
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
    tiga_status st = radius_common(&p, pos, feat, n, F, r, box, msg, ws, ws_bytes, &fill, &lay);
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
    const unsigned blocks = (unsigned)((p.ncells + RAD_WARPS - 1) / RAD_WARPS);
    radius_kernel<2><<<blocks, RAD_THREADS, 0, s>>>(p, msg->kind);
    return launch_status();
}

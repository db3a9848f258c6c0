// Source-block plan of a stored relation: one-time preprocessing that depends on (rowptr, col)
// only and makes the forward of a relation whose feature table is far larger than L2 an
// L2-resident gather.
//
// Why: with 16-byte feature rows and a table of a gigabyte, every gather of the plain row-major
// traversal (Sections 3.1, 4.3) is a random 32-byte DRAM sector; the traversal then moves several
// times the bytes it needs.  The plan regroups the edges by BLOCK of source rows (a slice of the
// feature table small enough to stay in L2) and, inside a block, by destination row, keeping the
// edge order of every row.  The forward then runs one pass per block: all gathers of a pass hit the
// same slice, the pass streams its edges once and adds one partial sum to every destination row
// that has an edge in the block.  A (destination row, source block) pair with at least one edge is a
// SEGMENT; the plan stores, per block, the segments' rows and their extents in the permuted edges.
//
// Build (all on the device, no inter-CTA waiting):
//   1. per tile of 2048 edges, the number of edges per block            -> counts[block][tile]
//   2. exclusive scan of counts (reduce-then-scan)                        -> first slot of (block, tile)
//   3. stable scatter: every warp ranks its 256 edges inside their blocks in edge order (warp match),
//      warps and tiles are offset by the scanned counts                  -> pcol, prow (and ppos)
//   4. segment heads: a permuted slot starts a segment when its (block, row) differs from its
//      predecessor's; heads are counted per tile, scanned and written out -> seg_row, seg_ptr
// The stable order makes the plan unique: it is the relation's edges sorted by (block, row, position).
#include "csr_shared.cuh"

namespace tiga {

constexpr int PLAN_TILE = 2048;
constexpr int PLAN_THREADS = 256;
constexpr int PLAN_WARPS = PLAN_THREADS / 32;
constexpr int PLAN_PER_WARP = PLAN_TILE / PLAN_WARPS;      // 256 edges = 8 rounds of 32
constexpr int PSCAN_BLOCK = 2048;

struct PlanParams {
    const void* rowptr;
    const int32_t* col;
    long long n_dst, n_edges;
    int nb, shift;
    long long ntiles;
    int32_t* counts;        // [nb * ntiles], scanned in place
    int32_t* prow;          // [n_edges] destination row of every permuted edge (scratch)
    int32_t* pcol;          // [n_edges]
    int32_t* ppos;          // [n_edges] or null
    int32_t* heads;         // [ntiles], scanned in place
    int32_t* seg_row;
    int32_t* seg_ptr;
    long long* seg_begin;   // [nb + 1] first segment of every block (-1: block without edges)
    long long* huge;        // [nb] segments above the whole-warp limit, per block
    long long* totals;      // [1] number of segments
};

// ---- generic exclusive scan of int32 (totals below 2^31), reduce-then-scan
__device__ __forceinline__ int plan_block_scan(int v, int* s_warp, int* total) {
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
        s_warp[lane] = winc - w;
        if (lane == 31) s_warp[32] = winc;
    }
    __syncthreads();
    const int r = s_warp[warp] + inc - v;
    *total = s_warp[32];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(256) pscan_reduce_kernel(const int32_t* __restrict__ a, long long n, int32_t* sums) {
    __shared__ int s_warp[33];
    const long long base = (long long)blockIdx.x * PSCAN_BLOCK;
    int v = 0;
    for (int k = threadIdx.x; k < PSCAN_BLOCK; k += blockDim.x)
        if (base + k < n) v += a[base + k];
    int total;
    plan_block_scan(v, s_warp, &total);
    if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

// one CTA turns the chunk totals into exclusive offsets (sequential over groups of blockDim.x)
__global__ void __launch_bounds__(1024) pscan_sums_kernel(int32_t* sums, long long nchunks) {
    __shared__ int s_warp[33];
    __shared__ int s_carry;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (long long base = 0; base < nchunks; base += blockDim.x) {
        const long long k = base + threadIdx.x;
        const int v = k < nchunks ? sums[k] : 0;
        int total;
        const int ex = plan_block_scan(v, s_warp, &total);
        const int carry = s_carry;
        if (k < nchunks) sums[k] = carry + ex;
        __syncthreads();
        if (threadIdx.x == 0) s_carry = carry + total;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) pscan_apply_kernel(int32_t* a, long long n, const int32_t* __restrict__ sums) {
    __shared__ int s_warp[33];
    constexpr int PER = PSCAN_BLOCK / 256;
    const long long base = (long long)blockIdx.x * PSCAN_BLOCK + (long long)threadIdx.x * PER;
    int v[PER];
    int sum = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        v[k] = (base + k < n) ? a[base + k] : 0;
        sum += v[k];
    }
    int total;
    int ex = plan_block_scan(sum, s_warp, &total) + sums[blockIdx.x];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        if (base + k < n) a[base + k] = ex;
        ex += v[k];
    }
}

// Exclusive scan of a[0..n) in place; `sums` holds ceil(n / 2048) + 1 ints of scratch.  Arrays of more
// than 2048 * 2^22 entries are not needed here (counts has at most 64 * 2^20 entries).
static tiga_status plan_scan(int32_t* a, long long n, int32_t* sums, cudaStream_t s) {
    if (n <= 0) return TIGA_OK;
    const long long nchunks = (n + PSCAN_BLOCK - 1) / PSCAN_BLOCK;
    pscan_reduce_kernel<<<counted((unsigned)nchunks), 256, 0, s>>>(a, n, sums);
    pscan_sums_kernel<<<counted(1), 1024, 0, s>>>(sums, nchunks);
    pscan_apply_kernel<<<counted((unsigned)nchunks), 256, 0, s>>>(a, n, sums);
    return launch_status();
}

// ---- 1. edges per (block, tile)
__global__ void __launch_bounds__(PLAN_THREADS) plan_count_kernel(const PlanParams p) {
    __shared__ int s_cnt[64];
    if (threadIdx.x < 64) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    const long long e0 = (long long)blockIdx.x * PLAN_TILE;
    for (int k = threadIdx.x; k < PLAN_TILE; k += PLAN_THREADS) {
        const long long e = e0 + k;
        if (e < p.n_edges) atomicAdd(&s_cnt[ld_stream(p.col + e) >> p.shift], 1);
    }
    __syncthreads();
    if (threadIdx.x < p.nb) p.counts[(long long)threadIdx.x * p.ntiles + blockIdx.x] = s_cnt[threadIdx.x];
}

// destination row of edge e: the last row i in [lo, hi] with rowptr[i] <= e
template <typename IT>
__device__ __forceinline__ long long row_of(const IT* __restrict__ rowptr, long long lo, long long hi, long long e) {
    while (lo < hi) {
        const long long mid = (lo + hi + 1) >> 1;
        if ((long long)rowptr[mid] <= e) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// ---- 3. stable scatter.  A warp owns 256 consecutive edges and walks them in 8 rounds of 32
// (coalesced); inside a round, lanes of the same block are ranked by lane index (warp match), rounds
// and warps add up in shared memory, tiles through the scanned counts.
template <typename IT>
__global__ void __launch_bounds__(PLAN_THREADS) plan_scatter_kernel(const PlanParams p) {
    constexpr unsigned FULL = 0xffffffffu;
    __shared__ int s_run[PLAN_WARPS][64];      // edges of (warp, block) seen so far
    __shared__ int s_base[PLAN_WARPS][64];     // first slot of (warp, block)
    __shared__ long long s_rows[2];
    const IT* __restrict__ rowptr = static_cast<const IT*>(p.rowptr);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long e0 = (long long)blockIdx.x * PLAN_TILE;
    const long long e1 = e0 + PLAN_TILE < p.n_edges ? e0 + PLAN_TILE : p.n_edges;
    for (int k = threadIdx.x; k < PLAN_WARPS * 64; k += PLAN_THREADS) (&s_run[0][0])[k] = 0;
    if (threadIdx.x == 0) s_rows[0] = row_of(rowptr, 0, p.n_dst - 1, e0);
    if (threadIdx.x == 32) s_rows[1] = row_of(rowptr, 0, p.n_dst - 1, e1 - 1);
    __syncthreads();
    const long long r_lo = s_rows[0], r_hi = s_rows[1];

    int cj[PLAN_PER_WARP / 32], rank[PLAN_PER_WARP / 32];
    const long long w0 = e0 + (long long)warp * PLAN_PER_WARP;
#pragma unroll
    for (int r = 0; r < PLAN_PER_WARP / 32; ++r) {
        const long long e = w0 + 32 * r + lane;
        const bool in = e < e1;
        cj[r] = in ? ld_stream(p.col + e) : -1;
        const int b = in ? (cj[r] >> p.shift) : 64 + 0;           // lanes past the end form a group of their own
        const unsigned m = __match_any_sync(FULL, b);
        rank[r] = 0;
        if (in) {
            rank[r] = s_run[warp][b] + __popc(m & ((1u << lane) - 1u));
        }
        __syncwarp();
        if (in && lane == __ffs(m) - 1) s_run[warp][b] += __popc(m);
        __syncwarp();
    }
    __syncthreads();
    // first slot of every (warp, block): scanned tile offset + edges of earlier warps
    if (threadIdx.x < p.nb) {
        int acc = p.counts[(long long)threadIdx.x * p.ntiles + blockIdx.x];
        for (int w = 0; w < PLAN_WARPS; ++w) { s_base[w][threadIdx.x] = acc; acc += s_run[w][threadIdx.x]; }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < PLAN_PER_WARP / 32; ++r) {
        const long long e = w0 + 32 * r + lane;
        if (e < e1) {
            const int b = cj[r] >> p.shift;
            const int dst = s_base[warp][b] + rank[r];
            p.pcol[dst] = cj[r];
            p.prow[dst] = (int32_t)row_of(rowptr, r_lo, r_hi, e);
            if (p.ppos) p.ppos[dst] = (int32_t)e;
        }
    }
}

// ---- 4. segment heads
__device__ __forceinline__ bool is_head(const PlanParams& p, long long d) {
    if (d == 0) return true;
    return p.prow[d] != p.prow[d - 1] || (p.pcol[d] >> p.shift) != (p.pcol[d - 1] >> p.shift);
}

__global__ void __launch_bounds__(PLAN_THREADS) plan_heads_count_kernel(const PlanParams p) {
    __shared__ int s_warp[33];
    const long long d0 = (long long)blockIdx.x * PLAN_TILE;
    int c = 0;
    for (int k = threadIdx.x; k < PLAN_TILE; k += PLAN_THREADS)
        if (d0 + k < p.n_edges && is_head(p, d0 + k)) ++c;
    int total;
    plan_block_scan(c, s_warp, &total);
    if (threadIdx.x == 0) p.heads[blockIdx.x] = total;
}

__global__ void __launch_bounds__(PLAN_THREADS) plan_heads_write_kernel(const PlanParams p) {
    __shared__ int s_warp[33];
    constexpr int PER = PLAN_TILE / PLAN_THREADS;
    const long long d0 = (long long)blockIdx.x * PLAN_TILE + (long long)threadIdx.x * PER;
    bool h[PER];
    int c = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        h[k] = d0 + k < p.n_edges && is_head(p, d0 + k);
        c += h[k] ? 1 : 0;
    }
    int total;
    long long s = (long long)p.heads[blockIdx.x] + plan_block_scan(c, s_warp, &total);
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        if (!h[k]) continue;
        const long long d = d0 + k;
        p.seg_row[s] = p.prow[d];
        p.seg_ptr[s] = (int32_t)d;
        const int b = p.pcol[d] >> p.shift;
        if (d == 0 || (p.pcol[d - 1] >> p.shift) != b) p.seg_begin[b] = s;
        ++s;
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == PLAN_THREADS - 1) {
        p.seg_ptr[s] = (int32_t)p.n_edges;          // s is the number of segments here
        p.totals[0] = s;
    }
}

// segments too long for one warp pass, per block (decides whether a pass needs the chunk kernels)
__global__ void plan_huge_kernel(const PlanParams p, long long nseg, int limit) {
    const long long s = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= nseg) return;
    if (p.seg_ptr[s + 1] - p.seg_ptr[s] > limit) atomicAdd(reinterpret_cast<unsigned long long*>(p.huge + (p.pcol[p.seg_ptr[s]] >> p.shift)), 1ULL);
}

static int ceil_log2(long long v) {
    int s = 0;
    while ((1LL << s) < v) ++s;
    return s;
}

}  // namespace tiga

using namespace tiga;

static bool plan_args_ok(const tiga_csr* g, int32_t n_blocks) {
    if (!g || g->n_dst <= 0 || g->n_src <= 0 || g->n_edges <= 0) return false;
    if (n_blocks < 1 || n_blocks > TIGA_PLAN_MAX_BLOCKS || (n_blocks & (n_blocks - 1))) return false;
    return g->n_edges < 0x7fffffffLL && g->n_dst <= 0x7fffffffLL && g->n_src <= 0x7fffffffLL;
}

extern "C" size_t tiga_csr_plan_bytes(const tiga_csr* g, int32_t n_blocks, int with_positions) {
    if (!plan_args_ok(g, n_blocks)) return 0;
    const size_t E = (size_t)g->n_edges;
    size_t smax = (size_t)g->n_dst * (size_t)n_blocks;
    if (smax > E) smax = E;
    return align_up(E * 4, 256) * (with_positions ? 2 : 1) + align_up(smax * 4, 256) + align_up((smax + 1) * 4, 256) + 256;
}

extern "C" size_t tiga_csr_plan_workspace_bytes(const tiga_csr* g, int32_t n_blocks) {
    if (!plan_args_ok(g, n_blocks)) return 0;
    const size_t E = (size_t)g->n_edges;
    const size_t ntiles = (E + PLAN_TILE - 1) / PLAN_TILE;
    const size_t ncount = ntiles * (size_t)n_blocks;
    return align_up(E * 4, 256) + align_up(ncount * 4, 256) + align_up((ncount / PSCAN_BLOCK + 2) * 4, 256) +
           align_up(ntiles * 4, 256) + align_up((ntiles / PSCAN_BLOCK + 2) * 4, 256) + align_up((2 * TIGA_PLAN_MAX_BLOCKS + 2) * 8, 256) + 256;
}

extern "C" tiga_status tiga_csr_plan_build(const tiga_csr* g, int32_t n_blocks, int with_positions,
                                           void* plan_buf, size_t plan_bytes, void* ws, size_t ws_bytes,
                                           tiga_csr_plan* plan, void* stream) {
    if (!plan) return TIGA_ERR_INVALID_ARG;
    if (!g || g->n_dst < 0 || g->n_src < 0 || g->n_edges < 0) return TIGA_ERR_INVALID_ARG;
    if (n_blocks < 1 || n_blocks > TIGA_PLAN_MAX_BLOCKS || (n_blocks & (n_blocks - 1))) return TIGA_ERR_INVALID_ARG;
    if (g->rowptr_type != TIGA_I32 && g->rowptr_type != TIGA_I64) return TIGA_ERR_INVALID_ARG;
    if (g->n_edges >= 0x7fffffffLL || g->n_dst > 0x7fffffffLL || g->n_src > 0x7fffffffLL) return TIGA_ERR_UNSUPPORTED;
    if (g->n_dst == 0 || g->n_src == 0 || g->n_edges == 0) return TIGA_ERR_INVALID_ARG;
    if (!g->rowptr || !g->col || !aligned16(g->rowptr) || !aligned16(g->col)) return TIGA_ERR_INVALID_ARG;
    if (!plan_buf || !aligned16(plan_buf) || plan_bytes < tiga_csr_plan_bytes(g, n_blocks, with_positions)) return TIGA_ERR_WORKSPACE;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_csr_plan_workspace_bytes(g, n_blocks)) return TIGA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    const size_t E = (size_t)g->n_edges;
    size_t smax = (size_t)g->n_dst * (size_t)n_blocks;
    if (smax > E) smax = E;
    PlanParams p{};
    p.rowptr = g->rowptr; p.col = g->col; p.n_dst = g->n_dst; p.n_edges = g->n_edges;
    p.nb = n_blocks;
    p.shift = ceil_log2((g->n_src + n_blocks - 1) / n_blocks);
    p.ntiles = (long long)((E + PLAN_TILE - 1) / PLAN_TILE);
    const size_t ncount = (size_t)p.ntiles * (size_t)n_blocks;

    Carver pc(plan_buf);
    *plan = tiga_csr_plan{};
    plan->off_col = (int64_t)pc.off; p.pcol = pc.take<int32_t>(E);
    plan->off_pos = -1;
    if (with_positions) { plan->off_pos = (int64_t)pc.off; p.ppos = pc.take<int32_t>(E); }
    plan->off_seg_row = (int64_t)pc.off; p.seg_row = pc.take<int32_t>(smax);
    plan->off_seg_ptr = (int64_t)pc.off; p.seg_ptr = pc.take<int32_t>(smax + 1);
    Carver wc(ws);
    p.prow = wc.take<int32_t>(E);
    p.counts = wc.take<int32_t>(ncount);
    int32_t* count_sums = wc.take<int32_t>(ncount / PSCAN_BLOCK + 2);
    p.heads = wc.take<int32_t>((size_t)p.ntiles);
    int32_t* head_sums = wc.take<int32_t>((size_t)p.ntiles / PSCAN_BLOCK + 2);
    long long* small = wc.take<long long>(2 * TIGA_PLAN_MAX_BLOCKS + 2);
    p.seg_begin = small; p.huge = small + TIGA_PLAN_MAX_BLOCKS + 1; p.totals = small + 2 * TIGA_PLAN_MAX_BLOCKS + 1;

    TIGA_CUDA_TRY(cudaMemsetAsync(small, 0xff, (TIGA_PLAN_MAX_BLOCKS + 1) * sizeof(long long), s));       // seg_begin = -1
    TIGA_CUDA_TRY(cudaMemsetAsync(p.huge, 0, (TIGA_PLAN_MAX_BLOCKS + 1) * sizeof(long long), s));
    plan_count_kernel<<<counted((unsigned)p.ntiles), PLAN_THREADS, 0, s>>>(p);
    tiga_status st = plan_scan(p.counts, (long long)ncount, count_sums, s);
    if (st != TIGA_OK) return st;
    if (g->rowptr_type == TIGA_I32) plan_scatter_kernel<int32_t><<<counted((unsigned)p.ntiles), PLAN_THREADS, 0, s>>>(p);
    else plan_scatter_kernel<int64_t><<<counted((unsigned)p.ntiles), PLAN_THREADS, 0, s>>>(p);
    plan_heads_count_kernel<<<counted((unsigned)p.ntiles), PLAN_THREADS, 0, s>>>(p);
    st = plan_scan(p.heads, p.ntiles, head_sums, s);
    if (st != TIGA_OK) return st;
    plan_heads_write_kernel<<<counted((unsigned)p.ntiles), PLAN_THREADS, 0, s>>>(p);
    if (launch_status() != TIGA_OK) return TIGA_ERR_CUDA;

    long long h_small[2 * TIGA_PLAN_MAX_BLOCKS + 2];
    TIGA_CUDA_TRY(cudaMemcpyAsync(h_small, small, sizeof(h_small), cudaMemcpyDeviceToHost, s));
    TIGA_CUDA_TRY(cudaStreamSynchronize(s));
    const long long nseg = h_small[2 * TIGA_PLAN_MAX_BLOCKS + 1];
    plan_huge_kernel<<<counted((unsigned)((nseg + 255) / 256)), 256, 0, s>>>(p, nseg, ROW_HUGE);
    if (launch_status() != TIGA_OK) return TIGA_ERR_CUDA;
    TIGA_CUDA_TRY(cudaMemcpyAsync(h_small, small, sizeof(h_small), cudaMemcpyDeviceToHost, s));
    TIGA_CUDA_TRY(cudaStreamSynchronize(s));

    plan->n_blocks = n_blocks; plan->block_shift = p.shift; plan->has_positions = with_positions ? 1 : 0;
    plan->n_dst = g->n_dst; plan->n_src = g->n_src; plan->n_edges = g->n_edges; plan->n_segments = nseg;
    // blocks without edges start where the next block with edges starts
    long long next = nseg;
    plan->seg_begin[n_blocks] = nseg;
    for (int b = n_blocks - 1; b >= 0; --b) {
        if (h_small[b] >= 0) next = h_small[b];
        plan->seg_begin[b] = next;
        plan->huge_segments[b] = h_small[TIGA_PLAN_MAX_BLOCKS + 1 + b];
    }
    plan->used_bytes = plan->off_seg_ptr + (int64_t)align_up(((size_t)nseg + 1) * 4, 256);
    return TIGA_OK;
}

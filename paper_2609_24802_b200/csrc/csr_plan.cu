// Hot-source plan of a stored relation: one-time preprocessing that depends on (rowptr, col) only
// and serves most gathers of a forward from L2 when the feature table is far larger than L2.
//
// Why: with 16-byte feature rows and a table of a gigabyte, most gathers of the row-major traversal
// (Sections 3.1, 4.3) miss L2 and each miss moves a 32-byte DRAM sector, so the traversal moves
// several times the bytes it needs.  In a skewed relation a small set of sources receives most of
// the edges (a sixteenth of the sources of an R-MAT graph is named by nine edges in ten), but those
// sources are scattered over the whole table.  The plan
//   * counts how often every source is gathered (its in-degree),
//   * selects the sources above a threshold, at most `max_hot_rows` of them, numbers them densely
//     (in source order) and lists them in `hot_id`,
//   * rewrites the index stream: col[e] -> rank of the source if it is hot, n_hot + col[e] otherwise.
// A forward then copies the hot rows into one compact table (tens of megabytes, L2 resident) and
// runs the unchanged row-major traversal over the rewritten indices: every edge is visited in the
// same order as without the plan, so sums, maxima and argmax positions are bit-identical.
//
// Build (device, no inter-CTA waiting): in-degree by atomics, a 4096-bin histogram of the
// in-degrees (read on the host to pick the threshold), flags + exclusive scan (reduce-then-scan)
// for the dense numbering, one pass that rewrites the indices.
#include "csr_shared.cuh"
#include <vector>

namespace tiga {

constexpr int PSCAN_BLOCK = 2048;
constexpr int PLAN_BINS = 4096;

// ---- exclusive scan of int32 (totals below 2^31), reduce-then-scan
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

// per chunk of 2048 sources: how many are hot
__global__ void __launch_bounds__(256) plan_hot_count_kernel(const int32_t* __restrict__ indeg, long long n, int thr, int32_t* sums) {
    __shared__ int s_warp[33];
    const long long base = (long long)blockIdx.x * PSCAN_BLOCK;
    int v = 0;
    for (int k = threadIdx.x; k < PSCAN_BLOCK; k += blockDim.x)
        if (base + k < n) v += indeg[base + k] >= thr ? 1 : 0;
    int total;
    plan_block_scan(v, s_warp, &total);
    if (threadIdx.x == 0) sums[blockIdx.x] = total;
}

// one CTA turns the chunk totals into exclusive offsets (sequential over groups of blockDim.x)
__global__ void __launch_bounds__(1024) plan_scan_sums_kernel(int32_t* sums, long long nchunks) {
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

// dense numbering: hot source j -> its rank, listed in hot_id; every source gets its new index
// (rank, or n_hot + j) written over its in-degree; the edges covered by hot sources are added up
__global__ void __launch_bounds__(256) plan_number_kernel(int32_t* indeg, long long n, int thr, const int32_t* __restrict__ sums,
                                                          int n_hot, int32_t* hot_id, unsigned long long* covered) {
    __shared__ int s_warp[33];
    __shared__ unsigned long long s_cov;
    constexpr int PER = PSCAN_BLOCK / 256;
    if (threadIdx.x == 0) s_cov = 0;
    const long long base = (long long)blockIdx.x * PSCAN_BLOCK + (long long)threadIdx.x * PER;
    int d[PER];
    int c = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        d[k] = base + k < n ? indeg[base + k] : -1;
        c += d[k] >= thr ? 1 : 0;
    }
    int total;
    int rank = plan_block_scan(c, s_warp, &total) + sums[blockIdx.x];
    unsigned long long cov = 0;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
        if (base + k >= n) break;
        if (d[k] >= thr) {
            hot_id[rank] = (int32_t)(base + k);
            indeg[base + k] = rank++;
            cov += (unsigned long long)d[k];
        } else {
            indeg[base + k] = n_hot + (int32_t)(base + k);
        }
    }
    if (cov) atomicAdd(&s_cov, cov);
    __syncthreads();
    if (threadIdx.x == 0 && s_cov) atomicAdd(covered, s_cov);
}

__global__ void __launch_bounds__(256) plan_indegree_kernel(const int32_t* __restrict__ col, long long n_edges, long long n_src, int32_t* indeg) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n_edges; e += stride)
        atomicAdd(indeg + checked(ld_stream(col + e), n_src, CHECK_SOURCE), 1);
}

// histogram of min(in-degree, PLAN_BINS - 1): per-CTA counts in shared memory, then global atomics
__global__ void __launch_bounds__(256) plan_degree_hist_kernel(const int32_t* __restrict__ indeg, long long n, unsigned long long* hist) {
    __shared__ unsigned int s_hist[PLAN_BINS];
    for (int k = threadIdx.x; k < PLAN_BINS; k += blockDim.x) s_hist[k] = 0;
    __syncthreads();
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride) {
        const int d = indeg[j];
        // sources that nobody names are the most common by far and never hot: not counted
        if (d > 0) atomicAdd(&s_hist[d < PLAN_BINS - 1 ? d : PLAN_BINS - 1], 1u);
    }
    __syncthreads();
    for (int k = threadIdx.x; k < PLAN_BINS; k += blockDim.x)
        if (s_hist[k]) atomicAdd(hist + k, (unsigned long long)s_hist[k]);
}

__global__ void __launch_bounds__(256) plan_rewrite_kernel(const int32_t* __restrict__ col, long long n_edges, long long n_src,
                                                           const int32_t* __restrict__ remap, int32_t* pcol) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n_edges; e += stride)
        st_stream(pcol + e, __ldg(remap + checked(ld_stream(col + e), n_src, CHECK_SOURCE)));
}

// compact copy of the hot source rows (16-byte vectors): hot[r, :] = x[hot_id[r], :]
__global__ void __launch_bounds__(256) plan_gather_hot_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ hot_id,
                                                              long long n_hot, int nvec, uint4* hot) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_hot * nvec) return;
    const long long r = t / nvec;
    const int v = (int)(t - r * nvec);
    hot[t] = __ldg(x + (long long)hot_id[r] * nvec + v);
}

tiga_status launch_gather_hot(const void* x, const int32_t* hot_id, long long n_hot, int nvec, void* hot, cudaStream_t s) {
    if (n_hot == 0) return TIGA_OK;
    const long long work = n_hot * nvec;
    plan_gather_hot_kernel<<<counted((unsigned)((work + 255) / 256)), 256, 0, s>>>(static_cast<const uint4*>(x), hot_id, n_hot, nvec,
                                                                                  static_cast<uint4*>(hot));
    return launch_status();
}

}  // namespace tiga

using namespace tiga;

static bool plan_sizes_ok(const tiga_csr* g, int64_t max_hot_rows) {
    if (!g || g->n_dst < 0 || g->n_src <= 0 || g->n_edges <= 0 || max_hot_rows < 0) return false;
    return g->n_src + max_hot_rows < 0x7fffffffLL && g->n_dst <= 0x7fffffffLL;
}

extern "C" size_t tiga_csr_plan_bytes(const tiga_csr* g, int64_t max_hot_rows) {
    if (!plan_sizes_ok(g, max_hot_rows)) return 0;
    return align_up((size_t)g->n_edges * 4, 256) + align_up((size_t)max_hot_rows * 4 + 4, 256) + 256;
}

extern "C" size_t tiga_csr_plan_workspace_bytes(const tiga_csr* g) {
    if (!plan_sizes_ok(g, 0)) return 0;
    const size_t n = (size_t)g->n_src;
    return align_up(n * 4, 256) + align_up((n / PSCAN_BLOCK + 2) * 4, 256) + align_up((PLAN_BINS + 1) * 8, 256) + 256;
}

extern "C" tiga_status tiga_csr_plan_build(const tiga_csr* g, int64_t max_hot_rows, void* plan_buf, size_t plan_bytes,
                                           void* ws, size_t ws_bytes, tiga_csr_plan* plan, void* stream) {
    if (!plan || !g) return TIGA_ERR_INVALID_ARG;
    if (g->n_dst < 0 || g->n_src <= 0 || g->n_edges <= 0 || max_hot_rows < 0) return TIGA_ERR_INVALID_ARG;
    if (!plan_sizes_ok(g, max_hot_rows)) return TIGA_ERR_UNSUPPORTED;
    if (!g->col || !aligned16(g->col)) return TIGA_ERR_INVALID_ARG;
    if (!plan_buf || !aligned16(plan_buf) || plan_bytes < tiga_csr_plan_bytes(g, max_hot_rows)) return TIGA_ERR_WORKSPACE;
    if (!ws || !aligned16(ws) || ws_bytes < tiga_csr_plan_workspace_bytes(g)) return TIGA_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long long n = g->n_src, E = g->n_edges;
    const long long nchunks = (n + PSCAN_BLOCK - 1) / PSCAN_BLOCK;

    Carver pc(plan_buf);
    *plan = tiga_csr_plan{};
    plan->off_col = (int64_t)pc.off;
    int32_t* pcol = pc.take<int32_t>((size_t)E);
    plan->off_hot_id = (int64_t)pc.off;
    int32_t* hot_id = pc.take<int32_t>((size_t)max_hot_rows + 1);
    plan->used_bytes = (int64_t)pc.off;
    Carver wc(ws);
    int32_t* indeg = wc.take<int32_t>((size_t)n);
    int32_t* sums = wc.take<int32_t>((size_t)nchunks + 2);
    unsigned long long* hist = wc.take<unsigned long long>(PLAN_BINS + 1);      // the last entry adds up the covered edges

    TIGA_CUDA_TRY(cudaMemsetAsync(indeg, 0, (size_t)n * sizeof(int32_t), s));
    TIGA_CUDA_TRY(cudaMemsetAsync(hist, 0, (PLAN_BINS + 1) * sizeof(unsigned long long), s));
    plan_indegree_kernel<<<counted(148 * 16), 256, 0, s>>>(g->col, E, n, indeg);
    plan_degree_hist_kernel<<<counted(148 * 4), 256, 0, s>>>(indeg, n, hist);
    if (launch_status() != TIGA_OK) return TIGA_ERR_CUDA;
    std::vector<unsigned long long> hh(PLAN_BINS + 1);
    TIGA_CUDA_TRY(cudaMemcpyAsync(hh.data(), hist, (PLAN_BINS + 1) * sizeof(unsigned long long), cudaMemcpyDeviceToHost, s));
    TIGA_CUDA_TRY(cudaStreamSynchronize(s));
    // the lowest threshold whose sources fit the budget; in-degrees of PLAN_BINS - 1 and more share a bin
    int thr = PLAN_BINS;                       // nothing is hot
    unsigned long long above = 0;
    for (int d = PLAN_BINS - 1; d >= 1; --d) {
        if (above + hh[d] > (unsigned long long)max_hot_rows) break;
        above += hh[d];
        thr = d;
    }
    const long long n_hot = (long long)above;
    if (thr == PLAN_BINS) thr = 0x7fffffff;

    plan_hot_count_kernel<<<counted((unsigned)nchunks), 256, 0, s>>>(indeg, n, thr, sums);
    plan_scan_sums_kernel<<<counted(1), 1024, 0, s>>>(sums, nchunks);
    plan_number_kernel<<<counted((unsigned)nchunks), 256, 0, s>>>(indeg, n, thr, sums, (int)n_hot, hot_id, hist + PLAN_BINS);
    plan_rewrite_kernel<<<counted(148 * 16), 256, 0, s>>>(g->col, E, n, indeg, pcol);
    if (launch_status() != TIGA_OK) return TIGA_ERR_CUDA;
    unsigned long long covered = 0;
    TIGA_CUDA_TRY(cudaMemcpyAsync(&covered, hist + PLAN_BINS, sizeof(covered), cudaMemcpyDeviceToHost, s));
    TIGA_CUDA_TRY(cudaStreamSynchronize(s));

    plan->n_dst = g->n_dst; plan->n_src = g->n_src; plan->n_edges = g->n_edges;
    plan->n_hot = n_hot; plan->min_hot_degree = n_hot ? thr : 0; plan->hot_edges = (int64_t)covered;
    return TIGA_OK;
}

namespace tiga { unsigned check_status_csr_plan(bool reset) { return read_check_status(reset); } }

// Pieces shared by the stored-relation kernels (csr.cu: sum / max reducers and their reverse mode;
// csr_attention.cu: online-softmax reducer): merge-path tile geometry, tile staging, feature traits.
#pragma once
#include "common.cuh"

namespace tiga {

constexpr int CSR_THREADS = 256;
constexpr int CSR_TILE = 2048;     // merge-path items per CTA (sum forward)
constexpr int CSR_TILE_ATT = 2048; // online-softmax reducer
constexpr int CSR_TILE_MAX = 1792; // max forward: a larger state per lane, more CTAs per SM with shorter tiles
constexpr int CSR_TILE_BWD = 1792; // sum backward: a fourth staged array (edge gradients)
constexpr int CSR_TILE_MIN = 1792; // the shortest of them: sizes the per-tile workspace arrays
constexpr int CSR_PAD = 8;         // readable entries behind a tile's staged edges

template <typename XT> struct XTraits;
template <> struct XTraits<float> {
    static constexpr int VW = 4;   // floats per 16-byte vector
    // acc[k] += x[k]  (a message with unit weight: fma(1, x, acc) rounds exactly like this sum)
    __device__ static __forceinline__ void add_to(const uint4& v, float* acc) {
        acc[0] += __uint_as_float(v.x); acc[1] += __uint_as_float(v.y);
        acc[2] += __uint_as_float(v.z); acc[3] += __uint_as_float(v.w);
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct XTraits<__half> {
    static constexpr int VW = 8;
    // acc[k] += x[k] with the mixed-precision add of sm_100 (the half is widened exactly, one rounding)
    __device__ static __forceinline__ void add_to(const uint4& v, float* acc) {
        const unsigned r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            unsigned short lo, hi;
            asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(r[k]));
            asm("add.rn.f32.f16 %0, %1, %0;" : "+f"(acc[2 * k]) : "h"(lo));
            asm("add.rn.f32.f16 %0, %1, %0;" : "+f"(acc[2 * k + 1]) : "h"(hi));
        }
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float* f) {
        const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float2 t = __half22float2(h[k]);
            f[2 * k] = t.x; f[2 * k + 1] = t.y;
        }
    }
};

struct CsrParams {
    const void* rowptr;
    const int32_t* col;
    const float* w;          // may be null (unit weights)
    const void* x;
    float* out;
    void* arg;               // int32 [n_dst, F], or int64 for the wide-position max reducer
    long long n_dst, n_edges;
    long long n_src;         // rows of x (checked build: bound of every gathered index; a planned relation adds n_hot)
    int F;                   // features per row
    int nvec;                // 16-byte vectors per feature row
    // workspace
    int32_t* carry_row;      // [ntiles]  row of the tile's trailing partial state, or -1
    float* carry_val;        // [ntiles, F]
    void* carry_arg;         // [ntiles, F] (max only; same element type as arg)
    long long ntiles;
    int* huge_count;         // narrow-row path: number of queued chunks of huge rows
    int4* huge_list;         // (row, chunk, chunks of the row, first slot of the row)
    int row_huge;            // rows above this many edges are cut into chunks of this length
    // planned apply (narrow rows): the most often gathered source rows are served from a compact copy
    const void* x_hot;       // [n_hot rows] copy of the hot source rows, or null
    int n_hot;               // col values below n_hot index x_hot, the others (minus n_hot) x
    // backward
    const float* gy;
    float* gx;
    float* gw;
    // online-softmax reducer (csr_attention.cu): destination queries, source keys (x holds the values)
    const float* q;
    const float* key;
    float scale;
    float* lse;              // [n_dst] log of the row's total mass (caller's array or workspace)
    float2* carry_ml;        // [ntiles] (running maximum, mass) of a tile's carry-out
};

// host side, defined in csr_plan.cu: compact copy of the hot source rows, hot[r, :] = x[hot_id[r], :]
tiga_status launch_gather_hot(const void* x, const int32_t* hot_id, long long n_hot, int nvec, void* hot, cudaStream_t s);

// Number of rows whose row-end item lies before merge diagonal d:
//   #{ i : rowptr[i+1] + i + 1 <= d }   (strictly increasing in i -> 32-ary search by one warp)
template <typename IT>
__device__ long long rows_done(const IT* __restrict__ rowptr, long long n, long long d) {
    long long lo = 0, hi = n;
    const int lane = threadIdx.x & 31;
    while (lo < hi) {
        const long long step = (hi - lo + 31) / 32;
        const long long q = lo + (long long)(lane + 1) * step;
        bool pred = false;
        if (q <= hi) pred = ((long long)rowptr[q] + q <= d);
        const int c = __popc(__ballot_sync(0xffffffffu, pred));
        const long long nhi = lo + (long long)(c + 1) * step - 1;
        lo = lo + (long long)c * step;
        hi = nhi < hi ? nhi : hi;
        if (lo > hi) lo = hi;
    }
    return lo;
}

struct Tile {
    long long i0, e0;   // first row / first edge of the tile
    int nfin;           // rows whose row-end item is in the tile: [i0, i0 + nfin)
    int nrows;          // rows staged: nfin (+1 when a trailing partial row exists)
    int ne;             // edges in the tile
};

// Stage the tile: s_ptr[k] = clamp(rowptr[i0+k] - e0, -1, ne+1) for k = 0..nrows, col and w.
// index with one pad word per 32: threads that read consecutive runs of 8 stay conflict free
static __device__ __forceinline__ int pad32(int i) { return i + (i >> 5); }

template <typename IT, bool PADDED = false, int TILE = CSR_TILE>
__device__ Tile stage_tile(const CsrParams& p, int* s_ptr, int* s_col, float* s_w, long long* s_coord) {
    const IT* rowptr = static_cast<const IT*>(p.rowptr);
    const long long total = p.n_dst + p.n_edges;
    const long long d0 = (long long)blockIdx.x * TILE;
    const long long d1 = (d0 + TILE < total) ? d0 + TILE : total;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        long long i = rows_done(rowptr, p.n_dst, d0);
        if ((threadIdx.x & 31) == 0) s_coord[0] = i;
    } else if (warp == 1) {
        long long i = rows_done(rowptr, p.n_dst, d1);
        if ((threadIdx.x & 31) == 0) s_coord[1] = i;
    }
    __syncthreads();
    Tile t;
    t.i0 = s_coord[0];
    const long long i1 = s_coord[1];
    t.e0 = d0 - t.i0;
    const long long e1 = d1 - i1;
    t.ne = (int)(e1 - t.e0);
    t.nfin = (int)(i1 - t.i0);
    t.nrows = t.nfin + (i1 < p.n_dst ? 1 : 0);
    for (int k = threadIdx.x; k <= t.nrows; k += CSR_THREADS) {
        long long v = (long long)rowptr[t.i0 + k] - t.e0;
        if (v < -1) v = -1;
        if (v > t.ne + 1) v = t.ne + 1;
        // a trailing partial row never ends inside this tile, whatever rowptr says
        if (k == t.nrows && t.nrows > t.nfin) v = t.ne + 1;
        s_ptr[k] = (int)v;
    }
    for (int k = threadIdx.x; k < t.ne; k += CSR_THREADS) {
        const int kk = PADDED ? pad32(k) : k;
        s_col[kk] = checked(ld_stream(p.col + t.e0 + k), p.n_src, CHECK_SOURCE);
        s_w[kk] = p.w ? ld_stream(p.w + t.e0 + k) : 1.f;
    }
    // a few valid entries behind the last edge: unrolled loops may load (never use) past their span
    if (threadIdx.x < CSR_PAD) { s_col[(PADDED ? pad32(t.ne) : t.ne) + threadIdx.x] = 0; s_w[(PADDED ? pad32(t.ne) : t.ne) + threadIdx.x] = 0.f; }
    __syncthreads();
    return t;
}

// last k in [0, nrows] with s_ptr[k] <= a   (s_ptr[0] <= 0 <= a always)
static __device__ __forceinline__ int row_of_edge(const int* s_ptr, int nrows, int a) {
    int lo = 0, hi = nrows;          // invariant: s_ptr[lo] <= a
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (s_ptr[mid] <= a) lo = mid; else hi = mid - 1;
    }
    return lo;
}

}  // namespace tiga

// Pieces of the generated-radius path shared by radius.cu (binning, Gaussian / distance /
// Lennard-Jones traversals) and radius_mlp.cu (edge-network message).
#pragma once
#include "common.cuh"
#include <math.h>

namespace tiga {

constexpr int TRAV_WARPS = 4;
constexpr int TRAV_THREADS = TRAV_WARPS * 32;
constexpr int STAGE_PAD = 32;           // sentinels behind the staged candidates: no bounds checks
constexpr int QB = 8;                   // queries per batch (kernels that run faster with four define their own width)
constexpr float FAR_AWAY = 1.0e18f;
constexpr int QDENSE = 64;              // a cell with more points than this is cut into slices of QSLICE queries:
constexpr int QSLICE = 16;              // its warp takes the first slice, the others wait in a queue that other warps walk
constexpr int QUEUE_BLOCKS = 148 * 8;   // most CTAs that walk the queued slices
constexpr int SORT_DENSE = 256;         // a cell with more points than this is ordered by a sorting network, not by rank counting

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
    float r2_mid, r2_band;    // its centre and half width
    double r2_exact;          // (double)r * (double)r
    float len[3];
    float inv_len[3];
    int periodic[3];
    int nc[3];
    float invh[3];
    float hcell[3];           // cell edge, len / nc
    int ncells;
    float p0, p1;             // message parameters
    // edge network (radius_mlp.cu): device pointers to W1 [H, 3+Fin], b1 [H], W2 [Fout, H], b2 [Fout]
    const float *W1, *b1, *W2, *b2;
    float *gW1, *gb1, *gW2, *gb2;
    int Fin, Fout;
    // plan (workspace)
    int32_t* cell;
    int32_t* cnt;
    int32_t* cell_start;
    int32_t* order_tmp;
    int32_t* order;
    float4* spos;             // positions in cell order, .w = original point id (bit pattern)
    int32_t* blocksum;
    // slices of cells with more than QDENSE points, queued by the binning scan
    int2* q_items;            // (cell, first query of the slice)
    int* q_count;
    int q_mode;               // two-launch form: 0 = one warp per cell, 1 = warps walk the queue
    int cell_blocks;          // one-launch form: CTAs [0, cell_blocks) take cells, the CTAs behind them walk the queue
    int32_t* b_items;         // cells with more than SORT_DENSE points (queued by the same scan), and how many
    int* b_count;
    // optional user copies of the plan
    int32_t* u_cell;
    int32_t* u_cell_start;
    int32_t* u_order;
};

struct RadiusLayout {
    size_t bytes;
    int nblocks;
};

// host side, defined in radius.cu
tiga_status fill_params(RadiusParams* p, long long n, float r, const tiga_box* box);
RadiusLayout carve_radius(RadiusParams* p, void* ws, int32_t** fill);
tiga_status run_binning(RadiusParams& p, int32_t* fill, int nblocks, cudaStream_t s);
// host side, defined in radius_lj.cu: zeroes out / count, then one launch (pairs visited once, rows summed by atomics)
tiga_status launch_lj_pairs(const RadiusParams& p, cudaStream_t s);

// The defining predicate in double precision (same operations as the plain definition).
static __device__ __noinline__ bool exact_within(const RadiusParams& p, const float4 a, const float4 b) {
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

// A cell with more than QDENSE points: the warp that owns it keeps the first QSLICE queries; the others
// are queued, QSLICE at a time, for the pass over the queue.  The queue is part of the binning plan
// (written where the cell offsets are, so the traversals carry no code for it).  (Short slices: a dense cell's queries meet
// thousands of candidates each, and many short slices fill the machine where a few long ones leave a tail.)
static __device__ __forceinline__ int slice_end(int qs, int cell_end) { return cell_end - qs > QSLICE ? qs + QSLICE : cell_end; }
static __device__ __forceinline__ void queue_extra_slices(const RadiusParams& p, int cell, int count) {
    if (count > QDENSE) {
        const int extra = (count - 1) / QSLICE;
        const int at = atomicAdd(p.q_count, extra);
        for (int k = 0; k < extra; ++k) p.q_items[at + k] = make_int2(cell, (k + 1) * QSLICE);
    }
    if (count > SORT_DENSE) p.b_items[atomicAdd(p.b_count, 1)] = cell;
}

// CTAs that walk the queue: no more than the queue can have items for (at most n / QSLICE slices exist)
static inline unsigned queue_blocks(long long n) {
    const long long need = n / ((long long)QSLICE * TRAV_WARPS) + 1;
    return (unsigned)(need < QUEUE_BLOCKS ? need : QUEUE_BLOCKS);
}

// One launch over the cells and, in the CTAs appended behind them, over the queue of slices (which the
// binning filled before the launch).
template <typename Launch>
static inline tiga_status cells_then_queue(const RadiusParams& p, cudaStream_t s, Launch launch) {
    RadiusParams q = p;
    q.cell_blocks = (p.ncells + TRAV_WARPS - 1) / TRAV_WARPS;
    launch(q, (unsigned)q.cell_blocks + queue_blocks(p.n));
    return launch_status();
}

// Runs a traversal kernel twice: over the cells, then over the queue of slices (for kernels whose
// register allocation suffers from carrying both loops).
template <typename Launch>
static inline tiga_status two_passes(const RadiusParams& p, cudaStream_t s, Launch launch) {
    RadiusParams q = p;
    q.q_mode = 0;
    launch(q, (unsigned)((p.ncells + TRAV_WARPS - 1) / TRAV_WARPS));
    q.q_mode = 1;
    launch(q, queue_blocks(p.n));
    return launch_status();
}

static __device__ __forceinline__ float fast_exp2(float x) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

static __device__ __forceinline__ float fast_rcp(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// two fp32 values per register pair: sm_100 executes add / mul / fma on both with one instruction
typedef unsigned long long f32x2;
static __device__ __forceinline__ f32x2 pack2(float a, float b) { f32x2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b)); return r; }
static __device__ __forceinline__ void unpack2(f32x2 v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
static __device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) { f32x2 r; asm("sub.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
static __device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) { f32x2 r; asm("mul.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
static __device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }

// Minimum-image displacement of two coordinates of a periodic dimension that is not split into enough
// cells for a frame shift: the subtraction that can lose bits (x near 0 against x near len) is replaced
// by an exact shift of the coordinate next to the upper face.
static __device__ __forceinline__ float mi_delta(float a, float b, float len, float half) {
    float t = a - b;
    if (t > half) t = (a - len) - b;
    else if (t < -half) t = a - (b - len);
    return t;
}

// exact predicate for the pair of original point ids (a, b)
static __device__ __noinline__ bool exact_pair(const RadiusParams& p, int a, int b) {
    const float4 pa = make_float4(p.pos[3 * (size_t)a], p.pos[3 * (size_t)a + 1], p.pos[3 * (size_t)a + 2], 0.f);
    const float4 pb = make_float4(p.pos[3 * (size_t)b], p.pos[3 * (size_t)b + 1], p.pos[3 * (size_t)b + 2], 0.f);
    return exact_within(p, pa, pb);
}

}  // namespace tiga

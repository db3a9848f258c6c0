/*
 * tiga.h -- C ABI of libtiga: the gf.apply gather / message / reduce hot path of
 * "Tiga: Compiling Graph Message Passing at Scale" as hand-written CUDA for sm_100a.
 *
 * Two traversals of the same operation (paper Section 3.1):
 *     m_e = f(x_s(e), a_e),     y_i = finalize( combine_{e : d(e) = i} lift(m_e) )
 *   1. a stored destination-oriented CSR relation with a sum or max segment reduce
 *      (Sections 3.1 and 4.3) and its reverse mode (Section 5);
 *   2. a generated radius relation N(i) = { j != i : |p_j - p_i| <= r } (Appendix A) that is
 *      produced on the fly through a cell directory and consumed by the message and a sum
 *      reducer without storing edges or messages (Section 4.9), and its reverse mode with
 *      the membership frozen (Section 5).
 *
 * Conventions for every entry point
 *   - All array arguments are DEVICE pointers (global memory of the current device) unless
 *     the comment says "host".  The small structs (tiga_csr, tiga_box, tiga_msg) are passed
 *     by HOST pointer and read before the call returns; no struct crosses the ABI by value.
 *   - The caller owns every buffer.  The library allocates nothing and keeps no state
 *     between calls except what it writes into the caller's workspace `ws`.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = the default
 *     stream) and return without synchronising unless stated otherwise.
 *   - Outputs are overwritten in full (empty rows and points without neighbours included);
 *     gradients are overwritten, not accumulated.  Rows of every output are in the
 *     caller's original row / point order.
 *   - Base pointers must be 16-byte aligned.  Feature rows are dense, row major.
 *   - Return value: TIGA_OK, or the first error found on the host.  Nothing is launched
 *     when an error is returned.  Errors never raise a device fault.
 */
#ifndef TIGA_H
#define TIGA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TIGA_OK = 0,
    TIGA_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, negative size, bad enum, bad box */
    TIGA_ERR_UNSUPPORTED = 2,   /* a combination this build has no kernel for */
    TIGA_ERR_WORKSPACE = 3,     /* ws is NULL or smaller than *_workspace_bytes() */
    TIGA_ERR_CUDA = 4,          /* a CUDA runtime call failed */
    TIGA_ERR_INVALID_GRAPH = 5, /* tiga_validate_csr found a malformed relation */
    TIGA_ERR_TOO_LARGE = 6,     /* the problem needs more scratch than the library's built-in array holds */
    TIGA_ERR_INVALID_POINTS = 7 /* tiga_validate_points found a coordinate that is not finite or lies outside the box */
} tiga_status;

typedef enum { TIGA_F32 = 0, TIGA_F16 = 1 } tiga_dtype;   /* feature storage; accumulation is fp32 */
typedef enum { TIGA_I32 = 0, TIGA_I64 = 1 } tiga_itype;   /* rowptr storage; col is always int32 */
/* TIGA_MAX64: the max reducer with 64-bit edge positions in argmax (an int64 array); any relation may use
 * it, relations of 2^31 edges or more must (TIGA_MAX keeps 32-bit positions). */
typedef enum { TIGA_SUM = 0, TIGA_MAX = 1, TIGA_MAX64 = 2 } tiga_reducer;

typedef enum {
    TIGA_MSG_COPY = 0,      /* CSR: m = x_j                         (w must be NULL)           */
    TIGA_MSG_WEIGHTED = 1,  /* CSR: m = w_e * x_j                   (Section 3.1 example)      */
    TIGA_MSG_GAUSS = 2,     /* radius: m = exp(-d^2 / (2 p0^2)) * x_j,  p0 = sigma             */
    TIGA_MSG_DIST = 3,      /* radius: m = d * x_j  (the paper's distance-weighted sum, Sec. 7) */
    TIGA_MSG_LJ = 4         /* radius: Lennard-Jones pair force and energy, p0 = eps, p1 = s   */
} tiga_msg_kind;

typedef struct {
    int32_t kind;           /* tiga_msg_kind */
    float p0, p1;
} tiga_msg;

/* Destination-oriented CSR relation (Section 3.1): rows enumerate destinations, col[e] is
 * the source of edge e, the edge position e indexes edge fields.  Duplicate edges are
 * separate messages, a self edge is ordinary, there is no implicit reverse edge. */
typedef struct {
    const void* rowptr;     /* device, int32 or int64 [n_dst + 1], rowptr[0] = 0, rowptr[n_dst] = n_edges */
    int32_t rowptr_type;    /* tiga_itype */
    const int32_t* col;     /* device, int32 [n_edges], values in [0, n_src) */
    int64_t n_dst, n_src, n_edges;
} tiga_csr;

/* Axis-aligned box with its origin at 0.  Points must lie in [0, len[d]] in every dimension.
 * periodic[d] != 0 selects the minimum image in that dimension and requires r < len[d] / 2. */
typedef struct {
    float len[3];
    int32_t periodic[3];
} tiga_box;

const char* tiga_status_string(tiga_status s);

/* Number of CUDA kernels this library has launched in this process so far (host-side counter,
 * all entry points, all devices).  No counterpart in the paper: benchmarks read it before and after
 * a timed region to state how many of the library's kernels ran inside it. */
int64_t tiga_kernel_launches(void);

/* Checked build (libtiga_checked.so, compiled with -DTIGA_CHECKED; no counterpart in the paper): every
 * index that is about to address a gathered source row, an edge or a point is range-checked on the device
 * first; a violation sets a bit of a status word and the access goes to element 0 instead, so nothing
 * faults.  tiga_checked_status synchronises the device and returns the bits seen since the last reset
 * (1 source index, 2 edge position, 4 point id, 8 slot of the cell-ordered points; 0x80000000 if the word
 * could not be read) and clears them when reset != 0.  The normal build checks nothing and returns 0.
 * tiga_is_checked_build tells the two apart. */
uint32_t tiga_checked_status(int reset);
int tiga_is_checked_build(void);

/* ------------------------------------------------------------------------------------ CSR */

/* Bytes of workspace tiga_apply_csr (backward = 0) or tiga_apply_csr_backward (backward = 1)
 * needs for this relation, feature width and reducer.  Host only, launches nothing. */
size_t tiga_csr_workspace_bytes(const tiga_csr* g, int32_t F, tiga_dtype x_dtype,
                                tiga_reducer reducer, int backward);

/* Full validation (Section 6, "Validation and trust boundaries": monotone row pointers,
 * endpoints, source-index bounds) when level = 1; metadata only when level = 0.
 * ws: at least 16 bytes of device memory.  level 1 launches a scan and SYNCHRONISES the
 * stream.  Returns TIGA_ERR_INVALID_GRAPH when a check fails. */
tiga_status tiga_validate_csr(const tiga_csr* g, int level, void* ws, size_t ws_bytes, void* stream);

/* Fused gather-message-reduce over a stored relation (Sections 3.1, 4.2, 4.3):
 *   sum : out[i,f] = sum over e in [rowptr[i], rowptr[i+1]) of w[e] * x[col[e], f]
 *   max : out[i,f] = max over the same edges; argmax[i,f] = the lowest edge position that
 *         attains it.  An empty row gives 0 (and argmax = -1).
 * No E x F message array is formed.
 *   x      : [n_src, F], x_dtype.  F must be a multiple of 4 (fp32) or 8 (fp16).
 *   w      : fp32 [n_edges] or NULL for unit weights (msg.kind = TIGA_MSG_COPY).
 *   out    : fp32 [n_dst, F].
 *   argmax : int32 [n_dst, F] for TIGA_MAX (needs n_edges < 2^31, else TIGA_ERR_UNSUPPORTED), int64 [n_dst, F] for
 *            TIGA_MAX64; required for both, ignored for TIGA_SUM.
 *   ws     : tiga_csr_workspace_bytes(g, F, x_dtype, reducer, 0) bytes; contents are scratch.
 * Long rows are split and their partial states merged in a fixed order (edge order for feature
 * rows of 64 bytes and more; a fixed lane-strided tree for narrower rows), without atomics, so
 * results are reproducible from run to run. */
tiga_status tiga_apply_csr(const tiga_csr* g, const void* x, tiga_dtype x_dtype, int32_t F,
                           const float* w, const tiga_msg* msg, tiga_reducer reducer,
                           float* out, void* argmax, void* ws, size_t ws_bytes, void* stream);

/* tiga_apply_csr for callers that cannot hand over a workspace.  (The paper has no counterpart;
 * this entry point exists for integration reasons only.)
 *
 * Who needs it: code that is given nothing but its input and output buffers and must not call
 * cudaMalloc -- a plug-in inside a host framework that owns the device allocator, a step
 * inside a latency-critical loop where an allocation would stall the device, a process whose
 * memory budget was fixed at start-up.  Such a caller cannot size and allocate the `ws` that
 * tiga_apply_csr wants, so here the scratch (one carry-out slot per tile) lives in a fixed
 * array inside the library's own device image: TIGA_BUILTIN_WS_BYTES (8 MiB) on every GPU that
 * loads the library, for as long as the process lives.
 *
 * Same arguments and results as tiga_apply_csr, minus ws / ws_bytes.  Differences:
 *   - Capacity: the call is refused with TIGA_ERR_TOO_LARGE, before anything is launched, when
 *     tiga_csr_workspace_bytes(g, F, x_dtype, reducer, 0) exceeds TIGA_BUILTIN_WS_BYTES
 *     (roughly (n_dst + n_edges) / 1792 * (4 F + 20) bytes plus about 1.5 KiB of padding, twice
 *     the F term for TIGA_MAX, three times for TIGA_MAX64; e.g. 16.8M edges at F = 64 need 2.7 MiB).
 *   - It never calls cudaMalloc, cudaFree or any other allocating routine.
 *   - The first call on each device looks up the array's device address (a host-side lookup,
 *     done with that device current and cached per device).  Make that first call before any
 *     stream capture begins.
 *   - All calls on one device share the one array, and it keeps whatever the previous call
 *     left in it.  What must start at zero (the length of the queue of chunks of very long
 *     rows) is cleared by the call itself; every tile writes its own slot before the fix-up pass
 *     reads it.  Two calls that overlap on the GPU (different streams, or
 *     different host threads) race on the array and corrupt each other's results; serialise
 *     them, or use tiga_apply_csr with separate workspaces. */
#define TIGA_BUILTIN_WS_BYTES (8u << 20)
tiga_status tiga_apply_csr_builtin_ws(const tiga_csr* g, const void* x, tiga_dtype x_dtype, int32_t F,
                                      const float* w, const tiga_msg* msg, tiga_reducer reducer,
                                      float* out, void* argmax, void* stream);

/* Hot-source plan: one-time preprocessing of a stored relation whose feature table is far larger
 * than the L2 cache (the billion-edge relation of Section 7 held in device memory).  It depends on
 * (rowptr, col) only -- the paper also treats relation set-up as untimed preprocessing (Section 7).
 * In a skewed relation a small set of sources receives most of the edges; the plan selects the
 * sources named by the most edges (at most max_hot_rows, all those with an in-degree of
 * min_hot_degree or more), numbers them densely and rewrites the index stream so that a hot source is
 * addressed by its rank and any other source j by n_hot + j.  tiga_apply_csr_planned copies the hot
 * rows of the feature table into one compact, L2-resident table and runs the unchanged row-major
 * traversal over the rewritten indices.  Edges are visited in the same order as without the plan:
 * sums, maxima and argmax positions are bit-identical to tiga_apply_csr's.
 * The struct is plain data on the HOST; the arrays it describes live in `plan_buf` on the device at the
 * byte offsets it records:
 *   col    int32 [n_edges]   rewritten source indices, in edge order
 *   hot_id int32 [n_hot]     source row of every hot rank, ascending */
typedef struct {
    int64_t n_dst, n_src, n_edges;
    int64_t n_hot;               /* hot sources */
    int64_t min_hot_degree;      /* every hot source is named by at least this many edges (0: none is hot) */
    int64_t hot_edges;           /* edges whose source is hot */
    int64_t off_col, off_hot_id; /* byte offsets in plan_buf */
    int64_t used_bytes;          /* bytes of plan_buf the plan occupies */
} tiga_csr_plan;

/* Bytes of plan_buf and of build scratch.  Host only. */
size_t tiga_csr_plan_bytes(const tiga_csr* g, int64_t max_hot_rows);
size_t tiga_csr_plan_workspace_bytes(const tiga_csr* g);

/* Builds the plan on the device and SYNCHRONISES the stream twice (the in-degree histogram and the
 * counts come back to the host).  Needs n_src + max_hot_rows < 2^31.  max_hot_rows: choose it so that
 * max_hot_rows * row bytes is about half the L2 size.  ws is scratch and may be freed afterwards.  In-
 * degrees of 4095 and more are not told apart: if more than max_hot_rows sources reach that, none is
 * hot.  The result is unique, so rebuilding gives the same plan. */
tiga_status tiga_csr_plan_build(const tiga_csr* g, int64_t max_hot_rows, void* plan_buf, size_t plan_bytes,
                                void* ws, size_t ws_bytes, tiga_csr_plan* plan /* host, out */, void* stream);

/* tiga_apply_csr through a plan built for this very relation (same arguments and results, bit for
 * bit).  Feature rows of at most 32 bytes (F <= 8 fp32, F <= 16 fp16; TIGA_ERR_UNSUPPORTED above:
 * wider rows are served by the tile kernels, which the plan does not change).
 *   ws : tiga_csr_planned_workspace_bytes(...) bytes: the compact table of hot rows plus the
 *        forward's own scratch. */
size_t tiga_csr_planned_workspace_bytes(const tiga_csr* g, const tiga_csr_plan* plan, int32_t F, tiga_dtype x_dtype,
                                        tiga_reducer reducer);
tiga_status tiga_apply_csr_planned(const tiga_csr* g, const tiga_csr_plan* plan, const void* plan_buf,
                                   const void* x, tiga_dtype x_dtype, int32_t F, const float* w, const tiga_msg* msg,
                                   tiga_reducer reducer, float* out, void* argmax,
                                   void* ws, size_t ws_bytes, void* stream);

/* Reverse mode of tiga_apply_csr for fixed relation indices (Section 5):
 *   sum : grad_w[e] = sum_f x[col[e],f] * grad_out[row(e),f]
 *         grad_x[j,:] = sum over edges e with col[e] = j of w[e] * grad_out[row(e),:]
 *   max : the cotangent of (i,f) flows only through edge argmax[i,f] (nothing if it is -1).
 *   grad_out : fp32 [n_dst, F];  argmax : the forward's output (int32 for TIGA_MAX, int64 for TIGA_MAX64).
 *   grad_x   : fp32 [n_src, F] or NULL to skip;  grad_w : fp32 [n_edges] or NULL to skip.
 * x is fp32 or fp16 (the forward's feature table; F % 8 == 0 for fp16); all gradients are fp32, and the
 * cotangent of an fp16 table is the fp32 grad_x (no rounding to fp16 is applied).  Repeated sources accumulate with floating-point atomics, so grad_x (and
 * grad_w for TIGA_MAX) may differ in the last bits between runs. */
tiga_status tiga_apply_csr_backward(const tiga_csr* g, const void* x, tiga_dtype x_dtype, int32_t F,
                                    const float* w, const tiga_msg* msg, tiga_reducer reducer,
                                    const float* grad_out, const void* argmax,
                                    float* grad_x, float* grad_w,
                                    void* ws, size_t ws_bytes, void* stream);

/* Degree histogram: deg_i = rowptr[i+1] - rowptr[i]; hist[d] = number of rows of degree d for
 * d < nbins - 1, hist[nbins-1] = number of rows with deg >= nbins - 1; *max_degree = max deg.
 *   hist : device int64 [nbins], 1 <= nbins <= 8192;  max_degree : device int64 [1]. */
tiga_status tiga_csr_degree_histogram(const tiga_csr* g, int64_t* hist, int64_t nbins,
                                      int64_t* max_degree, void* stream);

/* --------------------------------------------------------------------------------- radius */

/* Cell directory constants for n points, cutoff r and this box (host only):
 *   ncell[d] = clamp(floor(len[d] / (r (1 + 2^-10))), 1, min(1024, floor(cbrt(8 n)))),
 *   periodic dimensions with fewer than 3 cells use one cell,  invh[d] = (float)(ncell[d] / len[d]).
 * A point's cell is min(ncell[d]-1, (int)floorf(p[d] * invh[d])) with one fp32 multiply;
 * linear id = (c_z ncell[1] + c_y) ncell[0] + c_x.  Either output may be NULL. */
tiga_status tiga_radius_grid(int64_t n, float r, const tiga_box* box, int32_t ncell[3], float invh[3]);

/* Validation of point coordinates (Section 6, "Validation and trust boundaries", applied to the
 * generated relation): the apply calls trust that every coordinate is finite and lies in [0, len[d]];
 * a point outside is binned into an edge cell and silently misses neighbours.  level 0 checks the
 * arguments on the host only; level 1 scans the coordinates on the device and SYNCHRONISES the stream.
 *   pos : fp32 [n, 3];  ws : at least 16 bytes of device memory (level 1).
 * Returns TIGA_ERR_INVALID_POINTS when a coordinate fails the check. */
tiga_status tiga_validate_points(const float* pos, int64_t n, const tiga_box* box, int level,
                                 void* ws, size_t ws_bytes, void* stream);

/* Workspace bytes for tiga_radius_bin / tiga_apply_radius / tiga_apply_radius_backward. */
size_t tiga_radius_workspace_bytes(int64_t n, int32_t F, float r, const tiga_box* box, int backward);

/* Cell binning pass of the generated relation (Section 4.9): per-cell counts, exclusive scan,
 * stable scatter into cell order.
 *   pos        : fp32 [n, 3]
 *   cell       : int32 [n]            cell id of every point                 (NULL to skip)
 *   cell_start : int32 [ncells + 1]   exclusive scan of the per-cell counts  (NULL to skip)
 *   order      : int32 [n]            point ids sorted by (cell id, point id) (NULL to skip)
 * The same plan is left in ws for the apply calls. */
tiga_status tiga_radius_bin(const float* pos, int64_t n, float r, const tiga_box* box,
                            int32_t* cell, int32_t* cell_start, int32_t* order,
                            void* ws, size_t ws_bytes, void* stream);

/* Fused generated-relation apply (Section 4.9, Appendix A): bins the points, then for every
 * point i accumulates the messages of all j != i with |p_i - p_j| <= r (minimum image in
 * periodic dimensions; the predicate is decided exactly as in double precision) straight
 * into the sum reducer.  Neither an edge list nor per-edge messages are written.
 *   GAUSS / DIST : feat fp32 [n, F] (1 <= F <= 128; 128-bit accesses when F is a multiple
 *                  of 4, scalar accesses otherwise), out fp32 [n, F]
 *   LJ           : feat ignored, F ignored, out fp32 [n, 4] = (Fx, Fy, Fz, e_i) with
 *                  F_i = sum_j 24 eps (2 (s/d)^12 - (s/d)^6) (p_i - p_j) / d^2 and
 *                  e_i = (1/2) sum_j 4 eps ((s/d)^12 - (s/d)^6)
 *   count        : int32 [n] number of neighbours of every point, or NULL
 * A point without neighbours gets the zero vector. */
tiga_status tiga_apply_radius(const float* pos, const float* feat, int64_t n, int32_t F,
                              float r, const tiga_box* box, const tiga_msg* msg,
                              float* out, int32_t* count, void* ws, size_t ws_bytes, void* stream);

/* Reverse mode of tiga_apply_radius for TIGA_MSG_GAUSS with the membership frozen
 * (Section 5; Appendix A: positions enter through the displacement of selected edges):
 *   grad_feat[j,:] = sum over i with j in N(i) of g_ij grad_out[i,:]
 *   grad_pos[k,:]  = -(1/sigma^2) sum over j in N(k) of g_kj (p_k - p_j)
 *                                  (grad_out[k].feat[j] + grad_out[j].feat[k])
 *   grad_feat : fp32 [n, F] or NULL;  grad_pos : fp32 [n, 3] or NULL.  F must be a multiple of 4.
 *   reuse_plan != 0: ws still holds the bins of this very position snapshot (left there by
 *   tiga_apply_radius or tiga_radius_bin with the same n, r, box); otherwise it is rebuilt. */
tiga_status tiga_apply_radius_backward(const float* pos, const float* feat, int64_t n, int32_t F,
                                       float r, const tiga_box* box, const tiga_msg* msg,
                                       const float* grad_out, float* grad_feat, float* grad_pos,
                                       void* ws, size_t ws_bytes, int reuse_plan, void* stream);

/* ----------------------------------------------------------------- radius, edge network */

/* Shared edge-local network of the paper's Appendix A, evaluated per selected edge (i <- j):
 *     m_ij = W2 ReLU( W1 [p_j - p_i ; x_j] + b1 ) + b2
 * (displacement source minus destination, minimum image where periodic; the final bias is part
 * of every message).  All four arrays are DEVICE pointers, row major. */
typedef struct {
    int32_t f_in;       /* node feature width, 1..13 */
    int32_t hidden;     /* 8, 16 or 32 */
    int32_t f_out;      /* 1..4 */
    const float* W1;    /* [hidden, 3 + f_in]; columns 0..2 multiply the displacement */
    const float* b1;    /* [hidden] */
    const float* W2;    /* [f_out, hidden] */
    const float* b2;    /* [f_out] */
} tiga_edge_mlp;

/* Fused generated-relation apply with the edge network as the message (Appendix A, Section 4.9):
 *     out[i,:] = sum over j in N(i) of m_ij,   zero vector without neighbours.
 *   feat : fp32 [n, f_in];  out : fp32 [n, f_out];  count : int32 [n] or NULL.
 * Bins the points first (plan left in ws).  ws: tiga_radius_workspace_bytes(n, f_in, r, box, 0). */
tiga_status tiga_apply_radius_mlp(const float* pos, const float* feat, int64_t n, float r, const tiga_box* box,
                                  const tiga_edge_mlp* mlp, float* out, int32_t* count,
                                  void* ws, size_t ws_bytes, void* stream);

/* Reverse mode of tiga_apply_radius_mlp with the membership frozen (Section 5, Appendix A): the
 * activations are recomputed per pair, nothing of size E is stored.
 *   grad_out : fp32 [n, f_out]
 *   grad_feat [n, f_in], grad_pos [n, 3], grad_W1 [hidden, 3 + f_in], grad_b1 [hidden],
 *   grad_W2 [f_out, hidden], grad_b2 [f_out]: each fp32, overwritten, or NULL to skip.
 * Feature and position gradients are owner-computed (no atomics, reproducible); the parameter
 * gradients are summed with floating-point atomics and may differ in the last bits between runs.
 * ReLU'(0) = 0.  reuse_plan as in tiga_apply_radius_backward. */
tiga_status tiga_apply_radius_mlp_backward(const float* pos, const float* feat, int64_t n, float r, const tiga_box* box,
                                           const tiga_edge_mlp* mlp, const float* grad_out,
                                           float* grad_feat, float* grad_pos,
                                           float* grad_W1, float* grad_b1, float* grad_W2, float* grad_b2,
                                           void* ws, size_t ws_bytes, int reuse_plan, void* stream);

/* ----------------------------------------------------------------- stored relation, online-softmax reducer */

/* Online-softmax reducer over the rows of a stored relation (Section 5, "Online softmax and
 * approximation"; the attention appendix): the edge function supplies a score and a value,
 *     s_e = scale * <q[d(e),:], key[s(e),:]>,
 *     out[i,:] = sum_e exp(s_e) value[s(e),:] / sum_e exp(s_e)      over the edges e of row i,
 * evaluated with the streaming state (maximum, mass, accumulator) and the combine rule of that
 * section; the relation decides which interactions exist (a triangular relation with the diagonal
 * is causal attention).  Repeated edges are separate messages.  A row without edges yields the
 * zero vector and lse = -inf (the reducer's empty-row convention, as for the sum reducer).
 *   q : fp32 [n_dst, D];  key, value : fp32 [n_src, D];  D a multiple of 4, 4..128
 *       (TIGA_ERR_UNSUPPORTED above 128);  out : fp32 [n_dst, D], fully overwritten
 *   lse : fp32 [n_dst] or NULL, log of the row's total mass sum_e exp(s_e)
 *   ws  : tiga_csr_attention_workspace_bytes(g, D) bytes, 16-byte aligned.
 * All arrays are device pointers, g is read on the host.  Forward only (the paper has no
 * streaming backward for this reducer).  No atomics: results are reproducible. */
size_t tiga_csr_attention_workspace_bytes(const tiga_csr* g, int32_t D);
tiga_status tiga_apply_csr_attention(const tiga_csr* g, const float* q, const float* key, const float* value,
                                     int32_t D, float scale, float* out, float* lse,
                                     void* ws, size_t ws_bytes, void* stream);

/* ----------------------------------------------------------------- generated exact kNN */

#define TIGA_KNN_MAX_K 32

/* Generated exact k-nearest-neighbour relation consumed by a neighbour sum without storing an
 * adjacency (Section 4.9, generated kNN; Section 7: scalar neighbour sum with k = 16):
 *     N_k(i) = the k sources j != i with the smallest keys (d2_ij, j),
 *     out[i,:] = sum over j in N_k(i) of feat[j,:].
 * The key's squared distance is the fp32 value fl(fl(fl(dx*dx) + fl(dy*dy)) + fl(dz*dz)) of the
 * direct differences dx = fl(x_i - x_j), ... (the paper bounds this path to FP32 and uses direct
 * differences); equal distances are ordered by source index.  The result is exact for that key
 * on any input: a cell directory only orders the search (cells around the query first, farther
 * shells while the k-th key could still improve), it never replaces the comparison of keys.
 *   pos  : fp32 [n, 3] inside [0, len_d]; the box must not be periodic (TIGA_ERR_UNSUPPORTED)
 *   feat : fp32 [n, F], F >= 1;  k : 1..TIGA_KNN_MAX_K (TIGA_ERR_UNSUPPORTED above)
 *   out  : fp32 [n, F], fully overwritten
 *   nbr  : int32 [n, k] or NULL, source indices in key order; nbr_d2 : fp32 [n, k] or NULL.
 *          With fewer than k other points the missing entries are -1 and +inf and add nothing.
 *   ws   : tiga_knn_workspace_bytes(n, k, box) bytes, 16-byte aligned; holds the bins afterwards.
 * All array pointers are device pointers; the box is read on the host.  No backward exists for
 * this relation (the paper generates none for it either). */
size_t tiga_knn_workspace_bytes(int64_t n, int32_t k, const tiga_box* box);
tiga_status tiga_apply_knn(const float* pos, const float* feat, int64_t n, int32_t F, int32_t k,
                           const tiga_box* box, float* out, int32_t* nbr, float* nbr_d2,
                           void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TIGA_H */

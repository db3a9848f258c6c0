/*
 * CPU ORACLE -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow, fp64 restatement of what the gf.apply hot path computes, written from the
 * paper's definitions.  It shares no code, header, table or helper with the CUDA library;
 * only tests, the smoke check and the benchmark's cpu_baseline leg may call it.
 *
 * What is written out here, with the passage each function follows:
 *   - gather / message / reduce over a destination-oriented CSR relation
 *     (Section 3.1: m_e = f(x_s(e), a_e), y_i = finalize(combine over e with d(e)=i);
 *      Section 4.3: row_ptr gives edge ranges, the edge position indexes the weight,
 *      col_idx[e] supplies the source id; empty row -> reducer identity then finalize)
 *   - the weighted-sum adjoint (Section 5: xbar_j = sum_{e:s(e)=j} w_e ybar_d(e),
 *     wbar_e = x_s(e) . ybar_d(e); repeated sources accumulate)
 *   - the radius relation N(i) = { j != i : |p_j - p_i| <= r } (Appendix A) consumed by a
 *     message and a sum reducer without ever being stored (Section 4.9), by brute force
 *     over all ordered pairs, and its reverse mode with membership frozen (Section 5,
 *     Appendix A: the position derivative acts through the displacement of selected edges)
 *   - a cell directory (Section 4.9) used only to restrict candidates; the exact distance
 *     predicate is unchanged.
 *   - the online-softmax reducer over the rows of a stored relation (Section 5; attention
 *     appendix): the normalised exponential-weighted sum it evaluates, by the plain quotient.
 *   - the generated exact k-nearest-neighbour relation consumed by a neighbour sum
 *     (Section 4.9; keys are (squared distance, source index)), by brute force over all sources.
 * Readings where the paper is silent (max reducer: empty row finalizes to 0 with arg -1,
 * ties go to the lowest edge position; periodic boxes use the minimum image; Gaussian and
 * Lennard-Jones messages; the cell-grid constants) are the build's own and are listed in
 * the design notes.
 *
 * Precision: every floating-point input is converted exactly to double; sums run in edge
 * order / index order with no blocking, no fusion, no reordering.
 * Compile with -ffp-contract=off so that no multiply-add is contracted.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { DT_F32 = 0, DT_F16 = 1, DT_F64 = 2 };
enum { RED_SUM = 0, RED_MAX = 1 };
enum { MSG_GAUSS = 2, MSG_DIST = 3, MSG_LJ = 4 };

static double half_to_double(uint16_t h) {
    int s = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return s ? -v : v;
}

static inline double ld(const void* p, int dt, int64_t i) {
    if (dt == DT_F32) return (double)((const float*)p)[i];
    if (dt == DT_F64) return ((const double*)p)[i];
    return half_to_double(((const uint16_t*)p)[i]);
}

/* ------------------------------------------------------------------ CSR forward
 * Section 3.1 / 4.3.  message m = w[e] * x[col[e], f]  (w == NULL means weight 1).
 * sum : y = sum of m in edge order, A = sum of |m|.
 * max : y = largest m, arg = lowest edge position attaining it (strict '>' while
 *       scanning in edge order); empty row -> y = 0, arg = -1.  A = |y|.
 *       The selection is an integer decided by floating point, so it is taken in the
 *       precision the messages exist in: with fp32 / fp16 inputs (decide_fp32 != 0) every
 *       message is the fp64 product rounded once to fp32 before it is compared; two
 *       products that round to the same fp32 value are a tie and the earlier edge wins.
 */
int oracle_csr_forward(const int64_t* rowptr, const int32_t* col, int64_t n_dst,
                       const void* w, int w_dt, const void* x, int x_dt, int F, int reducer,
                       int decide_fp32, double* y, double* A, int64_t* arg) {
#pragma omp parallel for schedule(dynamic, 256)
    for (int64_t i = 0; i < n_dst; ++i) {
        for (int f = 0; f < F; ++f) {
            double acc = 0.0, absacc = 0.0;
            int64_t best = -1;
            for (int64_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
                double we = w ? ld(w, w_dt, e) : 1.0;
                double m = we * ld(x, x_dt, (int64_t)col[e] * F + f);
                if (reducer == RED_MAX && decide_fp32) m = (double)(float)m;
                if (reducer == RED_SUM) {
                    acc += m;
                    absacc += fabs(m);
                } else if (best < 0 || m > acc) {
                    acc = m;
                    best = e;
                }
            }
            y[i * F + f] = acc;
            if (A) A[i * F + f] = (reducer == RED_SUM) ? absacc : fabs(acc);
            if (arg) arg[i * F + f] = best;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ CSR backward, sum
 * Section 5: wbar_e = sum_f x[col[e],f] * ybar[row(e),f];
 *            xbar_j = sum over edges e with col[e] = j of w_e * ybar[row(e),:].
 * Aw / Ax hold the sums of absolute contributions.  Any output pointer may be NULL.
 * The scatter into xbar is applied in edge order; threads own disjoint source ranges.
 */
int oracle_csr_backward_sum(const int64_t* rowptr, const int32_t* col, int64_t n_dst, int64_t n_src,
                            const void* w, int w_dt, const void* x, int x_dt, int F,
                            const void* gy, int gy_dt,
                            double* gw, double* Aw, double* gx, double* Ax) {
    if (gw) {
#pragma omp parallel for schedule(dynamic, 256)
        for (int64_t i = 0; i < n_dst; ++i)
            for (int64_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
                double s = 0.0, a = 0.0;
                for (int f = 0; f < F; ++f) {
                    double t = ld(x, x_dt, (int64_t)col[e] * F + f) * ld(gy, gy_dt, i * F + f);
                    s += t;
                    a += fabs(t);
                }
                gw[e] = s;
                if (Aw) Aw[e] = a;
            }
    }
    if (gx) {
        memset(gx, 0, sizeof(double) * (size_t)n_src * F);
        if (Ax) memset(Ax, 0, sizeof(double) * (size_t)n_src * F);
        int nparts = 64;
#pragma omp parallel for schedule(dynamic, 1)
        for (int p = 0; p < nparts; ++p) {
            int64_t lo = n_src * p / nparts, hi = n_src * (p + 1) / nparts;
            for (int64_t i = 0; i < n_dst; ++i)
                for (int64_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
                    int64_t j = col[e];
                    if (j < lo || j >= hi) continue;
                    double we = w ? ld(w, w_dt, e) : 1.0;
                    for (int f = 0; f < F; ++f) {
                        double t = we * ld(gy, gy_dt, i * F + f);
                        gx[j * F + f] += t;
                        if (Ax) Ax[j * F + f] += fabs(t);
                    }
                }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ CSR backward, max
 * The cotangent of (i,f) flows only through the selected edge e* = arg[i,f] >= 0:
 *   wbar[e*] += x[col[e*],f] * ybar[i,f];  xbar[col[e*],f] += w[e*] * ybar[i,f].
 * Serial on purpose (scatter in (i,f) order).
 */
int oracle_csr_backward_max(const int32_t* col, int64_t n_dst, int64_t n_src, int64_t n_edges,
                            const void* w, int w_dt, const void* x, int x_dt, int F,
                            const void* gy, int gy_dt, const int64_t* arg,
                            double* gw, double* Aw, double* gx, double* Ax) {
    if (gw) memset(gw, 0, sizeof(double) * (size_t)n_edges);
    if (Aw) memset(Aw, 0, sizeof(double) * (size_t)n_edges);
    if (gx) memset(gx, 0, sizeof(double) * (size_t)n_src * F);
    if (Ax) memset(Ax, 0, sizeof(double) * (size_t)n_src * F);
    for (int64_t i = 0; i < n_dst; ++i)
        for (int f = 0; f < F; ++f) {
            int64_t e = arg[i * F + f];
            if (e < 0) continue;
            int64_t j = col[e];
            double g = ld(gy, gy_dt, i * F + f);
            double we = w ? ld(w, w_dt, e) : 1.0;
            double tw = ld(x, x_dt, j * F + f) * g, tx = we * g;
            if (gw) gw[e] += tw;
            if (Aw) Aw[e] += fabs(tw);
            if (gx) gx[j * F + f] += tx;
            if (Ax) Ax[j * F + f] += fabs(tx);
        }
    return 0;
}

/* ------------------------------------------------------------------ degree histogram
 * deg_i = rowptr[i+1]-rowptr[i]; hist[d] counts rows of degree d for d < nbins-1, the
 * last bin counts deg >= nbins-1.
 */
int oracle_degree_histogram(const int64_t* rowptr, int64_t n, int64_t nbins, int64_t* hist,
                            int64_t* max_degree) {
    int64_t mx = 0;
    for (int64_t b = 0; b < nbins; ++b) hist[b] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t d = rowptr[i + 1] - rowptr[i];
        if (d > mx) mx = d;
        hist[d < nbins - 1 ? d : nbins - 1] += 1;
    }
    *max_degree = mx;
    return 0;
}

/* ------------------------------------------------------------------ cell directory
 * Grid constants (the build's reading; the paper only says "a cell directory restricts
 * candidate traversal to nearby spatial cells", Section 4.9):
 *   n_d = clamp(floor(len_d / (r (1 + 2^-10))), 1, min(1024, icbrt(8 n)))  in double,
 *   periodic dimensions with n_d < 3 use n_d = 1,  invh_d = (float)(n_d / len_d).
 * Cell of a point: c_d = min(n_d - 1, (int)floorf(p_d * invh_d)) with ONE fp32 multiply;
 * linear id (c_z n_y + c_y) n_x + c_x.
 */
static int64_t icbrt64(int64_t v) {
    int64_t c = 0;
    while ((c + 1) * (c + 1) * (c + 1) <= v) ++c;
    return c;
}

int oracle_cell_grid(int64_t n, float r, const float* len, const int32_t* periodic,
                     int32_t* ncell, float* invh) {
    int64_t cap = icbrt64(8 * (n > 0 ? n : 1));
    if (cap > 1024) cap = 1024;
    if (cap < 1) cap = 1;
    for (int d = 0; d < 3; ++d) {
        double q = floor((double)len[d] / ((double)r * (1.0 + 1.0 / 1024.0)));
        int64_t nd = q < 1.0 ? 1 : (q > (double)cap ? cap : (int64_t)q);
        if (periodic[d] && nd < 3) nd = 1;
        ncell[d] = (int32_t)nd;
        invh[d] = (float)((double)nd / (double)len[d]);
    }
    return 0;
}

/* stable counting sort of the points by cell id (ties by original index) */
int oracle_bin(const float* pos, int64_t n, const int32_t* ncell, const float* invh,
               int32_t* cell, int32_t* cell_start, int32_t* order) {
    int64_t nc = (int64_t)ncell[0] * ncell[1] * ncell[2];
    for (int64_t c = 0; c <= nc; ++c) cell_start[c] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int32_t c[3];
        for (int d = 0; d < 3; ++d) {
            volatile float t = pos[3 * i + d] * invh[d];   /* one rounded fp32 product */
            int32_t k = (int32_t)floorf(t);
            if (k > ncell[d] - 1) k = ncell[d] - 1;
            if (k < 0) k = 0;
            c[d] = k;
        }
        cell[i] = (c[2] * ncell[1] + c[1]) * ncell[0] + c[0];
        cell_start[cell[i] + 1] += 1;
    }
    for (int64_t c = 0; c < nc; ++c) cell_start[c + 1] += cell_start[c];
    int32_t* fill = (int32_t*)malloc(sizeof(int32_t) * (size_t)(nc > 0 ? nc : 1));
    if (!fill) return 1;
    memcpy(fill, cell_start, sizeof(int32_t) * (size_t)nc);
    for (int64_t i = 0; i < n; ++i) order[fill[cell[i]]++] = (int32_t)i;
    free(fill);
    return 0;
}

/* ------------------------------------------------------------------ radius relation
 * Displacement of the ordered pair (i, j): D = p_i - p_j, minimum image in periodic
 * dimensions (D -= L rint(D / L)), d2 = Dx^2 + Dy^2 + Dz^2 summed left to right,
 * j is a neighbour of i iff j != i and d2 <= r*r (inclusive, Appendix A).
 */
typedef struct {
    const double* pos;
    int64_t n;
    double r2;
    double len[3];
    int periodic[3];
} rel_t;

static inline int pair_d2(const rel_t* R, int64_t i, int64_t j, double D[3], double* d2) {
    for (int d = 0; d < 3; ++d) {
        double t = R->pos[3 * i + d] - R->pos[3 * j + d];
        if (R->periodic[d]) t -= R->len[d] * rint(t / R->len[d]);
        D[d] = t;
    }
    *d2 = D[0] * D[0] + D[1] * D[1] + D[2] * D[2];
    return *d2 <= R->r2;
}

/* Optional candidate restriction: an fp64 cell directory of the oracle's own
 * (cell edge >= r, 27-cell stencil, wrapped or clipped).  It changes which pairs are
 * tested, never the predicate; the tests check it against the all-pairs loop. */
typedef struct {
    int nc[3];
    int64_t* start;   /* [ncells+1] */
    int64_t* items;   /* point ids grouped by cell, ascending inside a cell */
} grid_t;

static void cell_of(const rel_t* R, const grid_t* G, int64_t i, int c[3]) {
    for (int d = 0; d < 3; ++d) {
        int k = (int)floor(R->pos[3 * i + d] / R->len[d] * G->nc[d]);
        if (k < 0) k = 0;
        if (k > G->nc[d] - 1) k = G->nc[d] - 1;
        c[d] = k;
    }
}

static int grid_build(const rel_t* R, double r, grid_t* G) {
    int64_t total = 1;
    for (int d = 0; d < 3; ++d) {
        double q = floor(R->len[d] / r);
        int k = q < 1.0 ? 1 : (q > 512.0 ? 512 : (int)q);
        if (k < 3) k = 1;
        G->nc[d] = k;
        total *= k;
    }
    G->start = (int64_t*)calloc((size_t)total + 1, sizeof(int64_t));
    G->items = (int64_t*)malloc(sizeof(int64_t) * (size_t)(R->n > 0 ? R->n : 1));
    if (!G->start || !G->items) return 1;
    for (int64_t i = 0; i < R->n; ++i) {
        int c[3];
        cell_of(R, G, i, c);
        G->start[((int64_t)c[2] * G->nc[1] + c[1]) * G->nc[0] + c[0] + 1] += 1;
    }
    for (int64_t c = 0; c < total; ++c) G->start[c + 1] += G->start[c];
    int64_t* fill = (int64_t*)malloc(sizeof(int64_t) * (size_t)total);
    if (!fill) return 1;
    memcpy(fill, G->start, sizeof(int64_t) * (size_t)total);
    for (int64_t i = 0; i < R->n; ++i) {
        int c[3];
        cell_of(R, G, i, c);
        G->items[fill[((int64_t)c[2] * G->nc[1] + c[1]) * G->nc[0] + c[0]]++] = i;
    }
    free(fill);
    return 0;
}

/* candidate list of point i into buf (ascending ids are NOT guaranteed; callers that need
 * index order sort it).  Returns the number of candidates. */
static int cmp_i64(const void* a, const void* b) {
    int64_t x = *(const int64_t*)a, y = *(const int64_t*)b;
    return (x > y) - (x < y);
}

static int64_t candidates(const rel_t* R, const grid_t* G, int64_t i, int64_t** buf, int64_t* cap) {
    int c[3];
    cell_of(R, G, i, c);
    int64_t m = 0;
    int lo[3], hi[3];
    for (int d = 0; d < 3; ++d) {
        if (G->nc[d] == 1) { lo[d] = 0; hi[d] = 0; }
        else { lo[d] = -1; hi[d] = 1; }
    }
    for (int dz = lo[2]; dz <= hi[2]; ++dz)
        for (int dy = lo[1]; dy <= hi[1]; ++dy)
            for (int dx = lo[0]; dx <= hi[0]; ++dx) {
                int q[3] = { c[0] + dx, c[1] + dy, c[2] + dz };
                int ok = 1;
                for (int d = 0; d < 3; ++d) {
                    if (q[d] < 0 || q[d] >= G->nc[d]) {
                        if (R->periodic[d]) q[d] = (q[d] + G->nc[d]) % G->nc[d];
                        else ok = 0;
                    }
                }
                if (!ok) continue;
                int64_t id = ((int64_t)q[2] * G->nc[1] + q[1]) * G->nc[0] + q[0];
                for (int64_t t = G->start[id]; t < G->start[id + 1]; ++t) {
                    if (m == *cap) {
                        *cap = *cap ? *cap * 2 : 256;
                        *buf = (int64_t*)realloc(*buf, sizeof(int64_t) * (size_t)*cap);
                    }
                    (*buf)[m++] = G->items[t];
                }
            }
    qsort(*buf, (size_t)m, sizeof(int64_t), cmp_i64);
    return m;
}

static void rel_init(rel_t* R, const double* pos, int64_t n, double r, const double* len,
                     const int32_t* periodic) {
    R->pos = pos;
    R->n = n;
    R->r2 = r * r;
    for (int d = 0; d < 3; ++d) { R->len[d] = len[d]; R->periodic[d] = periodic[d]; }
}

/* ------------------------------------------------------------------ fused radius forward
 * For each requested row i (rows == NULL: all rows) and every neighbour j in index order:
 *   GAUSS : y_i += exp(-d2 / (2 p0^2)) x_j                       (Fout = F)
 *   DIST  : y_i += sqrt(d2) x_j                                  (Fout = F)
 *   LJ    : q = p1^2/d2, q3 = q^3, (Fx,Fy,Fz) += 24 p0 (2 q3^2 - q3)/d2 * D,
 *           e += (1/2) 4 p0 (q3^2 - q3)                          (Fout = 4, feat unused)
 * A receives the sums of absolute contributions, count the number of neighbours.
 * No neighbours -> zero vector (Appendix A).
 */
int oracle_radius_forward(const double* pos, const double* feat, int64_t n, int F,
                          double r, const double* len, const int32_t* periodic,
                          int kind, double p0, double p1,
                          const int64_t* rows, int64_t n_rows, int use_cells,
                          double* y, double* A, int32_t* count) {
    rel_t R;
    rel_init(&R, pos, n, r, len, periodic);
    grid_t G = { {0, 0, 0}, NULL, NULL };
    if (use_cells && grid_build(&R, r, &G)) return 1;
    const int Fo = (kind == MSG_LJ) ? 4 : F;
    if (!rows) n_rows = n;
#pragma omp parallel
    {
        int64_t* buf = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 16)
        for (int64_t t = 0; t < n_rows; ++t) {
            int64_t i = rows ? rows[t] : t;
            double* yi = y + t * Fo;
            double* Ai = A ? A + t * Fo : NULL;
            for (int f = 0; f < Fo; ++f) { yi[f] = 0.0; if (Ai) Ai[f] = 0.0; }
            int32_t cnt = 0;
            int64_t m = use_cells ? candidates(&R, &G, i, &buf, &cap) : n;
            for (int64_t u = 0; u < m; ++u) {
                int64_t j = use_cells ? buf[u] : u;
                if (j == i) continue;
                double D[3], d2;
                if (!pair_d2(&R, i, j, D, &d2)) continue;
                ++cnt;
                if (kind == MSG_LJ) {
                    double q = p1 * p1 / d2, q3 = q * q * q;
                    double fs = 24.0 * p0 * (2.0 * q3 * q3 - q3) / d2;
                    double e = 0.5 * 4.0 * p0 * (q3 * q3 - q3);
                    for (int d = 0; d < 3; ++d) {
                        yi[d] += fs * D[d];
                        if (Ai) Ai[d] += fabs(fs * D[d]);
                    }
                    yi[3] += e;
                    if (Ai) Ai[3] += fabs(e);
                } else {
                    double g = (kind == MSG_GAUSS) ? exp(-d2 / (2.0 * p0 * p0)) : sqrt(d2);
                    for (int f = 0; f < F; ++f) {
                        double c = g * feat[j * F + f];
                        yi[f] += c;
                        if (Ai) Ai[f] += fabs(c);
                    }
                }
            }
            if (count) count[t] = cnt;
        }
        free(buf);
    }
    free(G.start);
    free(G.items);
    return 0;
}

/* ------------------------------------------------------------------ fused radius backward
 * Gaussian message, membership frozen (Section 5).  With L = sum_i ybar_i . y_i
 *   = sum over ordered pairs (i, j in N(i)) of g_ij (ybar_i . x_j),  g_ij = exp(-|D_ij|^2/(2 s^2)),
 * the plain chain rule gives, for output row k,
 *   xbar_k  = sum over i with k in N(i) of g_ik ybar_i
 *   pbar_k  = sum over j in N(k)        of (-g_kj / s^2) D_kj (ybar_k . x_j)     [k is the query]
 *           + sum over i with k in N(i) of (+g_ik / s^2) D_ik (ybar_i . x_k)     [k is the source]
 * Both sums are evaluated separately, each pair from its own displacement.
 */
int oracle_radius_backward_gauss(const double* pos, const double* feat, const double* gy,
                                 int64_t n, int F, double r, const double* len,
                                 const int32_t* periodic, double sigma,
                                 const int64_t* rows, int64_t n_rows, int use_cells,
                                 double* gx, double* Agx, double* gp, double* Agp) {
    rel_t R;
    rel_init(&R, pos, n, r, len, periodic);
    grid_t G = { {0, 0, 0}, NULL, NULL };
    if (use_cells && grid_build(&R, r, &G)) return 1;
    if (!rows) n_rows = n;
    const double is2 = 1.0 / (sigma * sigma);
#pragma omp parallel
    {
        int64_t* buf = NULL;
        int64_t cap = 0;
#pragma omp for schedule(dynamic, 16)
        for (int64_t t = 0; t < n_rows; ++t) {
            int64_t k = rows ? rows[t] : t;
            if (gx) for (int f = 0; f < F; ++f) { gx[t * F + f] = 0.0; if (Agx) Agx[t * F + f] = 0.0; }
            if (gp) for (int d = 0; d < 3; ++d) { gp[t * 3 + d] = 0.0; if (Agp) Agp[t * 3 + d] = 0.0; }
            int64_t m = use_cells ? candidates(&R, &G, k, &buf, &cap) : n;
            for (int64_t u = 0; u < m; ++u) {
                int64_t o = use_cells ? buf[u] : u;
                if (o == k) continue;
                double D[3], d2;
                /* k as the query, o as its neighbour j */
                if (pair_d2(&R, k, o, D, &d2)) {
                    double g = exp(-d2 / (2.0 * sigma * sigma));
                    double dot = 0.0;
                    for (int f = 0; f < F; ++f) dot += gy[k * F + f] * feat[o * F + f];
                    if (gp) for (int d = 0; d < 3; ++d) {
                        double c = (-g * is2) * D[d] * dot;
                        gp[t * 3 + d] += c;
                        if (Agp) Agp[t * 3 + d] += fabs(c);
                    }
                }
                /* o as the query i, k as its neighbour (the source) */
                if (pair_d2(&R, o, k, D, &d2)) {
                    double g = exp(-d2 / (2.0 * sigma * sigma));
                    double dot = 0.0;
                    for (int f = 0; f < F; ++f) dot += gy[o * F + f] * feat[k * F + f];
                    if (gp) for (int d = 0; d < 3; ++d) {
                        double c = (g * is2) * D[d] * dot;
                        gp[t * 3 + d] += c;
                        if (Agp) Agp[t * 3 + d] += fabs(c);
                    }
                    if (gx) for (int f = 0; f < F; ++f) {
                        double c = g * gy[o * F + f];
                        gx[t * F + f] += c;
                        if (Agx) Agx[t * F + f] += fabs(c);
                    }
                }
            }
        }
        free(buf);
    }
    free(G.start);
    free(G.items);
    return 0;
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}

/* ------------------------------------------------------------------ edge neural network
 * Appendix A: over the radius relation N(i) = { j != i : |p_j - p_i| <= r },
 *     y_i = sum over j in N(i) of [ W2 ReLU( W1 [p_j - p_i ; x_j] + b1 ) + b2 ]
 * with the displacement taken source minus destination (minimum image where periodic) and the
 * final bias inside the sum.  W1 is [H, 3 + Fin] row major, W2 is [Fout, H].
 * Reverse mode with the membership frozen (Section 5), by the plain chain rule per ordered pair:
 *     mbar = ybar_i,  W2bar += mbar a^T,  b2bar += mbar,  abar = W2^T mbar,
 *     hbar = abar * [h > 0],  W1bar += hbar u^T,  b1bar += hbar,  ubar = W1^T hbar,
 *     pbar_j += ubar[0:3],  pbar_i -= ubar[0:3],  xbar_j += ubar[3:].
 * ReLU'(0) = 0.  Every output has a companion array with the sum of absolute contributions.
 * ReLU makes the gradient discontinuous where a pre-activation crosses zero; a lower-precision
 * evaluation can land on the other side there.  The backward therefore also reports, per
 * point, whether any pair it takes part in has a pre-activation with |h| < kink_eps, so that a
 * comparison can leave exactly those rows out (Section 5: ReLU-like kinks need appropriate
 * test points).
 */
typedef struct {
    int Fin, H, Fout;
    const double *W1, *b1, *W2, *b2;
} mlp_t;

/* forward of one ordered pair (i <- j); returns h (pre-activation) and u as well */
static void mlp_pair(const rel_t* R, const double* feat, const mlp_t* M, int64_t i, int64_t j,
                     const double D_ij[3], double* u, double* h, double* m) {
    const int K = 3 + M->Fin;
    for (int d = 0; d < 3; ++d) u[d] = -D_ij[d];              /* p_j - p_i */
    for (int f = 0; f < M->Fin; ++f) u[3 + f] = feat[j * M->Fin + f];
    for (int a = 0; a < M->H; ++a) {
        double s = M->b1[a];
        for (int k = 0; k < K; ++k) s += M->W1[a * K + k] * u[k];
        h[a] = s;
    }
    for (int o = 0; o < M->Fout; ++o) {
        double s = M->b2[o];
        for (int a = 0; a < M->H; ++a) s += M->W2[o * M->H + a] * (h[a] > 0.0 ? h[a] : 0.0);
        m[o] = s;
    }
    (void)R; (void)i;
}

int oracle_radius_mlp_forward(const double* pos, const double* feat, int64_t n, int Fin,
                              double r, const double* len, const int32_t* periodic,
                              const double* W1, const double* b1, const double* W2, const double* b2,
                              int H, int Fout, int use_cells, double* y, double* A, int32_t* count) {
    rel_t R;
    rel_init(&R, pos, n, r, len, periodic);
    grid_t G = { {0, 0, 0}, NULL, NULL };
    if (use_cells && grid_build(&R, r, &G)) return 1;
    mlp_t M = { Fin, H, Fout, W1, b1, W2, b2 };
#pragma omp parallel
    {
        int64_t* buf = NULL;
        int64_t cap = 0;
        double u[64], h[64], m[16];
#pragma omp for schedule(dynamic, 16)
        for (int64_t i = 0; i < n; ++i) {
            for (int o = 0; o < Fout; ++o) { y[i * Fout + o] = 0.0; if (A) A[i * Fout + o] = 0.0; }
            int32_t cnt = 0;
            int64_t mc = use_cells ? candidates(&R, &G, i, &buf, &cap) : n;
            for (int64_t t = 0; t < mc; ++t) {
                int64_t j = use_cells ? buf[t] : t;
                if (j == i) continue;
                double D[3], d2;
                if (!pair_d2(&R, i, j, D, &d2)) continue;
                ++cnt;
                mlp_pair(&R, feat, &M, i, j, D, u, h, m);
                for (int o = 0; o < Fout; ++o) { y[i * Fout + o] += m[o]; if (A) A[i * Fout + o] += fabs(m[o]); }
            }
            if (count) count[i] = cnt;
        }
        free(buf);
    }
    free(G.start);
    free(G.items);
    return 0;
}

/* Outputs (each with its abs-sum companion): gx [n,Fin], gp [n,3], gW1 [H,3+Fin], gb1 [H],
 * gW2 [Fout,H], gb2 [Fout].  Row k of gx / gp is gathered from the pairs in which k is the
 * destination and those in which it is the source; parameter gradients are summed over the
 * ordered pairs by their destination, per thread, and folded in thread order. */
int oracle_radius_mlp_backward(const double* pos, const double* feat, const double* gy, int64_t n, int Fin,
                               double r, const double* len, const int32_t* periodic,
                               const double* W1, const double* b1, const double* W2, const double* b2,
                               int H, int Fout, int use_cells, double kink_eps, int32_t* kink,
                               double* gx, double* Agx, double* gp, double* Agp,
                               double* gW1, double* AgW1, double* gb1, double* Agb1,
                               double* gW2, double* AgW2, double* gb2, double* Agb2) {
    rel_t R;
    rel_init(&R, pos, n, r, len, periodic);
    grid_t G = { {0, 0, 0}, NULL, NULL };
    if (use_cells && grid_build(&R, r, &G)) return 1;
    mlp_t M = { Fin, H, Fout, W1, b1, W2, b2 };
    const int K = 3 + Fin;
    const int NP = H * K + H + Fout * H + Fout;
    for (int e = 0; e < H * K; ++e) { gW1[e] = 0.0; AgW1[e] = 0.0; }
    for (int e = 0; e < H; ++e) { gb1[e] = 0.0; Agb1[e] = 0.0; }
    for (int e = 0; e < Fout * H; ++e) { gW2[e] = 0.0; AgW2[e] = 0.0; }
    for (int e = 0; e < Fout; ++e) { gb2[e] = 0.0; Agb2[e] = 0.0; }
#pragma omp parallel
    {
        int64_t* buf = NULL;
        int64_t cap = 0;
        double u[64], h[64], m[16], hb[64], ub[64];
        double* acc = (double*)calloc((size_t)2 * NP, sizeof(double));     /* gradients, then abs sums */
        double* aW1 = acc, *ab1 = aW1 + H * K, *aW2 = ab1 + H, *ab2 = aW2 + Fout * H;
        double* sW1 = acc + NP, *sb1 = sW1 + H * K, *sW2 = sb1 + H, *sb2 = sW2 + Fout * H;
#pragma omp for schedule(dynamic, 16)
        for (int64_t k = 0; k < n; ++k) {
            for (int f = 0; f < Fin; ++f) { gx[k * Fin + f] = 0.0; Agx[k * Fin + f] = 0.0; }
            for (int d = 0; d < 3; ++d) { gp[k * 3 + d] = 0.0; Agp[k * 3 + d] = 0.0; }
            if (kink) kink[k] = 0;
            int64_t mc = use_cells ? candidates(&R, &G, k, &buf, &cap) : n;
            for (int64_t t = 0; t < mc; ++t) {
                int64_t o = use_cells ? buf[t] : t;
                if (o == k) continue;
                double D[3], d2;
                for (int role = 0; role < 2; ++role) {
                    /* role 0: k is the destination i, o the source j; role 1: o destination, k source */
                    const int64_t i = role == 0 ? k : o, j = role == 0 ? o : k;
                    if (!pair_d2(&R, i, j, D, &d2)) continue;
                    mlp_pair(&R, feat, &M, i, j, D, u, h, m);
                    if (kink) for (int a = 0; a < H; ++a) if (fabs(h[a]) < kink_eps) kink[k] = 1;
                    for (int a = 0; a < H; ++a) {
                        double s = 0.0;
                        for (int q = 0; q < Fout; ++q) s += W2[q * H + a] * gy[i * Fout + q];
                        hb[a] = h[a] > 0.0 ? s : 0.0;
                    }
                    for (int c = 0; c < K; ++c) {
                        double s = 0.0;
                        for (int a = 0; a < H; ++a) s += W1[a * K + c] * hb[a];
                        ub[c] = s;
                    }
                    if (role == 0) {
                        for (int d = 0; d < 3; ++d) { gp[k * 3 + d] -= ub[d]; Agp[k * 3 + d] += fabs(ub[d]); }
                        for (int a = 0; a < H; ++a) {
                            for (int c = 0; c < K; ++c) { aW1[a * K + c] += hb[a] * u[c]; sW1[a * K + c] += fabs(hb[a] * u[c]); }
                            ab1[a] += hb[a]; sb1[a] += fabs(hb[a]);
                            const double act = h[a] > 0.0 ? h[a] : 0.0;
                            for (int q = 0; q < Fout; ++q) {
                                aW2[q * H + a] += gy[i * Fout + q] * act;
                                sW2[q * H + a] += fabs(gy[i * Fout + q] * act);
                            }
                        }
                        for (int q = 0; q < Fout; ++q) { ab2[q] += gy[i * Fout + q]; sb2[q] += fabs(gy[i * Fout + q]); }
                    } else {
                        for (int d = 0; d < 3; ++d) { gp[k * 3 + d] += ub[d]; Agp[k * 3 + d] += fabs(ub[d]); }
                        for (int f = 0; f < Fin; ++f) { gx[k * Fin + f] += ub[3 + f]; Agx[k * Fin + f] += fabs(ub[3 + f]); }
                    }
                }
            }
        }
#pragma omp critical
        {
            for (int e = 0; e < H * K; ++e) { gW1[e] += aW1[e]; AgW1[e] += sW1[e]; }
            for (int e = 0; e < H; ++e) { gb1[e] += ab1[e]; Agb1[e] += sb1[e]; }
            for (int e = 0; e < Fout * H; ++e) { gW2[e] += aW2[e]; AgW2[e] += sW2[e]; }
            for (int e = 0; e < Fout; ++e) { gb2[e] += ab2[e]; Agb2[e] += sb2[e]; }
        }
        free(acc);
        free(buf);
    }
    free(G.start);
    free(G.items);
    return 0;
}

/* ------------------------------------------------------------------ generated exact kNN + neighbour sum
 * Section 4.9 (generated kNN): every destination query examines all sources, keeps the k
 * smallest ordering keys and consumes the selected source features without storing an
 * adjacency.  A key is (squared distance, source index), so equal distances are ordered by
 * index.  The evaluated workload (Section 7) is a neighbour sum with k = 16.
 *
 * Precision: the paper bounds this path to FP32 and computes reference distances by direct
 * differences, not by the matrix-product identity.  The selection is an integer decision
 * made by floating point, so it is taken here in that precision: the squared distance is
 * the fp32 value  fl(fl(fl(dx*dx) + fl(dy*dy)) + fl(dz*dz))  with  dx = fl(x_i - x_j)  and
 * no contraction (this file is compiled with -ffp-contract=off).  The neighbour sum itself
 * is accumulated in double, in key order.
 *
 * Readings where the paper is silent: the query itself is not its own neighbour (j != i by
 * index, as for the radius relation of Appendix A); with fewer than k other points the
 * missing entries have index -1, distance +inf and contribute nothing.
 *
 * For each requested row (rows == NULL: all): idx [n_rows, k] and d2 [n_rows, k] in key
 * order, y [n_rows, F] the neighbour sum, A the sum of absolute contributions.
 */
int oracle_knn(const float* pos, const double* feat, int64_t n, int F, int k,
               const int64_t* rows, int64_t n_rows,
               int32_t* idx, float* d2, double* y, double* A) {
    if (k <= 0) return 1;
    if (!rows) n_rows = n;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t t = 0; t < n_rows; ++t) {
        const int64_t i = rows ? rows[t] : t;
        int32_t* bi = idx + t * k;
        float* bd = d2 + t * k;
        int have = 0;
        const float xi = pos[3 * i], yi = pos[3 * i + 1], zi = pos[3 * i + 2];
        for (int64_t j = 0; j < n; ++j) {
            if (j == i) continue;
            const float dx = xi - pos[3 * j], dy = yi - pos[3 * j + 1], dz = zi - pos[3 * j + 2];
            const float sx = dx * dx, sy = dy * dy, sz = dz * dz;
            float s = sx + sy;
            s = s + sz;
            /* sources arrive in index order, so a candidate goes behind retained keys of equal distance */
            if (have == k && !(s < bd[k - 1])) continue;
            int at = have < k ? have : k - 1;
            while (at > 0 && s < bd[at - 1]) { bd[at] = bd[at - 1]; bi[at] = bi[at - 1]; --at; }
            bd[at] = s;
            bi[at] = (int32_t)j;
            if (have < k) ++have;
        }
        for (int u = have; u < k; ++u) { bi[u] = -1; bd[u] = INFINITY; }
        for (int f = 0; f < F; ++f) {
            double acc = 0.0, ab = 0.0;
            for (int u = 0; u < have; ++u) {
                const double c = feat[(int64_t)bi[u] * F + f];
                acc += c;
                ab += fabs(c);
            }
            y[t * F + f] = acc;
            if (A) A[t * F + f] = ab;
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ online-softmax reducer over a stored relation
 * Section 5 ("Online softmax") and the attention appendix: the edge function supplies a score
 * and a value, s_e = scale * <q_d(e), k_s(e)> and v_s(e); the reducer's result for row i is
 *     y_i = sum_e exp(s_e) v_s(e) / sum_e exp(s_e)        over the edges e of row i,
 * the relation deciding which interactions are admissible (a triangular relation gives causal
 * attention).  The streaming state (maximum, mass, accumulator) and its combine rule are a way
 * of evaluating exactly this quotient, so the oracle is the quotient itself: per row the
 * scores, their maximum, then the normalised sum, all in double, in edge order.
 * Repeated edges are separate messages.  Reading for the empty row (the paper leaves it to the
 * reducer's convention): zero vector, as for the sum reducer; lse = -inf.
 *   q [n_dst, D], k [n_src, D], v [n_src, D];  y, A [n_dst, D];  lse [n_dst] = log sum_e exp(s_e).
 * A receives sum_e softmax_e |v_s(e)|, the scale of the rounding error of y.
 */
int oracle_csr_attention(const int64_t* rowptr, const int32_t* col, int64_t n_dst,
                         const double* q, const double* k, const double* v, int D, double scale,
                         double* y, double* A, double* lse) {
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < n_dst; ++i) {
        const int64_t b = rowptr[i], e = rowptr[i + 1];
        double* yi = y + i * D;
        double* Ai = A ? A + i * D : NULL;
        for (int d = 0; d < D; ++d) { yi[d] = 0.0; if (Ai) Ai[d] = 0.0; }
        if (b == e) { if (lse) lse[i] = -INFINITY; continue; }
        double* s = (double*)malloc((size_t)(e - b) * sizeof(double));
        double mx = -INFINITY;
        for (int64_t t = b; t < e; ++t) {
            const double* kj = k + (int64_t)col[t] * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += q[i * D + d] * kj[d];
            s[t - b] = scale * dot;
            if (s[t - b] > mx) mx = s[t - b];
        }
        double mass = 0.0;
        for (int64_t t = b; t < e; ++t) mass += exp(s[t - b] - mx);
        for (int64_t t = b; t < e; ++t) {
            const double pr = exp(s[t - b] - mx) / mass;
            const double* vj = v + (int64_t)col[t] * D;
            for (int d = 0; d < D; ++d) {
                yi[d] += pr * vj[d];
                if (Ai) Ai[d] += fabs(pr * vj[d]);
            }
        }
        if (lse) lse[i] = mx + log(mass);
        free(s);
    }
    return 0;
}

/*
 * Seeded synthetic graph generators shared by the CPU oracle's tests and the CUDA
 * library's tests/benchmarks.  This file holds NO message-passing arithmetic: it only
 * produces index arrays.  All randomness is counter based (a hash of seed, stream and
 * element index), so the bytes produced do not depend on the number of threads.
 *
 * R-MAT recipe: for every directed edge and every one of `scale` levels (most
 * significant bit first) one quadrant is drawn with probabilities (a,b,c,d):
 *   a -> (row bit 0, col bit 0), b -> (0,1), c -> (1,0), d -> (1,1).
 * row = destination, col = source (the CSR of the paper is destination oriented,
 * Section 3.1).  No noise, no label permutation; self loops and duplicates are kept
 * because duplicate edges are separate messages (Section 3.1).
 * The CSR is a stable counting sort by row: edges of one row keep generation order.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o libtigagen.so rmat.c
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline uint64_t mix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ULL;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* one 64-bit word for (seed, stream, index) */
static inline uint64_t ctr64(uint64_t seed, uint64_t stream, uint64_t idx) {
    return mix64(mix64(seed + 0x632BE59BD9B4E019ULL * (stream + 1)) ^ (idx * 0xD1342543DE82EF95ULL + stream));
}

/* Draw the (row, col) pair of edge `e`.  Each 64-bit word serves two levels (one
 * 32-bit uniform each); thresholds are compared in 32-bit fixed point. */
static inline void rmat_edge(uint64_t seed, int scale, uint32_t ta, uint32_t tab, uint32_t tabc,
                             uint64_t e, int64_t* row, int64_t* col) {
    int64_t r = 0, c = 0;
    for (int l = 0; l < scale; l += 2) {
        uint64_t word = ctr64(seed, (uint64_t)(l >> 1), e);
        for (int h = 0; h < 2 && l + h < scale; ++h) {
            uint32_t u = (uint32_t)(word >> (32 * h));
            int rb, cb;
            if (u < ta) { rb = 0; cb = 0; }
            else if (u < tab) { rb = 0; cb = 1; }
            else if (u < tabc) { rb = 1; cb = 0; }
            else { rb = 1; cb = 1; }
            r = (r << 1) | rb;
            c = (c << 1) | cb;
        }
    }
    *row = r;
    *col = c;
}

static inline uint32_t thr(double p) {
    double v = p * 4294967296.0;
    if (v >= 4294967295.0) return 0xFFFFFFFFu;
    if (v <= 0.0) return 0u;
    return (uint32_t)v;
}

/*
 * Destination-oriented CSR of an R-MAT graph with 2^scale rows and sources.
 *   rowptr : int64[2^scale + 1]  (out)
 *   col    : int32[n_edges]      (out)  sources, grouped by destination row,
 *                                       generation order inside a row
 * Returns 0, or 1 on a bad argument / allocation failure.
 */
int tigagen_rmat_csr(uint64_t seed, int scale, int64_t n_edges, double a, double b, double c,
                     int64_t* rowptr, int32_t* col) {
    if (scale < 1 || scale > 30 || n_edges < 0) return 1;
    const int64_t n = (int64_t)1 << scale;
    const uint32_t ta = thr(a), tab = thr(a + b), tabc = thr(a + b + c);
    memset(rowptr, 0, (size_t)(n + 1) * sizeof(int64_t));

    /* pass 1: degree of every row (edges are re-derived in pass 2, nothing is stored) */
    const int64_t BLK = (int64_t)1 << 22;
    int32_t* rbuf = (int32_t*)malloc((size_t)BLK * sizeof(int32_t));
    int32_t* cbuf = (int32_t*)malloc((size_t)BLK * sizeof(int32_t));
    if (!rbuf || !cbuf) { free(rbuf); free(cbuf); return 1; }
    for (int64_t e0 = 0; e0 < n_edges; e0 += BLK) {
        const int64_t m = (n_edges - e0 < BLK) ? n_edges - e0 : BLK;
#pragma omp parallel for schedule(static)
        for (int64_t k = 0; k < m; ++k) {
            int64_t r, cc;
            rmat_edge(seed, scale, ta, tab, tabc, (uint64_t)(e0 + k), &r, &cc);
            rbuf[k] = (int32_t)r;
        }
        for (int64_t k = 0; k < m; ++k) rowptr[(int64_t)rbuf[k] + 1] += 1;
    }
    for (int64_t i = 0; i < n; ++i) rowptr[i + 1] += rowptr[i];

    /* pass 2: stable scatter; `fill` starts as a copy of rowptr[0..n) */
    int64_t* fill = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    if (!fill) { free(rbuf); free(cbuf); return 1; }
    memcpy(fill, rowptr, (size_t)n * sizeof(int64_t));
    for (int64_t e0 = 0; e0 < n_edges; e0 += BLK) {
        const int64_t m = (n_edges - e0 < BLK) ? n_edges - e0 : BLK;
#pragma omp parallel for schedule(static)
        for (int64_t k = 0; k < m; ++k) {
            int64_t r, cc;
            rmat_edge(seed, scale, ta, tab, tabc, (uint64_t)(e0 + k), &r, &cc);
            rbuf[k] = (int32_t)r;
            cbuf[k] = (int32_t)cc;
        }
        for (int64_t k = 0; k < m; ++k) col[fill[rbuf[k]]++] = cbuf[k];
    }
    free(fill);
    free(rbuf);
    free(cbuf);
    return 0;
}

/* The raw (row, col) pair of one edge index, for spot checks of the generator. */
void tigagen_rmat_edge(uint64_t seed, int scale, double a, double b, double c, int64_t e,
                       int64_t* row, int64_t* col) {
    rmat_edge(seed, scale, thr(a), thr(a + b), thr(a + b + c), (uint64_t)e, row, col);
}

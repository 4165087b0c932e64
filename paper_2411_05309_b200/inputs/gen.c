/*
 * Seeded synthetic input generators for the five paged-memory workloads.
 *
 * This file only produces INPUT DATA (arrays of numbers, a graph, a list of row
 * ids).  It contains no page-table, paging, eviction or workload arithmetic, so
 * both the CUDA path and the independent CPU checker may be fed from it.
 *
 * Every value is a pure function of (seed, element index): element i of a stream
 * is derived from mix64(seed, i), a counter-based 64-bit mixer (splitmix64
 * finaliser), so any slice of any array can be regenerated on its own and the
 * result does not depend on the thread count.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC gen.c -o libgpuvm_inputs.so -lm
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

static inline uint64_t mix64(uint64_t seed, uint64_t i)
{
    uint64_t z = seed + (i + 1) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

uint64_t gvi_mix64(uint64_t seed, uint64_t i) { return mix64(seed, i); }

/* int32 values uniform in [0, 2^20): the streaming read-reduce array. */
void gvi_fill_i32_u20(int32_t *dst, uint64_t first, uint64_t n, uint64_t seed)
{
#pragma omp parallel for schedule(static)
    for (uint64_t k = 0; k < n; ++k)
        dst[k] = (int32_t)(mix64(seed, first + k) & 0xFFFFFu);
}

/* fp32 values on the grid j*2^-23 - 1, j in [0, 2^24): uniform in [-1, 1), every
 * value exactly representable in binary32. */
void gvi_fill_f32_pm1(float *dst, uint64_t first, uint64_t n, uint64_t seed)
{
#pragma omp parallel for schedule(static)
    for (uint64_t k = 0; k < n; ++k) {
        uint32_t j = (uint32_t)(mix64(seed, first + k) >> 40);
        dst[k] = (float)j * 0x1p-23f - 1.0f;
    }
}

/* int32 values uniform in [lo, lo + span): edge weights. */
void gvi_fill_i32_range(int32_t *dst, uint64_t first, uint64_t n, uint64_t seed, int32_t lo, uint32_t span)
{
#pragma omp parallel for schedule(static)
    for (uint64_t k = 0; k < n; ++k)
        dst[k] = lo + (int32_t)(mix64(seed, first + k) % span);
}

/* int64 indices uniform in [0, modulo). */
void gvi_fill_index_i64(int64_t *dst, uint64_t first, uint64_t n, uint64_t seed,
                        uint64_t modulo)
{
#pragma omp parallel for schedule(static)
    for (uint64_t k = 0; k < n; ++k)
        dst[k] = (int64_t)(mix64(seed, first + k) % modulo);
}

/*
 * RMAT edge list -> CSR.  2^scale vertices, n_edges directed edges.  Each edge
 * descends `scale` quadrant levels; at each level one 32-bit draw r selects
 * quadrant a (r < ta), b (r < tb), c (r < tc) or d, with integer thresholds so
 * that every platform takes the same branch.  Quadrant b sets the destination
 * bit, c the source bit, d both.  No noise, no vertex permutation; self loops and
 * duplicate edges are kept.  CSR is built by a stable counting sort on the source
 * vertex (edges of one vertex keep their generation order).
 *
 * row_off: int64[2^scale + 1], col: int32[n_edges].  Returns 0, or -1 when the
 * temporary arrays cannot be allocated.
 */
int gvi_rmat_csr(int scale, uint64_t n_edges, uint64_t seed,
                 uint32_t ta, uint32_t tb, uint32_t tc,
                 int64_t *row_off, int32_t *col)
{
    const uint64_t nv = 1ull << scale;
    uint32_t *src = (uint32_t *)malloc(n_edges * sizeof(uint32_t));
    uint32_t *dst = (uint32_t *)malloc(n_edges * sizeof(uint32_t));
    if (!src || !dst) { free(src); free(dst); return -1; }
    const uint64_t draws_per_edge = (uint64_t)((scale + 1) / 2);
#pragma omp parallel for schedule(static)
    for (uint64_t e = 0; e < n_edges; ++e) {
        uint32_t u = 0, v = 0;
        for (int lvl = 0; lvl < scale; ++lvl) {
            uint64_t h = mix64(seed, e * draws_per_edge + (uint64_t)(lvl >> 1));
            uint32_t r = (lvl & 1) ? (uint32_t)(h >> 32) : (uint32_t)h;
            uint32_t sb = 0, db = 0;
            if (r < ta)      { }
            else if (r < tb) { db = 1; }
            else if (r < tc) { sb = 1; }
            else             { sb = 1; db = 1; }
            u = (u << 1) | sb;
            v = (v << 1) | db;
        }
        src[e] = u;
        dst[e] = v;
    }
    memset(row_off, 0, (nv + 1) * sizeof(int64_t));
    for (uint64_t e = 0; e < n_edges; ++e) row_off[(uint64_t)src[e] + 1]++;
    for (uint64_t v = 0; v < nv; ++v) row_off[v + 1] += row_off[v];
    int64_t *cursor = (int64_t *)malloc(nv * sizeof(int64_t));
    if (!cursor) { free(src); free(dst); return -1; }
    memcpy(cursor, row_off, nv * sizeof(int64_t));
    for (uint64_t e = 0; e < n_edges; ++e) col[cursor[src[e]]++] = (int32_t)dst[e];
    free(cursor); free(src); free(dst);
    return 0;
}

/*
 * Zipf(s) ranks over {1..n_ranks} by rejection-inversion (Hoermann & Derflinger
 * 1996), all arithmetic in double; dst[k] = rank - 1.  The uniforms of sample k
 * come from mix64(seed, k * 64 + attempt), so sample k is independent of how many
 * attempts its neighbours needed.
 */
static inline double zipf_H(double x, double s)      /* integral of x^-s */
{
    return (s == 1.0) ? log(x) : (pow(x, 1.0 - s) - 1.0) / (1.0 - s);
}
static inline double zipf_Hinv(double y, double s)
{
    return (s == 1.0) ? exp(y) : pow(1.0 + y * (1.0 - s), 1.0 / (1.0 - s));
}

void gvi_fill_zipf_rows(int64_t *dst, uint64_t first, uint64_t n, uint64_t seed,
                        uint64_t n_ranks, double s)
{
    const double h_x1 = zipf_H(1.5, s) - 1.0;                 /* H(1.5) - h(1) */
    const double h_n = zipf_H((double)n_ranks + 0.5, s);
    const double thresh = 2.0 - zipf_Hinv(zipf_H(2.5, s) - pow(2.0, -s), s);
#pragma omp parallel for schedule(static)
    for (uint64_t k = 0; k < n; ++k) {
        uint64_t rank = 1;
        for (uint64_t attempt = 0; attempt < 64; ++attempt) {
            uint64_t h = mix64(seed, (first + k) * 64 + attempt);
            double u01 = ((double)(h >> 11) + 0.5) * 0x1p-53;  /* (0,1) */
            double u = h_n + u01 * (h_x1 - h_n);
            double x = zipf_Hinv(u, s);
            double kf = floor(x + 0.5);
            if (kf < 1.0) kf = 1.0;
            if (kf > (double)n_ranks) kf = (double)n_ranks;
            if (kf - x <= thresh || u >= zipf_H(kf + 0.5, s) - pow(kf, -s)) {
                rank = (uint64_t)kf;
                break;
            }
        }
        dst[k] = (int64_t)(rank - 1);
    }
}

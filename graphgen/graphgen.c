/*
 * graphgen — seeded synthetic inputs (graphs, features, attention vectors).
 *
 * Input data only: nothing here knows how an aggregation is computed.  Every
 * random value is a pure function of (seed, stream, index), so the output does
 * not depend on the number of threads or on the order of generation.
 *
 * Streams: 1 degrees, 2 sources, 3 edge shuffle, 4 features, 5 a_src,
 * 6 a_dst, 7 RMAT quadrants, 8 vertex relabelling.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ PRNG */

static inline uint64_t fin64(uint64_t z)
{
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27; z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}

/* counter-based generator: two rounds of a splitmix-style finaliser over a
 * key built from (seed, stream, index) */
uint64_t gg_mix64(uint64_t seed, uint64_t stream, uint64_t index)
{
    uint64_t z = fin64(seed * 0x9E3779B97F4A7C15ULL + 0x632BE59BD9B4E019ULL);
    z = fin64(z ^ (stream * 0xD1342543DE82EF95ULL + 0x2545F4914F6CDD1DULL));
    z = fin64(z + index * 0x9E3779B97F4A7C15ULL + 0x9E3779B97F4A7C15ULL);
    return z;
}

/* uniform in [0,1) from the top 53 bits */
static inline double u01(uint64_t seed, uint64_t stream, uint64_t index)
{
    return (double)(gg_mix64(seed, stream, index) >> 11) * (1.0 / 9007199254740992.0);
}

/* ---------------------------------------- keyed permutation of [0, n) */

typedef struct { uint64_t n; int half_bits; uint64_t half_mask; uint64_t seed, stream; } perm_t;

static perm_t perm_make(uint64_t n, uint64_t seed, uint64_t stream)
{
    perm_t p; int bits = 2;
    while (bits < 64 && (1ULL << bits) < n) bits += 2;
    p.n = n; p.half_bits = bits / 2; p.half_mask = (1ULL << p.half_bits) - 1;
    p.seed = seed; p.stream = stream;
    return p;
}

/* 4-round balanced Feistel network on 2*half_bits bits, cycle-walked into [0,n) */
static inline uint64_t perm_apply(const perm_t *p, uint64_t x)
{
    do {
        uint64_t l = x >> p->half_bits, r = x & p->half_mask;
        for (int round = 0; round < 4; ++round) {
            uint64_t f = gg_mix64(p->seed, p->stream, ((uint64_t)round << 56) | r) & p->half_mask;
            uint64_t t = l ^ f; l = r; r = t;
        }
        x = (l << p->half_bits) | r;
    } while (x >= p->n);
    return x;
}

/* ---------------------------------------------------------- power law */

static inline int64_t pl_degree(double u, double x0, double inv_am1, int64_t dmax)
{
    double d = floor(x0 * pow(1.0 - u, -inv_am1));
    if (!(d >= 1.0)) d = 1.0;
    if (d > (double)dmax) d = (double)dmax;
    return (int64_t)d;
}

static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * Power-law (Chung–Lu style) directed graph.
 *   in-degree d_v = clamp(floor(x0 (1-U_v)^(-1/(alpha-1))), 1, dmax); x0 is
 *   bisected until sum d_v is within 0.5 % of a draw budget;
 *   each of the d_v sources of row v is drawn in proportion to d_u (redrawn
 *   while u == v); duplicates inside a row are dropped;
 *   the draw budget starts at target_edges and is rescaled (at most 5 times)
 *   until the number of distinct edges is within 1 % of target_edges;
 *   vertex ids are relabelled by a keyed permutation and the edges are
 *   emitted in a keyed-permutation order.
 * src/dst must hold cap entries.  Returns the edge count, or -1 when cap is
 * too small, -2 on allocation failure, -3 on bad arguments.
 */
int64_t gg_powerlaw_graph(int64_t n, int64_t target_edges, double alpha, int64_t dmax,
                          uint64_t seed, int relabel, int32_t *src, int32_t *dst, int64_t cap)
{
    if (n < 2 || target_edges < n || dmax < 1 || alpha <= 1.0) return -3;
    if (dmax > n - 1) dmax = n - 1;
    const double inv_am1 = 1.0 / (alpha - 1.0);
    double *u = (double *)malloc(sizeof(double) * (size_t)n);
    int64_t *cum = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int64_t *kept = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int32_t *raw = NULL;
    if (!u || !cum || !kept) { free(u); free(cum); free(kept); return -2; }
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < n; ++v) u[v] = u01(seed, 1, (uint64_t)v);

    double budget = (double)target_edges;
    int64_t e = 0;
    for (int outer = 0; outer < 6; ++outer) {
        double lo = 1e-3, hi = (double)dmax + 1.0, x0 = 1.0;
        for (int it = 0; it < 200; ++it) {
            x0 = 0.5 * (lo + hi);
            int64_t total = 0;
#pragma omp parallel for schedule(static) reduction(+ : total)
            for (int64_t v = 0; v < n; ++v) total += pl_degree(u[v], x0, inv_am1, dmax);
            double rel = ((double)total - budget) / budget;
            if (fabs(rel) <= 0.005) break;
            if (rel > 0) hi = x0; else lo = x0;
        }
        cum[0] = 0;
        for (int64_t v = 0; v < n; ++v) cum[v + 1] = cum[v] + pl_degree(u[v], x0, inv_am1, dmax);
        const int64_t total = cum[n];
        free(raw);
        raw = (int32_t *)malloc(sizeof(int32_t) * (size_t)total);
        if (!raw) { free(u); free(cum); free(kept); return -2; }

#pragma omp parallel for schedule(dynamic, 64)
        for (int64_t v = 0; v < n; ++v) {
            const int64_t b = cum[v], d = cum[v + 1] - cum[v];
            int32_t *row = raw + b;
            for (int64_t k = 0; k < d; ++k) {
                int64_t s = v;
                for (uint64_t attempt = 0; s == v; ++attempt) {
                    double r = u01(seed, 2, (uint64_t)(b + k) + attempt * (uint64_t)total);
                    int64_t t = (int64_t)(r * (double)total);
                    if (t >= total) t = total - 1;
                    /* largest s with cum[s] <= t */
                    int64_t a = 0, c = n;
                    while (c - a > 1) { int64_t m = (a + c) >> 1; if (cum[m] <= t) a = m; else c = m; }
                    s = a;
                }
                row[k] = (int32_t)s;
            }
            qsort(row, (size_t)d, sizeof(int32_t), cmp_i32);
            int64_t w = 0;
            for (int64_t k = 0; k < d; ++k)
                if (k == 0 || row[k] != row[k - 1]) row[w++] = row[k];
            kept[v + 1] = w;
        }
        kept[0] = 0;
        for (int64_t v = 0; v < n; ++v) kept[v + 1] += kept[v];
        e = kept[n];
        double rel = ((double)e - (double)target_edges) / (double)target_edges;
        if (fabs(rel) <= 0.01) break;
        budget *= (double)target_edges / (double)e;
    }
    free(u);
    if (e > cap) { free(raw); free(kept); free(cum); return -1; }

    perm_t pv = perm_make((uint64_t)n, seed, 8);
    perm_t pe = perm_make((uint64_t)e, seed, 3);
    /* position of every kept edge in the emitted order */
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t v = 0; v < n; ++v) {
        const int32_t *row = raw + cum[v];
        const int32_t vd = relabel ? (int32_t)perm_apply(&pv, (uint64_t)v) : (int32_t)v;
        for (int64_t k = kept[v]; k < kept[v + 1]; ++k) {
            int32_t s = row[k - kept[v]];
            if (relabel) s = (int32_t)perm_apply(&pv, (uint64_t)s);
            uint64_t pos = perm_apply(&pe, (uint64_t)k);
            src[pos] = s; dst[pos] = vd;
        }
    }
    free(raw); free(kept); free(cum);
    return e;
}

/*
 * RMAT: e edges on 2^scale vertices; one quadrant draw per bit level per edge
 * with probabilities a, b, c, d = 1-a-b-c.  Quadrant (row bit, column bit):
 * a=(0,0) b=(0,1) c=(1,0) d=(1,1); the row is the source and the column the
 * destination.  Optional keyed relabelling of the vertex ids.
 */
int gg_rmat_graph(int scale, int64_t e, double a, double b, double c, uint64_t seed, int relabel,
                  int32_t *src, int32_t *dst)
{
    if (scale < 1 || scale > 30 || e < 0) return -3;
    perm_t pv = perm_make(1ULL << scale, seed, 8);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < e; ++i) {
        uint32_t s = 0, d = 0;
        for (int l = 0; l < scale; ++l) {
            double r = u01(seed, 7, (uint64_t)i * (uint64_t)scale + (uint64_t)l);
            uint32_t sb, db;
            if (r < a) { sb = 0; db = 0; }
            else if (r < a + b) { sb = 0; db = 1; }
            else if (r < a + b + c) { sb = 1; db = 0; }
            else { sb = 1; db = 1; }
            s = (s << 1) | sb; d = (d << 1) | db;
        }
        if (relabel) { s = (uint32_t)perm_apply(&pv, s); d = (uint32_t)perm_apply(&pv, d); }
        src[i] = (int32_t)s; dst[i] = (int32_t)d;
    }
    return 0;
}

/* uniformly random directed multigraph (tests: duplicates and self-loops occur) */
int gg_uniform_graph(int64_t n, int64_t e, uint64_t seed, int32_t *src, int32_t *dst)
{
    if (n < 1) return -3;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < e; ++i) {
        src[i] = (int32_t)(gg_mix64(seed, 2, (uint64_t)i) % (uint64_t)n);
        dst[i] = (int32_t)(gg_mix64(seed, 1, (uint64_t)i) % (uint64_t)n);
    }
    return 0;
}

/* ----------------------------------------------------------- features */

/* rows x cols fp32 matrix with leading dimension ld; element (r, c) uses
 * index r*cols + c of the stream; padding columns are set to pad.
 * dist 0: uniform [p0, p1); dist 1: normal(mean p0, std p1) by Box–Muller in fp64. */
int gg_fill_f32(float *out, int64_t rows, int64_t cols, int64_t ld, int dist, double p0, double p1,
                uint64_t seed, uint64_t stream, float pad)
{
    if (ld < cols) return -3;
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        float *row = out + r * ld;
        for (int64_t c = 0; c < cols; ++c) {
            uint64_t i = (uint64_t)(r * cols + c);
            double x;
            if (dist == 0) {
                x = p0 + (p1 - p0) * u01(seed, stream, i);
            } else {
                double u1 = 1.0 - u01(seed, stream, 2 * i);      /* (0,1] */
                double u2 = u01(seed, stream, 2 * i + 1);
                x = p0 + p1 * sqrt(-2.0 * log(u1)) * cos(two_pi * u2);
            }
            row[c] = (float)x;
        }
        for (int64_t c = cols; c < ld; ++c) row[c] = pad;
    }
    return 0;
}

/* fp32 -> bf16 bit patterns, round to nearest even (NaN kept quiet) */
void gg_f32_to_bf16(const float *in, uint16_t *out, int64_t count)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        uint32_t b; memcpy(&b, in + i, 4);
        if ((b & 0x7F800000u) == 0x7F800000u && (b & 0x007FFFFFu)) { out[i] = (uint16_t)((b >> 16) | 0x40u); continue; }
        b += 0x7FFFu + ((b >> 16) & 1u);
        out[i] = (uint16_t)(b >> 16);
    }
}

/* bf16 bit patterns -> fp32 (exact) */
void gg_bf16_to_f32(const uint16_t *in, float *out, int64_t count)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        uint32_t b = (uint32_t)in[i] << 16; memcpy(out + i, &b, 4);
    }
}

int gg_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

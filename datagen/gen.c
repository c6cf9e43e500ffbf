/*
 * Seeded synthetic-input generator (host side, plain C + OpenMP).
 *
 * Every value is a pure function of (seed, stream, index), so any slice of any
 * array can be produced anywhere, by any number of threads, with the same bits.
 * This file holds no arithmetic of the fused-operator method: it only makes
 * inputs.  Both the CUDA path's tests/benchmarks and the CPU checker read the
 * arrays it writes.
 *
 * Generator: a counter-based hash built on the SplitMix64 output function
 * (Steele, Lea, Flood: "Fast splittable pseudorandom number generators",
 * OOPSLA 2014):   z = c + 0x9E3779B97F4A7C15 * (index + 1)
 *                 z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9
 *                 z = (z ^ (z >> 27)) * 0x94D049BB133111EB
 *                 z =  z ^ (z >> 31)
 * where the stream constant c is the same mix applied to (seed, stream).
 *
 *   uniform  u = (z >> 11) * 2^-53                      in [0, 1)
 *   normal   Box-Muller on the pair (2p, 2p+1):  r = sqrt(-2 ln u1), u1 in (0,1]
 *            element 2p = r cos(2 pi u2), element 2p+1 = r sin(2 pi u2)
 *   CSR      independent Bernoulli(density) per cell, realised by geometric
 *            skipping along each row (gap = floor(ln u / ln(1-density)), u in
 *            (0,1]); columns come out strictly ascending, row lengths are
 *            Binomial(cols, density).
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

static inline uint64_t mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

static inline uint64_t stream_key(uint64_t seed, uint64_t stream)
{
    return mix64(mix64(seed + 0x9E3779B97F4A7C15ULL) ^ (stream * 0xD1B54A32D192ED03ULL + 1ULL));
}

static inline uint64_t draw(uint64_t key, uint64_t index)
{
    return mix64(key + 0x9E3779B97F4A7C15ULL * (index + 1ULL));
}

static inline double to_unit(uint64_t z) /* [0,1) */
{
    return (double)(z >> 11) * 0x1.0p-53;
}

static inline double to_unit_open0(uint64_t z) /* (0,1] */
{
    return (double)((z >> 11) + 1ULL) * 0x1.0p-53;
}

/* out[k] = lo + (hi-lo) * u(offset + k),  k in [0, count) */
void dg_uniform(uint64_t seed, uint64_t stream, int64_t offset, int64_t count,
                double lo, double hi, double *out)
{
    const uint64_t key = stream_key(seed, stream);
    const double span = hi - lo;
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < count; ++k)
        out[k] = lo + span * to_unit(draw(key, (uint64_t)(offset + k)));
}

/* out[k] = mean + std * z(offset + k),  k in [0, count) */
void dg_normal(uint64_t seed, uint64_t stream, int64_t offset, int64_t count,
               double mean, double std, double *out)
{
    const uint64_t key = stream_key(seed, stream);
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < count; ++k) {
        const uint64_t e = (uint64_t)(offset + k);
        const uint64_t p = e >> 1;
        const double u1 = to_unit_open0(draw(key, 2 * p));
        const double u2 = to_unit(draw(key, 2 * p + 1));
        const double r = sqrt(-2.0 * log(u1));
        const double a = two_pi * u2;
        out[k] = mean + std * r * ((e & 1) ? sin(a) : cos(a));
    }
}

/* Column of the next stored cell after `col` in a row (col = -1 to start). */
static inline int64_t next_col(uint64_t key, int64_t row, int64_t cols_, uint64_t k,
                               int64_t col, double inv_log1mp)
{
    (void)cols_;
    const uint64_t idx = ((uint64_t)row << 20) + k; /* rows hold far fewer than 2^20 draws */
    const double u = to_unit_open0(draw(key, idx));
    double gap = floor(log(u) * inv_log1mp);
    if (!(gap < 4.0e18)) gap = 4.0e18;
    return col + 1 + (int64_t)gap;
}

/* Row lengths of rows [row0, row0+nrows): counts[r] = number of stored cells. */
void dg_csr_count(uint64_t seed, uint64_t stream, int64_t row0, int64_t nrows,
                  int64_t cols, double density, int64_t *counts)
{
    const uint64_t key = stream_key(seed, stream);
    const double inv = (density >= 1.0) ? 0.0 : 1.0 / log1p(-density);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        int64_t c = -1, n = 0;
        uint64_t k = 0;
        if (density > 0.0) {
            for (;;) {
                c = (density >= 1.0) ? c + 1 : next_col(key, row0 + r, cols, k, c, inv);
                if (c >= cols) break;
                ++n; ++k;
            }
        }
        counts[r] = n;
    }
}

/*
 * Fill colidx / vals for rows [row0, row0+nrows).  rowptr holds nrows+1 offsets
 * relative to the first stored cell of row0 (rowptr[0] = 0), i.e. the exclusive
 * prefix sum of dg_csr_count's output.  Values are lo + (hi-lo) * u, drawn from
 * the stream `stream + 1` at index (row << 20) + position-in-row.
 */
void dg_csr_fill(uint64_t seed, uint64_t stream, int64_t row0, int64_t nrows,
                 int64_t cols, double density, double lo, double hi,
                 const int64_t *rowptr, int32_t *colidx, double *vals)
{
    const uint64_t key = stream_key(seed, stream);
    const uint64_t vkey = stream_key(seed, stream + 1);
    const double inv = (density >= 1.0) ? 0.0 : 1.0 / log1p(-density);
    const double span = hi - lo;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < nrows; ++r) {
        int64_t c = -1;
        uint64_t k = 0;
        int64_t p = rowptr[r];
        if (density <= 0.0) continue;
        for (;;) {
            c = (density >= 1.0) ? c + 1 : next_col(key, row0 + r, cols, k, c, inv);
            if (c >= cols) break;
            colidx[p] = (int32_t)c;
            vals[p] = lo + span * to_unit(draw(vkey, ((uint64_t)(row0 + r) << 20) + k));
            ++p; ++k;
        }
    }
}

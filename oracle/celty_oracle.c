/*
 * CPU oracle for the dual-sparse decode product y = W.x (Celty, Sections 3.1-3.3).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, obviously-correct fp64 C.  Nothing in the
 * product (the CUDA library and its Python binding) may include, link or call this file;
 * only the tests, the smoke check and the benchmark's cpu_baseline leg use it.  It shares
 * no code, header, table or helper with the CUDA path.
 *
 * What each function follows:
 *   orc_half_to_double      IEEE-754 binary16 -> binary64, exact (weights and activations
 *                           are FP16, Section 5 "Baselines").
 *   orc_masked_gemv         the plain definition of the result: the method only skips
 *                           multiplications by zero (Section 3.1, column skip; Section 3.2,
 *                           stored non-zeros), so y is the masked dense product restricted
 *                           to the surviving activations.
 *   orc_rlc_count/_fill     n-bit run-length coded CSC (Section 3.2): one run per stored
 *                           value = number of zeros preceding it; a gap larger than
 *                           2^n - 1 inserts zero-valued padding entries.  Worked example of
 *                           Section 3.2 (2-bit) is a test pin.
 *   orc_rlc_decode_rows     Algorithm 1 written as what it computes: inclusive prefix sum
 *                           of the runs plus the entry's ordinal (Section 3.3).
 *   orc_spmspv_rlc          the same product evaluated from the encoded arrays: decode,
 *                           then scatter-accumulate column by column (Section 3.3).
 *
 * Readings where the paper is silent (listed with reasons in the design notes):
 *   - a padding entry occupies one row itself and carries run = 2^n - 1; the first run of a
 *     column (or of a row tile) counts from the first row of that column (tile);
 *   - nothing is emitted after the last kept row; an empty column stores nothing;
 *   - tile_rows > 0 applies the same rule independently to consecutive row tiles of
 *     tile_rows rows (the paper partitions M across warps, Section 3.1); tile_rows = 0 is
 *     the whole column;
 *   - a kept entry whose value is +-0 is stored like any other; pads are flagged, not
 *     inferred from the value.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

double orc_half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1F;
    int frac = h & 0x3FF;
    double v;
    if (expo == 0) {
        v = ldexp((double)frac, -24);            /* subnormal or zero: frac * 2^-24 */
    } else if (expo == 31) {
        v = frac ? NAN : INFINITY;
    } else {
        v = ldexp((double)(1024 + frac), expo - 25); /* (1 + frac/1024) * 2^(expo-15) */
    }
    return sign ? -v : v;
}

int orc_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Plain definition (Section 3.1): for every row i,
 *   y[i] = sum over j ascending, mask[i][j] != 0 and keep[j] != 0, of W[i][j] * x[j]   (fp64)
 *   a[i] = the same sum of |W[i][j] * x[j]|                                           (fp64)
 * Masked-out and dropped terms are skipped, not multiplied.
 * W and mask are row-major with leading dimensions ldw / ldm (elements).
 * threads <= 1 runs serially; otherwise rows are split over that many OpenMP threads
 * (each row is still summed serially in ascending j, so the result does not depend on it).
 */
void orc_masked_gemv(const uint16_t *W, int64_t ldw, const uint8_t *mask, int64_t ldm,
                     int64_t M, int64_t K, const uint16_t *x, const uint8_t *keep,
                     double *y, double *a, int threads)
{
    int64_t i;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(threads > 1 ? threads : 1)
#endif
    for (i = 0; i < M; ++i) {
        double s = 0.0, sa = 0.0;
        for (int64_t j = 0; j < K; ++j) {
            if (!keep[j]) continue;
            if (!mask[i * ldm + j]) continue;
            double p = orc_half_to_double(W[i * ldw + j]) * orc_half_to_double(x[j]);
            s += p;
            sa += fabs(p);
        }
        y[i] = s;
        if (a) a[i] = sa;
    }
    (void)threads;
}

static int64_t n_tiles_of(int64_t M, int64_t tile_rows)
{
    return tile_rows > 0 ? (M + tile_rows - 1) / tile_rows : 1;
}

/*
 * Pass 1 of the encoder (Section 3.2): number of stored entries (non-zeros + pads) of
 * every block.  Block b = j * T + t is row tile t of column j, T = ceil(M / tile_rows)
 * (T = 1 when tile_rows == 0).  block_ptr has K*T + 1 slots and receives the exclusive
 * prefix sum of the block sizes.  Returns the total number of stored entries.
 */
int64_t orc_rlc_count(const uint8_t *mask, int64_t ldm, int64_t M, int64_t K,
                      int run_bits, int64_t tile_rows, int64_t *block_ptr)
{
    const int64_t max_run = ((int64_t)1 << run_bits) - 1;
    const int64_t T = n_tiles_of(M, tile_rows);
    const int64_t rows_per_tile = tile_rows > 0 ? tile_rows : M;
    int64_t total = 0;
    for (int64_t j = 0; j < K; ++j) {
        for (int64_t t = 0; t < T; ++t) {
            int64_t r0 = t * rows_per_tile;
            int64_t r1 = r0 + rows_per_tile < M ? r0 + rows_per_tile : M;
            int64_t gap = 0, n = 0;
            for (int64_t r = r0; r < r1; ++r) {
                if (!mask[r * ldm + j]) { gap += 1; continue; }
                while (gap > max_run) { n += 1; gap -= max_run + 1; } /* pad: max_run zeros + itself */
                n += 1;
                gap = 0;
            }
            block_ptr[j * T + t] = total;
            total += n;
        }
    }
    block_ptr[K * T] = total;
    return total;
}

/*
 * Pass 2 of the encoder (Section 3.2): for each block, in ascending row order, emit
 * (value, run) for every kept row, preceded by as many padding entries (value +0,
 * run 2^n - 1, flagged in is_pad) as the gap requires.  runs holds one run per byte.
 */
void orc_rlc_fill(const uint16_t *W, int64_t ldw, const uint8_t *mask, int64_t ldm,
                  int64_t M, int64_t K, int run_bits, int64_t tile_rows,
                  const int64_t *block_ptr, uint16_t *vals, uint8_t *runs, uint8_t *is_pad)
{
    const int64_t max_run = ((int64_t)1 << run_bits) - 1;
    const int64_t T = n_tiles_of(M, tile_rows);
    const int64_t rows_per_tile = tile_rows > 0 ? tile_rows : M;
    for (int64_t j = 0; j < K; ++j) {
        for (int64_t t = 0; t < T; ++t) {
            int64_t r0 = t * rows_per_tile;
            int64_t r1 = r0 + rows_per_tile < M ? r0 + rows_per_tile : M;
            int64_t e = block_ptr[j * T + t];
            int64_t gap = 0;
            for (int64_t r = r0; r < r1; ++r) {
                if (!mask[r * ldm + j]) { gap += 1; continue; }
                while (gap > max_run) {
                    vals[e] = 0; runs[e] = (uint8_t)max_run; is_pad[e] = 1; e += 1;
                    gap -= max_run + 1;
                }
                vals[e] = W[r * ldw + j]; runs[e] = (uint8_t)gap; is_pad[e] = 0; e += 1;
                gap = 0;
            }
        }
    }
}

/*
 * Decode (Algorithm 1 + "the absolute row index follows by adding each entry's ordinal",
 * Section 3.3): within a block, row of entry e = tile start + (run_0 + ... + run_e) + e.
 */
void orc_rlc_decode_rows(const uint8_t *runs, const int64_t *block_ptr, int64_t K,
                         int64_t M, int64_t tile_rows, int32_t *rows)
{
    const int64_t T = n_tiles_of(M, tile_rows);
    const int64_t rows_per_tile = tile_rows > 0 ? tile_rows : M;
    for (int64_t j = 0; j < K; ++j) {
        for (int64_t t = 0; t < T; ++t) {
            int64_t s = 0;
            int64_t b0 = block_ptr[j * T + t], b1 = block_ptr[j * T + t + 1];
            for (int64_t e = b0; e < b1; ++e) {
                s += runs[e];
                rows[e] = (int32_t)(t * rows_per_tile + s + (e - b0));
            }
        }
    }
}

/*
 * The product evaluated from the encoded arrays (Sections 3.1 and 3.3): for each
 * surviving column j in ascending order, every stored entry adds value * x[j] to the
 * output row it decodes to.  fp64; pads add +-0.  y (and a, if given) are overwritten.
 */
void orc_spmspv_rlc(const uint16_t *vals, const int32_t *rows, const int64_t *block_ptr,
                    int64_t K, int64_t M, int64_t tile_rows, const uint16_t *x,
                    const uint8_t *keep, double *y, double *a)
{
    const int64_t T = n_tiles_of(M, tile_rows);
    for (int64_t i = 0; i < M; ++i) { y[i] = 0.0; if (a) a[i] = 0.0; }
    for (int64_t j = 0; j < K; ++j) {
        if (!keep[j]) continue;
        double xj = orc_half_to_double(x[j]);
        for (int64_t e = block_ptr[j * T]; e < block_ptr[(j + 1) * T]; ++e) {
            double p = orc_half_to_double(vals[e]) * xj;
            y[rows[e]] += p;
            if (a) a[rows[e]] += fabs(p);
        }
    }
}

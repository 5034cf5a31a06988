/*
 * CPU oracle for the FluxBin decode linear layer  y = X * What^T.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64.  Shares no code with the CUDA
 * path; only tests, the smoke check and the benchmark's cpu_baseline leg may
 * call it.
 *
 * What is the weight?  (Def. 3.1 / Eq. 3, Eq. 9, with "one row scale per weight
 * group" of g columns and the storage model of the appendix):
 *
 *   What[i][j] = sum_{k<Kb} ar[k][i][j/g] * ac[k][j] * B[k][i][j]
 *              + sum_{k<Ks} sum_{v : idx[v]==j} asr[k][i][j/g] * ascd[k][v] * Bsd[k][i][v]
 *
 * with B in {-1,+1} stored as bits (1 <=> +1, Eq. 14's 2b-1), Bsd the dense
 * "virtual column" matrix of Eq. 12 and ascd the gathered column scale of Eq. 13.
 *
 * Functions
 *   fbo_dense_weight   materialise What in fp64 (brute force, tiny shapes)
 *   fbo_dense_linear   y = X What^T from the materialised matrix (brute force)
 *   fbo_linear_direct  THE oracle: Eq. 10 summed over bases, groups and columns
 *                      directly, never forming What, a table or the VCM gather
 *   fbo_lut_tables     Eq. 14: every table entry by its defining signed sum
 *   fbo_lut_linear     Eq. 13 (gather) + Eq. 14 (tables) + Eq. 15 (read, row scale)
 *
 * All fp16 inputs are converted exactly to double; all sums are fp64.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* IEEE binary16 bit pattern -> double, exact (subnormals, zeros, inf, nan). */
double fbo_half_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int m = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24);            /* subnormal: m * 2^-10 * 2^-14 */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp((double)(m | 0x400), e - 25); /* (1 + m/1024) * 2^(e-15) */
    return sign ? -v : v;
}

static inline double sgn(const uint32_t *words, int64_t bit)
{
    return ((words[bit >> 5] >> (bit & 31)) & 1u) ? 1.0 : -1.0;
}

int fbo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* What[M][N] in fp64.  Eq. 3 summed over k (global) + Eq. 9's masked salient refinement. */
void fbo_dense_weight(int M, int N, int Kb, int Ks, int g, int n_sal,
                      const uint32_t *bits, const uint16_t *row_scale, const uint16_t *col_scale,
                      const int32_t *sal_idx, const uint32_t *sal_bits,
                      const uint16_t *sal_row_scale, const uint16_t *sal_col_scale,
                      double *W)
{
    int ng = N / g, nw = N / 32, nws = (n_sal + 31) / 32;
    for (int64_t e = 0; e < (int64_t)M * N; ++e) W[e] = 0.0;
    for (int k = 0; k < Kb; ++k)
        for (int i = 0; i < M; ++i)
            for (int j = 0; j < N; ++j) {
                double ar = fbo_half_to_double(row_scale[((int64_t)k * M + i) * ng + j / g]);
                double ac = fbo_half_to_double(col_scale[(int64_t)k * N + j]);
                W[(int64_t)i * N + j] += (ar * ac) * sgn(bits + ((int64_t)k * M + i) * nw, j);
            }
    for (int k = 0; k < Ks; ++k)
        for (int i = 0; i < M; ++i)
            for (int v = 0; v < n_sal; ++v) {
                int j = sal_idx[v];
                double ar = fbo_half_to_double(sal_row_scale[((int64_t)k * M + i) * ng + j / g]);
                double ac = fbo_half_to_double(sal_col_scale[(int64_t)k * n_sal + v]);
                W[(int64_t)i * N + j] += (ar * ac) * sgn(sal_bits + ((int64_t)k * M + i) * nws, v);
            }
}

/* y[B][M] = X[B][N] * W^T, W given dense in fp64. */
void fbo_dense_linear(int M, int N, int B, const double *W, const uint16_t *x, int64_t ldx, double *y)
{
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < M; ++i) {
            double s = 0.0;
            for (int j = 0; j < N; ++j)
                s += fbo_half_to_double(x[(int64_t)b * ldx + j]) * W[(int64_t)i * N + j];
            y[(int64_t)b * M + i] = s;
        }
}

/*
 * THE oracle.  Eq. 10 written out: for every batch row b and output row i
 *
 *   y[b,i] = sum_k sum_G ar[k][i][G] * ( sum_{j in group G} x[b,j] * ac[k][j] * B[k][i][j] )
 *          + sum_k sum_v asr[k][i][idx[v]/g] * x[b,idx[v]] * ascd[k][v] * Bsd[k][i][v]
 *
 * Three nested loops, no blocking; OpenMP over output rows only.
 */
void fbo_linear_direct(int M, int N, int Kb, int Ks, int g, int n_sal,
                       const uint32_t *bits, const uint16_t *row_scale, const uint16_t *col_scale,
                       const int32_t *sal_idx, const uint32_t *sal_bits,
                       const uint16_t *sal_row_scale, const uint16_t *sal_col_scale,
                       const uint16_t *x, int B, int64_t ldx, double *y)
{
    int ng = N / g, nw = N / 32, nws = (n_sal + 31) / 32;
    for (int b = 0; b < B; ++b) {
        const uint16_t *xb = x + (int64_t)b * ldx;
#pragma omp parallel for schedule(static)
        for (int i = 0; i < M; ++i) {
            double acc = 0.0;
            for (int k = 0; k < Kb; ++k) {
                const uint32_t *brow = bits + ((int64_t)k * M + i) * nw;
                for (int G = 0; G < ng; ++G) {
                    double s = 0.0;
                    for (int j = G * g; j < (G + 1) * g; ++j)
                        s += fbo_half_to_double(xb[j]) * fbo_half_to_double(col_scale[(int64_t)k * N + j])
                             * sgn(brow, j);
                    acc += fbo_half_to_double(row_scale[((int64_t)k * M + i) * ng + G]) * s;
                }
            }
            for (int k = 0; k < Ks; ++k) {
                const uint32_t *brow = sal_bits + ((int64_t)k * M + i) * nws;
                for (int v = 0; v < n_sal; ++v) {
                    int j = sal_idx[v];
                    acc += fbo_half_to_double(sal_row_scale[((int64_t)k * M + i) * ng + j / g])
                           * (fbo_half_to_double(xb[j]) * fbo_half_to_double(sal_col_scale[(int64_t)k * n_sal + v])
                              * sgn(brow, v));
                }
            }
            y[(int64_t)b * M + i] = acc;
        }
    }
}

/*
 * Eq. 14.  a[ncols] are the fused activations x*alpha_c of one base (ncols % mu == 0).
 * tables[t][p] = sum_{n<mu} a[mu*t+n] * (2*bit_n(p) - 1), bit n of p <-> column mu*t+n.
 */
void fbo_lut_tables(int ncols, int mu, const double *a, double *tables)
{
    int nt = ncols / mu, np = 1 << mu;
    for (int t = 0; t < nt; ++t)
        for (int p = 0; p < np; ++p) {
            double s = 0.0;
            for (int n = 0; n < mu; ++n)
                s += a[mu * t + n] * (((p >> n) & 1) ? 1.0 : -1.0);
            tables[(int64_t)t * np + p] = s;
        }
}

/* mu bits starting at bit position `bit` of a row of packed words (zero beyond nbits). */
static inline unsigned pattern(const uint32_t *words, int64_t bit, int mu, int64_t nbits)
{
    unsigned p = 0;
    for (int n = 0; n < mu; ++n)
        if (bit + n < nbits && ((words[(bit + n) >> 5] >> ((bit + n) & 31)) & 1u)) p |= 1u << n;
    return p;
}

/*
 * The LUT way, in fp64 (Eq. 11, 13, 14, 15).  Global branch: per base, fuse the column scale
 * into x, build all tables, read them with each row's mu-bit patterns, and apply the row scale
 * once per (row, group) -- mu must divide g.  Salient branch: gather x and keep the virtual
 * columns of each row-scale group together, padding each group's run to a multiple of mu with
 * zero activations, so that a sub-vector never straddles two row scales.
 */
void fbo_lut_linear(int M, int N, int Kb, int Ks, int g, int n_sal, int mu,
                    const uint32_t *bits, const uint16_t *row_scale, const uint16_t *col_scale,
                    const int32_t *sal_idx, const uint32_t *sal_bits,
                    const uint16_t *sal_row_scale, const uint16_t *sal_col_scale,
                    const uint16_t *x, int B, int64_t ldx, double *y)
{
    int ng = N / g, nw = N / 32, nws = (n_sal + 31) / 32, np = 1 << mu;
    double *a = (double *)malloc(sizeof(double) * (size_t)(N > mu ? N : mu));
    double *tab = (double *)malloc(sizeof(double) * (size_t)(N / mu + 1) * np);
    for (int b = 0; b < B; ++b) {
        const uint16_t *xb = x + (int64_t)b * ldx;
        for (int i = 0; i < M; ++i) y[(int64_t)b * M + i] = 0.0;
        for (int k = 0; k < Kb; ++k) {
            for (int j = 0; j < N; ++j)   /* Eq. 11: column scale folds into the input */
                a[j] = fbo_half_to_double(xb[j]) * fbo_half_to_double(col_scale[(int64_t)k * N + j]);
            fbo_lut_tables(N, mu, a, tab);
            for (int i = 0; i < M; ++i) {
                const uint32_t *brow = bits + ((int64_t)k * M + i) * nw;
                double acc = 0.0;
                for (int G = 0; G < ng; ++G) {
                    double s = 0.0;
                    for (int t = G * g / mu; t < (G + 1) * g / mu; ++t)
                        s += tab[(int64_t)t * np + pattern(brow, (int64_t)t * mu, mu, N)];
                    acc += fbo_half_to_double(row_scale[((int64_t)k * M + i) * ng + G]) * s;
                }
                y[(int64_t)b * M + i] += acc;
            }
        }
        for (int k = 0; k < Ks; ++k) {
            int v0 = 0;
            while (v0 < n_sal) {           /* one run of virtual columns sharing a row-scale group */
                int G = sal_idx[v0] / g, v1 = v0;
                while (v1 < n_sal && sal_idx[v1] / g == G) ++v1;
                for (int c = v0; c < v1; c += mu) {
                    int w = (v1 - c < mu) ? v1 - c : mu;
                    for (int n = 0; n < mu; ++n)   /* Eq. 13 gather; zero padding past the run */
                        a[n] = (n < w) ? fbo_half_to_double(xb[sal_idx[c + n]])
                                         * fbo_half_to_double(sal_col_scale[(int64_t)k * n_sal + c + n]) : 0.0;
                    fbo_lut_tables(mu, mu, a, tab);
                    for (int i = 0; i < M; ++i) {
                        const uint32_t *brow = sal_bits + ((int64_t)k * M + i) * nws;
                        unsigned p = pattern(brow, c, w, n_sal);
                        y[(int64_t)b * M + i] += fbo_half_to_double(sal_row_scale[((int64_t)k * M + i) * ng + G])
                                                 * tab[p];
                    }
                }
                v0 = v1;
            }
        }
    }
    free(a);
    free(tab);
}

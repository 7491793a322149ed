/*
 * HIGGS oracle: a plain, slow, fp64 CPU statement of what the paper defines.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  It shares no
 * code, header, table or helper with the CUDA library and is never used as a
 * fallback.
 *
 * Everything is scalar double precision, loops in the order the paper states
 * the steps.  The only parallelism is an optional OpenMP "for" over rows
 * (rows of W are independent in Algorithm 1 and in Appendix F).
 *
 * Notation: N = output features (rows of W), K = input features, g = group
 * size (power of two), p = grid dimension, n = grid size, xi = RHT seed.
 * Codes are 0-based (Algorithm 1 prints them 1-based).
 *
 * Pins (see tests/test_oracle_*.py): Hadamard orthogonality / involution /
 * explicit (-1)^popcount(i&j) matrix; hand-worked g=4 example; brute-force
 * enumeration on tiny inputs; closed-form 1-D Lloyd-Max Gaussian MSEs;
 * Appendix E identity (relative error of the layer == grid MSE); dense path
 * == rotated path (Appendix F).  Exact positions of the points of a fitted
 * 2-D grid are "parity unpinned" by design: only stationarity, monotone MSE
 * and the MSE level are pinned.
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* Threads actually available to the OpenMP loops (1 without OpenMP).         */
int higgs_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void higgs_oracle_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* ------------------------------------------------------------------------- */
/* Sign of the RHT for input index j (Algorithm 1, "RHT seed xi").            */
/* The paper fixes no generator.  Reading used here: one independent          */
/* Rademacher sign per input index j, the same for every row and token, taken */
/* from the splitmix64 stream seeded with xi: output number m of that stream  */
/* is mix(xi + (m+1)*0x9E3779B97F4A7C15) with the splitmix64 finaliser, and    */
/* sign j is bit (j mod 64) of output number floor(j/64) (bit set -> -1).      */
static uint64_t splitmix64_output(uint64_t xi, uint64_t m) {
    uint64_t z = xi + (m + 1u) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

double higgs_oracle_sign(uint64_t xi, int64_t j) {
    uint64_t z = splitmix64_output(xi, (uint64_t)j >> 6);
    return ((z >> ((uint64_t)j & 63u)) & 1u) ? -1.0 : 1.0;
}

/* ------------------------------------------------------------------------- */
/* Randomised Hadamard transform of one group, in place (Algorithm 1 line     */
/* "RandomHadamardTransform", Appendix F):  v <- H * diag(signs) * v, with H   */
/* the Sylvester matrix H[i][j] = (-1)^popcount(i&j) (entries +-1).           */
/* normalised != 0 divides by sqrt(g), which makes the map a rotation.        */
void higgs_oracle_rht(double* v, int64_t g, const double* signs, int normalised) {
    for (int64_t j = 0; j < g; ++j) v[j] *= signs[j];
    for (int64_t h = 1; h < g; h *= 2) {
        for (int64_t base = 0; base < g; base += 2 * h) {
            for (int64_t j = base; j < base + h; ++j) {
                double a = v[j], b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
        }
    }
    if (normalised) {
        double r = 1.0 / sqrt((double)g);
        for (int64_t j = 0; j < g; ++j) v[j] *= r;
    }
}

/* ------------------------------------------------------------------------- */
/* Nearest grid point of one p-tuple by exhaustive search ("RoundToNearest",  */
/* Algorithm 1).  Ties go to the lowest index.  Also returns the runner-up    */
/* and the margin = distance from the point to the bisector hyperplane of     */
/* winner and runner-up: (d2^2 - d1^2) / (2 |G[c1]-G[c2]|).                    */
static void nearest_point(const double* t, int p, int n, const double* grid,
                          int* best, int* second, double* margin) {
    int c1 = -1, c2 = -1;
    double d1 = INFINITY, d2 = INFINITY;
    for (int c = 0; c < n; ++c) {
        double d = 0.0;
        for (int k = 0; k < p; ++k) {
            double e = t[k] - grid[(int64_t)c * p + k];
            d += e * e;
        }
        if (d < d1) {
            d2 = d1; c2 = c1;
            d1 = d;  c1 = c;
        } else if (d < d2) {
            d2 = d;  c2 = c;
        }
    }
    *best = c1;
    if (second) *second = c2;
    if (margin) {
        if (c2 < 0) {
            *margin = INFINITY;
        } else {
            double sep = 0.0;
            for (int k = 0; k < p; ++k) {
                double e = grid[(int64_t)c1 * p + k] - grid[(int64_t)c2 * p + k];
                sep += e * e;
            }
            sep = sqrt(sep);
            *margin = sep > 0.0 ? (d2 - d1) / (2.0 * sep) : 0.0;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Grid fit (Algorithm 2, "CLVQ(n,p), computed once").  The paper only names  */
/* the procedure; the reading used is the batch (Lloyd) fixed-point iteration  */
/* on a finite sample of N(0,I_p):                                            */
/*   centres <- first n samples;                                              */
/*   repeat: assign every sample to its nearest centre (ties -> lowest index); */
/*           every centre <- mean of its samples (empty cell keeps its centre) */
/*   until no assignment changes or max_iters is reached;                     */
/*   finally sort the centres lexicographically.                              */
/* mse_hist[it] (optional, length max_iters) receives the per-dimension MSE   */
/* of the assignment made in iteration it, measured against the centres that  */
/* assignment used.  Returns 0, or -1 on bad arguments.                       */
static int lex_cmp_p = 1;
static int lex_cmp(const void* a, const void* b) {
    const double* x = (const double*)a;
    const double* y = (const double*)b;
    for (int k = 0; k < lex_cmp_p; ++k) {
        if (x[k] < y[k]) return -1;
        if (x[k] > y[k]) return 1;
    }
    return 0;
}

int higgs_oracle_lloyd(int p, int n, const double* samples, int64_t m, int max_iters,
                       double* grid, double* mse_hist, int* iters_done, int* converged) {
    if (p < 1 || n < 1 || m < n || max_iters < 1) return -1;
    int32_t* assign = (int32_t*)malloc((size_t)m * sizeof(int32_t));
    double* sum = (double*)malloc((size_t)n * p * sizeof(double));
    int64_t* cnt = (int64_t*)malloc((size_t)n * sizeof(int64_t));
    if (!assign || !sum || !cnt) { free(assign); free(sum); free(cnt); return -1; }
    for (int64_t i = 0; i < m; ++i) assign[i] = -1;
    memcpy(grid, samples, (size_t)n * p * sizeof(double));
    int it = 0, done = 0;
    while (it < max_iters && !done) {
        int64_t changed = 0;
        double err = 0.0;
#pragma omp parallel for reduction(+ : changed, err) schedule(static)
        for (int64_t i = 0; i < m; ++i) {
            int c;
            nearest_point(samples + i * p, p, n, grid, &c, NULL, NULL);
            if (c != assign[i]) { ++changed; assign[i] = c; }
            for (int k = 0; k < p; ++k) {
                double e = samples[i * p + k] - grid[(int64_t)c * p + k];
                err += e * e;
            }
        }
        if (mse_hist) mse_hist[it] = err / ((double)m * p);
        ++it;
        if (changed == 0) { done = 1; break; }
        memset(sum, 0, (size_t)n * p * sizeof(double));
        memset(cnt, 0, (size_t)n * sizeof(int64_t));
        for (int64_t i = 0; i < m; ++i) {
            int c = assign[i];
            ++cnt[c];
            for (int k = 0; k < p; ++k) sum[(int64_t)c * p + k] += samples[i * p + k];
        }
        for (int c = 0; c < n; ++c)
            if (cnt[c] > 0)
                for (int k = 0; k < p; ++k) grid[(int64_t)c * p + k] = sum[(int64_t)c * p + k] / (double)cnt[c];
    }
    lex_cmp_p = p;
    qsort(grid, (size_t)n, (size_t)p * sizeof(double), lex_cmp);
    if (iters_done) *iters_done = it;
    if (converged) *converged = done;
    free(assign); free(sum); free(cnt);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Standard normal density and distribution.                                  */
static double phi(double x) { return exp(-0.5 * x * x) / sqrt(2.0 * M_PI); }
static double Phi(double x) { return 0.5 * erfc(-x / sqrt(2.0)); }

/* Per-dimension MSE of rounding N(0,1) to sorted 1-D levels, in closed form: */
/* cells are [a_i, a_{i+1}) with a_i the midpoints; for a cell with mass P,   */
/* first moment M1 = phi(a_i)-phi(a_{i+1}), second moment                     */
/* M2 = P + a_i phi(a_i) - a_{i+1} phi(a_{i+1}):  E(x-c)^2 = M2 - 2cM1 + c^2P. */
double higgs_oracle_gauss_mse_1d(const double* levels, int n) {
    double mse = 0.0;
    for (int i = 0; i < n; ++i) {
        int lo_inf = (i == 0), hi_inf = (i == n - 1);
        double a = lo_inf ? 0.0 : 0.5 * (levels[i - 1] + levels[i]);
        double b = hi_inf ? 0.0 : 0.5 * (levels[i] + levels[i + 1]);
        double Pa = lo_inf ? 0.0 : Phi(a), Pb = hi_inf ? 1.0 : Phi(b);
        double fa = lo_inf ? 0.0 : phi(a), fb = hi_inf ? 0.0 : phi(b);
        double afa = lo_inf ? 0.0 : a * fa, bfb = hi_inf ? 0.0 : b * fb;
        double P = Pb - Pa, M1 = fa - fb, M2 = P + afa - bfb;
        double c = levels[i];
        mse += M2 - 2.0 * c * M1 + c * c * P;
    }
    return mse;
}

/* Continuous Lloyd-Max iteration for N(0,1) (the textbook fixed point the    */
/* 1-D Gaussian-MSE-optimal grid satisfies): thresholds = midpoints, levels = */
/* conditional means (phi(a)-phi(b))/(Phi(b)-Phi(a)).  levels[n] out, sorted.  */
double higgs_oracle_lloyd_max_1d(int n, int iters, double* levels) {
    if (n < 1 || n > 4096) return NAN;
    double next[4096];
    for (int i = 0; i < n; ++i) levels[i] = -2.0 + 4.0 * (i + 0.5) / n;
    for (int it = 0; it < iters; ++it) {
        double prev_thr = 0.0;
        for (int i = 0; i < n; ++i) {
            int lo_inf = (i == 0), hi_inf = (i == n - 1);
            double a = lo_inf ? 0.0 : prev_thr;
            double b = hi_inf ? 0.0 : 0.5 * (levels[i] + levels[i + 1]);
            double Pa = lo_inf ? 0.0 : Phi(a), Pb = hi_inf ? 1.0 : Phi(b);
            double fa = lo_inf ? 0.0 : phi(a), fb = hi_inf ? 0.0 : phi(b);
            next[i] = (fa - fb) / (Pb - Pa);
            prev_thr = b;
        }
        for (int i = 0; i < n; ++i) levels[i] = next[i];
    }
    return higgs_oracle_gauss_mse_1d(levels, n);
}

/* Per-dimension MSE of rounding the given points (m x p) to the grid.        */
double higgs_oracle_grid_mse(int p, int n, const double* grid, const double* pts, int64_t m) {
    double err = 0.0;
#pragma omp parallel for reduction(+ : err) schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        int c;
        nearest_point(pts + i * p, p, n, grid, &c, NULL, NULL);
        for (int k = 0; k < p; ++k) {
            double e = pts[i * p + k] - grid[(int64_t)c * p + k];
            err += e * e;
        }
    }
    return err / ((double)m * p);
}

/* ------------------------------------------------------------------------- */
/* Encoder, Algorithm 1 (RHT-VQ), for a matrix W[N][K] whose rows are each     */
/* partitioned sequentially into K/g groups (Appendix F: groups span one       */
/* output row and g consecutive inputs).  Per (row, group):                   */
/*   s  = ||w||_2                                                             */
/*   w+ = H diag(sign(xi, .)) (w / s)        (H unnormalised: entries ~N(0,1)) */
/*   code_t = argmin_c || w+[tp:(t+1)p] - G[c] ||^2,  t = 0..ceil(g/p)-1       */
/*   stored scale = s / sqrt(g)                                               */
/* When p does not divide g (the paper's p = 3 grids with g = 1024; it does    */
/* not say how) the last tuple is completed with zeros and matched on all p   */
/* coordinates; reconstruction drops the completed coordinates.               */
/* A group of all zeros gets scale 0 and the code of the point nearest the    */
/* origin (the paper divides by zero there; this reading keeps it finite).    */
/* Outputs: codes/runner/margin [N][K/g][ceil(g/p)] (= [N][K/p] when p        */
/* divides g; int32 / double), scales[N][K/g]                                 */
/* (double, NOT yet rounded to the 16-bit storage type; the caller rounds).   */
int higgs_oracle_quantize(const double* W, int64_t N, int64_t K, int g, int p, int n,
                          const double* grid, uint64_t xi,
                          int32_t* codes, int32_t* runner, double* margin, double* scales) {
    if (g < 1 || (g & (g - 1)) || K % g || p < 1 || p > 16) return -1;
    int64_t groups = K / g, tup = (g + p - 1) / p;
    double* signs = (double*)malloc((size_t)K * sizeof(double));
    if (!signs) return -1;
    for (int64_t j = 0; j < K; ++j) signs[j] = higgs_oracle_sign(xi, j);
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < N; ++r) {
        double* v = (double*)calloc((size_t)g + 16, sizeof(double));   /* zeros behind the group complete a short tuple */
        if (!v) { fail = 1; continue; }
        for (int64_t i = 0; i < groups; ++i) {
            const double* w = W + r * K + i * g;
            double ss = 0.0;
            for (int j = 0; j < g; ++j) ss += w[j] * w[j];
            double s = sqrt(ss);
            for (int j = 0; j < g; ++j) v[j] = (s > 0.0) ? w[j] / s : 0.0;
            higgs_oracle_rht(v, g, signs + i * g, 0);
            for (int64_t t = 0; t < tup; ++t) {
                int c1, c2;
                double mg;
                nearest_point(v + t * p, p, n, grid, &c1, &c2, &mg);
                int64_t o = (r * groups + i) * tup + t;
                codes[o] = c1;
                if (runner) runner[o] = c2;
                if (margin) margin[o] = mg;
            }
            scales[r * groups + i] = s / sqrt((double)g);
        }
        free(v);
    }
    free(signs);
    return fail ? -1 : 0;
}

/* ------------------------------------------------------------------------- */
/* Dequantisation to the original space (Appendix F, "Dequantization"):       */
/* r = scale * G[codes] approximates Hn diag(sign) w with Hn = H/sqrt(g)      */
/* orthonormal and symmetric, so  w^ = diag(sign) Hn r.                       */
/* scales[N][K/g] are the stored (already rounded) scales, widened to double.  */
int higgs_oracle_dequantize(const int32_t* codes, const double* scales, int64_t N, int64_t K,
                            int g, int p, int n, const double* grid, uint64_t xi, double* What) {
    if (g < 1 || (g & (g - 1)) || K % g || p < 1 || p > 16) return -1;
    (void)n;
    int64_t groups = K / g, tup = (g + p - 1) / p;
    double* ones = (double*)malloc((size_t)g * sizeof(double));
    if (!ones) return -1;
    for (int j = 0; j < g; ++j) ones[j] = 1.0;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        for (int64_t i = 0; i < groups; ++i) {
            double* v = What + r * K + i * g;
            double sc = scales[r * groups + i];
            for (int64_t t = 0; t < tup; ++t) {
                int c = codes[(r * groups + i) * tup + t];
                for (int k = 0; k < p && t * p + k < g; ++k) v[t * p + k] = sc * grid[(int64_t)c * p + k];
            }
            higgs_oracle_rht(v, g, ones, 1);                 /* Hn r            */
            for (int j = 0; j < g; ++j) v[j] *= higgs_oracle_sign(xi, i * g + j); /* diag(sign) */
        }
    }
    free(ones);
    return 0;
}

/* y[B][N] = x[B][K] * What[N][K]^T : the plain definition of the layer.      */
void higgs_oracle_matmul_nt(const double* x, const double* What, int64_t B, int64_t N, int64_t K, double* y) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        for (int64_t b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int64_t j = 0; j < K; ++j) acc += x[b * K + j] * What[r * K + j];
            y[b * N + r] = acc;
        }
    }
}

/* The product computed entirely in the rotated space (Appendix F, "Rotating  */
/* Activations"): x+ = Hn diag(sign) x per group (same xi, same groups), then  */
/* y[b][r] = sum_i scale[r][i] * sum_t < G[code[r][i][t]], x+[b][i][tp:(t+1)p] > */
int higgs_oracle_linear_rotated(const double* x, int64_t B, const int32_t* codes, const double* scales,
                                int64_t N, int64_t K, int g, int p, int n, const double* grid,
                                uint64_t xi, double* y) {
    if (g < 1 || (g & (g - 1)) || K % g || g % p) return -1;
    (void)n;
    int64_t groups = K / g, tup = g / p;
    double* xr = (double*)malloc((size_t)B * K * sizeof(double));
    double* signs = (double*)malloc((size_t)K * sizeof(double));
    if (!xr || !signs) { free(xr); free(signs); return -1; }
    for (int64_t j = 0; j < K; ++j) signs[j] = higgs_oracle_sign(xi, j);
    memcpy(xr, x, (size_t)B * K * sizeof(double));
    for (int64_t b = 0; b < B; ++b)
        for (int64_t i = 0; i < groups; ++i) higgs_oracle_rht(xr + b * K + i * g, g, signs + i * g, 1);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        for (int64_t b = 0; b < B; ++b) {
            double acc = 0.0;
            for (int64_t i = 0; i < groups; ++i) {
                double part = 0.0;
                for (int64_t t = 0; t < tup; ++t) {
                    int c = codes[r * (K / p) + i * tup + t];
                    for (int k = 0; k < p; ++k)
                        part += grid[(int64_t)c * p + k] * xr[b * K + i * g + t * p + k];
                }
                acc += scales[r * groups + i] * part;
            }
            y[b * N + r] = acc;
        }
    }
    free(xr); free(signs);
    return 0;
}

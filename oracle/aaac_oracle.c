/*
 * AAAC CPU oracle  --  TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, double-precision restatement of the per-layer AAAC procedure
 * (Algorithm 1 of the paper) used only to check the CUDA library: the test
 * suite, the smoke check and the benchmark's CPU-baseline leg call it; the
 * product path never does.  It shares no code with the CUDA sources.
 *
 * Every function follows the paper's steps in the paper's order:
 *   oracle_act_stats      Eq. 7            I_k = sum_t X[t,k]^2
 *   oracle_scales         Alg. 1 line 1    per-group positive scale
 *   oracle_normalise      Eq. 2, line 2    w~ = w / s
 *   oracle_init_quantile  Eq. 9, Eq. 10    quantile initialisation of T0, T1
 *   oracle_init_grid      Sec. 3.1         the format's fixed table (INT4 grid / E2M1)
 *   oracle_fit_round      Alg. 1 lines 6-16 with n_inner = 1: assignment (Eq. 8),
 *                         weighted centroids (Eq. 11), keep-if-empty, sort
 *   oracle_assign         Alg. 1 lines 7-11  assignment step alone: sigma per group, objective
 *   oracle_inner_update   Alg. 1 lines 15-20 one inner k-means iteration with sigma frozen (no sort)
 *   oracle_sort_tables    Alg. 1 line 22     ascending sort of each table
 *   oracle_objective      Eq. 8 summed over all groups (no update)
 *   oracle_round_tables   Alg. 1 line 17   round tables to BF16
 *   oracle_pack           Alg. 1 lines 18-19, Eq. 6
 *   oracle_apply_sigma    Alg. 1 line 20   selection bit -> sign bit of the scale
 *   oracle_dequant        Eq. 5
 *   oracle_prescale       Sec. 4 "Combining AAAC with AWQ": per-input-channel scaling of W (and the
 *                         matching importance) before the fit
 *   oracle_pack_sigma_bits, oracle_dequant_sel, oracle_output_error_sel
 *                         the same with a selection group S smaller than the scale group g
 *                         (Sec. 3.1 "granularity"): sigma stored apart, 1/S bit per weight.
 *                         The fit and pack steps take the selection group size as their group
 *                         argument: they see normalised weights only, so g does not enter them.
 *   oracle_output_error   Sec. 3.2 "Activation importance": sum_k I_k (w - w^)^2
 *
 * Arithmetic.  Everything is double except the quantities that are *defined* as
 * single-precision numbers (they are stored formats or the definition of w~):
 *   - the scale s is a stored BF16 (INT4 mode) or E4M3 x FP32 tensor scale (NVFP4);
 *   - r = fl32(1/s) and w~ = fl32(w * r): one correctly rounded multiply;
 *   - I_k is the double sum rounded once to FP32.
 * No blocking, fusion or reordering: loops run in index order.  Rows are
 * independent, so per-row partial sums are formed (optionally by OpenMP threads)
 * and then added in row order; the result does not depend on the thread count.
 *
 * Readings of points the paper leaves open (each marked "parity unpinned by the
 * paper" where no printed number fixes it):
 *   - scale rule: INT4 s = bf16(absmax / 7), NVFP4 s = E4M3(absmax / (6 s_t)) * s_t,
 *     s_t = layer absmax / (448 * 6)                       [parity unpinned]
 *   - quantile = linear interpolation at q (n - 1)         [parity unpinned]
 *   - nibble order: element 2i -> low nibble of byte i     [parity unpinned]
 *   - separate selection bits (S < g): row-major, selection group j of a row in bit j mod 8 of
 *     byte j / 8 of the row's K / (8 S) bytes                [parity unpinned]
 *   - grid start ("init to the format's grid"): T0 = the format's table, T1 = T0 moved up
 *     half a step, the last step repeating half the last spacing   [parity unpinned by the paper:
 *     it starts from quantiles (Eq. 9-10) only; the half-step shift is Eq. 10's offset moved
 *     onto a grid]
 *   - argmin ties: of two equidistant entries the smaller one, of equal entries the lowest
 *     index (on an ascending table: the lowest index); sigma tie: table 0
 *   - an inner iteration (Alg. 1 lines 15-20) updates all entries of a table at once, from
 *     the cells of the table as it stood before the iteration (ordinary Lloyd / k-means)
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define M 16
enum { MODE_INT4 = 0, MODE_NVFP4 = 1 };
enum { OK = 0, ERR_ARG = 3, ERR_NONFINITE = 7 };

/* ---------------------------------------------------------------- formats */

static float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even FP32 -> BF16 (finite input) */
static uint16_t f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* E4M3 (the "FN" FP8 used for NVFP4 block scales): 1-4-3, bias 7, no infinity,
 * 0x7F = NaN, largest finite 0x7E = 448, subnormals m * 2^-9. */
static float e4m3_to_f32(uint8_t c) {
    int e = (c >> 3) & 15, m = c & 7;
    float v = (e == 0) ? ldexpf((float)m, -9) : ldexpf((float)(8 + m), e - 10);
    return (c & 0x80) ? -v : v;
}

/* nearest finite non-negative E4M3 code to x >= 0; ties to the even code; saturates at 448 */
static uint8_t e4m3_encode(float x) {
    int best = 0;
    double bd = fabs((double)x);
    for (int c = 1; c <= 0x7E; ++c) {
        double d = fabs((double)x - (double)e4m3_to_f32((uint8_t)c));
        if (d < bd || (d == bd && (c & 1) == 0)) { best = c; bd = d; }
    }
    return (uint8_t)best;
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

float oracle_e4m3_to_f32(uint8_t c) { return e4m3_to_f32(c); }
uint8_t oracle_e4m3_encode(float x) { return e4m3_encode(x); }

/* ------------------------------------------------------------ Eq. 7 */

/* I_k = sum_t X[t,k]^2, t ascending, double accumulation, one rounding to FP32. */
void oracle_act_stats(const uint16_t* X, int64_t T, int64_t K, int64_t ldx, float* I) {
    double* acc = (double*)calloc((size_t)K, sizeof(double));
    for (int64_t t = 0; t < T; ++t)
        for (int64_t k = 0; k < K; ++k) {
            double x = (double)bf16_to_f32(X[t * ldx + k]);
            acc[k] += x * x;
        }
    for (int64_t k = 0; k < K; ++k) I[k] = (float)acc[k];
    free(acc);
}

/* ------------------------------------------------------------ Alg. 1 line 1 */

/* effective positive scale of a stored scale (sign bit ignored) */
static float scale_value(const void* scales, int64_t j, int mode, float s_t) {
    if (mode == MODE_INT4) return bf16_to_f32(((const uint16_t*)scales)[j] & 0x7FFF);
    return e4m3_to_f32(((const uint8_t*)scales)[j] & 0x7F) * s_t;
}

/* Per-group scales.  INT4: bf16 [N][K/g].  NVFP4: E4M3 bytes [N][K/g] + tensor_scale[0]. */
int oracle_scales(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int g,
                  void* scales, float* tensor_scale) {
    if (K % g) return ERR_ARG;
    int64_t G = K / g;
    float A = 0.f;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            float w = bf16_to_f32(W[n * ldw + k]);
            if (!isfinite(w)) return ERR_NONFINITE;
            if (fabsf(w) > A) A = fabsf(w);
        }
    float s_t = 1.f, d6 = 6.f;
    if (mode == MODE_NVFP4) {
        s_t = (A == 0.f) ? 1.f : A / 2688.f;              /* 448 * 6 */
        if (s_t < 0x1p-96f) s_t = 0x1p-96f;
        d6 = 6.f * s_t;
        tensor_scale[0] = s_t;
    }
    for (int64_t n = 0; n < N; ++n)
        for (int64_t j = 0; j < G; ++j) {
            float a = 0.f;
            for (int k = 0; k < g; ++k) {
                float w = fabsf(bf16_to_f32(W[n * ldw + j * g + k]));
                if (w > a) a = w;
            }
            if (mode == MODE_INT4) {
                float s = 1.f;
                if (a != 0.f) {
                    s = bf16_to_f32(f32_to_bf16(a / 7.f));
                    if (s < FLT_MIN) s = FLT_MIN;          /* 2^-126 is a BF16 value */
                }
                ((uint16_t*)scales)[n * G + j] = f32_to_bf16(s);
            } else {
                float x = a / d6;
                uint8_t q = e4m3_encode(x);
                /* never store 0; keep |w~| <= 7.5 in the lowest subnormal step */
                if (q <= 1) q = (x > 1.25f * 0x1p-9f) ? 2 : 1;
                ((uint8_t*)scales)[n * G + j] = q;
            }
        }
    return OK;
}

/* ------------------------------------------------------------ Eq. 2 */

/* w~ = fl32(w * fl32(1/s)); wt is dense [N][K]. */
void oracle_normalise(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, int mode, int g,
                      const void* scales, const float* tensor_scale, float* wt) {
    int64_t G = K / g;
    float s_t = (mode == MODE_NVFP4) ? tensor_scale[0] : 1.f;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t j = 0; j < G; ++j) {
            float s = scale_value(scales, n * G + j, mode, s_t);
            float r = 1.0f / s;
            for (int k = 0; k < g; ++k) {
                float w = bf16_to_f32(W[n * ldw + j * g + k]);
                wt[n * K + j * g + k] = w * r;
            }
        }
}

/* ------------------------------------------------------------ Eq. 9, Eq. 10 */

static int cmp_float(const void* a, const void* b) {
    float x = *(const float*)a, y = *(const float*)b;
    return (x > y) - (x < y);
}

static double quantile_sorted(const float* x, int64_t n, double q) {
    double p = q * (double)(n - 1);
    int64_t lo = (int64_t)floor(p), hi = (int64_t)ceil(p);
    if (lo < 0) lo = 0;
    if (hi > n - 1) hi = n - 1;
    if (lo > hi) lo = hi;
    double f = p - (double)lo;
    double v = (double)x[lo] + f * ((double)x[hi] - (double)x[lo]);
    return (double)(float)v;                                /* tables start as FP32 numbers */
}

/* T0[i] = Quantile_{i/(M-1)}, T1[i] = Quantile_{d + (1-d) i/(M-1)}, d = 1/(2(M-1)),
 * over all n normalised weights. */
void oracle_init_quantile(const float* wt, int64_t n, double* T01) {
    float* s = (float*)malloc((size_t)n * sizeof(float));
    memcpy(s, wt, (size_t)n * sizeof(float));
    qsort(s, (size_t)n, sizeof(float), cmp_float);
    const double d = 1.0 / (2.0 * (M - 1));
    for (int i = 0; i < M; ++i) {
        T01[i] = quantile_sorted(s, n, (double)i / (double)(M - 1));
        T01[M + i] = quantile_sorted(s, n, d + (1.0 - d) * (double)i / (double)(M - 1));
    }
    free(s);
}

/* T0 = the format's table in normalised units (INT4: -8..7; NVFP4: signed E2M1 with
 * +0 and -0 both present), T1 = T0 moved up by half a step. */
void oracle_init_grid(int mode, double* T01) {
    static const double e2m1[M] = {-6, -4, -3, -2, -1.5, -1, -0.5, 0, 0, 0.5, 1, 1.5, 2, 3, 4, 6};
    for (int i = 0; i < M; ++i) T01[i] = (mode == MODE_INT4) ? (double)(i - 8) : e2m1[i];
    for (int i = 0; i < M - 1; ++i) T01[M + i] = 0.5 * (T01[i] + T01[i + 1]);
    T01[2 * M - 1] = T01[M - 1] + 0.5 * (T01[M - 1] - T01[M - 2]);
}

/* ------------------------------------------------------------ Eq. 4 */

/* index of the nearest entry; of two equidistant entries the smaller wins, of equal entries
 * the lowest index (tables are ascending except between the inner iterations of one table
 * update, where Alg. 1 sorts only after the last one; on an ascending table this is "the
 * lowest index wins") */
static int nearest(const double* T, double x) {
    int best = 0;
    double bd = fabs(x - T[0]);
    for (int i = 1; i < M; ++i) {
        double d = fabs(x - T[i]);
        if (d < bd || (d == bd && T[i] < T[best])) { bd = d; best = i; }
    }
    return best;
}

static void sort16(double* T) {
    for (int i = 1; i < M; ++i) {
        double v = T[i];
        int j = i - 1;
        while (j >= 0 && T[j] > v) { T[j + 1] = T[j]; --j; }
        T[j + 1] = v;
    }
}

/* Eq. 8 for one group: both weighted errors, the chosen table, the indices under it */
static int assign_group(const float* wt, const float* I, int g, const double* T01,
                        double* E0, double* E1, int* idx_sel) {
    int idx[2][128];
    double E[2] = {0.0, 0.0};
    for (int r = 0; r < 2; ++r)
        for (int k = 0; k < g; ++k) {
            double x = (double)wt[k];
            int i = nearest(T01 + r * M, x);
            double d = x - T01[r * M + i];
            E[r] += (double)I[k] * (d * d);
            idx[r][k] = i;
        }
    int sigma = (E[1] < E[0]) ? 1 : 0;
    for (int k = 0; k < g; ++k) idx_sel[k] = idx[sigma][k];
    *E0 = E[0];
    *E1 = E[1];
    return sigma;
}

/* One outer iteration with n_inner = 1 (Alg. 1 lines 6-16): assignment step, then each
 * entry becomes the activation-weighted centroid of its cell (kept if the cell has no
 * weight), then each table is sorted.  *E_out = the Eq. 8 objective of the assignment.
 * sigma_out (optional): [N*K/g]. */
int oracle_fit_round(const float* wt, const float* I, int64_t N, int64_t K, int g,
                     double* T01, double* E_out, uint8_t* sigma_out) {
    if (g > 128 || K % g) return ERR_ARG;
    int64_t G = K / g;
    const int P = 2 * M * 2 + 1;
    double* part = (double*)calloc((size_t)N * P, sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        double* p = part + n * P;                           /* [2][M] S, [2][M] Wt, E */
        int idx[128];
        for (int64_t j = 0; j < G; ++j) {
            const float* w = wt + n * K + j * g;
            const float* imp = I + j * g;
            double E0, E1;
            int sigma = assign_group(w, imp, g, T01, &E0, &E1, idx);
            for (int k = 0; k < g; ++k) {
                p[sigma * M + idx[k]] += (double)imp[k] * (double)w[k];
                p[2 * M + sigma * M + idx[k]] += (double)imp[k];
            }
            p[4 * M] += (E1 < E0) ? E1 : E0;
            if (sigma_out) sigma_out[n * G + j] = (uint8_t)sigma;
        }
    }
    double tot[2 * M * 2 + 1];
    for (int i = 0; i < P; ++i) tot[i] = 0.0;
    for (int64_t n = 0; n < N; ++n)
        for (int i = 0; i < P; ++i) tot[i] += part[n * P + i];
    free(part);
    for (int r = 0; r < 2; ++r) {
        for (int i = 0; i < M; ++i)
            if (tot[2 * M + r * M + i] > 0.0) T01[r * M + i] = tot[r * M + i] / tot[2 * M + r * M + i];
        sort16(T01 + r * M);
    }
    if (E_out) *E_out = tot[4 * M];
    return OK;
}

/* Assignment step alone (Alg. 1 lines 7-11): sigma[N*K/g] and the Eq. 8 objective. */
int oracle_assign(const float* wt, const float* I, int64_t N, int64_t K, int g,
                  const double* T01, uint8_t* sigma, double* E_out) {
    if (g > 128 || K % g) return ERR_ARG;
    int64_t G = K / g;
    double* rowE = (double*)calloc((size_t)N, sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        int idx[128];
        for (int64_t j = 0; j < G; ++j) {
            double E0, E1;
            sigma[n * G + j] = (uint8_t)assign_group(wt + n * K + j * g, I + j * g, g, T01, &E0, &E1, idx);
            rowE[n] += (E1 < E0) ? E1 : E0;
        }
    }
    double E = 0.0;
    for (int64_t n = 0; n < N; ++n) E += rowE[n];
    free(rowE);
    if (E_out) *E_out = E;
    return OK;
}

/* One inner iteration of the table update (Alg. 1 lines 15-20) with the selection frozen:
 * for r in {0, 1}, over the weights of the groups with sigma = r, every entry of T_r becomes the
 * activation-weighted centroid (Eq. 11) of its Voronoi cell under T_r as it stood on entry;
 * an entry whose denominator is zero keeps its value.  No sort (Alg. 1 sorts after the last
 * inner iteration only). */
int oracle_inner_update(const float* wt, const float* I, const uint8_t* sigma, int64_t N, int64_t K, int g,
                        double* T01) {
    if (g > 128 || K % g) return ERR_ARG;
    int64_t G = K / g;
    const int P = 2 * M * 2;
    double* part = (double*)calloc((size_t)N * P, sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        double* p = part + n * P;                           /* [2][M] S, [2][M] Wt */
        for (int64_t j = 0; j < G; ++j) {
            const int r = sigma[n * G + j] ? 1 : 0;
            for (int k = 0; k < g; ++k) {
                const double x = (double)wt[n * K + j * g + k], imp = (double)I[j * g + k];
                const int i = nearest(T01 + r * M, x);
                p[r * M + i] += imp * x;
                p[2 * M + r * M + i] += imp;
            }
        }
    }
    double tot[2 * M * 2];
    for (int i = 0; i < P; ++i) tot[i] = 0.0;
    for (int64_t n = 0; n < N; ++n)
        for (int i = 0; i < P; ++i) tot[i] += part[n * P + i];
    free(part);
    for (int i = 0; i < 2 * M; ++i)
        if (tot[2 * M + i] > 0.0) T01[i] = tot[i] / tot[2 * M + i];
    return OK;
}

/* Alg. 1 line 22 */
void oracle_sort_tables(double* T01) {
    sort16(T01);
    sort16(T01 + M);
}

/* sum over all groups of min_r (Eq. 8 error) for the given tables, no update */
double oracle_objective(const float* wt, const float* I, int64_t N, int64_t K, int g,
                        const double* T01) {
    int64_t G = K / g;
    double* rowE = (double*)calloc((size_t)N, sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        int idx[128];
        for (int64_t j = 0; j < G; ++j) {
            double E0, E1;
            assign_group(wt + n * K + j * g, I + j * g, g, T01, &E0, &E1, idx);
            rowE[n] += (E1 < E0) ? E1 : E0;
        }
    }
    double E = 0.0;
    for (int64_t n = 0; n < N; ++n) E += rowE[n];
    free(rowE);
    return E;
}

/* ------------------------------------------------------------ Alg. 1 line 17 */

/* Alg. 1 "Round T0, T1 to BF16".  The fitted tables are reported as FP32 numbers (the value
 * Tf) and the stored table is the BF16 rounding of that reported number, so the chain is
 * double -> FP32 -> BF16, both round-to-nearest-even.  It differs from a direct double -> BF16
 * rounding only when the FP32 rounding lands exactly on a BF16 half-way point, i.e. for a
 * double within 2^-25 relative of such a point (a 2^-17 fraction of all values); the pins
 * count how often that happens on the seeded layers.  Rounding is monotone; the sort is kept
 * for form. */
void oracle_round_tables(const double* T01, float* Tf, uint16_t* Tb) {
    double t[2 * M];
    for (int i = 0; i < 2 * M; ++i) {
        Tf[i] = (float)T01[i];
        Tb[i] = f32_to_bf16(Tf[i]);
        t[i] = (double)bf16_to_f32(Tb[i]);
    }
    for (int r = 0; r < 2; ++r) {
        sort16(t + r * M);
        for (int i = 0; i < M; ++i) Tb[r * M + i] = f32_to_bf16((float)t[r * M + i]);
    }
}

/* ------------------------------------------------------------ Alg. 1 lines 18-19 */

/* With the BF16 tables: sigma per group (Eq. 8), codes = nearest index under the chosen
 * table (Eq. 6), two codes per byte (even element in the low nibble).
 * ties[0] = groups with E0 == E1 exactly; ties[1] = weights exactly half-way between two
 * different entries of their chosen table. */
int oracle_pack(const float* wt, const float* I, int64_t N, int64_t K, int g,
                const uint16_t* Tb, uint8_t* codes, uint8_t* sigma_out, double* E_final,
                uint64_t* ties) {
    if (g > 128 || K % g || K % 2) return ERR_ARG;
    int64_t G = K / g;
    double T01[2 * M];
    for (int i = 0; i < 2 * M; ++i) T01[i] = (double)bf16_to_f32(Tb[i]);
    double* rowE = (double*)calloc((size_t)N, sizeof(double));
    uint64_t t0 = 0, t1 = 0;
#pragma omp parallel for schedule(static) reduction(+ : t0, t1)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t j = 0; j < G; ++j) {
            const float* w = wt + n * K + j * g;
            int idx[128];
            double E0, E1;
            int sigma = assign_group(w, I + j * g, g, T01, &E0, &E1, idx);
            if (E0 == E1) ++t0;
            rowE[n] += (E1 < E0) ? E1 : E0;
            sigma_out[n * G + j] = (uint8_t)sigma;
            for (int k = 0; k < g; ++k) {
                int64_t e = n * K + j * g + k;
                if (e & 1) codes[e >> 1] = (uint8_t)((codes[e >> 1] & 0x0F) | (idx[k] << 4));
                else codes[e >> 1] = (uint8_t)idx[k];
                double x = (double)w[k], d = fabs(x - T01[sigma * M + idx[k]]);
                for (int i = 0; i < M; ++i)
                    if (T01[sigma * M + i] != T01[sigma * M + idx[k]] && fabs(x - T01[sigma * M + i]) == d) { ++t1; break; }
            }
        }
    double E = 0.0;
    for (int64_t n = 0; n < N; ++n) E += rowE[n];
    free(rowE);
    if (E_final) *E_final = E;
    if (ties) { ties[0] = t0; ties[1] = t1; }
    return OK;
}

/* Alg. 1 line 20: the selection bit goes into the sign bit of the (positive) scale */
void oracle_apply_sigma(void* scales, const uint8_t* sigma, int64_t count, int mode) {
    for (int64_t j = 0; j < count; ++j) {
        if (mode == MODE_INT4) {
            uint16_t* s = (uint16_t*)scales;
            s[j] = (uint16_t)((s[j] & 0x7FFF) | (sigma[j] ? 0x8000 : 0));
        } else {
            uint8_t* s = (uint8_t*)scales;
            s[j] = (uint8_t)((s[j] & 0x7F) | (sigma[j] ? 0x80 : 0));
        }
    }
}

/* ------------------------------------------------------------ Eq. 5 */

/* w^ = T_sigma[c] * s with sigma = sign bit of the stored scale, s = its magnitude
 * (times the tensor scale for NVFP4); one FP32 multiply, then BF16 (nearest even). */
void oracle_dequant(const uint8_t* codes, const void* scales, const float* tensor_scale,
                    const uint16_t* Tb, int64_t N, int64_t K, int mode, int g, uint16_t* What,
                    int64_t ldo) {
    int64_t G = K / g;
    float s_t = (mode == MODE_NVFP4) ? tensor_scale[0] : 1.f;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            int64_t j = n * G + k / g, e = n * K + k;
            int sigma = (mode == MODE_INT4) ? (((const uint16_t*)scales)[j] >> 15)
                                            : (((const uint8_t*)scales)[j] >> 7);
            float s = scale_value(scales, j, mode, s_t);
            int c = (e & 1) ? (codes[e >> 1] >> 4) : (codes[e >> 1] & 0x0F);
            float v = bf16_to_f32(Tb[sigma * M + c]) * s;
            What[n * ldo + k] = f32_to_bf16(v);
        }
}

/* sum_k I_k (w - T_sigma[c] s)^2 over the layer, in weight units, all in double */
double oracle_output_error(const uint16_t* W, int64_t ldw, const uint8_t* codes, const void* scales,
                           const float* tensor_scale, const uint16_t* Tb, const float* I,
                           int64_t N, int64_t K, int mode, int g) {
    int64_t G = K / g;
    float s_t = (mode == MODE_NVFP4) ? tensor_scale[0] : 1.f;
    double E = 0.0;
    for (int64_t n = 0; n < N; ++n) {
        double rowE = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            int64_t j = n * G + k / g, e = n * K + k;
            int sigma = (mode == MODE_INT4) ? (((const uint16_t*)scales)[j] >> 15)
                                            : (((const uint8_t*)scales)[j] >> 7);
            double s = (double)scale_value(scales, j, mode, s_t);
            int c = (e & 1) ? (codes[e >> 1] >> 4) : (codes[e >> 1] & 0x0F);
            double d = (double)bf16_to_f32(W[n * ldw + k]) - (double)bf16_to_f32(Tb[sigma * M + c]) * s;
            rowE += (double)I[k] * (d * d);
        }
        E += rowE;
    }
    return E;
}

/* ------------------------------------------------------------ S < g: selection bits apart */

/* Alg. 1 line 20, S < g: the selection bits are stored separately, 1/S bit per weight.
 * sigma [N][GS] (one byte per selection group) -> bits [N][GS / 8], group j of a row in
 * bit j % 8 of the row's byte j / 8.  GS must be a multiple of 8. */
int oracle_pack_sigma_bits(const uint8_t* sigma, int64_t N, int64_t GS, uint8_t* bits) {
    if (GS % 8) return ERR_ARG;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t b = 0; b < GS / 8; ++b) {
            unsigned v = 0;
            for (int i = 0; i < 8; ++i) v |= (unsigned)(sigma[n * GS + b * 8 + i] ? 1 : 0) << i;
            bits[n * (GS / 8) + b] = (uint8_t)v;
        }
    return OK;
}

static int sigma_bit(const uint8_t* bits, int64_t n, int64_t GS, int64_t j) {
    return (bits[n * (GS / 8) + j / 8] >> (j % 8)) & 1;
}

/* Eq. 5 with sigma taken from the separate bits (selection group S) and the scale (sign bit
 * clear) from its own group of g weights. */
void oracle_dequant_sel(const uint8_t* codes, const void* scales, const float* tensor_scale,
                        const uint16_t* Tb, const uint8_t* sigma_bits, int S, int64_t N, int64_t K,
                        int mode, int g, uint16_t* What, int64_t ldo) {
    int64_t G = K / g, GS = K / S;
    float s_t = (mode == MODE_NVFP4) ? tensor_scale[0] : 1.f;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            int64_t e = n * K + k;
            int sigma = sigma_bit(sigma_bits, n, GS, k / S);
            float s = scale_value(scales, n * G + k / g, mode, s_t);
            int c = (e & 1) ? (codes[e >> 1] >> 4) : (codes[e >> 1] & 0x0F);
            What[n * ldo + k] = f32_to_bf16(bf16_to_f32(Tb[sigma * M + c]) * s);
        }
}

double oracle_output_error_sel(const uint16_t* W, int64_t ldw, const uint8_t* codes, const void* scales,
                               const float* tensor_scale, const uint16_t* Tb, const uint8_t* sigma_bits, int S,
                               const float* I, int64_t N, int64_t K, int mode, int g) {
    int64_t G = K / g, GS = K / S;
    float s_t = (mode == MODE_NVFP4) ? tensor_scale[0] : 1.f;
    double E = 0.0;
    for (int64_t n = 0; n < N; ++n) {
        double rowE = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            int64_t e = n * K + k;
            int sigma = sigma_bit(sigma_bits, n, GS, k / S);
            double s = (double)scale_value(scales, n * G + k / g, mode, s_t);
            int c = (e & 1) ? (codes[e >> 1] >> 4) : (codes[e >> 1] & 0x0F);
            double d = (double)bf16_to_f32(W[n * ldw + k]) - (double)bf16_to_f32(Tb[sigma * M + c]) * s;
            rowE += (double)I[k] * (d * d);
        }
        E += rowE;
    }
    return E;
}

/* ------------------------------------------------------------ channel scaling before the fit */

/* "AWQ first scales the weights, then AAAC learns codebooks on the scaled distribution": with a
 * positive multiplier a_k per input channel, W'[n][k] = bf16(w a_k) (one FP32 multiply, rounded to
 * the weights' storage type) and, because the layer's input is divided by a_k in exchange,
 * I'_k = sum_t (X[t][k] / a_k)^2 = I_k / a_k^2, formed in double and rounded once to FP32.
 * How the a_k are found (AWQ's search) is not part of the method.  I / I_out may be NULL. */
void oracle_prescale(const uint16_t* W, int64_t N, int64_t K, int64_t ldw, const float* a,
                     uint16_t* W_out, int64_t ldo, const float* I, float* I_out) {
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            W_out[n * ldo + k] = f32_to_bf16(bf16_to_f32(W[n * ldw + k]) * a[k]);
    if (I && I_out)
        for (int64_t k = 0; k < K; ++k) I_out[k] = (float)((double)I[k] / ((double)a[k] * (double)a[k]));
}

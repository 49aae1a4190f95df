/*
 * RMSMP CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, scalar restatement of the arithmetic of a row-wise mixed-scheme
 * (Power-of-Two 4-bit / Fixed-point 4-bit / Fixed-point 8-bit) quantized layer with
 * 4-bit fixed-point activations, written from the paper's Section 3 (Eq. 1-5,
 * Algorithm 1).  Only the test-suite, the smoke check and the CPU-baseline leg of the
 * benchmark may load this file.  It shares no code, table or header with the CUDA
 * library and never calls it.
 *
 * Arithmetic contract (the readings are listed where they are taken):
 *   - every fp32 step is ONE IEEE-754 binary32 operation, round-to-nearest-even;
 *     build with -ffp-contract=off and without fast-math;
 *   - integer accumulation is exact (int32, with an int64 checking variant).
 *
 * Build: gcc -O2 -std=c99 -ffp-contract=off -fopenmp -shared -fPIC rmsmp_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { O_SCHEME_POT = 0, O_SCHEME_FIXED = 1 };
enum { O_ACT_U4 = 0, O_ACT_S4 = 1 };
enum { O_POT_NEAREST = 0, O_POT_LOG2 = 1 };

/* Clip function of Eq. 3: w/alpha limited to [-1, +1].  One fp32 division. */
static float o_clip(float w, float alpha)
{
    float t = w / alpha;
    if (t < -1.0f) t = -1.0f;
    if (t > 1.0f) t = 1.0f;
    return t;
}

/*
 * Fixed-point quantizer.  Eq. 1 gives the level set  +-alpha * {0, 1/Q, 2/Q, ..., 1}
 * with Q = 2^(m-1) - 1; the quantizer is the projection of the clipped weight onto
 * that set (first line of Eq. 2).  Reading: Eq. 1's symmetric set is the authority
 * (the second line of Eq. 2, as printed, describes a 2^m-level grid without zero that
 * contradicts Eq. 1); "round" ties go to even.
 * Returns the signed integer level index q in [-Q, Q]; the weight is q * alpha / Q.
 */
int rmsmp_o_fixed_q(float w, float alpha, int bits)
{
    float Q = (float)((1 << (bits - 1)) - 1);
    float t = o_clip(w, alpha);
    float s = t * Q;               /* one fp32 multiply */
    return (int)rintf(s);          /* round half to even */
}

/*
 * Power-of-Two quantizer, m = 4.  Eq. 4 gives the level set
 *   +-alpha * {0, 2^-6, 2^-5, ..., 2^-1, 1}   (2^(m-1)-2 = 6).
 * The code is sign-magnitude: nibble = s<<3 | e, e = 0 is zero (sign forced to 0),
 * e = 1..7 is magnitude 2^(e-7).
 *
 * mode O_POT_NEAREST (default): projection of Eq. 5's first line -- the nearest level
 *   on the real line.  The decision points are the midpoints between neighbouring
 *   levels (2^-7 between 0 and 2^-6; 3*2^(e-9) between 2^(e-8) and 2^(e-7)), all exact
 *   in binary32.  Reading: a value exactly on a midpoint goes to the larger magnitude.
 * mode O_POT_LOG2: the printed rounding rule 2^round(log2 x) applied to x = |w/alpha|,
 *   with zero when round(log2 x) < -6.  round(log2 x) = -j  iff  2^-(j+1/2) <= x <
 *   2^-(j-1/2); the comparison is done exactly on x*x in double (x*x is exact there
 *   and 2^-(2j+1) is a power of two), so no logarithm is evaluated.
 */
int rmsmp_o_pot_nibble(float w, float alpha, int mode)
{
    float t = o_clip(w, alpha);
    int s = (t < 0.0f) ? 1 : 0;
    float x = fabsf(t);
    int e = 0;
    if (mode == O_POT_NEAREST) {
        if (x >= 0.0078125f) e = 1;                      /* 2^-7 : midpoint(0, 2^-6) */
        for (int k = 2; k <= 7; ++k) {
            float mid = ldexpf(3.0f, k - 9);              /* midpoint(2^(k-8), 2^(k-7)) */
            if (x >= mid) e = k;
        }
    } else {
        double xx = (double)x * (double)x;
        for (int k = 1; k <= 7; ++k) {
            double bound = ldexp(1.0, 2 * (k - 7) - 1);   /* (2^(k-7-1/2))^2 */
            if (xx >= bound) e = k;
        }
    }
    if (e == 0) s = 0;
    return (s << 3) | e;
}

/* Integer value carried by a PoT nibble: 0 or +-2^(e-1), i.e. level * 64. */
int rmsmp_o_pot_value(int nibble)
{
    int e = nibble & 7, s = (nibble >> 3) & 1;
    int v = (e == 0) ? 0 : (1 << (e - 1));
    return s ? -v : v;
}

/* Step that turns the integer value into the real weight: alpha/Q (Fixed), alpha/64 (PoT-4). */
float rmsmp_o_wstep(float alpha, int scheme, int bits)
{
    if (scheme == O_SCHEME_POT) return alpha / 64.0f;
    return alpha / (float)((1 << (bits - 1)) - 1);
}

/*
 * Quantize a whole weight matrix row by row (rows = filters, Section 3.1).
 * W[M][K] fp32 row-major; per-row scheme (0 PoT, 1 Fixed), bits (4 or 8), alpha.
 * values[M][K]: the integer each weight becomes (Fixed: q, PoT: +-2^(e-1) or 0).
 * wstep[M]: real weight = value * wstep.  Returns 0, or -1 on an invalid menu entry
 * (the method has exactly PoT-4, Fixed-4, Fixed-8) or a non-positive/non-finite alpha.
 */
int rmsmp_o_quantize_rows(const float *W, int M, int K, const uint8_t *scheme,
                          const uint8_t *bits, const float *alpha, int pot_mode,
                          int8_t *values, float *wstep)
{
    for (int r = 0; r < M; ++r) {
        int sc = scheme[r], b = bits[r];
        if (!((sc == O_SCHEME_POT && b == 4) || (sc == O_SCHEME_FIXED && (b == 4 || b == 8))))
            return -1;
        if (!(alpha[r] > 0.0f) || isinf(alpha[r])) return -1;
        for (int k = 0; k < K; ++k) {
            float w = W[(size_t)r * K + k];
            int v;
            if (sc == O_SCHEME_POT)
                v = rmsmp_o_pot_value(rmsmp_o_pot_nibble(w, alpha[r], pot_mode));
            else
                v = rmsmp_o_fixed_q(w, alpha[r], b);
            values[(size_t)r * K + k] = (int8_t)v;
        }
        wstep[r] = rmsmp_o_wstep(alpha[r], sc, b);
    }
    return 0;
}

/*
 * Activation quantizer: every activation is 4-bit fixed point, also for PoT rows
 * (Section 3.1; Figure 2 caption).  Reading: one clip value alpha_a per tensor;
 *   U4 (non-negative inputs):  a = round(clip(x/alpha_a, 0, 1) * 15), step alpha_a/15;
 *   S4: the Fixed-4 quantizer of Eq. 1 with alpha_a, step alpha_a/7.
 */
void rmsmp_o_quantize_act(const float *x, size_t count, float alpha_a, int kind,
                          int8_t *codes, float *act_step)
{
    for (size_t i = 0; i < count; ++i) {
        if (kind == O_ACT_U4) {
            float t = x[i] / alpha_a;
            if (t < 0.0f) t = 0.0f;
            if (t > 1.0f) t = 1.0f;
            float s = t * 15.0f;
            codes[i] = (int8_t)(int)rintf(s);
        } else {
            codes[i] = (int8_t)rmsmp_o_fixed_q(x[i], alpha_a, 4);
        }
    }
    *act_step = (kind == O_ACT_U4) ? alpha_a / 15.0f : alpha_a / 7.0f;
}

/* ---- row assignment (Section 3.1, Algorithm 1; ratio A:B:C of Section 3.3) ---- */

typedef struct { double var; int idx; } o_rank_t;

static int o_rank_cmp(const void *pa, const void *pb)
{
    const o_rank_t *a = (const o_rank_t *)pa, *b = (const o_rank_t *)pb;
    if (a->var < b->var) return -1;
    if (a->var > b->var) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

/* Population variance of one row, in double, plain two-pass sums in index order. */
double rmsmp_o_row_variance(const float *w, int K)
{
    double sum = 0.0;
    for (int k = 0; k < K; ++k) sum += (double)w[k];
    double mean = sum / (double)K;
    double acc = 0.0;
    for (int k = 0; k < K; ++k) {
        double d = (double)w[k] - mean;
        acc += d * d;
    }
    return acc / (double)K;
}

/*
 * Row counts for the ratio PoT-4 : Fixed-4 : Fixed-8 = A : B : C (A + B + C = 100).
 * Reading: n8 = floor(M*C/100 + 1/2), nP = floor(M*A/100 + 1/2) (limited to M - n8),
 * Fixed-4 takes the rest.
 */
void rmsmp_o_ratio_counts(int M, int A, int B, int C, int *nP, int *nF4, int *n8)
{
    (void)B;
    int c8 = (int)floor((double)M * (double)C / 100.0 + 0.5);
    if (c8 > M) c8 = M;
    int cP = (int)floor((double)M * (double)A / 100.0 + 0.5);
    if (cP > M - c8) cP = M - c8;
    *n8 = c8; *nP = cP; *nF4 = M - c8 - cP;
}

/*
 * Scheme/precision map of one layer.  The paper picks the Fixed-8 rows by a Hessian
 * eigenvalue (needs loss and data); the stand-in used by the synthetic workloads is the
 * variance itself: the n8 rows of highest variance become Fixed-8; of the others the nP
 * rows of lowest variance become PoT-4 and the remainder Fixed-4 ("smaller variance ->
 * PoT, otherwise Fixed").  Rank order = (variance, row index) ascending.
 */
void rmsmp_o_assign_rows(const float *W, int M, int K, int A, int B, int C,
                         uint8_t *scheme, uint8_t *bits)
{
    int nP, nF4, n8;
    rmsmp_o_ratio_counts(M, A, B, C, &nP, &nF4, &n8);
    o_rank_t *rk = (o_rank_t *)malloc(sizeof(o_rank_t) * (size_t)M);
    for (int r = 0; r < M; ++r) {
        rk[r].var = rmsmp_o_row_variance(W + (size_t)r * K, K);
        rk[r].idx = r;
    }
    qsort(rk, (size_t)M, sizeof(o_rank_t), o_rank_cmp);
    for (int i = 0; i < M; ++i) {
        int r = rk[i].idx;
        if (i < nP) { scheme[r] = O_SCHEME_POT; bits[r] = 4; }
        else if (i < nP + nF4) { scheme[r] = O_SCHEME_FIXED; bits[r] = 4; }
        else { scheme[r] = O_SCHEME_FIXED; bits[r] = 8; }
    }
    free(rk);
}

/*
 * Grouping: rows of one scheme are served by one GEMM core, so the packed order is all
 * PoT-4 rows, then Fixed-4, then Fixed-8, each group in original order (stable).
 * perm[p] = original row stored at packed position p.
 */
void rmsmp_o_group_rows(const uint8_t *scheme, const uint8_t *bits, int M, int32_t *perm)
{
    int p = 0;
    for (int g = 0; g < 3; ++g)
        for (int r = 0; r < M; ++r) {
            int key = (scheme[r] == O_SCHEME_POT) ? 0 : (bits[r] == 4 ? 1 : 2);
            if (key == g) perm[p++] = r;
        }
}

/* ---- the layer itself: out = proj(input) . proj(W)  (Algorithm 1, forward pass) ---- */

/* acc[n][r] = sum_k v[r][k] * a[n][k], int32.  v[M][K], a[N][K] (row pitch lda). */
void rmsmp_o_matmul(const int8_t *v, const int8_t *a, int M, int N, int K, int64_t lda,
                    int32_t *acc)
{
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n)
        for (int r = 0; r < M; ++r) {
            int32_t s = 0;
            for (int k = 0; k < K; ++k)
                s += (int32_t)v[(size_t)r * K + k] * (int32_t)a[(size_t)n * lda + k];
            acc[(size_t)n * M + r] = s;
        }
}

/* Same sum in int64: proves the int32 sum did not wrap. */
void rmsmp_o_matmul_i64(const int8_t *v, const int8_t *a, int M, int N, int K, int64_t lda,
                        int64_t *acc)
{
    for (int n = 0; n < N; ++n)
        for (int r = 0; r < M; ++r) {
            int64_t s = 0;
            for (int k = 0; k < K; ++k)
                s += (int64_t)v[(size_t)r * K + k] * (int64_t)a[(size_t)n * lda + k];
            acc[(size_t)n * M + r] = s;
        }
}

/*
 * The PoT rows done the multiplier-free way (Section 3.1: shifts replace multiplies):
 * acc +-= a << (e-1).  nib[M][K] are PoT nibbles.
 */
void rmsmp_o_matmul_pot_shift(const uint8_t *nib, const int8_t *a, int M, int N, int K,
                              int64_t lda, int32_t *acc)
{
    for (int n = 0; n < N; ++n)
        for (int r = 0; r < M; ++r) {
            int32_t s = 0;
            for (int k = 0; k < K; ++k) {
                int c = nib[(size_t)r * K + k];
                int e = c & 7;
                if (e == 0) continue;
                int32_t term = (int32_t)a[(size_t)n * lda + k] * (1 << (e - 1)); /* a << (e-1), sign-safe */
                s = (c & 8) ? s - term : s + term;
            }
            acc[(size_t)n * M + r] = s;
        }
}

/*
 * Direct convolution.  v[M][Cin][kh][kw] (filter-major, rows = filters), activations
 * a[B][H][W][Cin] (channels last), zero outside the image, output positions
 * Ho = (H + 2*pad - kh)/stride + 1 (same for Wo).  acc[B][Ho][Wo][M].
 */
void rmsmp_o_conv(const int8_t *v, const int8_t *a, int M, int Cin, int kh, int kw,
                  int B, int H, int W, int stride, int pad, int32_t *acc)
{
    int Ho = (H + 2 * pad - kh) / stride + 1;
    int Wo = (W + 2 * pad - kw) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int ho = 0; ho < Ho; ++ho)
            for (int wo = 0; wo < Wo; ++wo)
                for (int r = 0; r < M; ++r) {
                    int32_t s = 0;
                    for (int i = 0; i < kh; ++i) {
                        int y = ho * stride + i - pad;
                        if (y < 0 || y >= H) continue;
                        for (int j = 0; j < kw; ++j) {
                            int x = wo * stride + j - pad;
                            if (x < 0 || x >= W) continue;
                            for (int c = 0; c < Cin; ++c)
                                s += (int32_t)v[(((size_t)r * Cin + c) * kh + i) * kw + j] *
                                     (int32_t)a[(((size_t)b * H + y) * W + x) * Cin + c];
                        }
                    }
                    acc[(((size_t)b * Ho + ho) * Wo + wo) * M + r] = s;
                }
}

/*
 * Depthwise convolution (MobileNet-v2, one of the paper's models, Section 4.1; every filter is a
 * weight row of its own, Figure 2): channel c of the output sees channel c of the input only.
 * v[C][kh][kw], a[B][H][W][C], zero outside the image, acc[B][Ho][Wo][C].
 */
void rmsmp_o_conv_depthwise(const int8_t *v, const int8_t *a, int C, int kh, int kw,
                            int B, int H, int W, int stride, int pad, int32_t *acc)
{
    int Ho = (H + 2 * pad - kh) / stride + 1;
    int Wo = (W + 2 * pad - kw) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int ho = 0; ho < Ho; ++ho)
            for (int wo = 0; wo < Wo; ++wo)
                for (int c = 0; c < C; ++c) {
                    int32_t s = 0;
                    for (int i = 0; i < kh; ++i) {
                        int y = ho * stride + i - pad;
                        if (y < 0 || y >= H) continue;
                        for (int j = 0; j < kw; ++j) {
                            int x = wo * stride + j - pad;
                            if (x < 0 || x >= W) continue;
                            s += (int32_t)v[((size_t)c * kh + i) * kw + j] *
                                 (int32_t)a[(((size_t)b * H + y) * W + x) * C + c];
                        }
                    }
                    acc[(((size_t)b * Ho + ho) * Wo + wo) * C + c] = s;
                }
}

/* One output of the convolution at a time: (pixel index n = (b*Ho+ho)*Wo+wo, row r). */
void rmsmp_o_conv_points(const int8_t *v, const int8_t *a, int M, int Cin, int kh, int kw,
                         int B, int H, int W, int stride, int pad, const int64_t *n_idx,
                         const int32_t *r_idx, int64_t count, int32_t *acc)
{
    int Ho = (H + 2 * pad - kh) / stride + 1;
    int Wo = (W + 2 * pad - kw) / stride + 1;
    (void)B; (void)M;
#pragma omp parallel for schedule(static)
    for (int64_t q = 0; q < count; ++q) {
        int64_t n = n_idx[q];
        int r = r_idx[q];
        int wo = (int)(n % Wo), ho = (int)((n / Wo) % Ho);
        int64_t b = n / ((int64_t)Wo * Ho);
        int32_t s = 0;
        for (int i = 0; i < kh; ++i) {
            int y = ho * stride + i - pad;
            if (y < 0 || y >= H) continue;
            for (int j = 0; j < kw; ++j) {
                int x = wo * stride + j - pad;
                if (x < 0 || x >= W) continue;
                for (int c = 0; c < Cin; ++c)
                    s += (int32_t)v[(((size_t)r * Cin + c) * kh + i) * kw + j] *
                         (int32_t)a[(((size_t)b * H + y) * W + x) * Cin + c];
            }
        }
        acc[q] = s;
    }
}

/* One output of the linear layer at a time. */
void rmsmp_o_matmul_points(const int8_t *v, const int8_t *a, int K, int64_t lda,
                           const int64_t *n_idx, const int32_t *r_idx, int64_t count,
                           int32_t *acc)
{
    for (int64_t q = 0; q < count; ++q) {
        int32_t s = 0;
        for (int k = 0; k < K; ++k)
            s += (int32_t)v[(size_t)r_idx[q] * K + k] * (int32_t)a[(size_t)n_idx[q] * lda + k];
        acc[q] = s;
    }
}

/*
 * Scaling back to real numbers (the alpha of Eq. 1 / Eq. 4 times the activation step):
 * c_r = wstep_r * act_step (one fp32 multiply), y = (float)acc * c_r (exact conversion
 * while |acc| < 2^24, then one fp32 multiply).  acc and y are [N][M].
 */
void rmsmp_o_epilogue(const int32_t *acc, int64_t N, int M, const float *wstep, float act_step,
                      float *y)
{
    for (int64_t n = 0; n < N; ++n)
        for (int r = 0; r < M; ++r) {
            float c = wstep[r] * act_step;
            y[(size_t)n * M + r] = (float)acc[(size_t)n * M + r] * c;
        }
}

int rmsmp_o_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

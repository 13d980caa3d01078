/*
 * CPU oracle for the Ternary Weight Networks hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64.  It shares no code, header, table or constant with the
 * CUDA library; only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  Every function names the passage of the paper it follows.
 *
 * Conventions
 *   - master weights are fp32 and are widened exactly to double;
 *   - activations / gradients are bf16 bit patterns (uint16_t), widened exactly;
 *   - ternary codes are int8_t in {-1, 0, +1};
 *   - conv tensors are NHWC, filters are [Cout][kh][kw][Cin] (Cin fastest),
 *     convolution is cross-correlation with zero padding;
 *   - every contraction also returns A = sum_k |x_k * t_k| (no alpha, no
 *     epilogue), the quantity the parity tolerance is stated in.
 *
 * Pins (tests/test_oracle_*.py): closed form of alpha vs. Algorithm 1's
 * quotient (per layer and per filter), a hand-worked per-filter example, 3^n enumeration of Eq. 1, threshold sweeps vs. the paper's
 * closed forms for uniform / normal weights, pack round trip over all 3^16
 * words, numpy/torch fp64 matmul and conv2d, adjoint identities.
 * The binary-weight functions (ref_binarize, ref_pack1): a hand-worked example, the 2^n enumeration, the
 * closed form of alpha, every bit position of a word.
 * Parity unpinned: none of the functions below.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t B, H, W, Cin, Cout;
    int32_t kh, kw, stride_h, stride_w, pad_h, pad_w;
} ref_conv_desc;

typedef struct {
    double delta;        /* c * (1/n) * sum |W_i|                      */
    double alpha;        /* mean of |W_i| over |W_i| > delta, 0 if none */
    double sum_abs;      /* sum |W_i|                                   */
    double sum_abs_kept; /* sum of |W_i| over |W_i| > delta             */
    int64_t n_neg, n_zero, n_pos;
    int64_t n_boundary;  /* #{ i : | |W_i| - delta | <= 1e-12 * delta } */
    int32_t nonfinite;   /* 1 if any W_i is NaN or +-Inf                */
    int32_t pad_;
} ref_stats;

typedef struct {
    const float *scale;     /* [N] or NULL: per-output-channel multiplier */
    const float *shift;     /* [N] or NULL: per-output-channel offset     */
    const double *residual; /* same shape as the output, or NULL          */
    int32_t relu;
    int32_t pad_;
} ref_epilogue;

int ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double bf16_to_double(uint16_t b)
{
    uint32_t w = (uint32_t)b << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* Neumaier's compensated accumulator: s + c is the running sum. */
typedef struct { double s, c; } csum;
static void csum_add(csum *a, double x)
{
    double t = a->s + x;
    if (fabs(a->s) >= fabs(x)) a->c += (a->s - t) + x;
    else                       a->c += (x - t) + a->s;
    a->s = t;
}

/* ------------------------------------------------------------------------
 * Threshold ternarization.  Steps in the order of Algorithm 1:
 *   delta = c/n * ||W||_1            (Section 2.3 rule of thumb; Alg. 1)
 *   code_i = f(W_i | delta)          (Eq. 3: +1 if W_i > delta, -1 if
 *                                     W_i < -delta, 0 if |W_i| <= delta)
 *   alpha = mean of |W_i| over I_delta = { i : |W_i| > delta }   (Eq. 5)
 * n counts every weight, zeros included.  I_delta empty -> alpha = 0.
 * codes may be NULL.  Returns 0, or 1 when a weight is not finite.
 * ---------------------------------------------------------------------- */
int ref_ternarize(const float *W, int64_t n, double c, ref_stats *st, int8_t *codes)
{
    memset(st, 0, sizeof *st);
    csum S = {0.0, 0.0};
    for (int64_t i = 0; i < n; ++i) {
        double w = (double)W[i];
        if (!isfinite(w)) st->nonfinite = 1;
        csum_add(&S, fabs(w));
    }
    st->sum_abs = S.s + S.c;
    if (st->nonfinite) return 1;
    double delta = (n > 0) ? c * (st->sum_abs / (double)n) : 0.0;
    st->delta = delta;

    csum Kp = {0.0, 0.0};
    for (int64_t i = 0; i < n; ++i) {
        double w = (double)W[i];
        int8_t t;
        if (w > delta)       { t = +1; st->n_pos++; }
        else if (w < -delta) { t = -1; st->n_neg++; }
        else                 { t = 0;  st->n_zero++; }
        if (t != 0) csum_add(&Kp, fabs(w));
        if (fabs(fabs(w) - delta) <= 1e-12 * delta) st->n_boundary++;
        if (codes) codes[i] = t;
    }
    st->sum_abs_kept = Kp.s + Kp.c;
    int64_t kept = st->n_pos + st->n_neg;
    st->alpha = kept > 0 ? st->sum_abs_kept / (double)kept : 0.0;
    return 0;
}

/* ------------------------------------------------------------------------
 * Per-filter ternarization: Algorithm 1 as printed, whose first loop runs over
 * the filters of a layer.  Filter r (row r of W[rows][cols]) gets its own
 *   delta_r = c/cols * ||W_r||_1,   codes by Eq. 3 against delta_r,
 *   alpha_r = mean of |W_r,i| over |W_r,i| > delta_r            (Eq. 5)
 * n in the threshold rule is the element count of the filter.  st has `rows`
 * entries, codes (optional) rows*cols.  Returns the number of rows that hold
 * a non-finite weight.
 * ---------------------------------------------------------------------- */
int ref_ternarize_rows(const float *W, int64_t rows, int64_t cols, double c, ref_stats *st, int8_t *codes)
{
    int bad = 0;
    for (int64_t r = 0; r < rows; ++r)
        bad += ref_ternarize(W + r * cols, cols, c, st + r, codes ? codes + r * cols : NULL);
    return bad;
}

/* Algorithm 1's form of the scale: alpha = (W . W~) / (W~ . W~), in long double. */
double ref_alpha_alg1(const float *W, const int8_t *codes, int64_t n)
{
    long double num = 0.0L, den = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        num += (long double)W[i] * (long double)codes[i];
        den += (long double)codes[i] * (long double)codes[i];
    }
    return den > 0.0L ? (double)(num / den) : 0.0;
}

/* sum |W_i| in long double (cross-check of the compensated fp64 sum). */
double ref_sum_abs_ld(const float *W, int64_t n)
{
    long double s = 0.0L;
    for (int64_t i = 0; i < n; ++i) s += fabsl((long double)W[i]);
    return (double)s;
}

/* Eq. 1: J(alpha, W~) = || W - alpha W~ ||_2^2 */
double ref_objective(const float *W, const int8_t *codes, double alpha, int64_t n)
{
    long double j = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        long double d = (long double)W[i] - (long double)alpha * (long double)codes[i];
        j += d * d;
    }
    return (double)j;
}

/* ------------------------------------------------------------------------
 * 2-bit storage (Section 2.1, "2-bit storage requirement ... for a unit of
 * weight").  The paper fixes no encoding; this library's is:
 *   field   two's complement in two bits: 0 -> 00, +1 -> 01, -1 -> 11
 *           (10 is never produced);
 *   word    a row is cut into groups of 16 codes, one 32-bit word per group.
 *           Inside a group the even elements fill the low half-word and the
 *           odd elements the high half-word, each from its top bits down:
 *           element e (0..15) sits at bit position 14 - 2*(e/2) + 16*(e%2);
 *   row     ld_codes/16 words (ld_codes a multiple of 16 here), padded with 00.
 * ---------------------------------------------------------------------- */
static int field_pos(int64_t e) { return (int)(14 - 2 * (e / 2) + 16 * (e % 2)); }

int ref_pack(const int8_t *codes, int64_t rows, int64_t cols, int64_t ld_codes, uint32_t *packed)
{
    if (ld_codes % 16 != 0 || ld_codes < cols) return -1;
    int64_t wpr = ld_codes / 16;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t w = 0; w < wpr; ++w) packed[r * wpr + w] = 0u;
        for (int64_t j = 0; j < cols; ++j) {
            int8_t t = codes[r * cols + j];
            uint32_t f;
            if (t == 0) f = 0u; else if (t == 1) f = 1u; else if (t == -1) f = 3u; else return -2;
            packed[r * wpr + j / 16] |= f << field_pos(j % 16);
        }
    }
    return 0;
}

int ref_unpack(const uint32_t *packed, int64_t rows, int64_t cols, int64_t ld_codes, int8_t *codes)
{
    if (ld_codes % 16 != 0 || ld_codes < cols) return -1;
    int64_t wpr = ld_codes / 16;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < cols; ++j) {
            uint32_t f = (packed[r * wpr + j / 16] >> field_pos(j % 16)) & 3u;
            if (f == 2u) return -2;
            codes[r * cols + j] = (f == 0u) ? 0 : (f == 1u ? 1 : -1);
        }
    return 0;
}

/* ------------------------------------------------------------------------
 * Brute force on Eq. 1 / Eq. 4, used only to validate ref_ternarize.
 * ---------------------------------------------------------------------- */
static int cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

/* Threshold sweep.  Candidates: 0 and the midpoints of consecutive distinct
 * sorted |W| values.  For each, I = {|W_i| > delta}, alpha = mean_I |W|
 * (Eq. 5) and J = sum W^2 - (sum_I |W|)^2 / |I|  (Eq. 4 with Eq. 5
 * substituted).  Returns the minimiser: best_delta, best_alpha, best_J and
 * best_factor = best_delta / mean|W|. */
int ref_bruteforce_threshold(const float *W, int64_t n, double *best_delta,
                             double *best_alpha, double *best_J, double *best_factor)
{
    if (n <= 0) return -1;
    double *a = (double *)malloc((size_t)n * sizeof(double));
    if (!a) return -2;
    long double sq = 0.0L, tot = 0.0L;
    for (int64_t i = 0; i < n; ++i) {
        a[i] = fabs((double)W[i]);
        sq += (long double)a[i] * a[i];
        tot += a[i];
    }
    qsort(a, (size_t)n, sizeof(double), cmp_double);
    /* suffix[i] = sum of a[i..n-1] */
    long double *suffix = (long double *)malloc((size_t)(n + 1) * sizeof(long double));
    if (!suffix) { free(a); return -2; }
    suffix[n] = 0.0L;
    for (int64_t i = n - 1; i >= 0; --i) suffix[i] = suffix[i + 1] + a[i];

    double bJ = INFINITY, bD = 0.0, bA = 0.0;
    /* candidate index i: delta lies below a[i] and at/above a[i-1]; kept set = a[i..n-1] */
    for (int64_t i = 0; i < n; ++i) {
        double delta;
        if (i == 0) delta = 0.0;
        else {
            if (a[i] == a[i - 1]) continue;
            delta = 0.5 * (a[i] + a[i - 1]);
        }
        if (i == 0 && a[0] == 0.0) continue; /* delta = 0 keeps only |W| > 0 */
        long double k = suffix[i];
        long double cnt = (long double)(n - i);
        double J = (double)(sq - k * k / cnt);
        if (J < bJ) { bJ = J; bD = delta; bA = (double)(k / cnt); }
    }
    *best_delta = bD; *best_alpha = bA; *best_J = bJ;
    *best_factor = bD / (double)(tot / (long double)n);
    free(suffix); free(a);
    return 0;
}

/* Full enumeration of Eq. 1 for n <= 12: all 3^n ternary vectors, each with
 * its best alpha = max(0, W.W~ / W~.W~).  Writes the minimiser. */
int ref_bruteforce_enum(const float *W, int64_t n, int8_t *best_codes, double *best_alpha, double *best_J)
{
    if (n <= 0 || n > 12) return -1;
    int64_t total = 1;
    for (int64_t i = 0; i < n; ++i) total *= 3;
    int8_t t[12];
    double bJ = INFINITY;
    for (int64_t v = 0; v < total; ++v) {
        int64_t r = v;
        double num = 0.0, den = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            t[i] = (int8_t)(r % 3) - 1; r /= 3;
            num += (double)W[i] * t[i];
            den += (double)t[i] * t[i];
        }
        double alpha = den > 0.0 ? num / den : 0.0;
        if (alpha < 0.0) alpha = 0.0;
        double J = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double d = (double)W[i] - alpha * t[i];
            J += d * d;
        }
        if (J < bJ) {
            bJ = J; *best_alpha = alpha;
            memcpy(best_codes, t, (size_t)n);
        }
    }
    *best_J = bJ;
    return 0;
}

/* ------------------------------------------------------------------------
 * Binary precision weights (Section 3: the BPWN baseline "uses the sign
 * function to binarize the weights"), scaled like the ternary ones:
 *   B_i   = +1 if W_i >= 0, -1 if W_i < 0     (a two-valued code has no zero;
 *           the reading taken for W_i = 0, and for -0.0, is +1)
 *   alpha = (1/n) * sum |W_i|                  (the minimiser of ||W - alpha B||^2
 *           for B = sign(W): a 1-D quadratic in alpha, as Eq. 4 is for Eq. 1)
 * st: alpha, sum_abs, n_pos, n_neg and nonfinite are written; delta = 0,
 * n_zero = 0, sum_abs_kept = sum_abs.  Returns 0, or 1 when a weight is not finite.
 * ---------------------------------------------------------------------- */
int ref_binarize(const float *W, int64_t n, ref_stats *st, int8_t *codes)
{
    memset(st, 0, sizeof *st);
    csum S = {0.0, 0.0};
    for (int64_t i = 0; i < n; ++i) {
        double w = (double)W[i];
        if (!isfinite(w)) st->nonfinite = 1;
        csum_add(&S, fabs(w));
        int8_t b = (w < 0.0) ? -1 : +1;
        if (b > 0) st->n_pos++; else st->n_neg++;
        if (codes) codes[i] = b;
    }
    st->sum_abs = S.s + S.c;
    st->sum_abs_kept = st->sum_abs;
    if (st->nonfinite) return 1;
    st->alpha = n > 0 ? st->sum_abs / (double)n : 0.0;
    return 0;
}

/* Full enumeration of min over alpha >= 0 and B in {-1,+1}^n of ||W - alpha B||^2 for n <= 16: all 2^n
 * sign vectors, each with its best alpha = max(0, W.B / n).  Writes the minimiser. */
int ref_bruteforce_enum2(const float *W, int64_t n, int8_t *best_codes, double *best_alpha, double *best_J)
{
    if (n <= 0 || n > 16) return -1;
    int8_t b[16];
    double bJ = INFINITY;
    for (int64_t v = 0; v < ((int64_t)1 << n); ++v) {
        double num = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            b[i] = ((v >> i) & 1) ? -1 : +1;
            num += (double)W[i] * b[i];
        }
        double alpha = num / (double)n;
        if (alpha < 0.0) alpha = 0.0;
        double J = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double d = (double)W[i] - alpha * b[i];
            J += d * d;
        }
        if (J < bJ) {
            bJ = J; *best_alpha = alpha;
            memcpy(best_codes, b, (size_t)n);
        }
    }
    *best_J = bJ;
    return 0;
}

/* 1-bit storage of binary codes (the paper's model-compression argument with one bit per weight,
 * 32x smaller than fp32).  The paper fixes no encoding; this library's mirrors the 2-bit one:
 *   bit     1 for -1, 0 for +1;
 *   word    a row is cut into groups of 32 codes, one 32-bit word per group.  The even elements fill
 *           the low half-word and the odd elements the high half-word, each from its top bit down:
 *           element e (0..31) sits at bit position 15 - e/2 + 16*(e%2);
 *   row     ld_codes/32 words (ld_codes a multiple of 32 here); the padding bits are 0.
 * ---------------------------------------------------------------------- */
static int bit_pos(int64_t e) { return (int)(15 - (e / 2) + 16 * (e % 2)); }

int ref_pack1(const int8_t *codes, int64_t rows, int64_t cols, int64_t ld_codes, uint32_t *packed)
{
    if (ld_codes % 32 != 0 || ld_codes < cols) return -1;
    int64_t wpr = ld_codes / 32;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t w = 0; w < wpr; ++w) packed[r * wpr + w] = 0u;
        for (int64_t j = 0; j < cols; ++j) {
            int8_t t = codes[r * cols + j];
            if (t != 1 && t != -1) return -2;
            if (t == -1) packed[r * wpr + j / 32] |= 1u << bit_pos(j % 32);
        }
    }
    return 0;
}

int ref_unpack1(const uint32_t *packed, int64_t rows, int64_t cols, int64_t ld_codes, int8_t *codes)
{
    if (ld_codes % 32 != 0 || ld_codes < cols) return -1;
    int64_t wpr = ld_codes / 32;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < cols; ++j)
            codes[r * cols + j] = ((packed[r * wpr + j / 32] >> bit_pos(j % 32)) & 1u) ? -1 : +1;
    return 0;
}

/* ------------------------------------------------------------------------
 * Ternary block, forward (Eq. 2): Z = X * (alpha W~), then the epilogue
 *   y = relu?( scale[n] * (alpha * sum_k x_k t_k) + shift[n] + residual ).
 * ---------------------------------------------------------------------- */
static double apply_epilogue(double acc, double alpha, const ref_epilogue *e, int64_t ch, int64_t flat)
{
    double y = alpha * acc;
    if (e) {
        if (e->scale) y *= (double)e->scale[ch];
        if (e->shift) y += (double)e->shift[ch];
        if (e->residual) y += e->residual[flat];
        if (e->relu && y < 0.0) y = 0.0;
    }
    return y;
}

/* Inner product form: Y[m,n] = epi(alpha * sum_k X[m,k] * T[n,k]);
 * X is [M, ldx] bf16, T is int8 [N][K]. */
void ref_gemm(const uint16_t *X, int64_t ldx, const int8_t *T, double alpha,
              int64_t M, int64_t N, int64_t K, const ref_epilogue *e,
              double *Y, double *A)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0, mag = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double p = bf16_to_double(X[m * ldx + k]) * (double)T[n * K + k];
                acc += p;
                mag += fabs(p);
            }
            Y[m * N + n] = apply_epilogue(acc, alpha, e, n, m * N + n);
            if (A) A[m * N + n] = mag;
        }
    }
}

static int64_t out_extent(int64_t in, int k, int stride, int pad)
{
    return (in + 2 * (int64_t)pad - k) / stride + 1;
}

/* One output pixel (b, ho, wo), all Cout channels. */
static void conv_fwd_pixel(const ref_conv_desc *d, const uint16_t *X, const int8_t *T,
                           double alpha, const ref_epilogue *e,
                           int64_t b, int64_t ho, int64_t wo, int64_t flat_pix,
                           double *y, double *a)
{
    for (int64_t o = 0; o < d->Cout; ++o) {
        double acc = 0.0, mag = 0.0;
        for (int r = 0; r < d->kh; ++r) {
            int64_t h = ho * d->stride_h - d->pad_h + r;
            if (h < 0 || h >= d->H) continue;
            for (int s = 0; s < d->kw; ++s) {
                int64_t w = wo * d->stride_w - d->pad_w + s;
                if (w < 0 || w >= d->W) continue;
                const uint16_t *xp = X + ((b * d->H + h) * d->W + w) * d->Cin;
                const int8_t *tp = T + ((o * d->kh + r) * d->kw + s) * d->Cin;
                for (int64_t c = 0; c < d->Cin; ++c) {
                    double p = bf16_to_double(xp[c]) * (double)tp[c];
                    acc += p;
                    mag += fabs(p);
                }
            }
        }
        y[o] = apply_epilogue(acc, alpha, e, o, flat_pix * d->Cout + o);
        if (a) a[o] = mag;
    }
}

/* Convolution form, whole output [B, Ho, Wo, Cout]. */
void ref_conv2d_fwd(const ref_conv_desc *d, const uint16_t *X, const int8_t *T, double alpha,
                    const ref_epilogue *e, double *Y, double *A)
{
    int64_t Ho = out_extent(d->H, d->kh, d->stride_h, d->pad_h);
    int64_t Wo = out_extent(d->W, d->kw, d->stride_w, d->pad_w);
    int64_t npix = d->B * Ho * Wo;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < npix; ++p) {
        int64_t b = p / (Ho * Wo), ho = (p / Wo) % Ho, wo = p % Wo;
        conv_fwd_pixel(d, X, T, alpha, e, b, ho, wo, p, Y + p * d->Cout, A ? A + p * d->Cout : NULL);
    }
}

/* Same, for a list of flat output-pixel indices p = (b*Ho + ho)*Wo + wo.
 * Y, A are [npix][Cout]; the residual (if any) is still indexed by the full
 * output tensor. */
void ref_conv2d_fwd_pixels(const ref_conv_desc *d, const uint16_t *X, const int8_t *T, double alpha,
                           const ref_epilogue *e, const int64_t *pix, int64_t npix,
                           double *Y, double *A)
{
    int64_t Ho = out_extent(d->H, d->kh, d->stride_h, d->pad_h);
    int64_t Wo = out_extent(d->W, d->kw, d->stride_w, d->pad_w);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < npix; ++i) {
        int64_t p = pix[i];
        int64_t b = p / (Ho * Wo), ho = (p / Wo) % Ho, wo = p % Wo;
        conv_fwd_pixel(d, X, T, alpha, e, b, ho, wo, p, Y + i * d->Cout, A ? A + i * d->Cout : NULL);
    }
}

/* ------------------------------------------------------------------------
 * Ternary block, backward for data (Algorithm 1, TernaryBackward: ordinary
 * back-propagation with T = alpha W~ in place of W).  Written as the adjoint
 * of the forward sum in scatter form: every forward term
 *   Z[b,ho,wo,o] += alpha * X[b,h,w,c] * t[o,r,s,c]
 * contributes dX[b,h,w,c] += alpha * dZ[b,ho,wo,o] * t[o,r,s,c].
 * dZ is bf16 [B,Ho,Wo,Cout]; dX, A are double [B,H,W,Cin].
 * ---------------------------------------------------------------------- */
void ref_conv2d_bwd_data(const ref_conv_desc *d, const uint16_t *dZ, const int8_t *T, double alpha,
                         double *dX, double *A)
{
    int64_t Ho = out_extent(d->H, d->kh, d->stride_h, d->pad_h);
    int64_t Wo = out_extent(d->W, d->kw, d->stride_w, d->pad_w);
    int64_t img = d->H * d->W * d->Cin;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < d->B; ++b) {
        double *dx = dX + b * img;
        double *ax = A ? A + b * img : NULL;
        for (int64_t i = 0; i < img; ++i) { dx[i] = 0.0; if (ax) ax[i] = 0.0; }
        for (int64_t ho = 0; ho < Ho; ++ho)
        for (int64_t wo = 0; wo < Wo; ++wo)
        for (int64_t o = 0; o < d->Cout; ++o) {
            double g = bf16_to_double(dZ[((b * Ho + ho) * Wo + wo) * d->Cout + o]);
            for (int r = 0; r < d->kh; ++r) {
                int64_t h = ho * d->stride_h - d->pad_h + r;
                if (h < 0 || h >= d->H) continue;
                for (int s = 0; s < d->kw; ++s) {
                    int64_t w = wo * d->stride_w - d->pad_w + s;
                    if (w < 0 || w >= d->W) continue;
                    const int8_t *tp = T + ((o * d->kh + r) * d->kw + s) * d->Cin;
                    double *dp = dx + (h * d->W + w) * d->Cin;
                    double *ap = ax ? ax + (h * d->W + w) * d->Cin : NULL;
                    for (int64_t c = 0; c < d->Cin; ++c) {
                        double p = g * (double)tp[c];
                        dp[c] += p;
                        if (ap) ap[c] += fabs(p);
                    }
                }
            }
        }
        for (int64_t i = 0; i < img; ++i) dx[i] *= alpha;
    }
}

/* Gather form of the same adjoint for a list of flat input-pixel indices
 * q = (b*H + h)*W + w: dX[q,c] = alpha * sum over (r,s,o) with
 * ho*stride - pad + r == h (and likewise for w) of dZ[b,ho,wo,o] t[o,r,s,c].
 * Tests pin it to the scatter form above.  dX, A are [npix][Cin]. */
void ref_conv2d_bwd_data_pixels(const ref_conv_desc *d, const uint16_t *dZ, const int8_t *T, double alpha,
                                const int64_t *pix, int64_t npix, double *dX, double *A)
{
    int64_t Ho = out_extent(d->H, d->kh, d->stride_h, d->pad_h);
    int64_t Wo = out_extent(d->W, d->kw, d->stride_w, d->pad_w);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < npix; ++i) {
        int64_t q = pix[i];
        int64_t b = q / (d->H * d->W), h = (q / d->W) % d->H, w = q % d->W;
        for (int64_t c = 0; c < d->Cin; ++c) {
            double acc = 0.0, mag = 0.0;
            for (int r = 0; r < d->kh; ++r) {
                int64_t hn = h + d->pad_h - r;
                if (hn < 0 || hn % d->stride_h != 0) continue;
                int64_t ho = hn / d->stride_h;
                if (ho >= Ho) continue;
                for (int s = 0; s < d->kw; ++s) {
                    int64_t wn = w + d->pad_w - s;
                    if (wn < 0 || wn % d->stride_w != 0) continue;
                    int64_t wo = wn / d->stride_w;
                    if (wo >= Wo) continue;
                    const uint16_t *gp = dZ + ((b * Ho + ho) * Wo + wo) * d->Cout;
                    for (int64_t o = 0; o < d->Cout; ++o) {
                        double p = bf16_to_double(gp[o]) *
                                   (double)T[((o * d->kh + r) * d->kw + s) * d->Cin + c];
                        acc += p;
                        mag += fabs(p);
                    }
                }
            }
            dX[i * d->Cin + c] = alpha * acc;
            if (A) A[i * d->Cin + c] = mag;
        }
    }
}

/* ------------------------------------------------------------------------
 * Straight-through weight gradient (Algorithm 1, UpdateParameters; Fig. 1
 * caption): the gradient w.r.t. T, computed by ordinary back-propagation
 * and applied to the fp32 master copy unchanged -- no alpha factor, no mask:
 *   dW[o,r,s,c] = sum_{b,ho,wo} dZ[b,ho,wo,o] * X[b, ho*st-p+r, wo*st-p+s, c].
 * idx lists flat entries of dW ([Cout][kh][kw][Cin]); idx == NULL means all.
 * ---------------------------------------------------------------------- */
void ref_conv2d_bwd_weight(const ref_conv_desc *d, const uint16_t *X, const uint16_t *dZ,
                           const int64_t *idx, int64_t nidx, double *dW, double *A)
{
    int64_t Ho = out_extent(d->H, d->kh, d->stride_h, d->pad_h);
    int64_t Wo = out_extent(d->W, d->kw, d->stride_w, d->pad_w);
    int64_t total = d->Cout * d->kh * d->kw * d->Cin;
    int64_t cnt = idx ? nidx : total;
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t i = 0; i < cnt; ++i) {
        int64_t f = idx ? idx[i] : i;
        int64_t c = f % d->Cin;
        int64_t s = (f / d->Cin) % d->kw;
        int64_t r = (f / (d->Cin * d->kw)) % d->kh;
        int64_t o = f / (d->Cin * d->kw * d->kh);
        double acc = 0.0, mag = 0.0;
        for (int64_t b = 0; b < d->B; ++b)
        for (int64_t ho = 0; ho < Ho; ++ho) {
            int64_t h = ho * d->stride_h - d->pad_h + r;
            if (h < 0 || h >= d->H) continue;
            for (int64_t wo = 0; wo < Wo; ++wo) {
                int64_t w = wo * d->stride_w - d->pad_w + s;
                if (w < 0 || w >= d->W) continue;
                double p = bf16_to_double(dZ[((b * Ho + ho) * Wo + wo) * d->Cout + o]) *
                           bf16_to_double(X[((b * d->H + h) * d->W + w) * d->Cin + c]);
                acc += p;
                mag += fabs(p);
            }
        }
        dW[i] = acc;
        if (A) A[i] = mag;
    }
}

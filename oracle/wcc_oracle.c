/*
 * CPU oracle for the Wavelet Compressed Convolution (WCC) layer -- TEST INFRASTRUCTURE ONLY.
 *
 * Only the tests, the smoke check and the bench's CPU-baseline leg may call this
 * library.  It is deliberately plain and slow: the layer of Eq. 9 / Alg. 1 taken
 * step by step, with the signed symmetric quantizer of Eq. 1-2 placed on the
 * wavelet-domain activations and on the weights (Sec. 4, "Joint hard shrinkage").
 * Compile with contraction off (-ffp-contract=off): every written operation rounds once.
 *
 * Parity pins: the Haar steps, the norms, the selection, the quantizer and the integer
 * contraction are pinned by closed forms, an explicit orthonormal matrix, brute force and
 * the k = all / fixed-index-set invariants (tests/test_oracle_*.py).  The paper prints no
 * numeric input/output example of the layer, so the floating-point layer output on
 * realistic maps is "parity unpinned" beyond those invariants.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static int cmp_int_asc(const void *A, const void *B)
{
    const int32_t a = *(const int32_t *)A, b = *(const int32_t *)B;
    return (a > b) - (a < b);
}

#define REAL float
#define SUF(name) name##_f32
#define FMA(a, b, c) fmaf((a), (b), (c))
#include "wcc_oracle_impl.h"
#undef REAL
#undef SUF
#undef FMA

#define REAL double
#define SUF(name) name##_f64
#define FMA(a, b, c) fma((a), (b), (c))
#include "wcc_oracle_impl.h"
#undef REAL
#undef SUF
#undef FMA

/* fp32 -> bf16 -> fp32, round to nearest, ties to even (finite inputs). */
static float round_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    u &= 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return f;
}

void orc_round_bf16(const float *in, long n, float *out)
{
    for (long i = 0; i < n; ++i) out[i] = round_to_bf16(in[i]);
}

/*
 * Signed symmetric b-bit quantizer (Eq. 1-2, signed case): x_b = alpha * q_{b-1}(clip(x/alpha,-1,1)),
 * i.e. an integer code round(x * qmax/alpha) in [-qmax, qmax], qmax = 2^(b-1) - 1, times the
 * step alpha/qmax.  The clipping parameter alpha is the largest magnitude in the tensor, so
 * the clip never bites; x/alpha followed by the multiplication by qmax is taken as a single
 * multiplication by inv = qmax/alpha; round is to nearest, ties to even.
 * Returns the step (scale); codes are written to q.
 */
float orc_quantize_alpha(const float *x, long n, int bits, float alpha, int8_t *q);

float orc_quantize(const float *x, long n, int bits, int8_t *q)
{
    float amax = 0.0f;
    for (long i = 0; i < n; ++i) {
        const float a = fabsf(x[i]);
        if (a > amax) amax = a;
    }
    return orc_quantize_alpha(x, n, bits, amax, q);
}

/*
 * The same quantizer with the clipping parameter given (Eq. 2: alpha is a parameter of the layer, learned during
 * training; here it is an argument).  Values beyond +-alpha are clipped: their codes are +-qmax.
 */
float orc_quantize_alpha(const float *x, long n, int bits, float alpha, int8_t *q)
{
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const float amax = alpha;
    const float inv = (amax > 0.0f) ? qmax / amax : 0.0f;
    for (long i = 0; i < n; ++i) {
        float r = nearbyintf(x[i] * inv);
        if (r > qmax) r = qmax;
        if (r < -qmax) r = -qmax;
        q[i] = (int8_t)r;
    }
    return amax / qmax;
}

/* Weights: one clipping parameter per output channel (row of Wt[Cout][Cin]), the row's largest magnitude. */
void orc_quantize_weights(const float *Wt, int Cout, int Cin, int bits, int8_t *Wq, float *scale_w)
{
    for (int o = 0; o < Cout; ++o)
        scale_w[o] = orc_quantize(Wt + (size_t)o * Cin, Cin, bits, Wq + (size_t)o * Cin);
}

/*
 * The whole layer, WCC(K, x) = H^T T^T K T H x (Eq. 9), in the order of Alg. 1.
 *
 *  x        fp32 [N][Cin][H][W] (bf16 inputs are widened exactly by the caller)
 *  Wt       fp32 [Cout][Cin]
 *  k        kept positions per image
 *  bits     8 (or 2..7): quantized path; 0: no quantization, contraction in double
 *  out_bf16 non-zero: round the output to bf16 (kept in fp32 storage)
 *  idx_in   NULL, or a fixed index set [N][k] (ascending) used instead of the selection
 *  y        fp32 [N][Cout][H][W]
 * Optional taps (NULL to skip): coef [N][Cin][P], nrm2 [N][P], idx [N][k], Xq int8 [N][k][Cin],
 *  scale_a [1], Wq int8 [Cout][Cin], scale_w [Cout], acc int32 [N][k][Cout].
 */
int orc_forward_ex_f32(const float *x, const float *Wt, int N, int Cin, int Cout, int H, int W,
                       int levels, int k, int bits, int wbits, float alpha, const float *residual, int relu,
                       int out_bf16, const int32_t *idx_in, float *y,
                       float *coef_tap, float *nrm2_tap, int32_t *idx_tap, int8_t *Xq_tap,
                       float *scale_a_tap, int8_t *Wq_tap, float *scale_w_tap, int32_t *acc_tap);

int orc_forward_f32(const float *x, const float *Wt, int N, int Cin, int Cout, int H, int W,
                    int levels, int k, int bits, int out_bf16, const int32_t *idx_in, float *y,
                    float *coef_tap, float *nrm2_tap, int32_t *idx_tap, int8_t *Xq_tap,
                    float *scale_a_tap, int8_t *Wq_tap, float *scale_w_tap, int32_t *acc_tap)
{
    return orc_forward_ex_f32(x, Wt, N, Cin, Cout, H, W, levels, k, bits, bits, 0.0f, NULL, 0, out_bf16, idx_in, y,
                              coef_tap, nrm2_tap, idx_tap, Xq_tap, scale_a_tap, Wq_tap, scale_w_tap, acc_tap);
}

/*
 * The layer with the options a network built from it uses:
 *  wbits     bits of the weight codes (the paper also runs 4-bit weights with 8-bit activations, Tables 1-2)
 *  alpha     > 0: the clipping parameter of the activation quantizer (Eq. 2), one for the whole layer (Sec. 4);
 *            <= 0: the largest kept magnitude of this call
 *  residual  NULL, or a map [N][Cout][H][W] added to the layer's output (the skip connection of the inverted
 *            residual block, Eq. 13): one fp32 addition per element, after the inverse transform
 *  relu      non-zero: max(., 0) after the addition (the non-linearity between chained layers)
 * The output is rounded to bf16 last, when asked.
 */
int orc_forward_ex_f32(const float *x, const float *Wt, int N, int Cin, int Cout, int H, int W,
                       int levels, int k, int bits, int wbits, float alpha, const float *residual, int relu,
                       int out_bf16, const int32_t *idx_in, float *y,
                       float *coef_tap, float *nrm2_tap, int32_t *idx_tap, int8_t *Xq_tap,
                       float *scale_a_tap, int8_t *Wq_tap, float *scale_w_tap, int32_t *acc_tap)
{
    const long P = (long)H * W;
    if (k < 1 || k > P) return -1;
    if (!(bits == 0 || (bits >= 2 && bits <= 8))) return -1;
    if (bits > 0 && !(wbits >= 2 && wbits <= 8)) return -1;
    const size_t nk = (size_t)N * k;
    float *coef = (float *)malloc(sizeof(float) * (size_t)N * Cin * P);
    float *nrm2 = (float *)malloc(sizeof(float) * (size_t)N * P);
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * nk);
    float *Xc = (float *)malloc(sizeof(float) * nk * Cin);          /* [N][k][Cin] */
    float *Yc = (float *)malloc(sizeof(float) * nk * Cout);         /* [N][k][Cout] */
    float *Ywt = (float *)calloc((size_t)N * Cout * P, sizeof(float));
    int8_t *Xq = (int8_t *)malloc(nk * Cin);
    int8_t *Wq = (int8_t *)malloc((size_t)Cout * Cin);
    float *scale_w = (float *)malloc(sizeof(float) * Cout);
    int rc = -2;
    if (!coef || !nrm2 || !idx || !Xc || !Yc || !Ywt || !Xq || !Wq || !scale_w) goto done;

    /* A: Haar transform of every channel, all levels */
    rc = orc_haar_fwd_f32(x, N, Cin, H, W, levels, coef);
    if (rc) goto done;
    /* B: feature norms across channels, then the k positions of largest norm per image */
    orc_norms_f32(coef, N, Cin, P, nrm2);
    if (idx_in) memcpy(idx, idx_in, sizeof(int32_t) * nk);
    else { rc = orc_select_topk_f32(nrm2, N, P, k, idx, NULL); if (rc) goto done; }
    /* gather the kept columns: X[I] */
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < k; ++j)
            for (int c = 0; c < Cin; ++c)
                Xc[((size_t)n * k + j) * Cin + c] = coef[((size_t)n * Cin + c) * P + idx[(size_t)n * k + j]];

    /* C: the 1x1 convolution on the compressed columns */
    if (bits > 0) {
        const float scale_a = (alpha > 0.0f) ? orc_quantize_alpha(Xc, (long)(nk * Cin), bits, alpha, Xq)
                                             : orc_quantize(Xc, (long)(nk * Cin), bits, Xq);   /* one alpha for the layer */
        orc_quantize_weights(Wt, Cout, Cin, wbits, Wq, scale_w);
#pragma omp parallel for schedule(static)
        for (long r = 0; r < (long)nk; ++r)
            for (int o = 0; o < Cout; ++o) {
                int32_t acc = 0;
                for (int c = 0; c < Cin; ++c)
                    acc += (int32_t)Wq[(size_t)o * Cin + c] * (int32_t)Xq[(size_t)r * Cin + c];
                if (acc_tap) acc_tap[(size_t)r * Cout + o] = acc;
                Yc[(size_t)r * Cout + o] = (float)acc * (scale_a * scale_w[o]);
            }
        if (scale_a_tap) *scale_a_tap = scale_a;
        if (Xq_tap) memcpy(Xq_tap, Xq, nk * Cin);
        if (Wq_tap) memcpy(Wq_tap, Wq, (size_t)Cout * Cin);
        if (scale_w_tap) memcpy(scale_w_tap, scale_w, sizeof(float) * Cout);
    } else {
#pragma omp parallel for schedule(static)
        for (long r = 0; r < (long)nk; ++r)
            for (int o = 0; o < Cout; ++o) {
                double acc = 0.0;
                for (int c = 0; c < Cin; ++c)
                    acc += (double)Wt[(size_t)o * Cin + c] * (double)Xc[(size_t)r * Cin + c];
                Yc[(size_t)r * Cout + o] = (float)acc;
            }
    }

    /* D: zero map, Y[I] = Y_wt */
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < k; ++j)
            for (int o = 0; o < Cout; ++o)
                Ywt[((size_t)n * Cout + o) * P + idx[(size_t)n * k + j]] = Yc[((size_t)n * k + j) * Cout + o];
    /* E: inverse Haar transform */
    rc = orc_haar_inv_f32(Ywt, N, Cout, H, W, levels, y);
    if (rc) goto done;
    if (residual)
        for (size_t i = 0; i < (size_t)N * Cout * P; ++i) y[i] = y[i] + residual[i];
    if (relu)
        for (size_t i = 0; i < (size_t)N * Cout * P; ++i) y[i] = (y[i] > 0.0f) ? y[i] : 0.0f;
    if (out_bf16) orc_round_bf16(y, (long)N * Cout * P, y);

    if (coef_tap) memcpy(coef_tap, coef, sizeof(float) * (size_t)N * Cin * P);
    if (nrm2_tap) memcpy(nrm2_tap, nrm2, sizeof(float) * (size_t)N * P);
    if (idx_tap) memcpy(idx_tap, idx, sizeof(int32_t) * nk);
    rc = 0;
done:
    free(coef); free(nrm2); free(idx); free(Xc); free(Yc); free(Ywt); free(Xq); free(Wq); free(scale_w);
    return rc;
}

/* The same layer without quantization, entirely in double: used by the invariant tests. */
int orc_forward_f64(const double *x, const double *Wt, int N, int Cin, int Cout, int H, int W,
                    int levels, int k, const int32_t *idx_in, double *y, double *nrm2_tap, int32_t *idx_tap)
{
    const long P = (long)H * W;
    if (k < 1 || k > P) return -1;
    const size_t nk = (size_t)N * k;
    double *coef = (double *)malloc(sizeof(double) * (size_t)N * Cin * P);
    double *nrm2 = (double *)malloc(sizeof(double) * (size_t)N * P);
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * nk);
    double *Ywt = (double *)calloc((size_t)N * Cout * P, sizeof(double));
    int rc = -2;
    if (!coef || !nrm2 || !idx || !Ywt) goto done;
    rc = orc_haar_fwd_f64(x, N, Cin, H, W, levels, coef);
    if (rc) goto done;
    orc_norms_f64(coef, N, Cin, P, nrm2);
    if (idx_in) memcpy(idx, idx_in, sizeof(int32_t) * nk);
    else { rc = orc_select_topk_f64(nrm2, N, P, k, idx, NULL); if (rc) goto done; }
    for (long n = 0; n < N; ++n)
        for (long j = 0; j < k; ++j) {
            const long p = idx[(size_t)n * k + j];
            for (int o = 0; o < Cout; ++o) {
                double acc = 0.0;
                for (int c = 0; c < Cin; ++c)
                    acc += Wt[(size_t)o * Cin + c] * coef[((size_t)n * Cin + c) * P + p];
                Ywt[((size_t)n * Cout + o) * P + p] = acc;
            }
        }
    rc = orc_haar_inv_f64(Ywt, N, Cout, H, W, levels, y);
    if (rc) goto done;
    if (nrm2_tap) memcpy(nrm2_tap, nrm2, sizeof(double) * (size_t)N * P);
    if (idx_tap) memcpy(idx_tap, idx, sizeof(int32_t) * nk);
    rc = 0;
done:
    free(coef); free(nrm2); free(idx); free(Ywt);
    return rc;
}

/*
 * Depthwise 3x3 convolution (the K_dw of the inverted residual block, Eq. 13): every channel on its own, stride 1,
 * zero padding 1, no bias, cross-correlation.  w is [C][3][3].  fp32, one fused multiply-add per tap in row-major tap
 * order starting from +0; taps that fall outside the map contribute nothing.
 */
void orc_dwconv3x3_f32(const float *x, const float *w, int N, int C, int H, int W, float *y)
{
#pragma omp parallel for schedule(static)
    for (long pl = 0; pl < (long)N * C; ++pl) {
        const float *xp = x + (size_t)pl * H * W;
        const float *wp = w + (size_t)(pl % C) * 9;
        float *yp = y + (size_t)pl * H * W;
        for (int r = 0; r < H; ++r)
            for (int c = 0; c < W; ++c) {
                float acc = 0.0f;
                for (int i = 0; i < 3; ++i)
                    for (int j = 0; j < 3; ++j) {
                        const int rr = r + i - 1, cc = c + j - 1;
                        if (rr >= 0 && rr < H && cc >= 0 && cc < W) acc = fmaf(wp[i * 3 + j], xp[(size_t)rr * W + cc], acc);
                    }
                yp[(size_t)r * W + c] = acc;
            }
    }
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

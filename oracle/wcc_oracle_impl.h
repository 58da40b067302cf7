/*
 * CPU oracle for the Wavelet Compressed Convolution (WCC) layer -- TEST INFRASTRUCTURE ONLY.
 *
 * This file is included twice by wcc_oracle.c, once with REAL = float (the
 * precision the layer is defined in here) and once with REAL = double (used by
 * the invariant tests).  It is a plain, slow, loop-by-loop restatement of the
 * paper's definitions: one rounding per written operation, no blocking, no
 * fusion, no reordering.  It shares no code with the CUDA path.
 *
 * Required macros: REAL, SUF(name) (appends _f32 / _f64), FMA(a,b,c).
 */

/* ---------------------------------------------------------------------------
 * One level of the 2-D Haar transform (Eq. 3) on the top-left hc x wc corner of
 * an H x W plane.  The four 2x2 kernels of Eq. 3 are applied as a stride-2
 * cross-correlation:
 *     y1 = (a+b+c+d)/2   y2 = (a-b+c-d)/2   y3 = (a+b-c-d)/2   y4 = (a-b-c+d)/2
 * with a=x[2i][2j], b=x[2i][2j+1], c=x[2i+1][2j], d=x[2i+1][2j+1], evaluated
 * horizontally first (s0=a+b, d0=a-b, s1=c+d, d1=c-d) and then vertically.
 * The sub-bands are written as the four quadrants of the same corner
 * (y1 top-left, y2 top-right, y3 bottom-left, y4 bottom-right).
 * ------------------------------------------------------------------------- */
static void SUF(haar_level_fwd)(const REAL *src, REAL *dst, int W, int hc, int wc)
{
    const int h = hc / 2, w = wc / 2;
    const REAL half = (REAL)0.5;
    for (int i = 0; i < h; ++i) {
        for (int j = 0; j < w; ++j) {
            const REAL a = src[(size_t)(2 * i) * W + 2 * j];
            const REAL b = src[(size_t)(2 * i) * W + 2 * j + 1];
            const REAL c = src[(size_t)(2 * i + 1) * W + 2 * j];
            const REAL d = src[(size_t)(2 * i + 1) * W + 2 * j + 1];
            const REAL s0 = a + b, d0 = a - b, s1 = c + d, d1 = c - d;
            dst[(size_t)i * W + j]           = (s0 + s1) * half;   /* y1 */
            dst[(size_t)i * W + j + w]       = (d0 + d1) * half;   /* y2 */
            dst[(size_t)(i + h) * W + j]     = (s0 - s1) * half;   /* y3 */
            dst[(size_t)(i + h) * W + j + w] = (d0 - d1) * half;   /* y4 */
        }
    }
}

/* Transposed convolution with the same kernels (Eq. 4): the exact inverse of the level above. */
static void SUF(haar_level_inv)(const REAL *src, REAL *dst, int W, int hc, int wc)
{
    const int h = hc / 2, w = wc / 2;
    const REAL half = (REAL)0.5;
    for (int i = 0; i < h; ++i) {
        for (int j = 0; j < w; ++j) {
            const REAL y1 = src[(size_t)i * W + j];
            const REAL y2 = src[(size_t)i * W + j + w];
            const REAL y3 = src[(size_t)(i + h) * W + j];
            const REAL y4 = src[(size_t)(i + h) * W + j + w];
            const REAL t0 = y1 + y3, t1 = y1 - y3, u0 = y2 + y4, u1 = y2 - y4;
            dst[(size_t)(2 * i) * W + 2 * j]         = (t0 + u0) * half;   /* a */
            dst[(size_t)(2 * i) * W + 2 * j + 1]     = (t0 - u0) * half;   /* b */
            dst[(size_t)(2 * i + 1) * W + 2 * j]     = (t1 + u1) * half;   /* c */
            dst[(size_t)(2 * i + 1) * W + 2 * j + 1] = (t1 - u1) * half;   /* d */
        }
    }
}

/* Multi-level transform of one plane (Eq. 5-6): level l works on the low-pass corner left by level l-1. */
static void SUF(haar_plane_fwd)(const REAL *x, REAL *coef, REAL *scratch, int H, int W, int levels)
{
    memcpy(coef, x, sizeof(REAL) * (size_t)H * W);
    for (int l = 1; l <= levels; ++l) {
        const int hc = H >> (l - 1), wc = W >> (l - 1);
        for (int r = 0; r < hc; ++r)
            memcpy(scratch + (size_t)r * W, coef + (size_t)r * W, sizeof(REAL) * (size_t)wc);
        SUF(haar_level_fwd)(scratch, coef, W, hc, wc);
    }
}

/* Inverse: the transposed operations in the opposite order (coarsest level first). */
static void SUF(haar_plane_inv)(const REAL *coef, REAL *x, REAL *scratch, int H, int W, int levels)
{
    memcpy(x, coef, sizeof(REAL) * (size_t)H * W);
    for (int l = levels; l >= 1; --l) {
        const int hc = H >> (l - 1), wc = W >> (l - 1);
        for (int r = 0; r < hc; ++r)
            memcpy(scratch + (size_t)r * W, x + (size_t)r * W, sizeof(REAL) * (size_t)wc);
        SUF(haar_level_inv)(scratch, x, W, hc, wc);
    }
}

/* x[N][C][H][W] -> coef[N][C][H][W], every plane on its own.  Returns 0, or -1 on a bad shape. */
int SUF(orc_haar_fwd)(const REAL *x, int N, int C, int H, int W, int levels, REAL *coef)
{
    if (levels < 1 || H <= 0 || W <= 0 || (H % (1 << levels)) || (W % (1 << levels))) return -1;
    const long planes = (long)N * C;
    const size_t P = (size_t)H * W;
    int bad = 0;
#pragma omp parallel
    {
        REAL *scratch = (REAL *)malloc(sizeof(REAL) * P);
        if (!scratch) {
#pragma omp atomic write
            bad = 1;
        }
#pragma omp for schedule(static)
        for (long p = 0; p < planes; ++p)
            if (scratch) SUF(haar_plane_fwd)(x + (size_t)p * P, coef + (size_t)p * P, scratch, H, W, levels);
        free(scratch);
    }
    return bad ? -2 : 0;
}

int SUF(orc_haar_inv)(const REAL *coef, int N, int C, int H, int W, int levels, REAL *x)
{
    if (levels < 1 || H <= 0 || W <= 0 || (H % (1 << levels)) || (W % (1 << levels))) return -1;
    const long planes = (long)N * C;
    const size_t P = (size_t)H * W;
    int bad = 0;
#pragma omp parallel
    {
        REAL *scratch = (REAL *)malloc(sizeof(REAL) * P);
        if (!scratch) {
#pragma omp atomic write
            bad = 1;
        }
#pragma omp for schedule(static)
        for (long p = 0; p < planes; ++p)
            if (scratch) SUF(haar_plane_inv)(coef + (size_t)p * P, x + (size_t)p * P, scratch, H, W, levels);
        free(scratch);
    }
    return bad ? -2 : 0;
}

/* ---------------------------------------------------------------------------
 * Other wavelets (App. F compares Haar with db2, db3, coif1, bior1.3, bior2.2, sym4: filters of 4 to 8 taps).
 * A two-channel filter bank with T taps per filter (T even), periodic extension, so that an n-sample signal gives
 * n/2 + n/2 coefficients and the transformed map has the size of the input (what the in-place compression needs;
 * the paper does not name the extension).  One 2-D level on the hc x wc corner, as a stride-2 cross-correlation with
 * the outer products of the 1-D decomposition filters, origin c0 = T/2 - 1:
 *     band[i][j] = sum_{tr, tc} f_row[tr] * f_col[tc] * x[(2i + tr - c0) mod hc][(2j + tc - c0) mod wc]
 * y1 = (lo, lo), y2 = (lo along the height, hi along the width), y3 = (hi, lo), y4 = (hi, hi); same quadrant
 * placement as the Haar level above.  w2 holds the four T x T tap products, rounded once to REAL; one fused
 * multiply-add per tap, row-major tap order, from +0.  With lo = [1, 1]/sqrt 2, hi = [1, -1]/sqrt 2 this is Eq. 3.
 * ------------------------------------------------------------------------- */
static void SUF(dwt_level_fwd)(const REAL *src, REAL *dst, int W, int hc, int wc, const REAL *w2, int T)
{
    const int h = hc / 2, w = wc / 2, c0 = T / 2 - 1;
    for (int i = 0; i < h; ++i)
        for (int j = 0; j < w; ++j)
            for (int b = 0; b < 4; ++b) {
                REAL acc = (REAL)0;
                for (int tr = 0; tr < T; ++tr) {
                    const int rr = ((2 * i + tr - c0) % hc + hc) % hc;
                    for (int tc = 0; tc < T; ++tc) {
                        const int cc = ((2 * j + tc - c0) % wc + wc) % wc;
                        acc = FMA(w2[(b * T + tr) * T + tc], src[(size_t)rr * W + cc], acc);
                    }
                }
                dst[(size_t)(i + (b >> 1) * h) * W + j + (b & 1) * w] = acc;
            }
}

/* The synthesis step: the adjoint structure with the reconstruction filters (for an orthogonal wavelet they are the
 * decomposition filters and this is the transpose, Eq. 4):
 *     x[r][c] = sum over bands b, taps (tr, tc) with (r - tr + c0) mod hc and (c - tc + c0) mod wc both even
 *               of g_row[tr] * g_col[tc] * band_b[((r - tr + c0) mod hc) / 2][((c - tc + c0) mod wc) / 2]
 * summed in the order tr, tc, b, one fused multiply-add each, from +0. */
static void SUF(dwt_level_inv)(const REAL *src, REAL *dst, int W, int hc, int wc, const REAL *v2, int T)
{
    const int h = hc / 2, w = wc / 2, c0 = T / 2 - 1;
    for (int r = 0; r < hc; ++r)
        for (int c = 0; c < wc; ++c) {
            REAL acc = (REAL)0;
            for (int tr = 0; tr < T; ++tr) {
                const int mr = ((r - tr + c0) % hc + hc) % hc;
                if (mr & 1) continue;
                for (int tc = 0; tc < T; ++tc) {
                    const int mc = ((c - tc + c0) % wc + wc) % wc;
                    if (mc & 1) continue;
                    const int i = mr / 2, j = mc / 2;
                    for (int b = 0; b < 4; ++b)
                        acc = FMA(v2[(b * T + tr) * T + tc], src[(size_t)(i + (b >> 1) * h) * W + j + (b & 1) * w], acc);
                }
            }
            dst[(size_t)r * W + c] = acc;
        }
}

/* The four T x T tap products of a filter pair: [0] lo x lo, [1] lo (rows) x hi (columns), [2] hi x lo, [3] hi x hi. */
static void SUF(tap_products)(const REAL *lo, const REAL *hi, int T, REAL *out)
{
    for (int b = 0; b < 4; ++b)
        for (int tr = 0; tr < T; ++tr)
            for (int tc = 0; tc < T; ++tc)
                out[(b * T + tr) * T + tc] = ((b >> 1) ? hi[tr] : lo[tr]) * ((b & 1) ? hi[tc] : lo[tc]);
}

/* Multi-level transform of every plane with a given filter pair (taps T <= 16, even); dir = 0 forward (decomposition
 * filters), 1 inverse (reconstruction filters).  Returns 0, -1 on a bad shape. */
int SUF(orc_dwt)(const REAL *in, int N, int C, int H, int W, int levels, const REAL *lo, const REAL *hi, int T, int dir, REAL *out)
{
    if (levels < 1 || T < 2 || T > 16 || (T & 1) || H <= 0 || W <= 0 || (H % (1 << levels)) || (W % (1 << levels))) return -1;
    const long planes = (long)N * C;
    const size_t P = (size_t)H * W;
    REAL w2[4 * 16 * 16];
    SUF(tap_products)(lo, hi, T, w2);
    int bad = 0;
#pragma omp parallel
    {
        REAL *scratch = (REAL *)malloc(sizeof(REAL) * P);
        if (!scratch) {
#pragma omp atomic write
            bad = 1;
        }
#pragma omp for schedule(static)
        for (long p = 0; p < planes; ++p) {
            if (!scratch) continue;
            REAL *o = out + (size_t)p * P;
            memcpy(o, in + (size_t)p * P, sizeof(REAL) * P);
            for (int step = 0; step < levels; ++step) {
                const int l = dir ? levels - step : step + 1;
                const int hc = H >> (l - 1), wc = W >> (l - 1);
                for (int r = 0; r < hc; ++r) memcpy(scratch + (size_t)r * W, o + (size_t)r * W, sizeof(REAL) * (size_t)wc);
                if (dir) SUF(dwt_level_inv)(scratch, o, W, hc, wc, w2, T);
                else SUF(dwt_level_fwd)(scratch, o, W, hc, wc, w2, T);
            }
        }
        free(scratch);
    }
    return bad ? -2 : 0;
}

/*
 * Re-read one transformed plane (quadrant layout) as the concatenated vector of Eq. 6:
 * [y1^L, y2^L, y3^L, y4^L, y2^(L-1), y3^(L-1), y4^(L-1), ..., y2^1, y3^1, y4^1],
 * each sub-band row-major.
 */
void SUF(orc_concat_order)(const REAL *coef, int H, int W, int levels, REAL *vec)
{
    size_t o = 0;
    {
        const int h = H >> levels, w = W >> levels;
        for (int i = 0; i < h; ++i)
            for (int j = 0; j < w; ++j) vec[o++] = coef[(size_t)i * W + j];
    }
    for (int l = levels; l >= 1; --l) {
        const int h = H >> l, w = W >> l;
        for (int i = 0; i < h; ++i)
            for (int j = 0; j < w; ++j) vec[o++] = coef[(size_t)i * W + j + w];         /* y2^l */
        for (int i = 0; i < h; ++i)
            for (int j = 0; j < w; ++j) vec[o++] = coef[(size_t)(i + h) * W + j];       /* y3^l */
        for (int i = 0; i < h; ++i)
            for (int j = 0; j < w; ++j) vec[o++] = coef[(size_t)(i + h) * W + j + w];   /* y4^l */
    }
}

/*
 * Feature norm across channels at every wavelet-domain position (Alg. 1, norm step): the squared l2 norm, accumulated as one fused
 * multiply-add per channel in ascending channel order starting from +0.
 * Ranking by the squared norm equals ranking by the norm.
 */
void SUF(orc_norms)(const REAL *coef, int N, int C, long P, REAL *nrm2)
{
#pragma omp parallel for schedule(static)
    for (long n = 0; n < N; ++n)
        for (long p = 0; p < P; ++p) {
            REAL acc = (REAL)0;
            for (int c = 0; c < C; ++c) {
                const REAL v = coef[((size_t)n * C + c) * P + p];
                acc = FMA(v, v, acc);
            }
            nrm2[(size_t)n * P + p] = acc;
        }
}

/*
 * Joint shrinkage T (Eq. 7 with the joint rule of Sec. 4; Alg. 1, index-set step with
 * k = ceil(gamma n_w n_h)): for every image, order the positions by (norm descending, position
 * ascending), keep the first k, and report them in ascending position.  tau[n] is the
 * k-th largest norm.  A full sort: nothing clever.
 */
typedef struct { REAL v; int p; } SUF(keyed);

static int SUF(cmp_desc)(const void *A, const void *B)
{
    const SUF(keyed) *a = (const SUF(keyed) *)A, *b = (const SUF(keyed) *)B;
    if (a->v > b->v) return -1;
    if (a->v < b->v) return 1;
    return (a->p > b->p) - (a->p < b->p);
}

static int cmp_int_asc(const void *A, const void *B);

int SUF(orc_select_topk)(const REAL *nrm2, int N, long P, int k, int32_t *idx, REAL *tau)
{
    if (k < 1 || k > P) return -1;
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (long n = 0; n < N; ++n) {
        SUF(keyed) *a = (SUF(keyed) *)malloc(sizeof(SUF(keyed)) * (size_t)P);
        if (!a) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        for (long p = 0; p < P; ++p) { a[p].v = nrm2[(size_t)n * P + p]; a[p].p = (int)p; }
        qsort(a, (size_t)P, sizeof(SUF(keyed)), SUF(cmp_desc));
        for (int j = 0; j < k; ++j) idx[(size_t)n * k + j] = a[j].p;
        if (tau) tau[n] = a[k - 1].v;
        qsort(idx + (size_t)n * k, (size_t)k, sizeof(int32_t), cmp_int_asc);
        free(a);
    }
    return bad ? -2 : 0;
}

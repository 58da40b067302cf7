// WCC with other wavelets than Haar (App. F: db2, db3, coif1, bior1.3, bior2.2, sym4 -- filters of 4 to 8 taps): a
// generic two-channel filter bank with periodic extension, one launch per level.  These kernels are plain (one thread
// per output, every tap a global load through L1/L2): the longer filters are the paper's ablation, not its hot path.
//
// One 2-D level on the hc x wc low-pass corner of every plane, as a stride-2 cross-correlation with the outer products
// of the 1-D filters, origin c0 = T/2 - 1:
//     band[i][j] = sum_{tr, tc} f_row[tr] * f_col[tc] * x[(2i + tr - c0) mod hc][(2j + tc - c0) mod wc]
// y1 = (lo, lo) top-left, y2 = (lo along the height, hi along the width) top-right, y3 = (hi, lo) bottom-left, y4 =
// (hi, hi) bottom-right: the quadrant layout of the Haar kernels.  The synthesis is the adjoint structure with the
// reconstruction filters.  fp32, one fused multiply-add per tap in a fixed order (row-major taps; synthesis: taps, then
// bands), tap products rounded once: the same arithmetic as the plain CPU statement, so coefficients are bit-identical.
#pragma once

#include "common.cuh"

namespace wcc {
namespace wv {

constexpr int MAX_TAPS = 8;

struct TapProducts {
    float w[4 * MAX_TAPS * MAX_TAPS];   // [band][tr][tc], stride T
    int T;
};

inline TapProducts tap_products(const float* lo, const float* hi, int T)
{
    TapProducts tp = {};
    tp.T = T;
    for (int b = 0; b < 4; ++b)
        for (int tr = 0; tr < T; ++tr)
            for (int tc = 0; tc < T; ++tc) {
                volatile float p = ((b >> 1) ? hi[tr] : lo[tr]) * ((b & 1) ? hi[tc] : lo[tc]);     // one fp32 rounding
                tp.w[(b * T + tr) * T + tc] = p;
            }
    return tp;
}

__device__ __forceinline__ float load_as_float(const float* p) { return *p; }
__device__ __forceinline__ float load_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store_from_float(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_from_float(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// src: planes of pitch W holding the hc x wc corner to transform (a copy: dst's corner is overwritten); dst: fp32.
template <typename TI>
__global__ void __launch_bounds__(256)
dwt_level_fwd_kernel(const TI* __restrict__ src, float* __restrict__ dst, long long planes, int H, int W, int hc, int wc,
                     const TapProducts tp)
{
    const int h = hc >> 1, w = wc >> 1, T = tp.T, c0 = T / 2 - 1;
    const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= planes * h * w) return;
    const int j = (int)(id % w);
    const long long t = id / w;
    const int i = (int)(t % h);
    const long long pl = t / h;
    const TI* s = src + (size_t)pl * H * W;
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int tr = 0; tr < T; ++tr) {
        const int rr = ((2 * i + tr - c0) % hc + hc) % hc;
        for (int tc = 0; tc < T; ++tc) {
            const int cc = ((2 * j + tc - c0) % wc + wc) % wc;
            const float v = load_as_float(s + (size_t)rr * W + cc);
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[b] = __fmaf_rn(tp.w[(b * T + tr) * T + tc], v, acc[b]);
        }
    }
    float* d = dst + (size_t)pl * H * W;
#pragma unroll
    for (int b = 0; b < 4; ++b) d[(size_t)(i + (b >> 1) * h) * W + j + (b & 1) * w] = acc[b];
}

// src: planes of pitch W holding the four quadrants of the hc x wc corner (a copy); dst: the reconstructed corner.
template <typename TO>
__global__ void __launch_bounds__(256)
dwt_level_inv_kernel(const float* __restrict__ src, TO* __restrict__ dst, long long planes, int H, int W, int hc, int wc,
                     const TapProducts tp)
{
    const int h = hc >> 1, w = wc >> 1, T = tp.T, c0 = T / 2 - 1;
    const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= planes * hc * wc) return;
    const int c = (int)(id % wc);
    const long long t = id / wc;
    const int r = (int)(t % hc);
    const long long pl = t / hc;
    const float* s = src + (size_t)pl * H * W;
    float acc = 0.0f;
    for (int tr = 0; tr < T; ++tr) {
        const int mr = ((r - tr + c0) % hc + hc) % hc;
        if (mr & 1) continue;
        for (int tc = 0; tc < T; ++tc) {
            const int mc = ((c - tc + c0) % wc + wc) % wc;
            if (mc & 1) continue;
            const int i = mr >> 1, j = mc >> 1;
#pragma unroll
            for (int b = 0; b < 4; ++b)
                acc = __fmaf_rn(tp.w[(b * T + tr) * T + tc], s[(size_t)(i + (b >> 1) * h) * W + j + (b & 1) * w], acc);
        }
    }
    store_from_float(dst + (size_t)pl * H * W + (size_t)r * W + c, acc);
}

// Dequantize the accumulators of the kept positions into the (zeroed) wavelet-domain output map:
// Ywt[n][o][idx[n][j]] = float(acc[n*k + j][o]) * (scale_a * scale_w[o])   (or the fp32 products when ACCF).
template <bool ACCF>
__global__ void __launch_bounds__(256)
scatter_coef_kernel(const int32_t* __restrict__ acc, int ldc, const int32_t* __restrict__ idx, const float* __restrict__ amax_kept,
                    float qmax, const float* __restrict__ scale_w, int N, int Cout, long long P, int k, float* __restrict__ Ywt)
{
    const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;          // one thread per (row, output channel)
    if (id >= (long long)N * k * Cout) return;
    const int o = (int)(id % Cout);
    const long long row = id / Cout;
    const long long n = row / k;
    const int p = idx[row];
    const int32_t a = acc[row * ldc + o];
    float v;
    if (ACCF) v = __int_as_float(a);
    else v = __fmul_rn((float)a, __fmul_rn(__fdiv_rn(*amax_kept, qmax), scale_w[o]));
    Ywt[((size_t)n * Cout + o) * P + p] = v;
}

// Copy the left `wc` columns of every row of every plane (pitch W): the corner a level is about to overwrite.
static wcc_status copy_corner(const float* src, float* dst, long long planes, int H, int W, int wc, cudaStream_t st)
{
    WCC_CUDA_TRY(cudaMemcpy2DAsync(dst, (size_t)W * 4, src, (size_t)W * 4, (size_t)wc * 4, (size_t)planes * H,
                                   cudaMemcpyDeviceToDevice, st));
    return WCC_OK;
}

}  // namespace wv

// x [planes][H][W] of dt -> coef fp32 (quadrant layout); scratch: fp32 [planes][H][W].
static wcc_status launch_dwt_fwd(const void* x, long long planes, int H, int W, int L, wcc_dtype dt, const wv::TapProducts& tp,
                                 float* coef, float* scratch, cudaStream_t st)
{
    for (int l = 1; l <= L; ++l) {
        const int hc = H >> (l - 1), wc = W >> (l - 1);
        const long long outs = planes * (hc / 2) * (wc / 2);
        const unsigned blocks = (unsigned)((outs + 255) / 256);
        if (l == 1) {
            if (dt == WCC_BF16)
                wv::dwt_level_fwd_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), coef, planes, H, W, hc, wc, tp);
            else
                wv::dwt_level_fwd_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(x), coef, planes, H, W, hc, wc, tp);
        } else {
            wcc_status s = wv::copy_corner(coef, scratch, planes, H, W, wc, st);
            if (s != WCC_OK) return s;
            wv::dwt_level_fwd_kernel<float><<<blocks, 256, 0, st>>>(scratch, coef, planes, H, W, hc, wc, tp);
        }
        WCC_LAUNCH_CHECK();
    }
    return WCC_OK;
}

// work fp32 [planes][H][W] holds the coefficients and is overwritten; out [planes][H][W] of dt; scratch as above.
static wcc_status launch_dwt_inv(float* work, long long planes, int H, int W, int L, wcc_dtype dt, const wv::TapProducts& tp,
                                 void* out, float* scratch, cudaStream_t st)
{
    for (int l = L; l >= 1; --l) {
        const int hc = H >> (l - 1), wc = W >> (l - 1);
        const long long outs = planes * hc * wc;
        const unsigned blocks = (unsigned)((outs + 255) / 256);
        wcc_status s = wv::copy_corner(work, scratch, planes, H, W, wc, st);
        if (s != WCC_OK) return s;
        if (l > 1)
            wv::dwt_level_inv_kernel<float><<<blocks, 256, 0, st>>>(scratch, work, planes, H, W, hc, wc, tp);
        else if (dt == WCC_BF16)
            wv::dwt_level_inv_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(scratch, static_cast<__nv_bfloat16*>(out), planes, H, W, hc, wc, tp);
        else
            wv::dwt_level_inv_kernel<float><<<blocks, 256, 0, st>>>(scratch, static_cast<float*>(out), planes, H, W, hc, wc, tp);
        WCC_LAUNCH_CHECK();
    }
    return WCC_OK;
}

}  // namespace wcc

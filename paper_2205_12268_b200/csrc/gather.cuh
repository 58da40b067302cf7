// Quantization of the weights and gather + quantization of the kept wavelet-domain columns
// (signed symmetric scheme of Eq. 1-2 placed on the transformed activations and on the weights, Sec. 4).
#pragma once

#include "common.cuh"

namespace wcc {

__device__ __forceinline__ int quant_code(float v, float inv, float qmax)
{
    float r = rintf(__fmul_rn(v, inv));          // round to nearest, ties to even
    r = fminf(fmaxf(r, -qmax), qmax);
    return (int)r;
}

// One warp per output channel o.  bits >= 2: Wq int8 [Cout][kpad] (zero padded) and scale_w[o] = max|w| / qmax.
// bits == 0: bf16 copy of the row, zero padded.
__device__ __forceinline__ void weight_prep_row(const float* __restrict__ Wt, int o, int Cin, int kpad, int bits,
                                                void* __restrict__ Wq, float* __restrict__ scale_w)
{
    const int lane = threadIdx.x & 31;
    const float* w = Wt + (size_t)o * Cin;
    if (bits == 0) {
        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(Wq) + (size_t)o * kpad;
        for (int c = lane; c < kpad; c += 32) dst[c] = __float2bfloat16_rn(c < Cin ? w[c] : 0.0f);
        return;
    }
    float m = 0.0f;
    for (int c = lane; c < Cin; c += 32) m = fmaxf(m, fabsf(w[c]));
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
    const float qmax = (float)((1 << (bits - 1)) - 1);
    const float inv = (m > 0.0f) ? __fdiv_rn(qmax, m) : 0.0f;
    int8_t* dst = static_cast<int8_t*>(Wq) + (size_t)o * kpad;
    for (int c = lane; c < kpad; c += 32) dst[c] = (c < Cin) ? (int8_t)quant_code(w[c], inv, qmax) : (int8_t)0;
    if (lane == 0) scale_w[o] = __fdiv_rn(m, qmax);
}

__global__ void __launch_bounds__(128)
weight_prep_kernel(const float* __restrict__ Wt, int Cout, int Cin, int kpad, int bits,
                   void* __restrict__ Wq, float* __restrict__ scale_w)
{
    const int o = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (o < Cout) weight_prep_row(Wt, o, Cin, kpad, bits, Wq, scale_w);
}

// One thread per kept position (row r = n*k + j of the compressed matrix) and chunk of `cpc` channels (blockIdx.y; a
// multiple of 64): reads coef[n][c][idx[n][j]] for its channels and writes that part of one K-major row.  Consecutive
// rows are consecutive kept positions, so a warp's reads of one channel are contiguous wherever the kept set is dense
// (the low-pass corner) and sector-sparse elsewhere.
template <bool QUANT>
__global__ void __launch_bounds__(128)
gather_quant_kernel(const float* __restrict__ coef, const int32_t* __restrict__ idx, const float* __restrict__ amax_kept,
                    int M, int Cin, int P, int k, int kpad, int cpc, float qmax, void* __restrict__ Xq)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= M) return;
    const int n = r / k;
    const int p = idx[r];
    const float* src = coef + (size_t)n * Cin * P + p;
    float inv = 0.0f;
    if (QUANT) {
        const float amax = *amax_kept;
        inv = (amax > 0.0f) ? __fdiv_rn(qmax, amax) : 0.0f;
    }
    constexpr int CH = QUANT ? 16 : 8;      // channels per 16-byte store
    uint4* dst = reinterpret_cast<uint4*>(static_cast<char*>(Xq) + (size_t)r * kpad * (QUANT ? 1 : 2));
    const int c_lo = (int)blockIdx.y * cpc, c_hi = min(kpad, c_lo + cpc);
    for (int c0 = c_lo; c0 < c_hi; c0 += CH) {
        float v[CH];
#pragma unroll
        for (int i = 0; i < CH; ++i) v[i] = (c0 + i < Cin) ? src[(size_t)(c0 + i) * P] : 0.0f;
        uint32_t w[4];
        if (QUANT) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t b0 = (uint32_t)quant_code(v[4 * i + 0], inv, qmax) & 0xFFu;
                const uint32_t b1 = (uint32_t)quant_code(v[4 * i + 1], inv, qmax) & 0xFFu;
                const uint32_t b2 = (uint32_t)quant_code(v[4 * i + 2], inv, qmax) & 0xFFu;
                const uint32_t b3 = (uint32_t)quant_code(v[4 * i + 3], inv, qmax) & 0xFFu;
                w[i] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = pack_bf16x2(v[2 * i], v[2 * i + 1]);
        }
        dst[c0 / CH] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

wcc_status launch_weight_prep(const float* Wt, int Cout, int Cin, int kpad, int bits,
                              void* Wq, float* scale_w, cudaStream_t st)
{
    weight_prep_kernel<<<ceil_div(Cout, 4), 128, 0, st>>>(Wt, Cout, Cin, kpad, bits, Wq, scale_w);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

wcc_status launch_gather_quant(const float* coef, const int32_t* idx, const float* amax_kept,
                               int N, int Cin, int P, int k, int kpad, int bits, void* Xq, cudaStream_t st)
{
    const int M = N * k;
    const float qmax = (bits >= 2) ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    // rows alone fill the GPU from about 150 K kept positions on; below that the channels are split as well
    const int cpc = (M >= 148 * 1024) ? kpad : 64;
    const dim3 grid(ceil_div(M, 128), ceil_div(kpad, cpc));
    if (bits >= 2)
        gather_quant_kernel<true><<<grid, 128, 0, st>>>(coef, idx, amax_kept, M, Cin, P, k, kpad, cpc, qmax, Xq);
    else
        gather_quant_kernel<false><<<grid, 128, 0, st>>>(coef, idx, amax_kept, M, Cin, P, k, kpad, cpc, qmax, Xq);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

}  // namespace wcc

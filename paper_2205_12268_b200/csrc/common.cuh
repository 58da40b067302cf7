// Shared declarations of the WCC CUDA library (sm_100a).  Internal: not part of the C ABI.
// The library is one translation unit (libwcc.cu includes every *.cuh), so device globals are defined here.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "wcc.h"

namespace wcc {

// Device status word: WCC_OK, or WCC_ERR_TIMEOUT once a bounded wait inside a kernel gave up.
__device__ int g_status = 0;

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

#define WCC_CUDA_TRY(expr)                         \
    do {                                           \
        cudaError_t e__ = (expr);                  \
        if (e__ != cudaSuccess) return WCC_ERR_CUDA; \
    } while (0)

// host-side count of kernel launches (reported by wcc_kernel_launches)
static unsigned long long g_launches = 0;

#define WCC_LAUNCH_CHECK()                                   \
    do {                                                     \
        ++g_launches;                                        \
        if (cudaPeekAtLastError() != cudaSuccess) {          \
            (void)cudaGetLastError();                        \
            return WCC_ERR_CUDA;                             \
        }                                                    \
    } while (0)

// ---- element access -------------------------------------------------------------------------
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Order-preserving map float -> uint32 (larger float = larger key); -0 is folded onto +0.
__device__ __forceinline__ uint32_t float_key(float v)
{
    uint32_t b = __float_as_uint(v);
    if ((b << 1) == 0u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// Digits of a norm for the histograms that the producers of the norms hand to the selection.  A norm is a sum of squares,
// never negative, so its sign bit carries nothing: the digits are the 11 and the 16 bits below it (digit16 >> 5 ==
// digit11).  The masks keep a non-finite value with a sign bit inside the tables.
__device__ __forceinline__ uint32_t norm_digit11(float v) { return (__float_as_uint(v) >> 20) & 0x7FFu; }
__device__ __forceinline__ uint32_t norm_digit16(float v) { return (__float_as_uint(v) >> 15) & 0xFFFFu; }

// Histogram increment with warp aggregation: lanes of a warp that hit the same bin elect one lane that adds their
// count, so a bin that attracts most keys (typical for the leading digit of the norms) costs one shared-memory
// atomic per warp instead of up to 32 serialized ones.  Must be reached by all 32 lanes (pred selects the ones that count).
__device__ __forceinline__ void hist_add(uint32_t* h, uint32_t bin, bool pred)
{
    const unsigned active = __ballot_sync(0xFFFFFFFFu, pred);
    if (pred) {
        const unsigned peers = __match_any_sync(active, bin);
        if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&h[bin], (uint32_t)__popc(peers));
    }
}

// ---- geometry of one call -------------------------------------------------------------------
struct Geom {
    int N, C, H, W, L;
    int P;          // H*W
};

// ---- stage launchers (each enqueues on `st`, returns a wcc_status) ---------------------------
// Forward Haar + norms (+ per-position max |coef| over channels when amaxpos != NULL).
wcc_status launch_haar_fwd(const void* x, int N, int C, int H, int W, int L, wcc_dtype dt,
                           float* coef, float* nrm2, float* amaxpos, cudaStream_t st);
// Plain inverse Haar.
wcc_status launch_haar_inv(const float* coef, int N, int C, int H, int W, int L, wcc_dtype dt,
                           void* out, cudaStream_t st);
// Dequantize + scatter into a zero map + inverse Haar.  acc rows have pitch ldc (int32 or fp32 bits).
wcc_status launch_scatter_inv(const int32_t* acc, int ldc, bool acc_is_float, const int32_t* rank,
                              const float* amax_kept, int bits, const float* scale_w,
                              int N, int Cout, int H, int W, int L, int k, wcc_dtype dt, void* y, cudaStream_t st,
                              const void* residual = nullptr, int relu = 0);

// Radix select + ordered compaction.  rank (int32 [N][P], -1 = dropped), amaxpos / amax_kept (max over the
// kept positions of amaxpos, as float bits, must be zeroed by this call) are optional.
size_t select_ws_bytes(int N, int P);
wcc_status launch_select(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau,
                         int32_t* rank, const float* amaxpos, bool want_amax,
                         void* ws, size_t ws_bytes, cudaStream_t st, bool hist1_ready = false,
                         const uint32_t* fine = nullptr, uint32_t* thr = nullptr, bool want_rank = true);

// Weight quantization (bits >= 2: int8 codes + per-row scale; bits == 0: bf16 copy), rows padded to kpad.
wcc_status launch_weight_prep(const float* Wt, int Cout, int Cin, int kpad, int bits,
                              void* Wq, float* scale_w, cudaStream_t st);
// Gather the kept columns and quantize them (bits >= 2) or round them to bf16 (bits == 0).
wcc_status launch_gather_quant(const float* coef, const int32_t* idx, const float* amax_kept,
                               int N, int Cin, int P, int k, int kpad, int bits, void* Xq, cudaStream_t st);

// Tensor-core contraction acc[M][ldc] = Xq[M][kpad] * Wq[Cout][kpad]^T.
wcc_status launch_contract(const void* Xq, const void* Wq, int M, int Cout, int kpad, int bits,
                           int32_t* acc, int ldc, cudaStream_t st);

}  // namespace wcc

// Gather + quantization of the kept columns straight from the input (no stored coefficient map): the path of layers
// whose channel counts exceed one operand tile of the fused kernels (Alg. 1, steps A-B of the kept columns only).
#pragma once

#include "common.cuh"
#include "gather.cuh"
#include "haar.cuh"

namespace wcc {

// The same rows without a stored coefficient map: one warp per (image, tile, chunk of 16 / 8 channels) transforms its
// channels of x again (as the first pass did) and writes, for every slot of the lane whose position is kept, that
// chunk of the position's row (rank[n][p] = row of position p inside image n, or -1).  Same codes as gather_quant_kernel.
template <typename T, int L, bool VEC, bool QUANT>
__global__ void __launch_bounds__(128)
regather_quant_kernel(const T* __restrict__ x, const int32_t* __restrict__ rank, const float* __restrict__ amax_kept,
                      int N, int C, int H, int W, int k, int kpad, float qmax, void* __restrict__ Xq)
{
    using TT = HaarTile<L>;
    constexpr int CH = QUANT ? 16 : 8;                 // channels per 16-byte store
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const int chunks = kpad / CH;
    const long long gw = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (gw >= (long long)N * tiles_x * tiles_y * chunks) return;
    const int lane = threadIdx.x & 31;
    const int chunk = (int)(gw % chunks);
    int n, ty, tx;
    tile_coords((int)(gw / chunks), tiles_x, tiles_y, n, ty, tx);
    const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
    const size_t P = (size_t)H * W;
    int rk[8];
    bool any = false;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        rk[s] = slot_ok<L>(lp, s) ? rank[(size_t)n * P + lp.pos[s]] : -1;
        any = any || rk[s] >= 0;
    }
    if (!__any_sync(0xFFFFFFFFu, any ? 1 : 0)) return;                // nothing kept in this tile
    float inv = 0.0f;
    if (QUANT) {
        const float amax = *amax_kept;
        inv = (amax > 0.0f) ? __fdiv_rn(qmax, amax) : 0.0f;
    }
    const T* xin = x + (size_t)n * C * P;
    uint32_t packed[8][4];
#pragma unroll
    for (int g = 0; g < CH / 4; ++g) {
        RawPatch raw[4];
#pragma unroll
        for (int d = 0; d < 4; ++d) {
            const int c = chunk * CH + g * 4 + d;
#pragma unroll
            for (int i = 0; i < 8; ++i) raw[d].w[i] = 0u;
            if (c < C) load_patch<T, VEC>(xin + (size_t)c * P, W, lp, raw[d]);       // channels of the padding are zero
        }
        float o[4][8];
#pragma unroll
        for (int d = 0; d < 4; ++d) {
            float p[2][4];
            unpack_patch<T>(raw[d], p);
            haar_fwd_lane<L>(p, o[d], lane);
        }
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            if (QUANT) {
                const uint32_t b0 = (uint32_t)quant_code(o[0][s], inv, qmax) & 0xFFu;
                const uint32_t b1 = (uint32_t)quant_code(o[1][s], inv, qmax) & 0xFFu;
                const uint32_t b2 = (uint32_t)quant_code(o[2][s], inv, qmax) & 0xFFu;
                const uint32_t b3 = (uint32_t)quant_code(o[3][s], inv, qmax) & 0xFFu;
                packed[s][g] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
            } else {
                packed[s][2 * g] = pack_bf16x2(o[0][s], o[1][s]);
                packed[s][2 * g + 1] = pack_bf16x2(o[2][s], o[3][s]);
            }
        }
    }
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        if (rk[s] >= 0) {
            char* row = static_cast<char*>(Xq) + ((size_t)n * k + rk[s]) * kpad * (QUANT ? 1 : 2);
            *reinterpret_cast<uint4*>(row + (size_t)chunk * 16) = make_uint4(packed[s][0], packed[s][1], packed[s][2], packed[s][3]);
        }
    }
}

template <typename T, int L, bool VEC>
static wcc_status regather_dispatch(const void* x, const int32_t* rank, const float* amax_kept, int N, int C, int H, int W,
                                    int k, int kpad, int bits, void* Xq, cudaStream_t st)
{
    using TT = HaarTile<L>;
    const float qmax = (bits >= 2) ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    const long long warps = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH) * (kpad / (bits >= 2 ? 16 : 8));
    if (warps > 0x7FFFFFFFLL * 4) return WCC_ERR_SHAPE;
    const unsigned blocks = (unsigned)((warps + 3) / 4);
    if (bits >= 2)
        regather_quant_kernel<T, L, VEC, true><<<blocks, 128, 0, st>>>(static_cast<const T*>(x), rank, amax_kept, N, C, H, W, k, kpad, qmax, Xq);
    else
        regather_quant_kernel<T, L, VEC, false><<<blocks, 128, 0, st>>>(static_cast<const T*>(x), rank, amax_kept, N, C, H, W, k, kpad, qmax, Xq);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

wcc_status launch_regather_quant(const void* x, const int32_t* rank, const float* amax_kept, int N, int C, int H, int W, int L,
                                 int k, int kpad, int bits, wcc_dtype dt, void* Xq, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;
    WCC_DISPATCH_TLV(regather_dispatch, dt, L, vec, x, rank, amax_kept, N, C, H, W, k, kpad, bits, Xq, st);
}

}  // namespace wcc

// Haar kernels: forward transform + channel norms, plain inverse, and the fused
// dequantize + scatter + inverse (steps A, B-norms, D, E of the WCC workflow; Eq. 3-6, Alg. 1).
//
// Work decomposition (all three kernels).  One warp owns a tile of 2^L rows x TW columns of one image,
// TW = 4 * CG, CG = 32 / 2^(L-1).  Lane (rp, cg) = (lane / CG, lane % CG) holds the 2 x 4 patch at rows
// 2rp, 2rp+1 and columns 4cg..4cg+3 of the tile: level 1 is computed inside the lane, level 2 pairs the
// lanes rp and rp^1 (lane ^ CG), level 3 combines the four lanes {rp, rp^2} x {cg, cg^1}.  After the
// transform every lane owns exactly eight wavelet-domain positions ("slots"):
//   0,1  y2 of level 1 (two quads)      2,3  y3 of level 1       4,5  y4 of level 1
//   6,7  L=1: y1 of level 1 (two quads)
//        L>=2, rp even: slot 6 = y2 of level 2, slot 7 = y1 of level 2 (L=2) or one of y1..y4 of level 3,
//                       by (rp & 2, cg & 1): (0,0) y1, (0,1) y2, (2,0) y3, (2,1) y4
//        L>=2, rp odd : slot 6 = y3 of level 2, slot 7 = y4 of level 2
// so the per-position norm accumulators live in registers across the whole channel loop, which keeps the
// channel order of the fused multiply-add chain fixed (ascending), and nothing is exchanged through
// shared memory.  Arithmetic follows the order written in wcc.h so that results are bit-identical to a
// plain fp32 evaluation.
#pragma once

#include "common.cuh"

namespace wcc {

template <int L>
struct HaarTile {
    static constexpr int RP = 1 << (L - 1);   // lane rows
    static constexpr int CG = 32 / RP;        // lane columns
    static constexpr int TH = 2 * RP;         // tile rows  (= 2^L)
    static constexpr int TW = 4 * CG;         // tile columns
};

struct LanePos {
    int pos[8];       // position (row * W + col) of each owned slot inside a plane
    bool ok0, ok1;    // quad 0 / quad 1 of the patch lies inside the image
    int r0, c0;       // top-left of the patch
};

template <int L>
__device__ __forceinline__ LanePos lane_positions(int H, int W, int tile_y, int tile_x, int lane)
{
    using T = HaarTile<L>;
    const int rp = lane / T::CG, cg = lane % T::CG;
    LanePos lp;
    lp.r0 = tile_y * T::TH + 2 * rp;
    lp.c0 = tile_x * T::TW + 4 * cg;
    lp.ok0 = lp.c0 < W;
    lp.ok1 = lp.c0 + 2 < W;
    const int i1 = lp.r0 >> 1, j1 = lp.c0 >> 1, h1 = H >> 1, w1 = W >> 1;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        lp.pos[0 + q] = i1 * W + w1 + j1 + q;
        lp.pos[2 + q] = (h1 + i1) * W + j1 + q;
        lp.pos[4 + q] = (h1 + i1) * W + w1 + j1 + q;
    }
    if (L == 1) {
        lp.pos[6] = i1 * W + j1;
        lp.pos[7] = i1 * W + j1 + 1;
    } else {
        const int i2 = i1 >> 1, j2 = j1 >> 1, h2 = H >> 2, w2 = W >> 2;
        if ((rp & 1) == 0) {
            lp.pos[6] = i2 * W + w2 + j2;
            if (L == 2) {
                lp.pos[7] = i2 * W + j2;
            } else {
                const int i3 = i2 >> 1, j3 = j2 >> 1, h3 = H >> 3, w3 = W >> 3;
                const bool top = (rp & 2) == 0, left = (cg & 1) == 0;
                lp.pos[7] = (top ? i3 : h3 + i3) * W + (left ? j3 : w3 + j3);
            }
        } else {
            lp.pos[6] = (h2 + i2) * W + j2;
            lp.pos[7] = (h2 + i2) * W + w2 + j2;
        }
    }
    return lp;
}

// slot validity: the second quad's level-1 slots (1, 3, 5 and, for L = 1, 7) need ok1
template <int L>
__device__ __forceinline__ bool slot_ok(const LanePos& lp, int s)
{
    if (s < 6) return (s & 1) ? lp.ok1 : lp.ok0;
    if (L == 1) return (s == 7) ? lp.ok1 : lp.ok0;
    return lp.ok0;
}

// Forward transform of the lane's patch p[row][col] into its eight slots.
template <int L>
__device__ __forceinline__ void haar_fwd_lane(const float (&p)[2][4], float (&o)[8], int lane)
{
    using T = HaarTile<L>;
    float ll[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const float a = p[0][2 * q], b = p[0][2 * q + 1], c = p[1][2 * q], d = p[1][2 * q + 1];
        const float s0 = __fadd_rn(a, b), d0 = __fsub_rn(a, b), s1 = __fadd_rn(c, d), d1 = __fsub_rn(c, d);
        ll[q] = __fmul_rn(__fadd_rn(s0, s1), 0.5f);
        o[0 + q] = __fmul_rn(__fadd_rn(d0, d1), 0.5f);
        o[2 + q] = __fmul_rn(__fsub_rn(s0, s1), 0.5f);
        o[4 + q] = __fmul_rn(__fsub_rn(d0, d1), 0.5f);
    }
    if (L == 1) {
        o[6] = ll[0];
        o[7] = ll[1];
        return;
    }
    const int rp = lane / T::CG, cg = lane % T::CG;
    const bool even = (rp & 1) == 0;
    const float s = __fadd_rn(ll[0], ll[1]), d = __fsub_rn(ll[0], ll[1]);
    const float ps = __shfl_xor_sync(0xFFFFFFFFu, s, T::CG);
    const float pd = __shfl_xor_sync(0xFFFFFFFFu, d, T::CG);
    float ll2 = 0.0f;
    if (even) {
        ll2 = __fmul_rn(__fadd_rn(s, ps), 0.5f);       // y1 = (s0 + s1) / 2
        o[6] = __fmul_rn(__fadd_rn(d, pd), 0.5f);      // y2 = (d0 + d1) / 2
        o[7] = ll2;
    } else {
        o[6] = __fmul_rn(__fsub_rn(ps, s), 0.5f);      // y3 = (s0 - s1) / 2, s0 from the even lane
        o[7] = __fmul_rn(__fsub_rn(pd, d), 0.5f);      // y4 = (d0 - d1) / 2
    }
    if (L == 3) {
        const float v = ll2;
        const float h = __shfl_xor_sync(0xFFFFFFFFu, v, 1);
        const float v2 = __shfl_xor_sync(0xFFFFFFFFu, v, 2 * T::CG);
        const float h2 = __shfl_xor_sync(0xFFFFFFFFu, h, 2 * T::CG);
        const bool top = (rp & 2) == 0, left = (cg & 1) == 0;
        const float a = top ? (left ? v : h) : (left ? v2 : h2);
        const float b = top ? (left ? h : v) : (left ? h2 : v2);
        const float c = top ? (left ? v2 : h2) : (left ? v : h);
        const float dd = top ? (left ? h2 : v2) : (left ? h : v);
        const float s0 = __fadd_rn(a, b), d0 = __fsub_rn(a, b), s1 = __fadd_rn(c, dd), d1 = __fsub_rn(c, dd);
        const float r = top ? (left ? __fadd_rn(s0, s1) : __fadd_rn(d0, d1))
                            : (left ? __fsub_rn(s0, s1) : __fsub_rn(d0, d1));
        if (even) o[7] = __fmul_rn(r, 0.5f);
    }
}

// Inverse transform of the lane's eight slots into its patch.
template <int L>
__device__ __forceinline__ void haar_inv_lane(const float (&o)[8], float (&p)[2][4], int lane)
{
    using T = HaarTile<L>;
    float ll[2];
    if (L == 1) {
        ll[0] = o[6];
        ll[1] = o[7];
    } else {
        const int rp = lane / T::CG, cg = lane % T::CG;
        const bool even = (rp & 1) == 0;
        float ll2 = o[7];
        if (L == 3) {
            const float v = o[7];
            const float h = __shfl_xor_sync(0xFFFFFFFFu, v, 1);
            const float v2 = __shfl_xor_sync(0xFFFFFFFFu, v, 2 * T::CG);
            const float h2 = __shfl_xor_sync(0xFFFFFFFFu, h, 2 * T::CG);
            const bool top = (rp & 2) == 0, left = (cg & 1) == 0;
            const float y1 = top ? (left ? v : h) : (left ? v2 : h2);
            const float y2 = top ? (left ? h : v) : (left ? h2 : v2);
            const float y3 = top ? (left ? v2 : h2) : (left ? v : h);
            const float y4 = top ? (left ? h2 : v2) : (left ? h : v);
            const float t0 = __fadd_rn(y1, y3), t1 = __fsub_rn(y1, y3), u0 = __fadd_rn(y2, y4), u1 = __fsub_rn(y2, y4);
            const float r = top ? (left ? __fadd_rn(t0, u0) : __fsub_rn(t0, u0))
                                : (left ? __fadd_rn(t1, u1) : __fsub_rn(t1, u1));
            ll2 = __fmul_rn(r, 0.5f);
        }
        const float m0 = even ? ll2 : o[6];
        const float m1 = even ? o[6] : o[7];
        const float p0 = __shfl_xor_sync(0xFFFFFFFFu, m0, T::CG);
        const float p1 = __shfl_xor_sync(0xFFFFFFFFu, m1, T::CG);
        if (even) {       // y1 = m0, y2 = m1, y3 = p0, y4 = p1 -> first row of the 2x2 output
            const float t0 = __fadd_rn(m0, p0), u0 = __fadd_rn(m1, p1);
            ll[0] = __fmul_rn(__fadd_rn(t0, u0), 0.5f);
            ll[1] = __fmul_rn(__fsub_rn(t0, u0), 0.5f);
        } else {          // y1 = p0, y2 = p1, y3 = m0, y4 = m1 -> second row
            const float t1 = __fsub_rn(p0, m0), u1 = __fsub_rn(p1, m1);
            ll[0] = __fmul_rn(__fadd_rn(t1, u1), 0.5f);
            ll[1] = __fmul_rn(__fsub_rn(t1, u1), 0.5f);
        }
    }
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const float y1 = ll[q], y2 = o[0 + q], y3 = o[2 + q], y4 = o[4 + q];
        const float t0 = __fadd_rn(y1, y3), t1 = __fsub_rn(y1, y3), u0 = __fadd_rn(y2, y4), u1 = __fsub_rn(y2, y4);
        p[0][2 * q] = __fmul_rn(__fadd_rn(t0, u0), 0.5f);
        p[0][2 * q + 1] = __fmul_rn(__fsub_rn(t0, u0), 0.5f);
        p[1][2 * q] = __fmul_rn(__fadd_rn(t1, u1), 0.5f);
        p[1][2 * q + 1] = __fmul_rn(__fsub_rn(t1, u1), 0.5f);
    }
}

// ---- patch load / store ------------------------------------------------------------------------
struct RawPatch { uint32_t w[8]; };   // fp32: 2 rows x 4 words; bf16: 2 rows x 2 words (w[0..1], w[4..5])

template <typename T, bool VEC>
__device__ __forceinline__ void load_patch(const T* __restrict__ plane, int W, const LanePos& lp, RawPatch& r)
{
#pragma unroll
    for (int row = 0; row < 2; ++row) {
        const T* src = plane + (size_t)(lp.r0 + row) * W + lp.c0;
        uint32_t* w = r.w + 4 * row;
        if (sizeof(T) == 4) {
            if (VEC) {
                if (lp.ok0) {
                    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(src));
                    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
                } else { w[0] = w[1] = w[2] = w[3] = 0u; }
            } else {
                uint2 a = make_uint2(0u, 0u), b = make_uint2(0u, 0u);
                if (lp.ok0) a = __ldcs(reinterpret_cast<const uint2*>(src));
                if (lp.ok1) b = __ldcs(reinterpret_cast<const uint2*>(src + 2));
                w[0] = a.x; w[1] = a.y; w[2] = b.x; w[3] = b.y;
            }
        } else {
            if (VEC) {
                uint2 v = make_uint2(0u, 0u);
                if (lp.ok0) v = __ldcs(reinterpret_cast<const uint2*>(src));
                w[0] = v.x; w[1] = v.y;
            } else {
                w[0] = lp.ok0 ? __ldcs(reinterpret_cast<const uint32_t*>(src)) : 0u;
                w[1] = lp.ok1 ? __ldcs(reinterpret_cast<const uint32_t*>(src + 2)) : 0u;
            }
        }
    }
}

template <typename T>
__device__ __forceinline__ void unpack_patch(const RawPatch& r, float (&p)[2][4])
{
#pragma unroll
    for (int row = 0; row < 2; ++row) {
        const uint32_t* w = r.w + 4 * row;
        if (sizeof(T) == 4) {
#pragma unroll
            for (int i = 0; i < 4; ++i) p[row][i] = __uint_as_float(w[i]);
        } else {
            p[row][0] = bf16lo(w[0]); p[row][1] = bf16hi(w[0]);
            p[row][2] = bf16lo(w[1]); p[row][3] = bf16hi(w[1]);
        }
    }
}

template <typename T, bool VEC>
__device__ __forceinline__ void store_patch(T* __restrict__ plane, int W, const LanePos& lp, const float (&p)[2][4])
{
#pragma unroll
    for (int row = 0; row < 2; ++row) {
        T* dst = plane + (size_t)(lp.r0 + row) * W + lp.c0;
        if (sizeof(T) == 4) {
            if (VEC) {
                if (lp.ok0) *reinterpret_cast<float4*>(dst) = make_float4(p[row][0], p[row][1], p[row][2], p[row][3]);
            } else {
                if (lp.ok0) *reinterpret_cast<float2*>(dst) = make_float2(p[row][0], p[row][1]);
                if (lp.ok1) *reinterpret_cast<float2*>(dst + 2) = make_float2(p[row][2], p[row][3]);
            }
        } else {
            const uint32_t lo = pack_bf16x2(p[row][0], p[row][1]), hi = pack_bf16x2(p[row][2], p[row][3]);
            if (VEC) {
                if (lp.ok0) *reinterpret_cast<uint2*>(dst) = make_uint2(lo, hi);
            } else {
                if (lp.ok0) *reinterpret_cast<uint32_t*>(dst) = lo;
                if (lp.ok1) *reinterpret_cast<uint32_t*>(dst + 2) = hi;
            }
        }
    }
}

// Store the eight slots of a lane into a quadrant-layout fp32 plane.
template <int L, bool VEC>
__device__ __forceinline__ void store_slots(float* __restrict__ plane, const LanePos& lp, const float (&o)[8])
{
    if (VEC) {   // W % 4 == 0: both quads valid together and the pairs are 8-byte aligned
        if (lp.ok0) {
            *reinterpret_cast<float2*>(plane + lp.pos[0]) = make_float2(o[0], o[1]);
            *reinterpret_cast<float2*>(plane + lp.pos[2]) = make_float2(o[2], o[3]);
            *reinterpret_cast<float2*>(plane + lp.pos[4]) = make_float2(o[4], o[5]);
            if (L == 1) {
                *reinterpret_cast<float2*>(plane + lp.pos[6]) = make_float2(o[6], o[7]);
            } else {
                plane[lp.pos[6]] = o[6];
                plane[lp.pos[7]] = o[7];
            }
        }
    } else {
#pragma unroll
        for (int s = 0; s < 8; ++s)
            if (slot_ok<L>(lp, s)) plane[lp.pos[s]] = o[s];
    }
}

template <int L, bool VEC>
__device__ __forceinline__ void load_slots(const float* __restrict__ plane, const LanePos& lp, float (&o)[8])
{
    if (VEC) {
        if (lp.ok0) {
            const float2 a = *reinterpret_cast<const float2*>(plane + lp.pos[0]);
            const float2 b = *reinterpret_cast<const float2*>(plane + lp.pos[2]);
            const float2 c = *reinterpret_cast<const float2*>(plane + lp.pos[4]);
            o[0] = a.x; o[1] = a.y; o[2] = b.x; o[3] = b.y; o[4] = c.x; o[5] = c.y;
            if (L == 1) {
                const float2 d = *reinterpret_cast<const float2*>(plane + lp.pos[6]);
                o[6] = d.x; o[7] = d.y;
            } else {
                o[6] = plane[lp.pos[6]];
                o[7] = plane[lp.pos[7]];
            }
        } else {
#pragma unroll
            for (int s = 0; s < 8; ++s) o[s] = 0.0f;
        }
    } else {
#pragma unroll
        for (int s = 0; s < 8; ++s) o[s] = slot_ok<L>(lp, s) ? plane[lp.pos[s]] : 0.0f;
    }
}

__device__ __forceinline__ void tile_coords(int warp, int tiles_x, int tiles_y, int& n, int& ty, int& tx)
{
    tx = warp % tiles_x;
    const int t = warp / tiles_x;
    ty = t % tiles_y;
    n = t / tiles_y;
}

// ---- forward: Haar + norms ---------------------------------------------------------------------
// One warp per (image, tile); the warp walks the channels in ascending order, D channels of loads in
// flight at a time.  Writes coef (optional), nrm2 (optional) and amaxpos = max_c |coef| (optional).
template <typename T, int L, bool VEC, int D>
__global__ void __launch_bounds__(128)
haar_fwd_kernel(const T* __restrict__ x, int N, int C, int H, int W,
                float* __restrict__ coef, float* __restrict__ nrm2, float* __restrict__ amaxpos)
{
    using TT = HaarTile<L>;
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const int warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (warp >= N * tiles_x * tiles_y) return;
    const int lane = threadIdx.x & 31;
    int n, ty, tx;
    tile_coords(warp, tiles_x, tiles_y, n, ty, tx);
    const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
    const size_t P = (size_t)H * W;
    const T* xin = x + (size_t)n * C * P;
    float* cout = coef ? coef + (size_t)n * C * P : nullptr;

    float nacc[8], amax[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) { nacc[s] = 0.0f; amax[s] = 0.0f; }

    for (int c0 = 0; c0 < C; c0 += D) {
        RawPatch raw[D];
#pragma unroll
        for (int d = 0; d < D; ++d) {
            if (c0 + d < C) load_patch<T, VEC>(xin + (size_t)(c0 + d) * P, W, lp, raw[d]);
        }
#pragma unroll
        for (int d = 0; d < D; ++d) {
            if (c0 + d < C) {
                float p[2][4], o[8];
                unpack_patch<T>(raw[d], p);
                haar_fwd_lane<L>(p, o, lane);
                if (cout) store_slots<L, VEC>(cout + (size_t)(c0 + d) * P, lp, o);
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    nacc[s] = __fmaf_rn(o[s], o[s], nacc[s]);
                    amax[s] = fmaxf(amax[s], fabsf(o[s]));
                }
            }
        }
    }
    if (nrm2) store_slots<L, VEC>(nrm2 + (size_t)n * P, lp, nacc);
    if (amaxpos) store_slots<L, VEC>(amaxpos + (size_t)n * P, lp, amax);
}

// ---- plain inverse -------------------------------------------------------------------------------
// One warp per (plane, tile).
template <typename T, int L, bool VEC>
__global__ void __launch_bounds__(128)
haar_inv_kernel(const float* __restrict__ coef, int planes, int H, int W, T* __restrict__ out)
{
    using TT = HaarTile<L>;
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (warp >= (long long)planes * tiles_x * tiles_y) return;
    const int lane = threadIdx.x & 31;
    int pl, ty, tx;
    tile_coords((int)warp, tiles_x, tiles_y, pl, ty, tx);
    const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
    const size_t P = (size_t)H * W;
    float o[8], p[2][4];
    load_slots<L, VEC>(coef + (size_t)pl * P, lp, o);
    haar_inv_lane<L>(o, p, lane);
    store_patch<T, VEC>(out + (size_t)pl * P, W, lp, p);
}

// ---- fused dequantize + scatter + inverse ----------------------------------------------------
// One warp per (image, tile, group of OCW output channels).  rank[n][p] is the row of position p in the
// compressed matrix (or -1 when p was dropped: the zero map).  acc row r = n*k + rank holds the int32
// accumulators (or fp32 products when ACCF) of all output channels, pitch ldc (multiple of 4).
template <typename T, int L, bool VEC, bool ACCF, int OCW>
__global__ void __launch_bounds__(128)
scatter_inv_kernel(const int32_t* __restrict__ acc, int ldc, const int32_t* __restrict__ rank,
                   const float* __restrict__ amax_kept, float qmax, const float* __restrict__ scale_w,
                   int N, int Cout, int H, int W, int k, T* __restrict__ y)
{
    using TT = HaarTile<L>;
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const int groups = (Cout + OCW - 1) / OCW;
    const long long gw = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (gw >= (long long)N * tiles_x * tiles_y * groups) return;
    const int lane = threadIdx.x & 31;
    const int g = (int)(gw % groups);
    int n, ty, tx;
    tile_coords((int)(gw / groups), tiles_x, tiles_y, n, ty, tx);
    const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
    const size_t P = (size_t)H * W;

    const int32_t* rk = rank + (size_t)n * P;
    const int32_t* rowp[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        int r = -1;
        if (slot_ok<L>(lp, s)) r = rk[lp.pos[s]];
        rowp[s] = (r >= 0) ? acc + ((size_t)n * k + r) * ldc : nullptr;
    }
    float scale_a = 1.0f;
    if (!ACCF) scale_a = __fdiv_rn(*amax_kept, qmax);

    const int o_end = min(Cout, (g + 1) * OCW);
    for (int o0 = g * OCW; o0 < o_end; o0 += 4) {
        int4 v[8];
#pragma unroll
        for (int s = 0; s < 8; ++s)
            v[s] = rowp[s] ? *reinterpret_cast<const int4*>(rowp[s] + o0) : make_int4(0, 0, 0, 0);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = o0 + j;
            if (o < o_end) {      // warp-uniform
                float sc = 1.0f;
                if (!ACCF) sc = __fmul_rn(scale_a, scale_w[o]);
                float sl[8], p[2][4];
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    const int a = (j == 0) ? v[s].x : (j == 1) ? v[s].y : (j == 2) ? v[s].z : v[s].w;
                    sl[s] = ACCF ? __int_as_float(a) : __fmul_rn((float)a, sc);
                }
                haar_inv_lane<L>(sl, p, lane);
                store_patch<T, VEC>(y + ((size_t)n * Cout + o) * P, W, lp, p);
            }
        }
    }
}

// ---- launchers -------------------------------------------------------------------------------
template <typename T, int L, bool VEC>
static wcc_status haar_fwd_dispatch(const void* x, int N, int C, int H, int W, float* coef, float* nrm2,
                                    float* amaxpos, cudaStream_t st)
{
    using TT = HaarTile<L>;
    constexpr int D = (sizeof(T) == 4) ? 4 : 8;
    const long long warps = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    const int blocks = (int)((warps + 3) / 4);
    haar_fwd_kernel<T, L, VEC, D><<<blocks, 128, 0, st>>>(static_cast<const T*>(x), N, C, H, W, coef, nrm2, amaxpos);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

#define WCC_DISPATCH_TLV(FN, dt, L, vec, ...)                                                        \
    do {                                                                                             \
        if ((dt) == WCC_F32) {                                                                       \
            if ((L) == 1) return (vec) ? FN<float, 1, true>(__VA_ARGS__) : FN<float, 1, false>(__VA_ARGS__); \
            if ((L) == 2) return FN<float, 2, true>(__VA_ARGS__);                                    \
            return FN<float, 3, true>(__VA_ARGS__);                                                  \
        } else {                                                                                     \
            if ((L) == 1) return (vec) ? FN<__nv_bfloat16, 1, true>(__VA_ARGS__) : FN<__nv_bfloat16, 1, false>(__VA_ARGS__); \
            if ((L) == 2) return FN<__nv_bfloat16, 2, true>(__VA_ARGS__);                            \
            return FN<__nv_bfloat16, 3, true>(__VA_ARGS__);                                          \
        }                                                                                            \
    } while (0)

wcc_status launch_haar_fwd(const void* x, int N, int C, int H, int W, int L, wcc_dtype dt,
                           float* coef, float* nrm2, float* amaxpos, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;   // always true for L >= 2
    WCC_DISPATCH_TLV(haar_fwd_dispatch, dt, L, vec, x, N, C, H, W, coef, nrm2, amaxpos, st);
}

template <typename T, int L, bool VEC>
static wcc_status haar_inv_dispatch(const float* coef, int planes, int H, int W, void* out, cudaStream_t st)
{
    using TT = HaarTile<L>;
    const long long warps = (long long)planes * ceil_div(W, TT::TW) * (H / TT::TH);
    const int blocks = (int)((warps + 3) / 4);
    haar_inv_kernel<T, L, VEC><<<blocks, 128, 0, st>>>(coef, planes, H, W, static_cast<T*>(out));
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

wcc_status launch_haar_inv(const float* coef, int N, int C, int H, int W, int L, wcc_dtype dt,
                           void* out, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;
    WCC_DISPATCH_TLV(haar_inv_dispatch, dt, L, vec, coef, N * C, H, W, out, st);
}

template <typename T, int L, bool VEC>
static wcc_status scatter_inv_dispatch(const int32_t* acc, int ldc, bool accf, const int32_t* rank,
                                       const float* amax_kept, float qmax, const float* scale_w,
                                       int N, int Cout, int H, int W, int k, void* y, cudaStream_t st)
{
    using TT = HaarTile<L>;
    constexpr int OCW = 8;
    const long long warps = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH) * ceil_div(Cout, OCW);
    const int blocks = (int)((warps + 3) / 4);
    if (accf)
        scatter_inv_kernel<T, L, VEC, true, OCW><<<blocks, 128, 0, st>>>(acc, ldc, rank, amax_kept, qmax, scale_w,
                                                                          N, Cout, H, W, k, static_cast<T*>(y));
    else
        scatter_inv_kernel<T, L, VEC, false, OCW><<<blocks, 128, 0, st>>>(acc, ldc, rank, amax_kept, qmax, scale_w,
                                                                           N, Cout, H, W, k, static_cast<T*>(y));
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

wcc_status launch_scatter_inv(const int32_t* acc, int ldc, bool acc_is_float, const int32_t* rank,
                              const float* amax_kept, int bits, const float* scale_w,
                              int N, int Cout, int H, int W, int L, int k, wcc_dtype dt, void* y, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;
    const float qmax = (bits >= 2) ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    WCC_DISPATCH_TLV(scatter_inv_dispatch, dt, L, vec, acc, ldc, acc_is_float, rank, amax_kept, qmax, scale_w,
                     N, Cout, H, W, k, y, st);
}

}  // namespace wcc

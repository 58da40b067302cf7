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
//        L>=2, rp even: slot 7 = y2 of level 2, slot 6 = y1 of level 2 (L=2) or one of y1..y4 of level 3,
//                       by (rp & 2, cg & 1): (0,0) y1, (0,1) y2, (2,0) y3, (2,1) y4
//        L>=2, rp odd : slot 6 = y3 of level 2, slot 7 = y4 of level 2
// In haar_fwd_kernel the per-position norm accumulators live in registers across the whole channel loop, which keeps
// the channel order of the fused multiply-add chain fixed (ascending); the first pass of the fused layer
// (haar_norms_token_kernel) keeps that order too while several warps share a tile: the partial sums are handed from
// warp to warp.  Arithmetic follows the order written in wcc.h so that results are bit-identical to a plain fp32
// evaluation.
#pragma once

#include "common.cuh"
#include "tma.cuh"

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
            lp.pos[7] = i2 * W + w2 + j2;
            if (L == 2) {
                lp.pos[6] = i2 * W + j2;
            } else {
                const int i3 = i2 >> 1, j3 = j2 >> 1, h3 = H >> 3, w3 = W >> 3;
                const bool top = (rp & 2) == 0, left = (cg & 1) == 0;
                lp.pos[6] = (top ? i3 : h3 + i3) * W + (left ? j3 : w3 + j3);
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

// Packed fp32 pairs (Blackwell f32x2 pipe): each operation rounds both halves once, to nearest even, exactly like
// the scalar operation.  a - b is written fma(b, -1, a): one rounding of the exact difference.
// add2 / mul2 are written in PTX with an explicit rounding modifier so that a product followed by a sum is never
// contracted into one fused operation (that would round once instead of twice and change quantization codes).
__device__ __forceinline__ float2 add2(float2 a, float2 b)
{
    float2 r;
    asm("{\n .reg .b64 ra, rb, rc;\n mov.b64 ra, {%2, %3};\n mov.b64 rb, {%4, %5};\n add.rn.f32x2 rc, ra, rb;\n mov.b64 {%0, %1}, rc;\n}\n"
        : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return r;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b)
{
    float2 r;
    asm("{\n .reg .b64 ra, rb, rc;\n mov.b64 ra, {%2, %3};\n mov.b64 rb, {%4, %5};\n mul.rn.f32x2 rc, ra, rb;\n mov.b64 {%0, %1}, rc;\n}\n"
        : "=f"(r.x), "=f"(r.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return r;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) { return __ffma2_rn(b, make_float2(-1.0f, -1.0f), a); }
__device__ __forceinline__ float2 half2x(float2 a) { return mul2(a, make_float2(0.5f, 0.5f)); }

// Forward transform of the lane's patch p[row][col] into its eight slots.  The two quads of the patch are processed
// side by side in packed pairs: (quad 0, quad 1).
template <int L>
__device__ __forceinline__ void haar_fwd_lane(const float (&p)[2][4], float (&o)[8], int lane)
{
    using T = HaarTile<L>;
    const float2 a = make_float2(p[0][0], p[0][2]), b = make_float2(p[0][1], p[0][3]);
    const float2 c = make_float2(p[1][0], p[1][2]), d = make_float2(p[1][1], p[1][3]);
    const float2 s0 = add2(a, b), d0 = sub2(a, b), s1 = add2(c, d), d1 = sub2(c, d);
    const float2 ll = half2x(add2(s0, s1));            // y1 of both quads
    const float2 y2 = half2x(add2(d0, d1));
    const float2 y3 = half2x(sub2(s0, s1));
    const float2 y4 = half2x(sub2(d0, d1));
    o[0] = y2.x; o[1] = y2.y; o[2] = y3.x; o[3] = y3.y; o[4] = y4.x; o[5] = y4.y;
    if (L == 1) {
        o[6] = ll.x;
        o[7] = ll.y;
        return;
    }
    // Level 2: the lane pair (rp, rp^1) holds the 2x2 block of level-1 low-pass values, one row each.  With
    // sg = +1 on the upper (even) lane and -1 on the lower one, fma(own, sg, other) is own+other on the upper lane
    // (s0+s1, d0+d1 -> y1, y2) and other-own on the lower lane (s0-s1, d0-d1 -> y3, y4): one rounding, as an add.
    const int rp = lane / T::CG, cg = lane % T::CG;
    const bool even = (rp & 1) == 0;
    const float sg = even ? 1.0f : -1.0f;
    const float s = __fadd_rn(ll.x, ll.y), dd = __fsub_rn(ll.x, ll.y);
    const float ps = __shfl_xor_sync(0xFFFFFFFFu, s, T::CG);
    const float pd = __shfl_xor_sync(0xFFFFFFFFu, dd, T::CG);
    const float2 l2 = half2x(__ffma2_rn(make_float2(s, dd), make_float2(sg, sg), make_float2(ps, pd)));
    o[6] = l2.x;                                       // even: y1, odd: y3
    o[7] = l2.y;                                       // even: y2, odd: y4
    if (L == 3) {
        // Level 3: the four even lanes {rp, rp^2} x {cg, cg^1} hold a, b / c, d.  Horizontal step: left lane a+b (c+d),
        // right lane a-b (c-d); vertical step: top lanes sum (y1, y2), bottom lanes difference (y3, y4).
        const float sgh = (cg & 1) == 0 ? 1.0f : -1.0f;
        const float sgv = (rp & 2) == 0 ? 1.0f : -1.0f;
        const float v = o[6];
        const float h = __shfl_xor_sync(0xFFFFFFFFu, v, 1);
        const float t = __fmaf_rn(v, sgh, h);
        const float q = __shfl_xor_sync(0xFFFFFFFFu, t, 2 * T::CG);
        const float r = __fmul_rn(__fmaf_rn(t, sgv, q), 0.5f);
        if (even) o[6] = r;
    }
}

// Inverse transform of the lane's eight slots into its patch.
template <int L>
__device__ __forceinline__ void haar_inv_lane(const float (&o)[8], float (&p)[2][4], int lane)
{
    using T = HaarTile<L>;
    float2 ll;
    if (L == 1) {
        ll = make_float2(o[6], o[7]);
    } else {
        const int rp = lane / T::CG, cg = lane % T::CG;
        const float sg = (rp & 1) == 0 ? 1.0f : -1.0f;
        float m0 = o[6];
        if (L == 3) {
            // vertical step: top lanes y1+y3 (y2+y4), bottom lanes y1-y3 (y2-y4); horizontal step: left lanes sum
            // (a, c), right lanes difference (b, d)
            const float sgh = (cg & 1) == 0 ? 1.0f : -1.0f;
            const float sgv = (rp & 2) == 0 ? 1.0f : -1.0f;
            const float pv = __shfl_xor_sync(0xFFFFFFFFu, m0, 2 * T::CG);
            const float w = __fmaf_rn(m0, sgv, pv);
            const float q = __shfl_xor_sync(0xFFFFFFFFu, w, 1);
            const float r = __fmul_rn(__fmaf_rn(w, sgh, q), 0.5f);
            if ((rp & 1) == 0) m0 = r;
        }
        // level 2: upper lane holds (y1, y2), lower lane (y3, y4)
        const float m1 = o[7];
        const float p0 = __shfl_xor_sync(0xFFFFFFFFu, m0, T::CG);
        const float p1 = __shfl_xor_sync(0xFFFFFFFFu, m1, T::CG);
        // upper: (t0, u0) = (y1 + y3, y2 + y4); lower: (t1, u1) = (y1 - y3, y2 - y4)
        const float2 tu = __ffma2_rn(make_float2(m0, m1), make_float2(sg, sg), make_float2(p0, p1));
        ll = make_float2(__fmul_rn(__fadd_rn(tu.x, tu.y), 0.5f), __fmul_rn(__fsub_rn(tu.x, tu.y), 0.5f));
    }
    const float2 y2 = make_float2(o[0], o[1]), y3 = make_float2(o[2], o[3]), y4 = make_float2(o[4], o[5]);
    const float2 t0 = add2(ll, y3), t1 = sub2(ll, y3), u0 = add2(y2, y4), u1 = sub2(y2, y4);
    const float2 a = half2x(add2(t0, u0)), b = half2x(sub2(t0, u0));
    const float2 c = half2x(add2(t1, u1)), d = half2x(sub2(t1, u1));
    p[0][0] = a.x; p[0][1] = b.x; p[0][2] = a.y; p[0][3] = b.y;
    p[1][0] = c.x; p[1][1] = d.x; p[1][2] = c.y; p[1][3] = d.y;
}

// The same transforms on U independent channels at once, stage by stage: the shuffles of one stage are issued back to
// back for all U channels, so their latencies overlap (shuffles keep their program order; channel after channel they
// would form one long dependent chain).  Arithmetic per channel is exactly that of haar_fwd_lane / haar_inv_lane.
template <int L, int U>
__device__ __forceinline__ void haar_fwd_lanes(const float (&p)[U][2][4], float (&o)[U][8], int lane)
{
    using T = HaarTile<L>;
    float2 ll[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const float2 a = make_float2(p[u][0][0], p[u][0][2]), b = make_float2(p[u][0][1], p[u][0][3]);
        const float2 c = make_float2(p[u][1][0], p[u][1][2]), d = make_float2(p[u][1][1], p[u][1][3]);
        const float2 s0 = add2(a, b), d0 = sub2(a, b), s1 = add2(c, d), d1 = sub2(c, d);
        ll[u] = half2x(add2(s0, s1));
        const float2 y2 = half2x(add2(d0, d1));
        const float2 y3 = half2x(sub2(s0, s1));
        const float2 y4 = half2x(sub2(d0, d1));
        o[u][0] = y2.x; o[u][1] = y2.y; o[u][2] = y3.x; o[u][3] = y3.y; o[u][4] = y4.x; o[u][5] = y4.y;
        if (L == 1) { o[u][6] = ll[u].x; o[u][7] = ll[u].y; }
    }
    if (L == 1) return;
    const int rp = lane / T::CG, cg = lane % T::CG;
    const bool even = (rp & 1) == 0;
    const float sg = even ? 1.0f : -1.0f;
    float s[U], dd[U], ps[U], pd[U];
#pragma unroll
    for (int u = 0; u < U; ++u) { s[u] = __fadd_rn(ll[u].x, ll[u].y); dd[u] = __fsub_rn(ll[u].x, ll[u].y); }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        ps[u] = __shfl_xor_sync(0xFFFFFFFFu, s[u], T::CG);
        pd[u] = __shfl_xor_sync(0xFFFFFFFFu, dd[u], T::CG);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const float2 l2 = half2x(__ffma2_rn(make_float2(s[u], dd[u]), make_float2(sg, sg), make_float2(ps[u], pd[u])));
        o[u][6] = l2.x;
        o[u][7] = l2.y;
    }
    if (L == 3) {
        const float sgh = (cg & 1) == 0 ? 1.0f : -1.0f;
        const float sgv = (rp & 2) == 0 ? 1.0f : -1.0f;
        float h[U], t[U], q[U];
#pragma unroll
        for (int u = 0; u < U; ++u) h[u] = __shfl_xor_sync(0xFFFFFFFFu, o[u][6], 1);
#pragma unroll
        for (int u = 0; u < U; ++u) t[u] = __fmaf_rn(o[u][6], sgh, h[u]);
#pragma unroll
        for (int u = 0; u < U; ++u) q[u] = __shfl_xor_sync(0xFFFFFFFFu, t[u], 2 * T::CG);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float r = __fmul_rn(__fmaf_rn(t[u], sgv, q[u]), 0.5f);
            if (even) o[u][6] = r;
        }
    }
}

template <int L, int U>
__device__ __forceinline__ void haar_inv_lanes(const float (&o)[U][8], float (&p)[U][2][4], int lane)
{
    using T = HaarTile<L>;
    float2 ll[U];
    if (L == 1) {
#pragma unroll
        for (int u = 0; u < U; ++u) ll[u] = make_float2(o[u][6], o[u][7]);
    } else {
        const int rp = lane / T::CG, cg = lane % T::CG;
        const float sg = (rp & 1) == 0 ? 1.0f : -1.0f;
        float m0[U];
#pragma unroll
        for (int u = 0; u < U; ++u) m0[u] = o[u][6];
        if (L == 3) {
            const float sgh = (cg & 1) == 0 ? 1.0f : -1.0f;
            const float sgv = (rp & 2) == 0 ? 1.0f : -1.0f;
            float pv[U], w[U], q[U];
#pragma unroll
            for (int u = 0; u < U; ++u) pv[u] = __shfl_xor_sync(0xFFFFFFFFu, m0[u], 2 * T::CG);
#pragma unroll
            for (int u = 0; u < U; ++u) w[u] = __fmaf_rn(m0[u], sgv, pv[u]);
#pragma unroll
            for (int u = 0; u < U; ++u) q[u] = __shfl_xor_sync(0xFFFFFFFFu, w[u], 1);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float r = __fmul_rn(__fmaf_rn(w[u], sgh, q[u]), 0.5f);
                if ((rp & 1) == 0) m0[u] = r;
            }
        }
        float p0[U], p1[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            p0[u] = __shfl_xor_sync(0xFFFFFFFFu, m0[u], T::CG);
            p1[u] = __shfl_xor_sync(0xFFFFFFFFu, o[u][7], T::CG);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float2 tu = __ffma2_rn(make_float2(m0[u], o[u][7]), make_float2(sg, sg), make_float2(p0[u], p1[u]));
            ll[u] = make_float2(__fmul_rn(__fadd_rn(tu.x, tu.y), 0.5f), __fmul_rn(__fsub_rn(tu.x, tu.y), 0.5f));
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const float2 y2 = make_float2(o[u][0], o[u][1]), y3 = make_float2(o[u][2], o[u][3]), y4 = make_float2(o[u][4], o[u][5]);
        const float2 t0 = add2(ll[u], y3), t1 = sub2(ll[u], y3), u0 = add2(y2, y4), u1 = sub2(y2, y4);
        const float2 a = half2x(add2(t0, u0)), b = half2x(sub2(t0, u0));
        const float2 c = half2x(add2(t1, u1)), d = half2x(sub2(t1, u1));
        p[u][0][0] = a.x; p[u][0][1] = b.x; p[u][0][2] = a.y; p[u][0][3] = b.y;
        p[u][1][0] = c.x; p[u][1][1] = d.x; p[u][1][2] = c.y; p[u][1][3] = d.y;
    }
}

// ---- transforms with the halvings taken out ------------------------------------------------------------
// Multiplying by a power of two commutes with every rounding (barring overflow and subnormal results), so the forward
// transform can run on sums and differences alone and leave one exact multiplication per slot to the consumer:
// true coefficient of slot s = raw value * slot_scale[s], where |slot_scale| = 2^-level.  The same holds for squares
// (norm = raw norm * scale^2) and maxima.  Results are bit-identical to haar_fwd_lanes for inputs whose partial sums stay
// below 2^125 and above the subnormal range.
// `swapped`: the lane passes its two patch rows in exchanged order (a shared-memory bank trick of the TMA rings); the sums
// over rows are unchanged and the differences over rows (y3, y4 of level 1) change sign, which goes into the scale.
template <int L>
__device__ __forceinline__ void slot_scales(int lane, bool swapped, float (&sc)[8])
{
    using T = HaarTile<L>;
    const int rp = lane / T::CG;
    const float h = 0.5f, hs = swapped ? -0.5f : 0.5f;
    sc[0] = h; sc[1] = h; sc[2] = hs; sc[3] = hs; sc[4] = hs; sc[5] = hs;
    if (L == 1) { sc[6] = h; sc[7] = h; }
    else {
        sc[7] = 0.25f;
        sc[6] = (L == 3 && (rp & 1) == 0) ? 0.125f : 0.25f;
    }
}

template <int L, int U>
__device__ __forceinline__ void haar_fwd_lanes_raw(const float (&p)[U][2][4], float (&o)[U][8], int lane)
{
    using T = HaarTile<L>;
    float2 ll[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const float2 a = make_float2(p[u][0][0], p[u][0][2]), b = make_float2(p[u][0][1], p[u][0][3]);
        const float2 c = make_float2(p[u][1][0], p[u][1][2]), d = make_float2(p[u][1][1], p[u][1][3]);
        const float2 s0 = add2(a, b), d0 = sub2(a, b), s1 = add2(c, d), d1 = sub2(c, d);
        ll[u] = add2(s0, s1);
        const float2 y2 = add2(d0, d1), y3 = sub2(s0, s1), y4 = sub2(d0, d1);
        o[u][0] = y2.x; o[u][1] = y2.y; o[u][2] = y3.x; o[u][3] = y3.y; o[u][4] = y4.x; o[u][5] = y4.y;
        if (L == 1) { o[u][6] = ll[u].x; o[u][7] = ll[u].y; }
    }
    if (L == 1) return;
    const int rp = lane / T::CG, cg = lane % T::CG;
    const bool even = (rp & 1) == 0;
    const float sg = even ? 1.0f : -1.0f;
    float s[U], dd[U], ps[U], pd[U];
#pragma unroll
    for (int u = 0; u < U; ++u) { s[u] = __fadd_rn(ll[u].x, ll[u].y); dd[u] = __fsub_rn(ll[u].x, ll[u].y); }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        ps[u] = __shfl_xor_sync(0xFFFFFFFFu, s[u], T::CG);
        pd[u] = __shfl_xor_sync(0xFFFFFFFFu, dd[u], T::CG);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const float2 l2 = __ffma2_rn(make_float2(s[u], dd[u]), make_float2(sg, sg), make_float2(ps[u], pd[u]));
        o[u][6] = l2.x;
        o[u][7] = l2.y;
    }
    if (L == 3) {
        const float sgh = (cg & 1) == 0 ? 1.0f : -1.0f;
        const float sgv = (rp & 2) == 0 ? 1.0f : -1.0f;
        float h[U], t[U], q[U];
#pragma unroll
        for (int u = 0; u < U; ++u) h[u] = __shfl_xor_sync(0xFFFFFFFFu, o[u][6], 1);
#pragma unroll
        for (int u = 0; u < U; ++u) t[u] = __fmaf_rn(o[u][6], sgh, h[u]);
#pragma unroll
        for (int u = 0; u < U; ++u) q[u] = __shfl_xor_sync(0xFFFFFFFFu, t[u], 2 * T::CG);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float r = __fmaf_rn(t[u], sgv, q[u]);
            if (even) o[u][6] = r;
        }
    }
}

// Inverse on slots that the caller has already multiplied by slot_scales (not swapped): sums and differences only.
template <int L, int U>
__device__ __forceinline__ void haar_inv_lanes_raw(const float (&o)[U][8], float (&p)[U][2][4], int lane)
{
    using T = HaarTile<L>;
    float2 ll[U];
    if (L == 1) {
#pragma unroll
        for (int u = 0; u < U; ++u) ll[u] = make_float2(o[u][6], o[u][7]);
    } else {
        const int rp = lane / T::CG, cg = lane % T::CG;
        const float sg = (rp & 1) == 0 ? 1.0f : -1.0f;
        float m0[U];
#pragma unroll
        for (int u = 0; u < U; ++u) m0[u] = o[u][6];
        if (L == 3) {
            const float sgh = (cg & 1) == 0 ? 1.0f : -1.0f;
            const float sgv = (rp & 2) == 0 ? 1.0f : -1.0f;
            float pv[U], w[U], q[U];
#pragma unroll
            for (int u = 0; u < U; ++u) pv[u] = __shfl_xor_sync(0xFFFFFFFFu, m0[u], 2 * T::CG);
#pragma unroll
            for (int u = 0; u < U; ++u) w[u] = __fmaf_rn(m0[u], sgv, pv[u]);
#pragma unroll
            for (int u = 0; u < U; ++u) q[u] = __shfl_xor_sync(0xFFFFFFFFu, w[u], 1);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float r = __fmaf_rn(w[u], sgh, q[u]);
                if ((rp & 1) == 0) m0[u] = r;
            }
        }
        float p0[U], p1[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            p0[u] = __shfl_xor_sync(0xFFFFFFFFu, m0[u], T::CG);
            p1[u] = __shfl_xor_sync(0xFFFFFFFFu, o[u][7], T::CG);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const float2 tu = __ffma2_rn(make_float2(m0[u], o[u][7]), make_float2(sg, sg), make_float2(p0[u], p1[u]));
            ll[u] = make_float2(__fadd_rn(tu.x, tu.y), __fsub_rn(tu.x, tu.y));
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const float2 y2 = make_float2(o[u][0], o[u][1]), y3 = make_float2(o[u][2], o[u][3]), y4 = make_float2(o[u][4], o[u][5]);
        const float2 t0 = add2(ll[u], y3), t1 = sub2(ll[u], y3), u0 = add2(y2, y4), u1 = sub2(y2, y4);
        const float2 a = add2(t0, u0), b = sub2(t0, u0);
        const float2 c = add2(t1, u1), d = sub2(t1, u1);
        p[u][0][0] = a.x; p[u][0][1] = b.x; p[u][0][2] = a.y; p[u][0][3] = b.y;
        p[u][1][0] = c.x; p[u][1][1] = d.x; p[u][1][2] = c.y; p[u][1][3] = d.y;
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
// One warp per (image, tile, chunk of cpc channels; blockIdx.y = chunk); the warp walks its channels in ascending
// order, D channels of loads in flight at a time.  Writes coef (optional) and, when one chunk holds all channels,
// nrm2 (optional) and amaxpos = max_c |coef| (optional): the norm is one chain of fused multiply-adds over all
// channels, so with several chunks it is taken from the stored coefficients afterwards (coef_norms_kernel).
template <typename T, int L, bool VEC, int D>
__global__ void __launch_bounds__(128)
haar_fwd_kernel(const T* __restrict__ x, int N, int C, int H, int W, int cpc,
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
    const int c_lo = (int)blockIdx.y * cpc, c_hi = min(C, c_lo + cpc);
    if (gridDim.y > 1) { nrm2 = nullptr; amaxpos = nullptr; }

    float nacc[8], amax[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) { nacc[s] = 0.0f; amax[s] = 0.0f; }

    for (int c0 = c_lo; c0 < c_hi; c0 += D) {
        RawPatch raw[D];
#pragma unroll
        for (int d = 0; d < D; ++d) {
            if (c0 + d < c_hi) load_patch<T, VEC>(xin + (size_t)(c0 + d) * P, W, lp, raw[d]);
        }
#pragma unroll
        for (int d = 0; d < D; ++d) {
            if (c0 + d < c_hi) {
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


// ---- depthwise 3x3 convolution fused with the forward transform ------------------------------------------
// The input of the block's second pointwise layer is a depthwise convolution of the expanded map (Eq. 13); both are
// separable per channel, so the convolution's output never goes to memory: every lane computes the convolution at the
// eight pixels of its patch (from a 4 x 6 neighbourhood of the input, zeros outside the map) and transforms them right
// away.  Per output pixel: one fused multiply-add per tap, row-major tap order, starting from +0 (taps outside the map
// contribute nothing).  Same work decomposition (channel chunks included) and outputs as haar_fwd_kernel; w is fp32
// [C][3][3].

// One channel's input of the convolution as loaded: rows r0-1 .. r0+2, columns c0-1 .. c0+4 of the lane's patch (zeros
// outside the map), and the channel's nine taps.  With W % 4 == 0 the four middle columns are one aligned vector; bf16
// rows then stay packed (two words of middle columns, one word holding the left and the right neighbour).
template <typename T, bool VEC>
struct DwRaw {
    static constexpr bool PACKED = VEC && sizeof(T) == 2;
    static constexpr int RW = PACKED ? 3 : 6;
    uint32_t v[4][RW];
    float k[9];
};

// ER / EC: the tile touches the top or bottom / the left or right border of the map (or hangs over it), so rows / columns
// of the neighbourhood can fall outside; tiles in the interior load without any bounds test.
template <typename T, bool VEC, bool ER = true, bool EC = true>
__device__ __forceinline__ void dwconv_load(const T* __restrict__ plane, const float* __restrict__ w9, const LanePos& lp,
                                            int H, int W, DwRaw<T, VEC>& r)
{
#pragma unroll
    for (int i = 0; i < 9; ++i) r.k[i] = __ldg(w9 + i);
    auto load1 = [&](int rr, int cc) -> uint32_t {         // one element as fp32 bits (bf16: the upper half)
        if (sizeof(T) == 4) return __ldg(reinterpret_cast<const uint32_t*>(plane) + (size_t)rr * W + cc);
        return (uint32_t)__ldg(reinterpret_cast<const unsigned short*>(plane) + (size_t)rr * W + cc) << 16;
    };
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        const int rr = lp.r0 + a - 1;
        const bool row_in = !ER || (rr >= 0 && rr < H);
        if constexpr (VEC) {
            const uint32_t left = (row_in && (!EC || (lp.c0 > 0 && lp.c0 - 1 < W))) ? load1(rr, lp.c0 - 1) : 0u;
            const uint32_t right = (row_in && (!EC || lp.c0 + 4 < W)) ? load1(rr, lp.c0 + 4) : 0u;
            if constexpr (sizeof(T) == 4) {
                uint4 m = make_uint4(0u, 0u, 0u, 0u);
                if (row_in && (!EC || lp.ok0)) m = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint32_t*>(plane) + (size_t)rr * W + lp.c0));
                r.v[a][0] = left; r.v[a][1] = m.x; r.v[a][2] = m.y; r.v[a][3] = m.z; r.v[a][4] = m.w; r.v[a][5] = right;
            } else {
                uint2 m = make_uint2(0u, 0u);
                if (row_in && (!EC || lp.ok0)) m = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned short*>(plane) + (size_t)rr * W + lp.c0));
                r.v[a][0] = m.x; r.v[a][1] = m.y; r.v[a][2] = (left >> 16) | right;
            }
        } else {
#pragma unroll
            for (int b = 0; b < 6; ++b) {
                const int cc = lp.c0 + b - 1;
                r.v[a][b] = (row_in && cc >= 0 && cc < W) ? load1(rr, cc) : 0u;
            }
        }
    }
}

// The convolution at the eight pixels of the lane's patch: one fused multiply-add per tap, row-major tap order, from +0.
template <typename T, bool VEC>
__device__ __forceinline__ void dwconv_compute(const DwRaw<T, VEC>& r, float (&p)[2][4])
{
    float in[4][6];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        if constexpr (DwRaw<T, VEC>::PACKED) {
            in[a][0] = bf16lo(r.v[a][2]);
            in[a][1] = bf16lo(r.v[a][0]); in[a][2] = bf16hi(r.v[a][0]);
            in[a][3] = bf16lo(r.v[a][1]); in[a][4] = bf16hi(r.v[a][1]);
            in[a][5] = bf16hi(r.v[a][2]);
        } else {
#pragma unroll
            for (int b = 0; b < 6; ++b) in[a][b] = __uint_as_float(r.v[a][b]);
        }
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            float acc = 0.0f;
#pragma unroll
            for (int i = 0; i < 3; ++i)
#pragma unroll
                for (int j = 0; j < 3; ++j) acc = __fmaf_rn(r.k[i * 3 + j], in[a + i][b + j], acc);
            p[a][b] = acc;
        }
}

// Channels [c_lo, c_hi) of one tile, two at a time: while one channel is convolved and transformed the next one's input
// is in flight (two register buffers that swap roles).
template <typename T, int L, bool VEC, bool NORMS, bool ER, bool EC>
__device__ __forceinline__ void dwconv_channels(const T* __restrict__ uin, const float* __restrict__ w, float* __restrict__ cout,
                                                int c_lo, int c_hi, const LanePos& lp, int lane, int n, int H, int W,
                                                float* __restrict__ nrm2, float* __restrict__ amaxpos)
{
    const size_t P = (size_t)H * W;
    float nacc[8], amax[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) { nacc[s] = 0.0f; amax[s] = 0.0f; }
    auto finish = [&](const DwRaw<T, VEC>& r, int c) {
        float p[2][4], o[8];
        dwconv_compute<T, VEC>(r, p);
        haar_fwd_lane<L>(p, o, lane);
        if (cout) store_slots<L, VEC>(cout + (size_t)c * P, lp, o);
        if (NORMS) {
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                nacc[s] = __fmaf_rn(o[s], o[s], nacc[s]);
                amax[s] = fmaxf(amax[s], fabsf(o[s]));
            }
        }
    };
    DwRaw<T, VEC> a, b;
    if (c_lo < c_hi) dwconv_load<T, VEC, ER, EC>(uin + (size_t)c_lo * P, w + (size_t)c_lo * 9, lp, H, W, a);
    for (int c = c_lo; c < c_hi; c += 2) {
        if (c + 1 < c_hi) dwconv_load<T, VEC, ER, EC>(uin + (size_t)(c + 1) * P, w + (size_t)(c + 1) * 9, lp, H, W, b);
        finish(a, c);
        if (c + 1 < c_hi) {
            if (c + 2 < c_hi) dwconv_load<T, VEC, ER, EC>(uin + (size_t)(c + 2) * P, w + (size_t)(c + 2) * 9, lp, H, W, a);
            finish(b, c + 1);
        }
    }
    if (NORMS) {
        if (nrm2) store_slots<L, VEC>(nrm2 + (size_t)n * P, lp, nacc);
        if (amaxpos) store_slots<L, VEC>(amaxpos + (size_t)n * P, lp, amax);
    }
}

// NORMS = false: a chunk of the channels (blockIdx.y), coefficients only.
template <typename T, int L, bool VEC, bool NORMS>
__global__ void __launch_bounds__(128)
dwconv_haar_fwd_kernel(const T* __restrict__ u, const float* __restrict__ w, int N, int C, int H, int W, int cpc,
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
    const T* uin = u + (size_t)n * C * P;
    float* cout = coef ? coef + (size_t)n * C * P : nullptr;
    const int c_lo = (int)blockIdx.y * cpc, c_hi = min(C, c_lo + cpc);

    // border tests only where the tile needs them
    const int ty0 = ty * TT::TH, tx0 = tx * TT::TW;
    const bool er = !(ty0 >= 1 && ty0 + TT::TH < H), ec = !(tx0 >= 1 && tx0 + TT::TW < W);
    if (!VEC || (er && ec)) dwconv_channels<T, L, VEC, NORMS, true, true>(uin, w, cout, c_lo, c_hi, lp, lane, n, H, W, nrm2, amaxpos);
    else if (er) dwconv_channels<T, L, VEC, NORMS, true, false>(uin, w, cout, c_lo, c_hi, lp, lane, n, H, W, nrm2, amaxpos);
    else if (ec) dwconv_channels<T, L, VEC, NORMS, false, true>(uin, w, cout, c_lo, c_hi, lp, lane, n, H, W, nrm2, amaxpos);
    else dwconv_channels<T, L, VEC, NORMS, false, false>(uin, w, cout, c_lo, c_hi, lp, lane, n, H, W, nrm2, amaxpos);
}

// Channel norms of a stored coefficient map: one thread per position builds the chain of fused multiply-adds over the
// channels in ascending order, from +0, and max |coef|.  Thirty-two channels of loads in flight per thread.
__global__ void __launch_bounds__(256)
coef_norms_kernel(const float* __restrict__ coef, int N, int C, long long P, float* __restrict__ nrm2, float* __restrict__ amaxpos)
{
    const long long id = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (id >= (long long)N * P) return;
    const long long n = id / P, p = id - n * P;
    const float* src = coef + (size_t)n * C * P + p;
    constexpr int UN = 32;
    float acc = 0.0f, am = 0.0f;
    int c = 0;
    for (; c + UN <= C; c += UN) {
        float v[UN];
#pragma unroll
        for (int i = 0; i < UN; ++i) v[i] = __ldcs(src + (size_t)(c + i) * P);
#pragma unroll
        for (int i = 0; i < UN; ++i) {
            acc = __fmaf_rn(v[i], v[i], acc);
            am = fmaxf(am, fabsf(v[i]));
        }
    }
    for (; c < C; ++c) {
        const float v = __ldcs(src + (size_t)c * P);
        acc = __fmaf_rn(v, v, acc);
        am = fmaxf(am, fabsf(v));
    }
    if (nrm2) nrm2[id] = acc;
    if (amaxpos) amaxpos[id] = am;
}

// Channels per chunk of the forward kernels: one chunk (norms in the same pass) when the tiles alone fill the GPU or no
// coefficient map is stored; otherwise chunks of a multiple of `unit` channels, about 64 warps for each of the 148 SMs.
static int forward_chunk_channels(long long tile_warps, int C, int unit, bool has_coef)
{
    constexpr long long want = 148 * 64;              // measured on the block's shapes: 24 to 96 warps per SM tried
    if (!has_coef || tile_warps >= want || C <= 2 * unit) return C;
    const long long chunks = std::min<long long>((C + unit - 1) / unit, (want + tile_warps - 1) / tile_warps);
    int cpc = (int)((C + chunks - 1) / chunks);
    cpc = (cpc + unit - 1) / unit * unit;
    return std::min(cpc, C);
}

static wcc_status launch_coef_norms(const float* coef, int N, int C, long long P, float* nrm2, float* amaxpos, cudaStream_t st)
{
    if (!nrm2 && !amaxpos) return WCC_OK;
    coef_norms_kernel<<<(unsigned)(((long long)N * P + 255) / 256), 256, 0, st>>>(coef, N, C, P, nrm2, amaxpos);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

// ---- per-warp asynchronous patch ring ------------------------------------------------------------
// Each lane copies its own 2 x 4 patch of a few channels ahead of use with cp.async (global -> shared, no
// registers held while the copy flies) and later reads back exactly the bytes it copied, so no barrier is needed:
// only the thread's own cp.async groups are waited for.  A stage holds LU channels; slot of (stage, channel d,
// row r, lane) = ((stage * LU + d) * 2 + r) * 32 + lane, ROWB bytes each (conflict-free: lanes are contiguous).
template <typename T, int LU_ = (sizeof(T) == 2) ? 4 : 2>
struct PatchRing {
    static constexpr int ROWB = 4 * (int)sizeof(T);              // bytes of one patch row: 8 (bf16) or 16 (fp32)
    static constexpr int LU = LU_;                               // channels per stage (default: 2 KB per warp and stage)
    static constexpr int STAGE_BYTES = LU * 2 * 32 * ROWB;

    // start the copies of channels [c0, c0 + LU) of one image into `stage`; always commits one group
    static __device__ __forceinline__ void issue(uint32_t ring, int stage, const T* __restrict__ xin, size_t P, int W,
                                                 int C, int c0, const LanePos& lp, int lane)
    {
#pragma unroll
        for (int d = 0; d < LU; ++d) {
            const int c = c0 + d;
            const bool valid = (c < C) && lp.ok0;
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                const T* src = valid ? xin + (size_t)c * P + (size_t)(lp.r0 + r) * W + lp.c0 : xin;
                const uint32_t dst = ring + (uint32_t)((((stage * LU + d) * 2 + r) * 32 + lane) * ROWB);
                const int nbytes = valid ? ROWB : 0;              // 0: the slot is zero-filled
                if (ROWB == 16)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
                else
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(nbytes) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }

    template <int PENDING>
    static __device__ __forceinline__ void wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

    static __device__ __forceinline__ void read(const uint8_t* ring, int stage, int d, int lane, RawPatch& raw)
    {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const uint8_t* src = ring + (size_t)((((stage * LU + d) * 2 + r) * 32 + lane) * ROWB);
            if (ROWB == 16) {
                const uint4 v = *reinterpret_cast<const uint4*>(src);
                raw.w[4 * r + 0] = v.x; raw.w[4 * r + 1] = v.y; raw.w[4 * r + 2] = v.z; raw.w[4 * r + 3] = v.w;
            } else {
                const uint2 v = *reinterpret_cast<const uint2*>(src);
                raw.w[4 * r + 0] = v.x; raw.w[4 * r + 1] = v.y;
            }
        }
    }
};

// ---- first pass of the fused layer without TMA (rows that are no multiple of 16 bytes, unaligned x) -----------
// Norms only, inputs through per-warp cp.async rings.
// One CTA of 4 warps per (image, tile).  The warps split the channels: in every round of 4 * LU channels warp w
// transforms channels [w * LU, (w + 1) * LU) of the round in registers and hands the slot values over through shared
// memory; then the 128 threads run the fused multiply-add chain of two positions each (warp w: slots 2w and 2w+1
// of every lane) over the round's channels in ascending order, so the sum is the same sequential chain a single
// thread would build.  Inputs arrive through the per-warp cp.async ring (RING stages ahead).  Only the norms and
// the per-position max |coef| are written, plus on request (NormsExtra): the coefficient map (tests), round 1 of
// the select's histogram (the 11 bits below the sign of every norm), and, in extra CTAs appended to
// the grid, the quantized weights (one warp per output channel), which saves a launch of its own.
struct NormsExtra {
    float* coef;          // fp32 [N][C][P] or NULL
    uint32_t* hist1;      // [N][3][2048] (round 1 first), zeroed by the caller, or NULL
    uint32_t* fine;       // [N][65536]: histogram of the 16 bits below the sign of every norm, zeroed by the caller, or NULL
    const float* Wt;      // weights to prepare in the extra CTAs, or NULL
    void* Wq;
    float* scale_w;
    int Cout, kpad, bits;
    int tiles;            // CTAs that transform; CTAs beyond prepare weights
};

// Last step of the first pass for warps 0..3: thread (warp, lane) owns slot pair `warp` of its lane; write the norms and
// the max |coef|, and count the norms in the select's histograms.
template <int L, bool VEC>
__device__ __forceinline__ void norms_finish(const LanePos& lp, int warp, int n, size_t P, float n0, float n1, float a0, float a1,
                                             float* __restrict__ nrm2, float* __restrict__ amaxpos, const NormsExtra& ex)
{
    int p0 = 0, p1 = 0;
    bool ok0 = false, ok1 = false;
#pragma unroll
    for (int s = 0; s < 8; s += 2) {
        if (s == 2 * warp) {
            p0 = lp.pos[s]; p1 = lp.pos[s + 1];
            ok0 = slot_ok<L>(lp, s); ok1 = slot_ok<L>(lp, s + 1);
        }
    }
    const bool pair = VEC && (L == 1 || warp < 3);     // adjacent, 8-byte aligned positions
    float* nr = nrm2 + (size_t)n * P;
    if (pair) {
        if (ok0) *reinterpret_cast<float2*>(nr + p0) = make_float2(n0, n1);
    } else {
        if (ok0) nr[p0] = n0;
        if (ok1) nr[p1] = n1;
    }
    if (amaxpos) {
        float* am = amaxpos + (size_t)n * P;
        if (pair) {
            if (ok0) *reinterpret_cast<float2*>(am + p0) = make_float2(a0, a1);
        } else {
            if (ok0) am[p0] = a0;
            if (ok1) am[p1] = a1;
        }
    }
    if (ex.hist1) {                                    // norms are >= +0: the digit is the 11 bits below the sign
        uint32_t* h = ex.hist1 + (size_t)n * 3 * 2048;
        hist_add(h, norm_digit11(n0), ok0 && n0 != 0.0f);             // zero norms are not counted (see the token kernel)
        hist_add(h, norm_digit11(n1), ok1 && n1 != 0.0f);
    }
    if (ex.fine) {                                     // 16-bit digits are spread out: plain atomics
        uint32_t* f = ex.fine + (size_t)n * 65536;
        if (ok0 && n0 != 0.0f) atomicAdd(&f[norm_digit16(n0)], 1u);
        if (ok1 && n1 != 0.0f) atomicAdd(&f[norm_digit16(n1)], 1u);
    }
}

constexpr int NORMS_WARPS = 8;     // warps per CTA: the transform is issue-latency bound, more warps hide it

template <typename T, int L, bool VEC>
__global__ void __launch_bounds__(NORMS_WARPS * 32)
haar_norms_kernel(const T* __restrict__ x, int N, int C, int H, int W,
                  float* __restrict__ nrm2, float* __restrict__ amaxpos, const NormsExtra ex)
{
    if ((int)blockIdx.x >= ex.tiles) {                 // weight preparation CTAs
        const int o = ((int)blockIdx.x - ex.tiles) * NORMS_WARPS + (int)(threadIdx.x >> 5);
        if (o < ex.Cout) weight_prep_row(ex.Wt, o, C, ex.kpad, ex.bits, ex.Wq, ex.scale_w);
        return;
    }
    using TT = HaarTile<L>;
    using Ring = PatchRing<T, (sizeof(T) == 2) ? 2 : 1>;
    constexpr int LU = Ring::LU, RC = NORMS_WARPS * LU;   // channels per warp and per round
    constexpr int RING = 4;                            // stages per warp
    __shared__ float2 buf[RC][4][32];                  // [channel of the round][slot pair][lane]
    __shared__ __align__(16) uint8_t ring_mem[VEC ? NORMS_WARPS * RING * Ring::STAGE_BYTES : 16];
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int n, ty, tx;
    tile_coords(blockIdx.x, tiles_x, tiles_y, n, ty, tx);
    const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
    const size_t P = (size_t)H * W;
    const T* xin = x + (size_t)n * C * P;
    uint8_t* my_ring = ring_mem + (VEC ? warp * RING * Ring::STAGE_BYTES : 0);
    const uint32_t my_ring_s = (uint32_t)__cvta_generic_to_shared(my_ring);

    float2 nn = make_float2(0.0f, 0.0f);
    float a0 = 0.0f, a1 = 0.0f;
    const int rounds = (C + RC - 1) / RC;
    if (VEC) {
#pragma unroll
        for (int r = 0; r < RING - 1; ++r) Ring::issue(my_ring_s, r, xin, P, W, C, r * RC + warp * LU, lp, lane);
    }
    for (int r = 0; r < rounds; ++r) {
        if (VEC) {
            Ring::issue(my_ring_s, (r + RING - 1) % RING, xin, P, W, C, (r + RING - 1) * RC + warp * LU, lp, lane);
            Ring::template wait<RING - 1>();
        }
        float p[LU][2][4], o[LU][8];
#pragma unroll
        for (int d = 0; d < LU; ++d) {
            const int c = r * RC + warp * LU + d;
            RawPatch raw;
            if (VEC) {
                Ring::read(my_ring, r % RING, d, lane, raw);          // channels beyond C arrive as zeros
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) raw.w[i] = 0u;
                if (c < C) load_patch<T, VEC>(xin + (size_t)c * P, W, lp, raw);
            }
            unpack_patch<T>(raw, p[d]);
        }
        haar_fwd_lanes<L, LU>(p, o, lane);
#pragma unroll
        for (int d = 0; d < LU; ++d) {
            const int c = r * RC + warp * LU + d;
#pragma unroll
            for (int s = 0; s < 8; s += 2) buf[warp * LU + d][s >> 1][lane] = make_float2(o[d][s], o[d][s + 1]);
            if (ex.coef && c < C) store_slots<L, VEC>(ex.coef + ((size_t)n * C + c) * P, lp, o[d]);
        }
        __syncthreads();
        // the chain: warps 0..3 own slot pair `warp` of every lane.  Channels beyond C contribute fma(0, 0, acc) = acc
        // and max(acc, 0) = acc: no special case needed
        if (warp < 4) {
#pragma unroll
            for (int c = 0; c < RC; ++c) {
                const float2 v = buf[c][warp][lane];
                nn = __ffma2_rn(v, v, nn);
                a0 = fmaxf(a0, fabsf(v.x));
                a1 = fmaxf(a1, fabsf(v.y));
            }
        }
        __syncthreads();
    }
    if (VEC) Ring::template wait<0>();
    if (warp >= 4) return;
    norms_finish<L, VEC>(lp, warp, n, P, nn.x, nn.y, a0, a1, nrm2, amaxpos, ex);
}

// ---- per-warp ring of TMA boxes --------------------------------------------------------------------
// One lane of a warp asks the TMA unit for boxes of CB channels x (tile rows) x (tile columns) of one image
// (cp.async.bulk.tensor, completion counted on an mbarrier per stage); no thread spends instructions or registers on
// addresses, and the copies bypass the load/store pipe.  A stage is laid out [channel][row][column], dense.  Only the
// owning warp reads a stage and only its lane 0 refills it (after __syncwarp), so no "empty" barrier is needed.
template <typename T, int L, int CB_, int S_>
struct TileRing {
    using TT = HaarTile<L>;
    static constexpr int CB = CB_, S = S_;
    static constexpr int ROW_BYTES = TT::TW * (int)sizeof(T);
    static constexpr int CH_BYTES = TT::TH * ROW_BYTES;          // 256 positions: 512 (bf16) or 1024 (fp32) bytes
    static constexpr int STAGE_BYTES = CB * CH_BYTES;
    static constexpr int BYTES = S * STAGE_BYTES;
    // bf16, L = 3: rows are 64 bytes, so the rows 2rp of the four lane rows would all start in the same banks; lanes
    // with odd rp read their second row first, which spreads one load over all 32 banks
    static constexpr bool ALT = (sizeof(T) == 2 && L == 3);

    uint32_t ring_s, bar_s;      // shared-space addresses of the stages and of the S mbarriers
    const uint8_t* ring;
    int off_a, off_b;            // byte offsets (inside a channel) of the row this lane reads first / second
    bool swap;                   // the first row read is the patch's second row

    // the same without touching the barriers (another thread initializes them and a block-wide barrier follows)
    __device__ __forceinline__ void attach(uint8_t* stages, uint64_t* bars, int lane)
    {
        ring = stages;
        ring_s = tc::smem_u32(stages);
        bar_s = tc::smem_u32(bars);
        set_lane(lane);
    }
    __device__ __forceinline__ void init(uint8_t* stages, uint64_t* bars, int lane)
    {
        ring = stages;
        ring_s = tc::smem_u32(stages);
        bar_s = tc::smem_u32(bars);
        set_lane(lane);
        if (lane == 0) {
#pragma unroll
            for (int i = 0; i < S; ++i) tc::mbar_init(bar_s + 8 * i, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
    }
    __device__ __forceinline__ void set_lane(int lane)
    {
        const int rp = lane / TT::CG, cg = lane % TT::CG;
        swap = ALT && (rp & 1);
        const int base = 2 * rp * ROW_BYTES + 4 * cg * (int)sizeof(T);
        off_a = base + (swap ? ROW_BYTES : 0);
        off_b = base + (swap ? 0 : ROW_BYTES);
    }
    // lane 0 only: request channels [c0, c0 + CB) of image n at tile origin (x0, y0) into `stage`
    __device__ __forceinline__ void issue(const CUtensorMap* tm, int stage, int x0, int y0, int c0, int n) const
    {
        tc::mbar_expect_tx(bar_s + 8 * stage, STAGE_BYTES);
        tc::tma_load_4d(ring_s + stage * STAGE_BYTES, tm, x0, y0, c0, n, bar_s + 8 * stage);
    }
    __device__ __forceinline__ bool wait(int stage, uint32_t parity) const { return tc::mbar_wait(bar_s + 8 * stage, parity); }

    // rows in the order they were read: for lanes with `swap` set the patch's second row comes first
    __device__ __forceinline__ void read_raw(int stage, int d, RawPatch& raw) const
    {
        const uint8_t* ch = ring + stage * STAGE_BYTES + d * CH_BYTES;
        if (sizeof(T) == 4) {
            const uint4 a = *reinterpret_cast<const uint4*>(ch + off_a);
            const uint4 b = *reinterpret_cast<const uint4*>(ch + off_b);
            raw.w[0] = a.x; raw.w[1] = a.y; raw.w[2] = a.z; raw.w[3] = a.w;
            raw.w[4] = b.x; raw.w[5] = b.y; raw.w[6] = b.z; raw.w[7] = b.w;
        } else {
            const uint2 a = *reinterpret_cast<const uint2*>(ch + off_a);
            const uint2 b = *reinterpret_cast<const uint2*>(ch + off_b);
            raw.w[0] = a.x; raw.w[1] = a.y; raw.w[4] = b.x; raw.w[5] = b.y;
        }
    }
    __device__ __forceinline__ void read(int stage, int d, RawPatch& raw) const
    {
        const uint8_t* ch = ring + stage * STAGE_BYTES + d * CH_BYTES;
        if (sizeof(T) == 4) {
            const uint4 a = *reinterpret_cast<const uint4*>(ch + off_a);
            const uint4 b = *reinterpret_cast<const uint4*>(ch + off_b);
            raw.w[0] = a.x; raw.w[1] = a.y; raw.w[2] = a.z; raw.w[3] = a.w;
            raw.w[4] = b.x; raw.w[5] = b.y; raw.w[6] = b.z; raw.w[7] = b.w;
        } else {
            const uint2 a = *reinterpret_cast<const uint2*>(ch + off_a);
            const uint2 b = *reinterpret_cast<const uint2*>(ch + off_b);
            raw.w[0] = (ALT && swap) ? b.x : a.x; raw.w[1] = (ALT && swap) ? b.y : a.y;
            raw.w[4] = (ALT && swap) ? a.x : b.x; raw.w[5] = (ALT && swap) ? a.y : b.y;
        }
    }
};

// After a wait ran out: report it and give copies that may still be in flight time to land before the CTA's shared
// memory is handed to another CTA.
__device__ __noinline__ void tma_timeout(int* status)
{
    if ((threadIdx.x & 31) == 0) atomicExch(status, (int)WCC_ERR_TIMEOUT);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
}

// ---- first pass, TMA-fed, the norm chain handed from warp to warp ------------------------------------------
// One CTA of W warps per tile.  The warps take the boxes of CB channels in turn (box r goes to warp r % W): each transforms
// its box on its own, fed by its own ring of TMA boxes, and only the chain of fused multiply-adds that builds the norms
// (one per position, ascending channel order) runs in sequence: the eight partial sums of every lane travel from the warp
// of box r to the warp of box r + 1 through shared memory (a "token", signalled on an mbarrier).  So the sums are the
// same sequential chains a single thread would build, while loads, unpacking, transforms and maxima of different boxes
// overlap.  The transform runs without its halvings (haar_fwd_lanes_raw); one exact multiplication per slot at the end.
// NW warps share a tile (one CTA = one tile at a time): 4 when tiles are few and deep in channels, so that enough warps
// are in flight; 1 when there are many tiles, which needs no hand-over at all (C4-like maps: 20.5 us instead of 24.5).
template <typename T, int L, int NW_>
struct NormsTokCfg {
    static constexpr int W = NW_;                                 // warps per tile
    static constexpr int CB = (sizeof(T) == 2) ? 8 : 4;           // channels per box: 4 KB
    static constexpr int S = 3;                                   // boxes in flight per warp
    using Ring = TileRing<T, L, CB, S>;
    static constexpr size_t SMEM = 128 + (size_t)W * Ring::BYTES + 8 * 32 * 4 + (size_t)W * 8 * 32 * 4 + (size_t)W * S * 8 + W * 8;
};

template <typename T, int L, int NW_>
__global__ void __launch_bounds__(NW_ * 32, 16 / NW_)
haar_norms_token_kernel(const __grid_constant__ CUtensorMap tmx, int N, int C, int H, int W, int tiles_total, int tile_ctas,
                        float* __restrict__ nrm2, float* __restrict__ amaxpos, const NormsExtra ex, int* __restrict__ status)
{
    using TT = HaarTile<L>;
    using Cfg = NormsTokCfg<T, L, NW_>;
    using Ring = typename Cfg::Ring;
    constexpr int CB = Cfg::CB, S = Cfg::S, NW = Cfg::W;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((int)blockIdx.x >= tile_ctas) {                // weight preparation CTAs
        const int o = ((int)blockIdx.x - tile_ctas) * NW + warp;
        if (o < ex.Cout) weight_prep_row(ex.Wt, o, C, ex.kpad, ex.bits, ex.Wq, ex.scale_w);
        return;
    }
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_s = tc::smem_u32(smem_raw);
    uint8_t* sm = smem_raw + (((raw_s + 127u) & ~127u) - raw_s);
    uint8_t* stages = sm + (size_t)warp * Ring::BYTES;
    float4* token = reinterpret_cast<float4*>(sm + (size_t)NW * Ring::BYTES);                 // [2][32] float4: 8 sums per lane
    float* amax_sm = reinterpret_cast<float*>(token + 2 * 32);                                 // [NW][8][32]
    uint64_t* ring_bars = reinterpret_cast<uint64_t*>(amax_sm + NW * 8 * 32);                   // [NW][S]
    uint64_t* tok_bars = ring_bars + NW * S;                                                    // [NW]

    // The CTA walks the tiles blockIdx.x, blockIdx.x + tile_ctas, ...; a warp's ring of boxes runs on across tiles, so
    // the first boxes of the next tile are in flight while the current one is finished.
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const size_t P = (size_t)H * W;
    const int iters = (tiles_total - (int)blockIdx.x + tile_ctas - 1) / tile_ctas;
    const int rounds = (C + CB - 1) / CB;
    const int mine = (rounds - warp + NW - 1) / NW;    // boxes of this warp per tile: r = warp + m * NW
    const int total = iters * mine;
    Ring ring;
    ring.init(stages, ring_bars + warp * S, lane);
    // The next box to request, kept as running counters (a division per box would cost more issue slots than the
    // transform of the box's channels): box `iss_mi` of this warp in tile (iss_n, iss_ty, iss_tx), into stage `iss_stage`.
    int iss_mi = 0, iss_it = 0, iss_stage = 0, iss_n = 0, iss_ty = 0, iss_tx = 0, issued = 0;
    tile_coords((int)blockIdx.x, tiles_x, tiles_y, iss_n, iss_ty, iss_tx);
    auto issue_next = [&]() {                          // all lanes keep the counters, lane 0 talks to the TMA unit
        if (issued >= total) return;
        if (lane == 0) ring.issue(&tmx, iss_stage, iss_tx * TT::TW, iss_ty * TT::TH, (warp + iss_mi * NW) * CB, iss_n);
        ++issued;
        if (++iss_stage == S) iss_stage = 0;
        if (++iss_mi == mine) {
            iss_mi = 0;
            ++iss_it;
            tile_coords((int)blockIdx.x + iss_it * tile_ctas, tiles_x, tiles_y, iss_n, iss_ty, iss_tx);
        }
    };
#pragma unroll
    for (int m = 0; m < S; ++m) issue_next();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < NW; ++i) tc::mbar_init(tc::smem_u32(&tok_bars[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    float sc[8];
    slot_scales<L>(lane, ring.swap, sc);
    bool ok = true;
    int tok_seen = 0;                                  // tokens received so far
    int stage = 0;                                     // stage of the next box to consume, and its barrier's parity
    uint32_t parity = 0;
    for (int it = 0; it < iters; ++it) {
        int n, ty, tx;
        tile_coords((int)blockIdx.x + it * tile_ctas, tiles_x, tiles_y, n, ty, tx);
        const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
        float amax[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) amax[s] = 0.0f;
        for (int m = 0; m < mine && ok; ++m) {
            const int r = warp + m * NW;
            ok = ring.wait(stage, parity);
            RawPatch raw[CB];
#pragma unroll
            for (int d = 0; d < CB; ++d) ring.read_raw(stage, d, raw[d]);      // channels beyond C arrive as zeros: fma(0, 0, acc) = acc
            if (ex.coef) {                             // test tap: the plain transform (also gets the signs of zeros right)
#pragma unroll
                for (int d = 0; d < CB; ++d) {
                    if (r * CB + d < C) {
                        RawPatch rw;
                        float pp[2][4], oc[8];
                        ring.read(stage, d, rw);
                        unpack_patch<T>(rw, pp);
                        haar_fwd_lane<L>(pp, oc, lane);
                        store_slots<L, true>(ex.coef + ((size_t)n * C + r * CB + d) * P, lp, oc);
                    }
                }
            }
            __syncwarp();                              // every lane is done reading the stage
            issue_next();                              // refills exactly this stage (S boxes are always in flight)
            if (++stage == S) { stage = 0; parity ^= 1u; }
            float o[CB][8];
#pragma unroll
            for (int g = 0; g < CB / 4; ++g) {
                float p[4][2][4];
#pragma unroll
                for (int d = 0; d < 4; ++d) unpack_patch<T>(raw[g * 4 + d], p[d]);
                haar_fwd_lanes_raw<L, 4>(p, *reinterpret_cast<float(*)[4][8]>(&o[g * 4]), lane);
            }
#pragma unroll
            for (int d = 0; d < CB; ++d)
#pragma unroll
                for (int s = 0; s < 8; ++s) amax[s] = fmaxf(amax[s], fabsf(o[d][s]));
            // the token: partial sums of the boxes before this one
            float2 acc[4];
            if (r > 0) {
                ok = ok && tc::mbar_wait(tc::smem_u32(&tok_bars[warp]), (uint32_t)tok_seen & 1u);
                ++tok_seen;
                const float4 t0 = token[lane], t1 = token[32 + lane];
                acc[0] = make_float2(t0.x, t0.y); acc[1] = make_float2(t0.z, t0.w);
                acc[2] = make_float2(t1.x, t1.y); acc[3] = make_float2(t1.z, t1.w);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[i] = make_float2(0.0f, 0.0f);
            }
#pragma unroll
            for (int d = 0; d < CB; ++d)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 v = make_float2(o[d][2 * i], o[d][2 * i + 1]);
                    acc[i] = __ffma2_rn(v, v, acc[i]);
                }
            if (r + 1 < rounds) {
                token[lane] = make_float4(acc[0].x, acc[0].y, acc[1].x, acc[1].y);
                token[32 + lane] = make_float4(acc[2].x, acc[2].y, acc[3].x, acc[3].y);
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(tc::smem_u32(&tok_bars[(warp + 1) % NW]));
            } else if (ok) {                           // last box: these are the norms
                float nacc[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    nacc[2 * i] = __fmul_rn(acc[i].x, __fmul_rn(sc[2 * i], sc[2 * i]));
                    nacc[2 * i + 1] = __fmul_rn(acc[i].y, __fmul_rn(sc[2 * i + 1], sc[2 * i + 1]));
                }
                store_slots<L, true>(nrm2 + (size_t)n * P, lp, nacc);
                // Norms that are exactly zero are not counted: after a ReLU whole regions of a map are zero, and their
                // positions would all hit one bin (thousands of atomics on one address).  The selection knows the number
                // of positions, so the zeros are what the bins leave out; they rank below everything else.
                if (ex.hist1) {                        // norms are >= +0: the digit is the 11 bits below the sign
                    uint32_t* h = ex.hist1 + (size_t)n * 3 * 2048;
#pragma unroll
                    for (int s = 0; s < 8; ++s) hist_add(h, norm_digit11(nacc[s]), lp.ok0 && nacc[s] != 0.0f);
                }
                if (ex.fine && lp.ok0) {               // 16-bit digits of non-zero norms are spread out: plain atomics
                    uint32_t* f = ex.fine + (size_t)n * 65536;
#pragma unroll
                    for (int s = 0; s < 8; ++s)
                        if (nacc[s] != 0.0f) atomicAdd(&f[norm_digit16(nacc[s])], 1u);
                }
            }
        }
        // per-position max |coef|: combine the warps' maxima.  The two block-wide barriers also keep every token of
        // this tile ahead of any token of the next one (a single token buffer is enough).
#pragma unroll
        for (int s = 0; s < 8; ++s) amax_sm[(warp * 8 + s) * 32 + lane] = amax[s];
        __syncthreads();
        if (warp == 0 && amaxpos) {
            float am[8];
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                float v = amax_sm[s * 32 + lane];
#pragma unroll
                for (int w2 = 1; w2 < NW; ++w2) v = fmaxf(v, amax_sm[(w2 * 8 + s) * 32 + lane]);
                am[s] = __fmul_rn(v, fabsf(sc[s]));
            }
            store_slots<L, true>(amaxpos + (size_t)n * P, lp, am);
        }
        __syncthreads();
    }
    if (!__all_sync(0xFFFFFFFFu, ok ? 1 : 0)) tma_timeout(status);
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
// One warp per (image, tile, group of ocw output channels; ocw a multiple of 4).  rank[n][p] is the row of position p
// in the compressed matrix (or -1 when p was dropped: the zero map).  acc row r = n*k + rank holds the int32
// accumulators (or fp32 products when ACCF) of all output channels, pitch ldc (multiple of 4).  The accumulators of
// the next four channels are gathered while the current four are transformed.
template <typename T, int L, bool VEC, bool ACCF>
__global__ void __launch_bounds__(128, 5)
scatter_inv_kernel(const int32_t* __restrict__ acc, int ldc, const int32_t* __restrict__ rank,
                   const float* __restrict__ amax_kept, float qmax, const float* __restrict__ scale_w,
                   int N, int Cout, int ocw, int H, int W, int k, T* __restrict__ y, const T* __restrict__ residual, int relu)
{
    using TT = HaarTile<L>;
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    const int groups = (Cout + ocw - 1) / ocw;
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

    // Four channels at a time: dequantize straight into the pre-scaled slots of haar_inv_lanes_raw, acc * (scale * 2^-level)
    // (the halvings of the inverse transform are exact powers of two and commute with every rounding).
    const bool coarse6 = L == 3 && ((lane / TT::CG) & 1) == 0;         // slot 6 holds a level-3 coefficient
    const int o_end = min(Cout, (g + 1) * ocw);
    int4 v[8], vn[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        v[s] = rowp[s] ? __ldg(reinterpret_cast<const int4*>(rowp[s] + g * ocw)) : make_int4(0, 0, 0, 0);
        vn[s] = v[s];
    }
    for (int o0 = g * ocw; o0 < o_end; o0 += 4) {
        if (o0 + 4 < o_end) {
#pragma unroll
            for (int s = 0; s < 8; ++s)
                vn[s] = rowp[s] ? __ldg(reinterpret_cast<const int4*>(rowp[s] + o0 + 4)) : make_int4(0, 0, 0, 0);
        }
        float sl[4][8], p[4][2][4];
#pragma unroll
        for (int d = 0; d < 4; ++d) {
            const int o = o0 + d;
            float sc = 1.0f;
            if (!ACCF) sc = (o < o_end) ? __fmul_rn(scale_a, scale_w[o]) : 0.0f;
            const float s1 = __fmul_rn(sc, 0.5f), s2 = __fmul_rn(sc, 0.25f);
            const float s6 = (L == 1) ? s1 : (coarse6 ? __fmul_rn(sc, 0.125f) : s2), s7 = (L == 1) ? s1 : s2;
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                const int a = (d == 0) ? v[s].x : (d == 1) ? v[s].y : (d == 2) ? v[s].z : v[s].w;
                const float f = ACCF ? __int_as_float(a) : __int2float_rn(a);
                sl[d][s] = __fmul_rn(f, s < 6 ? s1 : (s == 6 ? s6 : s7));
            }
        }
        haar_inv_lanes_raw<L, 4>(sl, p, lane);
#pragma unroll
        for (int d = 0; d < 4; ++d) {
            const int o = o0 + d;
            if (o < o_end) {      // warp-uniform
                if (residual) {                        // the skip connection (Eq. 13): one fp32 addition per element
                    RawPatch rr;
                    float rp[2][4];
#pragma unroll
                    for (int i = 0; i < 8; ++i) rr.w[i] = 0u;
                    load_patch<T, VEC>(residual + ((size_t)n * Cout + o) * P, W, lp, rr);
                    unpack_patch<T>(rr, rp);
#pragma unroll
                    for (int a = 0; a < 2; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) p[d][a][b] = __fadd_rn(p[d][a][b], rp[a][b]);
                }
                if (relu) {
#pragma unroll
                    for (int a = 0; a < 2; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) p[d][a][b] = fmaxf(p[d][a][b], 0.0f);
                }
                store_patch<T, VEC>(y + ((size_t)n * Cout + o) * P, W, lp, p[d]);
            }
        }
#pragma unroll
        for (int s = 0; s < 8; ++s) v[s] = vn[s];
    }
}

// ---- launchers -------------------------------------------------------------------------------
template <typename T, int L, bool VEC>
static wcc_status haar_norms_dispatch(const void* x, int N, int C, int H, int W, float* nrm2, float* amaxpos,
                                      NormsExtra ex, cudaStream_t st);

template <typename T, int L, bool VEC>
static wcc_status haar_fwd_dispatch(const void* x, int N, int C, int H, int W, float* coef, float* nrm2,
                                    float* amaxpos, cudaStream_t st)
{
    using TT = HaarTile<L>;
    constexpr int D = (sizeof(T) == 4) ? 4 : 8;
    const long long warps = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    if (!coef && nrm2) return haar_norms_dispatch<T, L, VEC>(x, N, C, H, W, nrm2, amaxpos, NormsExtra{}, st);   // norms only
    const int blocks = (int)((warps + 3) / 4);
    const int cpc = forward_chunk_channels(warps, C, D, coef != nullptr);
    const dim3 grid(blocks, ceil_div(C, cpc));
    haar_fwd_kernel<T, L, VEC, D><<<grid, 128, 0, st>>>(static_cast<const T*>(x), N, C, H, W, cpc, coef, nrm2, amaxpos);
    WCC_LAUNCH_CHECK();
    if (grid.y > 1) return launch_coef_norms(coef, N, C, (long long)H * W, nrm2, amaxpos, st);
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

template <typename T, int L, bool VEC>
static wcc_status haar_norms_dispatch(const void* x, int N, int C, int H, int W, float* nrm2, float* amaxpos,
                                      NormsExtra ex, cudaStream_t st)
{
    using TT = HaarTile<L>;
    const long long tiles = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    if (VEC && tc::tma_ok_x(x, (int)sizeof(T), W)) {
        if (tiles > 0x7FFFFFFFLL) return WCC_ERR_SHAPE;
        static int sm_count[64] = {0};
        int dev = 0;
        WCC_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return WCC_ERR_CUDA;
        if (!sm_count[dev]) WCC_CUDA_TRY(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
        int* status = nullptr;
        WCC_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_status));
        ex.tiles = (int)tiles;
        // sixteen warps per SM are resident whatever the split: as many warps per tile as keeps them all busy
        const long long warps = 16LL * sm_count[dev];
        auto launch = [&](auto kern, auto cfg) -> wcc_status {
            using Cfg = decltype(cfg);
            CUtensorMap tmx;
            if (!tc::make_map_x(&tmx, x, (int)sizeof(T), N, C, H, W, TT::TW, TT::TH, Cfg::CB)) return WCC_ERR_CUDA;
            WCC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM));
            const long long resident = warps / Cfg::W;                  // every tile CTA is resident at once
            const int tile_ctas = (int)(tiles < resident ? tiles : resident);
            const long long grid = tile_ctas + (ex.Wt ? ceil_div(ex.Cout, Cfg::W) : 0);
            kern<<<(unsigned)grid, Cfg::W * 32, Cfg::SMEM, st>>>(tmx, N, C, H, W, (int)tiles, tile_ctas, nrm2, amaxpos, ex, status);
            WCC_LAUNCH_CHECK();
            return WCC_OK;
        };
        if (tiles * 2 > warps) return launch(haar_norms_token_kernel<T, L, 1>, NormsTokCfg<T, L, 1>{});
        if (tiles * 4 > warps) return launch(haar_norms_token_kernel<T, L, 2>, NormsTokCfg<T, L, 2>{});
        return launch(haar_norms_token_kernel<T, L, 4>, NormsTokCfg<T, L, 4>{});
    }
    ex.tiles = (int)tiles;
    const long long grid = tiles + (ex.Wt ? ceil_div(ex.Cout, NORMS_WARPS) : 0);
    haar_norms_kernel<T, L, VEC><<<(unsigned)grid, NORMS_WARPS * 32, 0, st>>>(static_cast<const T*>(x), N, C, H, W, nrm2, amaxpos, ex);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

// First pass of the fused layer (see haar_norms_kernel); ex.tiles is filled in here.
wcc_status launch_haar_norms(const void* x, int N, int C, int H, int W, int L, wcc_dtype dt,
                             float* nrm2, float* amaxpos, const NormsExtra& ex, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;
    WCC_DISPATCH_TLV(haar_norms_dispatch, dt, L, vec, x, N, C, H, W, nrm2, amaxpos, ex, st);
}

template <typename T, int L, bool VEC>
static wcc_status dwconv_haar_dispatch(const void* u, const float* w, int N, int C, int H, int W, float* coef, float* nrm2,
                                       float* amaxpos, cudaStream_t st)
{
    using TT = HaarTile<L>;
    const long long warps = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    const int blocks = (int)((warps + 3) / 4);
    const int cpc = forward_chunk_channels(warps, C, 8, coef != nullptr);
    const dim3 grid(blocks, ceil_div(C, cpc));
    if (grid.y > 1)
        dwconv_haar_fwd_kernel<T, L, VEC, false><<<grid, 128, 0, st>>>(static_cast<const T*>(u), w, N, C, H, W, cpc, coef, nullptr, nullptr);
    else
        dwconv_haar_fwd_kernel<T, L, VEC, true><<<grid, 128, 0, st>>>(static_cast<const T*>(u), w, N, C, H, W, cpc, coef, nrm2, amaxpos);
    WCC_LAUNCH_CHECK();
    if (grid.y > 1) return launch_coef_norms(coef, N, C, (long long)H * W, nrm2, amaxpos, st);
    return WCC_OK;
}

// Depthwise 3x3 convolution + forward Haar + norms (+ per-position max |coef|) in one pass over u.
wcc_status launch_dwconv_haar_fwd(const void* u, const float* w, int N, int C, int H, int W, int L, wcc_dtype dt,
                                  float* coef, float* nrm2, float* amaxpos, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;
    WCC_DISPATCH_TLV(dwconv_haar_dispatch, dt, L, vec, u, w, N, C, H, W, coef, nrm2, amaxpos, st);
}

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
                                       int N, int Cout, int H, int W, int k, void* y, const void* residual, int relu,
                                       cudaStream_t st)
{
    using TT = HaarTile<L>;
    // channels per warp: as many as still leave about 32 warps for each of the 148 SMs (8 to 64)
    const long long tiles = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    int ocw = 64;
    while (ocw > 8 && tiles * ceil_div(Cout, ocw) < 148 * 32) ocw >>= 1;
    const long long warps = tiles * ceil_div(Cout, ocw);
    const int blocks = (int)((warps + 3) / 4);
    if (accf)
        scatter_inv_kernel<T, L, VEC, true><<<blocks, 128, 0, st>>>(acc, ldc, rank, amax_kept, qmax, scale_w,
                                                                     N, Cout, ocw, H, W, k, static_cast<T*>(y),
                                                                     static_cast<const T*>(residual), relu);
    else
        scatter_inv_kernel<T, L, VEC, false><<<blocks, 128, 0, st>>>(acc, ldc, rank, amax_kept, qmax, scale_w,
                                                                      N, Cout, ocw, H, W, k, static_cast<T*>(y),
                                                                      static_cast<const T*>(residual), relu);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

wcc_status launch_scatter_inv(const int32_t* acc, int ldc, bool acc_is_float, const int32_t* rank,
                              const float* amax_kept, int bits, const float* scale_w,
                              int N, int Cout, int H, int W, int L, int k, wcc_dtype dt, void* y, cudaStream_t st,
                              const void* residual, int relu)
{
    const bool vec = (W % 4) == 0;
    const float qmax = (bits >= 2) ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    WCC_DISPATCH_TLV(scatter_inv_dispatch, dt, L, vec, acc, ldc, acc_is_float, rank, amax_kept, qmax, scale_w,
                     N, Cout, H, W, k, y, residual, relu, st);
}

}  // namespace wcc

// Second pass of the fused layer, one tile per CTA.  wcc_forward uses it for the shapes that the four-tile kernel of
// fused_tiles.cuh does not cover (input rows that cannot be a TMA map, many output channels together with many K steps);
// that kernel also borrows the descriptor and TMEM helpers below.
// For one warp tile of one image, recompute the Haar transform from x, keep the
// selected positions (zero the others), quantize, run the pointwise convolution on tensor cores, dequantize,
// apply the inverse transform and store y (steps A, C, D, E of the WCC workflow, Eq. 9 / Alg. 1, with the index
// set and the activation scale of step B already known).  Neither the coefficient map, nor the compressed matrix,
// nor the accumulators, nor the zero-filled map ever reach HBM.
//
// One CTA = 4 warps = one warp tile (32 lanes x 8 slots = 256 wavelet-domain positions, see haar.cuh).
//  phase 1  the four warps split the input channels in units of 8; every lane transforms its 2x4 patch of each
//           channel in registers and writes the eight quantized (or bf16) slot values into the A operand in shared
//           memory.  Row of a position in A: slot * 32 + lane, so one MMA block of 128 rows is four slots.
//           Dropped positions are written as zeros: their accumulators are zero, which is the zero-filled map.
//  phase 2  one thread issues tcgen05.mma (kind::i8, int32 accumulate; or kind::f16 on bf16, fp32 accumulate):
//           D[256 x Cout] = A[256 x Cin] * Wq[Cout x Cin]^T, two M blocks, output channels in chunks of <= 64.
//  phase 3  warp w reads TMEM lane quarter w (slots w and w+4 of all lanes) with tcgen05.ld, dequantizes and
//           transposes through shared memory so that every lane gets its own eight slots back; inverse transform
//           by warp shuffles, stores of y.
// Operands use the no-swizzle K-major core-matrix layout (8 rows x 16 bytes contiguous): element (row, 16-byte
// K chunk j) at j * rows * 16 + row * 16, i.e. leading (K) offset rows*16 bytes, stride (M/N) offset 128 bytes.
// The single mbarrier wait is bounded and reports WCC_ERR_TIMEOUT.
#pragma once

#include "common.cuh"
#include "contract.cuh"
#include "haar.cuh"

namespace wcc {
namespace fz {

constexpr int ROWS = 256;            // positions per CTA
constexpr int SUB = 16;              // output channels per transpose round
constexpr int RING2 = 3;             // cp.async stages per warp in phase 1
constexpr float MAGIC = 12582912.0f; // 1.5 * 2^23: adding it rounds to the nearest integer, ties to even

__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | ((lbo_bytes >> 4) << 16);
    const uint32_t hi = (sbo_bytes >> 4) | (1u << 14);      // version 1, layout type 0 (no swizzle)
    return ((uint64_t)hi << 32) | lo;
}

__device__ __forceinline__ void tmem_ld8_nowait(uint32_t taddr, uint32_t (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
}

// y = WCC(x) + residual: one fp32 addition per element of the lane's patch (Eq. 13)
template <typename T, bool VEC>
__device__ __forceinline__ void add_residual(const T* __restrict__ plane, int W, const LanePos& lp, float (&p)[2][4])
{
    RawPatch rr;
    float rp[2][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) rr.w[i] = 0u;
    load_patch<T, VEC>(plane, W, lp, rr);
    unpack_patch<T>(rr, rp);
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) p[a][b] = __fadd_rn(p[a][b], rp[a][b]);
}
__device__ __forceinline__ void relu_patch(float (&p)[2][4])
{
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) p[a][b] = fmaxf(p[a][b], 0.0f);
}

struct Ctl {
    uint64_t mma_done;
    uint32_t tmem_base;
    int pad;
};

template <typename T, int L, bool VEC, bool I8>
__global__ void __launch_bounds__(128, 4)
fused_pass2_kernel(const T* __restrict__ x, const uint8_t* __restrict__ Wq, const int32_t* __restrict__ rank,
                   const float* __restrict__ nrm2, const uint32_t* __restrict__ thr, const float* __restrict__ amax_kept, float qmax, const float* __restrict__ scale_w,
                   int N, int Cin, int Cout, int H, int W, int k, int kpad, int npad, int nchunk, int tmem_cols, int a_ksteps,
                   T* __restrict__ y, uint8_t* __restrict__ xq_tap, int32_t* __restrict__ acc_tap, int* __restrict__ status,
                   float alpha, int relu, const T* __restrict__ residual)
{
    using TT = HaarTile<L>;
    constexpr int ES = I8 ? 1 : 2;                    // operand element size
    constexpr int UNIT_BYTES = 8 * ES;                // 8 channels of one position
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = tc::smem_u32(smem_raw);
    const uint32_t base = (raw + 127u) & ~127u;
    uint8_t* sm = smem_raw + (base - raw);
    const int krow = kpad * ES;                       // bytes of K per row
    const int kchunks = krow / 16;
    using Ring = PatchRing<T>;
    uint8_t* sA = sm;                                                   // [2 * a_ksteps][256][16]
    uint8_t* sB = sA + (size_t)a_ksteps * 2 * ROWS * 16;                // [kchunks][npad][16]
    int32_t* srank = reinterpret_cast<int32_t*>(sB + (size_t)kchunks * npad * 16);      // [8][32]
    Ctl* ctl = reinterpret_cast<Ctl*>(srank + 8 * 32);
    uint8_t* shared_region = reinterpret_cast<uint8_t*>(ctl + 1);       // phase 1: input rings; phase 3: transpose buffer
    float* stage = reinterpret_cast<float*>(shared_region);             // [SUB][8][32]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_x = (W + TT::TW - 1) / TT::TW, tiles_y = H / TT::TH;
    int n, ty, tx;
    tile_coords(blockIdx.x, tiles_x, tiles_y, n, ty, tx);
    const LanePos lp = lane_positions<L>(H, W, ty, tx, lane);
    const size_t P = (size_t)H * W;

    // ---- phase 0: barrier, TMEM, ranks, weights ---------------------------------------------------
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&ctl->mma_done), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(tc::smem_u32(&ctl->tmem_base)), "r"((uint32_t)tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // start the first ring stages before the (slower) scattered loads of the keep / drop decisions
    const T* xin = x + (size_t)n * Cin * P;
    constexpr int LU = Ring::LU, SUBS = 8 / LU;
    constexpr int UPK = 32 / UNIT_BYTES;               // units per K step
    const int ksteps = krow / 32;
    const int halves = (a_ksteps < ksteps) ? 2 : 1;
    uint8_t* my_ring = shared_region + (VEC ? warp * RING2 * Ring::STAGE_BYTES : 0);
    const uint32_t my_ring_s = tc::smem_u32(my_ring);
    // units of half h taken by this warp: u0 + warp, u0 + warp + 4, ... below ur (units from ur on are zero padding)
    auto half_units = [&](int h, int& u0, int& u1, int& ur, int& my_units) {
        const int ks0 = h * a_ksteps, ks1 = min(ksteps, ks0 + a_ksteps);
        u0 = ks0 * UPK; u1 = ks1 * UPK;
        ur = min(u1, max(u0, (Cin + 7) / 8));
        my_units = max(0, (ur - u0 - warp + 3) / 4);
    };
    auto ring_prologue = [&](int h) {
        if (!VEC) return;
        int u0, u1, ur, my_units;
        half_units(h, u0, u1, ur, my_units);
        const int nq = my_units * SUBS;
#pragma unroll
        for (int q = 0; q < RING2 - 1; ++q)
            Ring::issue(my_ring_s, q, xin, P, W, q < nq ? Cin : 0, (u0 + warp + 4 * (q / SUBS)) * 8 + (q % SUBS) * LU, lp, lane);
    };
    ring_prologue(0);
    // kept or dropped: from the rank map when the select wrote one (thr[n][2] != 0: partial ties, or a test wants
    // the ranks), else by comparing the position's norm with the threshold key
    const uint32_t tkey = thr[n * 4], use_rank = thr[n * 4 + 2];
    int rk[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        rk[s] = -1;
        if (slot_ok<L>(lp, s)) {
            if (use_rank) rk[s] = rank[(size_t)n * P + lp.pos[s]];
            else rk[s] = (float_key(nrm2[(size_t)n * P + lp.pos[s]]) >= tkey) ? 0 : -1;
        }
        if (warp == 0) srank[s * 32 + lane] = rk[s];
    }
    for (int i = threadIdx.x; i < npad * kchunks; i += 128) {
        const int row = i / kchunks, j = i - row * kchunks;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row < Cout) v = *reinterpret_cast<const uint4*>(Wq + (size_t)row * krow + j * 16);
        *reinterpret_cast<uint4*>(sB + ((size_t)j * npad + row) * 16) = v;
    }
    float inv = 0.0f, scale_a = 1.0f;
    if (I8) {
        const float amax = (alpha > 0.0f) ? alpha : *amax_kept;
        inv = (amax > 0.0f) ? __fdiv_rn(qmax, amax) : 0.0f;
        scale_a = __fdiv_rn(amax, qmax);
    } else {
        inv = 1.0f;
    }
    float mul[8];                      // per slot: the quantization factor, or 0 for a dropped position
#pragma unroll
    for (int s = 0; s < 8; ++s) mul[s] = (rk[s] >= 0) ? inv : 0.0f;

    // ---- phases 1 + 2: transform + quantize into the A operand, tensor-core contraction ----------------
    // A holds a_ksteps K steps (32 bytes of K each).  When the input channels need more than that (and there is a
    // single chunk of output channels) the K range is done in two halves that accumulate into the same TMEM tile, so
    // that A stays small enough for four CTAs per SM.
    // Warp w takes the 8-channel units w, w+4, ... of a half; inputs arrive LU channels at a time through its ring.
    const uint32_t a_addr = tc::smem_u32(sA), b_addr = tc::smem_u32(sB);
    volatile int no_abort = 0;
    uint32_t commits = 0;                              // MMA batches committed so far (same value in every thread)
    uint32_t tmem = 0;
    bool ok = true;
    auto issue_mmas = [&](int ks0, int ks1, int ks_base, int n0, int cur) {   // thread 0 only
        const uint32_t idesc = (I8 ? (2u << 4) : (1u << 4)) | (1u << 7) | (1u << 10) |
                               ((uint32_t)(cur >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        for (int b = 0; b < 2; ++b) {
            for (int ks = ks0; ks < ks1; ++ks) {
                const uint64_t ad = smem_desc_plain(a_addr + (uint32_t)((ks - ks_base) * 2 * ROWS * 16 + b * 128 * 16), ROWS * 16, 128);
                const uint64_t bd = smem_desc_plain(b_addr + (uint32_t)(ks * 2 * npad * 16 + n0 * 16), (uint32_t)npad * 16, 128);
                tc::mma_ss<I8>(tmem + (uint32_t)(b * nchunk), ad, bd, idesc, ks > 0 ? 1u : 0u);
            }
        }
        tc::mma_commit(tc::smem_u32(&ctl->mma_done));
    };

    for (int h = 0; h < halves; ++h) {
        const int ks0 = h * a_ksteps, ks1 = min(ksteps, ks0 + a_ksteps);
        int u0, u1, ur, my_units;
        half_units(h, u0, u1, ur, my_units);
        if (h > 0) {                                   // the tensor core still reads A: wait for the first half
            ok = tc::mbar_wait(tc::smem_u32(&ctl->mma_done), (commits - 1u) & 1u, &no_abort);
            ok = __syncthreads_and(ok ? 1 : 0) != 0;
            if (!ok) break;
            tc::fence_after();
        }
        const int nq = my_units * SUBS;                // ring stages this warp consumes in this half (first ones in flight)
        auto chan0 = [&](int q) { return (u0 + warp + 4 * (q / SUBS)) * 8 + (q % SUBS) * LU; };
        for (int ui = 0; ui < my_units; ++ui) {
            const int u = u0 + warp + 4 * ui;
            uint32_t packed[8][4];     // per slot: 8 int8 codes (2 words) or 8 bf16 values (4 words)
#pragma unroll
            for (int g = 0; g < 2; ++g) {                  // two groups of 4 channels
                uint32_t code[4][8];                       // int8: float bits whose low byte is the code; bf16: value bits
                float p[4][2][4], o[4][8];
#pragma unroll
                for (int dd4 = 0; dd4 < 4; ++dd4) {
                    const int d = g * 4 + dd4;             // channel within the unit
                    const int sub = d / LU, dd = d % LU;   // ring stage within the unit, channel within the stage
                    const int q = ui * SUBS + sub;
                    if (VEC && dd == 0) {
                        const int qn = q + RING2 - 1;
                        Ring::issue(my_ring_s, qn % RING2, xin, P, W, qn < nq ? Cin : 0, chan0(qn), lp, lane);
                        Ring::template wait<RING2 - 1>();
                    }
                    const int c = u * 8 + d;
                    RawPatch rawp;
                    if (VEC) {
                        Ring::read(my_ring, q % RING2, dd, lane, rawp);      // channels beyond Cin arrive as zeros
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) rawp.w[i] = 0u;
                        if (c < Cin) load_patch<T, VEC>(xin + (size_t)c * P, W, lp, rawp);
                    }
                    unpack_patch<T>(rawp, p[dd4]);
                }
                haar_fwd_lanes<L, 4>(p, o, lane);
#pragma unroll
                for (int dd4 = 0; dd4 < 4; ++dd4) {
#pragma unroll
                    for (int s = 0; s < 8; s += 2) {
                        float2 t = mul2(make_float2(o[dd4][s], o[dd4][s + 1]), make_float2(mul[s], mul[s + 1]));
                        if (I8 && alpha > 0.0f) {          // a given clipping parameter can be exceeded: clamp to the grid
                            t.x = fminf(fmaxf(t.x, -qmax), qmax);
                            t.y = fminf(fmaxf(t.y, -qmax), qmax);
                        }
                        // int8: the low byte of (t + 1.5*2^23) is the two's complement code of rint(t); |t| <= qmax by
                        // construction.  Scalar adds on purpose: a packed add right after the packed product gets
                        // contracted into one fused operation, which rounds once and changes half-way codes.
                        if (I8) t = make_float2(__fadd_rn(t.x, MAGIC), __fadd_rn(t.y, MAGIC));
                        code[dd4][s] = __float_as_uint(t.x);
                        code[dd4][s + 1] = __float_as_uint(t.y);
                    }
                }
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    if (I8) {
                        const uint32_t lo = __byte_perm(code[0][s], code[1][s], 0x0040);
                        const uint32_t hi = __byte_perm(code[2][s], code[3][s], 0x0040);
                        packed[s][g] = __byte_perm(lo, hi, 0x5410);
                    } else {
                        packed[s][2 * g] = pack_bf16x2(__uint_as_float(code[0][s]), __uint_as_float(code[1][s]));
                        packed[s][2 * g + 1] = pack_bf16x2(__uint_as_float(code[2][s]), __uint_as_float(code[3][s]));
                    }
                }
            }
            const int j = ((u - u0) * UNIT_BYTES) >> 4;    // 16-byte K chunk inside this half's A
            const int off = (u * UNIT_BYTES) & 15;         // 0 or 8 (int8); always 0 (bf16)
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                uint8_t* dst = sA + ((size_t)j * ROWS + s * 32 + lane) * 16 + off;
                if (I8) *reinterpret_cast<uint2*>(dst) = make_uint2(packed[s][0], packed[s][1]);
                else *reinterpret_cast<uint4*>(dst) = make_uint4(packed[s][0], packed[s][1], packed[s][2], packed[s][3]);
                if (xq_tap && rk[s] >= 0) {
                    uint8_t* g = xq_tap + ((size_t)n * k + rk[s]) * krow + (size_t)u * UNIT_BYTES;
                    if (I8) *reinterpret_cast<uint2*>(g) = make_uint2(packed[s][0], packed[s][1]);
                    else *reinterpret_cast<uint4*>(g) = make_uint4(packed[s][0], packed[s][1], packed[s][2], packed[s][3]);
                }
            }
        }
        for (int u = ur + warp; u < u1; u += 4) {          // padding of K up to a multiple of 32 bytes: zeros
            const int j = ((u - u0) * UNIT_BYTES) >> 4;
            const int off = (u * UNIT_BYTES) & 15;
#pragma unroll
            for (int s = 0; s < 8; ++s) {
                uint8_t* dst = sA + ((size_t)j * ROWS + s * 32 + lane) * 16 + off;
                if (I8) *reinterpret_cast<uint2*>(dst) = make_uint2(0u, 0u);
                else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
                if (xq_tap && rk[s] >= 0) {
                    uint8_t* g = xq_tap + ((size_t)n * k + rk[s]) * krow + (size_t)u * UNIT_BYTES;
                    if (I8) *reinterpret_cast<uint2*>(g) = make_uint2(0u, 0u);
                    else *reinterpret_cast<uint4*>(g) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
        }
        if (VEC) Ring::template wait<0>();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> visible to the tensor core
        tc::fence_before();
        __syncthreads();
        tc::fence_after();
        tmem = ctl->tmem_base;
        if (h + 1 < halves) {                          // first half of K: start accumulating now (single chunk of N)
            if (threadIdx.x == 0) issue_mmas(ks0, ks1, ks0, 0, npad);
            ++commits;
            ring_prologue(h + 1);                      // the second half's inputs fly while the tensor core works
        }
    }

    // ---- phases 2 (last K range) + 3, per chunk of output channels -----------------------------------
    const int ks_last = (halves - 1) * a_ksteps;
    for (int n0 = 0; ok && n0 < npad; n0 += nchunk) {
        const int cur = min(nchunk, npad - n0);
        if (threadIdx.x == 0) issue_mmas(ks_last, ksteps, ks_last, n0, cur);
        ++commits;
        ok = tc::mbar_wait(tc::smem_u32(&ctl->mma_done), (commits - 1u) & 1u, &no_abort);
        ok = __syncthreads_and(ok ? 1 : 0) != 0;
        if (!ok) break;
        tc::fence_after();

        for (int s0 = 0; s0 < cur; s0 += SUB) {
            uint32_t r0[SUB], r1[SUB];
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)s0;
#pragma unroll
            for (int q8 = 0; q8 < SUB / 8; ++q8) {
                tmem_ld8_nowait(taddr + 8 * q8, *reinterpret_cast<uint32_t(*)[8]>(&r0[8 * q8]));                      // slot `warp`
                tmem_ld8_nowait(taddr + (uint32_t)nchunk + 8 * q8, *reinterpret_cast<uint32_t(*)[8]>(&r1[8 * q8]));   // slot `warp + 4`
            }
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            const int rka = srank[warp * 32 + lane], rkb = srank[(warp + 4) * 32 + lane];
#pragma unroll
            for (int j = 0; j < SUB; ++j) {
                const int o = n0 + s0 + j;
                float fa, fb;
                if (I8) {
                    const float sc = (o < Cout) ? __fmul_rn(scale_a, scale_w[o]) : 0.0f;
                    // exact int -> float for |acc| < 2^22: bits(1.5*2^23) + acc, minus 1.5*2^23
                    fa = __fmul_rn(__fsub_rn(__uint_as_float(0x4B400000u + r0[j]), MAGIC), sc);
                    fb = __fmul_rn(__fsub_rn(__uint_as_float(0x4B400000u + r1[j]), MAGIC), sc);
                } else {
                    fa = __uint_as_float(r0[j]);
                    fb = __uint_as_float(r1[j]);
                }
                stage[(j * 8 + warp) * 32 + lane] = fa;
                stage[(j * 8 + warp + 4) * 32 + lane] = fb;
                if (acc_tap && o < Cout) {
                    if (rka >= 0) acc_tap[((size_t)n * k + rka) * Cout + o] = (int32_t)r0[j];
                    if (rkb >= 0) acc_tap[((size_t)n * k + rkb) * Cout + o] = (int32_t)r1[j];
                }
            }
            __syncthreads();
            {
                float sl[SUB / 4][8], p[SUB / 4][2][4];
#pragma unroll
                for (int jj = 0; jj < SUB / 4; ++jj) {
#pragma unroll
                    for (int s = 0; s < 8; ++s) sl[jj][s] = stage[((warp + 4 * jj) * 8 + s) * 32 + lane];
                }
                haar_inv_lanes<L, SUB / 4>(sl, p, lane);
#pragma unroll
                for (int jj = 0; jj < SUB / 4; ++jj) {
                    const int o = n0 + s0 + warp + 4 * jj;
                    if (o < Cout) {
                        const size_t plane = ((size_t)n * Cout + o) * P;
                        if (residual) add_residual<T, VEC>(residual + plane, W, lp, p[jj]);
                        if (relu) relu_patch(p[jj]);
                        store_patch<T, VEC>(y + plane, W, lp, p[jj]);
                    }
                }
            }
            __syncthreads();
        }
        tc::fence_before();
        __syncthreads();
    }
    if (!ok && threadIdx.x == 0) atomicExch(status, (int)WCC_ERR_TIMEOUT);
    tc::fence_before();
    __syncthreads();
    if (warp == 0) {
        tc::fence_after();
        tmem = ctl->tmem_base;
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)tmem_cols) : "memory");
    }
}

}  // namespace fz

static inline size_t vmax(size_t a, size_t b) { return a > b ? a : b; }

// Options of the fused second pass beyond Alg. 1: a given clipping parameter, residual add and ReLU on the way out.
struct FusedExtra { float alpha; int relu; const void* residual; };

// Host-side plan of the one-tile kernel (pure arithmetic; ok = the problem fits its shared memory).
struct FzPlan { int npad, nchunk, tmem_cols, a_ksteps; size_t smem; bool ok; };

static FzPlan fz_plan(int esz, int Cout, int kpad, int bits)
{
    FzPlan p = {};
    const bool i8 = bits >= 2;
    const int es = i8 ? 1 : 2;
    p.npad = ceil_div(Cout, 16) * 16;
    p.nchunk = p.npad < 64 ? p.npad : 64;
    p.tmem_cols = 32;
    while (p.tmem_cols < 2 * p.nchunk) p.tmem_cols <<= 1;
    const int kchunks = kpad * es / 16;
    const int ksteps = kpad * es / 32;
    // two K halves when that brings A down enough for a fourth CTA per SM (single chunk of output channels only)
    p.a_ksteps = (p.npad <= p.nchunk && ksteps >= 4) ? (ksteps + 1) / 2 : ksteps;
    const size_t stage_bytes = (size_t)((esz == 2) ? 4 : 2) * 2 * 32 * 4 * esz;          // PatchRing<T>::STAGE_BYTES
    const size_t region = vmax((size_t)fz::SUB * 8 * 32 * 4, (size_t)4 * fz::RING2 * stage_bytes);
    p.smem = 128 + (size_t)p.a_ksteps * 2 * fz::ROWS * 16 + (size_t)kchunks * p.npad * 16 + 8 * 32 * 4 + sizeof(fz::Ctl) +
             region + 16;
    p.ok = p.smem <= 200 * 1024 && (kpad * es) % 32 == 0;
    return p;
}

template <typename T, int L, bool VEC>
static wcc_status fused_pass2_dispatch(const void* x, const void* Wq, const int32_t* rank, const float* nrm2,
                                       const uint32_t* thr, const float* amax_kept, int bits,
                                       const float* scale_w, int N, int Cin, int Cout, int H, int W, int k, int kpad,
                                       void* y, void* xq_tap, int32_t* acc_tap, const FusedExtra& fx, cudaStream_t st)
{
    using TT = HaarTile<L>;
    static_assert(PatchRing<T>::STAGE_BYTES == ((sizeof(T) == 2) ? 4 : 2) * 2 * 32 * 4 * (int)sizeof(T), "fz_plan mirrors PatchRing");
    const bool i8 = bits >= 2;
    const FzPlan plan = fz_plan((int)sizeof(T), Cout, kpad, bits);
    if (!plan.ok) return WCC_ERR_SHAPE;
    const int npad = plan.npad, nchunk = plan.nchunk, tmem_cols = plan.tmem_cols, a_ksteps = plan.a_ksteps;
    const size_t smem = plan.smem;
    const float qmax = i8 ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    int* status = nullptr;
    WCC_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_status));
    const long long ctas = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    if (ctas > 0x7FFFFFFFLL) return WCC_ERR_SHAPE;
    auto launch = [&](auto kern) -> wcc_status {
        WCC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        kern<<<(unsigned)ctas, 128, smem, st>>>(static_cast<const T*>(x), static_cast<const uint8_t*>(Wq), rank, nrm2, thr, amax_kept,
                                                qmax, scale_w, N, Cin, Cout, H, W, k, kpad, npad, nchunk, tmem_cols, a_ksteps,
                                                static_cast<T*>(y), static_cast<uint8_t*>(xq_tap), acc_tap, status,
                                                fx.alpha, fx.relu, static_cast<const T*>(fx.residual));
        WCC_LAUNCH_CHECK();
        return WCC_OK;
    };
    if (i8) return launch(fz::fused_pass2_kernel<T, L, VEC, true>);
    return launch(fz::fused_pass2_kernel<T, L, VEC, false>);
}

// Fused second pass.  xq_tap ([N*k][kpad] of int8 or bf16) and acc_tap (int32 [N*k][Cout]) may be NULL.
wcc_status launch_fused_pass2(const void* x, const void* Wq, const int32_t* rank, const float* nrm2, const uint32_t* thr,
                              const float* amax_kept, int bits,
                              const float* scale_w, int N, int Cin, int Cout, int H, int W, int L, int k, int kpad,
                              wcc_dtype dt, void* y, void* xq_tap, int32_t* acc_tap, const FusedExtra& fx, cudaStream_t st)
{
    const bool vec = (W % 4) == 0;
    WCC_DISPATCH_TLV(fused_pass2_dispatch, dt, L, vec, x, Wq, rank, nrm2, thr, amax_kept, bits, scale_w, N, Cin, Cout, H, W, k, kpad,
                     y, xq_tap, acc_tap, fx, st);
}

}  // namespace wcc

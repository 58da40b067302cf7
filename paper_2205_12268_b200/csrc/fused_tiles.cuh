// Second pass of the fused layer, four tiles per CTA (steps A, C, D, E of the WCC workflow, Eq. 9 / Alg. 1, with the
// index set and the activation scale of step B already known): transform from x, keep / drop, quantize, pointwise
// convolution on tensor cores, dequantize, inverse transform, store y.
//
// A CTA owns four warp tiles (4 x 256 = 1024 wavelet-domain positions, see haar.cuh) and runs 4 * WPT compute warps
// plus one warp that issues the tensor-core instructions.  Compute warp w works for tile t = w % 4; the WPT warps of a
// tile split the input channels (in 16-byte chunks of an operand row) on the way in and the output channels (in groups
// of eight) on the way out.  Rows of the A operand are ordered  slot * 128 + t * 32 + lane,  so MMA block b (128 rows)
// holds slot b of all four tiles and the accumulators of tile t's lanes sit in TMEM lanes 32t .. 32t+31: exactly the
// lane quarter that warp w = t (mod 4) may read.  Every thread therefore reads back its own eight slots of an output
// channel with tcgen05.ld and runs the inverse transform in registers; nothing is transposed through shared memory.
//
// Inputs arrive through a per-warp ring of TMA boxes (CB channels of the warp's tile each); the A operand is handed to
// the tensor core one K step (32 bytes of K per row, 32 KB) at a time through mbarriers:
//   full_a[buf]  8 arrivals (4 tiles x 2 chunks)  -> the issuing warp runs 8 MMAs (one per block) on that K step
//   empty_a[buf] tcgen05.commit                   -> the buffer may be overwritten
//   ready[tb]    tcgen05.commit                   -> accumulator buffer tb holds a finished chunk of output channels
//   tfree[tb]    one arrival per compute warp     -> accumulator buffer tb has been read back
// With one chunk of output channels (<= 64) K steps stream through two A buffers; with several chunks (32 channels each,
// two accumulator buffers) every K step stays resident.  No block-wide barrier between set-up and tear-down.
// Every mbarrier wait is bounded and reports WCC_ERR_TIMEOUT.
#pragma once

#include "common.cuh"
#include "contract.cuh"
#include "fused.cuh"
#include "haar.cuh"

namespace wcc {
namespace ft {

constexpr int TILES = 4;                    // warp tiles per CTA
constexpr int ROWS = TILES * 256;           // operand rows per CTA
constexpr int KSTEP_BYTES = ROWS * 32;      // one K step of A
constexpr int MAX_NA = 4;

struct Ctl {
    uint64_t full_a[MAX_NA];
    uint64_t empty_a[MAX_NA];
    uint64_t ready[2];
    uint64_t tfree[2];
    uint64_t tok[TILES][2];      // NEXT: token of the norm chain has arrived for warp q of tile t
    uint32_t tmem_base;
    int abort_flag;
};

// With these pointers set (kernel variant NEXT) the kernel is also the first pass of the NEXT layer of a chain: the
// output tile it has just computed (after the residual add / ReLU, rounded to the activation type as it is stored) is
// transformed forward again while still in registers, and the channel norms, the per-position max |coefficient| and the
// selection's histograms of the next layer's input come out of the same launch; the next layer never reads its input
// for a first pass (App. H, "Memory bandwidth and traffic": consecutive separable steps done on a tile in one go).
struct NextNorms {
    float* nrm2;          // fp32 [N][P]
    float* amaxpos;       // fp32 [N][P]
    uint32_t* hist1;      // [N][3][2048], zero on entry (round 1 is filled)
    uint32_t* fine;       // [N][65536], zero on entry
};
constexpr int TOKEN_BYTES = 32 * 16 * 4;     // per lane: 8 partial sums + 8 running maxima

template <typename T, bool I8, int WPT>
struct Cfg {
    static constexpr int CWARPS = TILES * WPT;
    static constexpr int THREADS = (CWARPS + 1) * 32;
    static constexpr int CB = (sizeof(T) == 2) ? 8 : 4;          // channels per TMA box: 4 KB
    static constexpr int S = (WPT >= 4) ? 2 : 4;                  // boxes in flight per warp
    static constexpr int CCH = I8 ? 16 : 8;                       // channels per 16-byte operand chunk
    static constexpr int BPC = CCH / CB;                          // boxes per chunk
    static constexpr int GROUPS = CCH / 4;                        // groups of four channels per chunk
};

struct Params {
    const uint8_t* Wq; const int32_t* rank; const float* nrm2; const uint32_t* thr; const float* amax_kept;
    const float* scale_w; float qmax;
    float alpha;                 // > 0: given clipping parameter of the activation quantizer (codes are clamped)
    int relu;                    // non-zero: y = max(., 0)
    const void* residual;        // NULL, or [N][Cout][H][W] of the activation type, added before the ReLU
    NextNorms nx;                // kernel variant NEXT only
    int N, Cin, Cout, H, W, k, kpad, npad, nchunk, nn, nbuf, tmem_cols, na, tiles_total;
    int split_from, parts;       // CTAs from split_from on share a tile group `parts` ways by output channels
    void* y; uint8_t* xq_tap; int32_t* acc_tap; int* status;
};

// MODE is a set of compiled-in features: 1 = ReLU on the way out, 2 = the next layer's norms (chain), 4 = a given clipping
// parameter (codes are clamped), 8 = residual add.  A compiled-in feature is still switched by its run-time argument; a
// feature that is not compiled in costs nothing: as run-time branches in one kernel the options cost the plain layer
// 7-18 %, and the mere presence of the residual code costs a ReLU-only layer with 192 output channels 6 us of 80.
// Instantiated: 0 (plain), 1, 3, 5, 7 and 15 (everything); a request runs on the smallest variant that contains it.
template <typename T, int L, bool I8, int WPT, int MODE>
__global__ void __launch_bounds__(Cfg<T, I8, WPT>::THREADS, 1)
fused_tiles_kernel(const __grid_constant__ CUtensorMap tmx, const Params pr)
{
    constexpr bool RELU = (MODE & 1) != 0, NEXT = (MODE & 2) != 0, CLAMP = (MODE & 4) != 0, RES = (MODE & 8) != 0;
    static_assert(!NEXT || WPT == 2, "the norm chain alternates between the two warps of a tile");
    using TT = HaarTile<L>;
    using C = Cfg<T, I8, WPT>;
    using Ring = TileRing<T, L, C::CB, C::S>;
    constexpr int ES = I8 ? 1 : 2;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = tc::smem_u32(smem_raw);
    uint8_t* sm = smem_raw + (((raw + 127u) & ~127u) - raw);
    const int krow = pr.kpad * ES, kchunks = krow / 16, ksteps = krow / 32;
    uint8_t* sA = sm;                                                         // [na][2][ROWS][16]
    uint8_t* sRing = sA + (size_t)pr.na * KSTEP_BYTES;                        // [CWARPS][S][4 KB]
    uint8_t* sB = sRing + (size_t)C::CWARPS * Ring::BYTES;                    // [kchunks][npad][16]
    uint64_t* ring_bars = reinterpret_cast<uint64_t*>(sB + (size_t)kchunks * pr.npad * 16);   // [CWARPS][S]
    Ctl* ctl = reinterpret_cast<Ctl*>(ring_bars + C::CWARPS * C::S);
    float* sscale = reinterpret_cast<float*>(ctl + 1);                        // [npad]
    float4* stok = reinterpret_cast<float4*>((reinterpret_cast<uintptr_t>(sscale + pr.npad) + 15) & ~(uintptr_t)15);   // NEXT: [TILES][2][4][32]
    volatile int* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool is_mma = warp == C::CWARPS;
    const int t = warp & 3, q = warp >> 2;
    // The last, partial wave of tile groups is spread over the SMs that would idle: `parts` CTAs take one group each,
    // all of them build the whole operand (the transform and quantization are repeated) and each runs the contraction and
    // the way out for its own share of the output channels.
    int grp = (int)blockIdx.x, o_lo = 0, o_cnt = pr.npad;
    if ((int)blockIdx.x >= pr.split_from) {
        const int r = (int)blockIdx.x - pr.split_from;
        grp = pr.split_from + r / pr.parts;
        o_cnt = pr.npad / pr.parts;
        o_lo = (r % pr.parts) * o_cnt;
    }

    // ---- set-up -------------------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_NA; ++i) { tc::mbar_init(tc::smem_u32(&ctl->full_a[i]), 2 * TILES); tc::mbar_init(tc::smem_u32(&ctl->empty_a[i]), 1); }
        for (int i = 0; i < 2; ++i) { tc::mbar_init(tc::smem_u32(&ctl->ready[i]), 1); tc::mbar_init(tc::smem_u32(&ctl->tfree[i]), C::CWARPS); }
        for (int i = 0; i < TILES; ++i) { tc::mbar_init(tc::smem_u32(&ctl->tok[i][0]), 1); tc::mbar_init(tc::smem_u32(&ctl->tok[i][1]), 1); }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int tiles_x = (pr.W + TT::TW - 1) / TT::TW, tiles_y = pr.H / TT::TH;
    if (is_mma) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(tc::smem_u32(&ctl->tmem_base)), "r"((uint32_t)pr.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        // Lane w of this warp starts the input ring of compute warp w (barriers and the first S boxes), so that the
        // compute warps spend the set-up on their own global loads instead of waiting for the first TMA issue.
        if (lane < C::CWARPS) {
            const int t2 = lane & 3, q2 = lane >> 2, tile2 = grp * TILES + t2;
            const uint32_t bar2 = tc::smem_u32(ring_bars + lane * C::S);
            const uint32_t ring2 = tc::smem_u32(sRing + (size_t)lane * Ring::BYTES);
#pragma unroll
            for (int i = 0; i < C::S; ++i) tc::mbar_init(bar2 + 8 * i, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            if (tile2 < pr.tiles_total) {
                int n2, ty2, tx2;
                tile_coords(tile2, tiles_x, tiles_y, n2, ty2, tx2);
                const int boxes2 = ((kchunks - q2 + WPT - 1) / WPT) * C::BPC;
#pragma unroll
                for (int m = 0; m < C::S; ++m) {
                    if (m < boxes2) {
                        tc::mbar_expect_tx(bar2 + 8 * m, Ring::STAGE_BYTES);
                        tc::tma_load_4d(ring2 + m * Ring::STAGE_BYTES, &tmx, tx2 * TT::TW, ty2 * TT::TH,
                                        (q2 + (m / C::BPC) * WPT) * C::CCH + (m % C::BPC) * C::CB, n2, bar2 + 8 * m);
                    }
                }
            }
        }
        __syncwarp();
    }
    const int tile = grp * TILES + t;
    const bool live = !is_mma && tile < pr.tiles_total;
    int n = 0, ty = 0, tx = 0;
    if (live) tile_coords(tile, tiles_x, tiles_y, n, ty, tx);
    const LanePos lp = lane_positions<L>(pr.H, pr.W, ty, tx, lane);
    const size_t P = (size_t)pr.H * pr.W;
    const int x0 = tx * TT::TW, y0 = ty * TT::TH;

    // this warp's operand chunks: j = q, q + WPT, ... < kchunks; boxes in consumption order: m -> chunk m / BPC
    const int my_chunks = is_mma ? 0 : (kchunks - q + WPT - 1) / WPT;
    const int my_boxes = live ? my_chunks * C::BPC : 0;
    auto box_c0 = [&](int m) { return (q + (m / C::BPC) * WPT) * C::CCH + (m % C::BPC) * C::CB; };
    Ring ring;
    if (!is_mma) ring.attach(sRing + (size_t)warp * Ring::BYTES, ring_bars + warp * C::S, lane);
    // weights -> B operand (core-matrix layout), all threads
    for (int i = threadIdx.x; i < o_cnt * kchunks; i += C::THREADS) {      // rows o_lo .. o_lo + o_cnt of the weights
        const int row = i / kchunks, j = i - row * kchunks;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (o_lo + row < pr.Cout) v = *reinterpret_cast<const uint4*>(pr.Wq + (size_t)(o_lo + row) * krow + j * 16);
        *reinterpret_cast<uint4*>(sB + ((size_t)j * pr.npad + row) * 16) = v;
    }
    // kept or dropped: from the rank map when the select wrote one (thr[n][2] != 0), else by the threshold key
    float mul[8];
    int rk[8];
#pragma unroll
    for (int s = 0; s < 8; ++s) { mul[s] = 0.0f; rk[s] = -1; }
    // all independent loads first (threshold, norms, max |kept|), so that their latencies overlap
    float amax = 0.0f;
    if (I8) amax = (CLAMP && pr.alpha > 0.0f) ? pr.alpha : *pr.amax_kept;
    if (live) {
        const uint4 th = *reinterpret_cast<const uint4*>(pr.thr + n * 4);      // {threshold key, ties kept, use-rank flag, -}
        float nv[8];
#pragma unroll
        for (int s = 0; s < 8; ++s) nv[s] = slot_ok<L>(lp, s) ? pr.nrm2[(size_t)n * P + lp.pos[s]] : 0.0f;
        float inv = 1.0f;
        if (I8) inv = (amax > 0.0f) ? __fdiv_rn(pr.qmax, amax) : 0.0f;
        const uint32_t tkey = th.x, use_rank = th.z;
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            if (slot_ok<L>(lp, s)) {
                if (use_rank) rk[s] = pr.rank[(size_t)n * P + lp.pos[s]];
                else rk[s] = (float_key(nv[s]) >= tkey) ? 0 : -1;
            }
            mul[s] = (rk[s] >= 0) ? inv : 0.0f;
        }
        // the transform runs without its halvings: they go into the per-slot factor (exact, a power of two)
        float sc[8];
        slot_scales<L>(lane, ring.swap, sc);
#pragma unroll
        for (int s = 0; s < 8; ++s) mul[s] = __fmul_rn(mul[s], sc[s]);
    }
    if (I8) {                                          // dequantization factor of every output channel
        const float scale_a = __fdiv_rn(amax, pr.qmax);
        for (int o = threadIdx.x; o < pr.npad; o += C::THREADS) sscale[o] = (o < pr.Cout) ? __fmul_rn(scale_a, pr.scale_w[o]) : 0.0f;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // B operand -> visible to the tensor core
    tc::fence_before();
    __syncthreads();
    tc::fence_after();
    const uint32_t tmem = ctl->tmem_base;
    const uint32_t a_addr = tc::smem_u32(sA), b_addr = tc::smem_u32(sB);
    bool ok = true;

    if (is_mma) {
        // ---- tensor-core issue ------------------------------------------------------------------------
        if (lane == 0) {
            auto idesc_of = [&](int cur) {
                return (I8 ? (2u << 4) : (1u << 4)) | (1u << 7) | (1u << 10) | ((uint32_t)(cur >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            };
            auto mma_kstep = [&](int ks, int buf, int n0, int cur, uint32_t d0, bool first) {
#pragma unroll 1
                for (int b = 0; b < 8; ++b) {
                    const uint64_t ad = fz::smem_desc_plain(a_addr + (uint32_t)(buf * KSTEP_BYTES + b * 128 * 16), ROWS * 16, 128);
                    const uint64_t bd = fz::smem_desc_plain(b_addr + (uint32_t)((ks * 2 * pr.npad + n0) * 16), (uint32_t)pr.npad * 16, 128);
                    tc::mma_ss<I8>(d0 + (uint32_t)(b * pr.nchunk), ad, bd, idesc_of(cur), first ? 0u : 1u);
                }
            };
            if (pr.nn == 1) {
                for (int ks = 0; ks < ksteps && ok; ++ks) {
                    const int buf = ks % pr.na;
                    ok = tc::mbar_wait(tc::smem_u32(&ctl->full_a[buf]), (uint32_t)(ks / pr.na) & 1u, abort_flag);
                    if (!ok) break;
                    tc::fence_after();
                    mma_kstep(ks, buf, 0, o_cnt, tmem, ks == 0);
                    tc::mma_commit(tc::smem_u32(&ctl->empty_a[buf]));
                }
                if (ok) tc::mma_commit(tc::smem_u32(&ctl->ready[0]));
            } else {
                for (int ks = 0; ks < ksteps && ok; ++ks) ok = tc::mbar_wait(tc::smem_u32(&ctl->full_a[ks]), 0u, abort_flag);
                tc::fence_after();
                for (int c = 0; c < pr.nn && ok; ++c) {
                    const int tb = c % pr.nbuf;
                    if (c >= pr.nbuf) {
                        ok = tc::mbar_wait(tc::smem_u32(&ctl->tfree[tb]), (uint32_t)(c / pr.nbuf - 1) & 1u, abort_flag);
                        if (!ok) break;
                        tc::fence_after();
                    }
                    const int n0 = c * pr.nchunk, cur = min(pr.nchunk, pr.npad - n0);
                    for (int ks = 0; ks < ksteps; ++ks) mma_kstep(ks, ks, n0, cur, tmem + (uint32_t)(tb * 8 * pr.nchunk), ks == 0);
                    tc::mma_commit(tc::smem_u32(&ctl->ready[tb]));
                }
            }
        }
        __syncwarp();
    } else {
        // ---- phase 1: transform + quantize into the A operand ---------------------------------------------
        const bool clamp = CLAMP && I8 && pr.alpha > 0.0f;     // a given clipping parameter can be exceeded
        const float qmax = pr.qmax;
        int m = 0;                                     // boxes consumed so far
        for (int ci = 0; ci < my_chunks && ok; ++ci) {
            const int j = q + ci * WPT, ks = j >> 1, jj = j & 1, buf = ks % pr.na;
            uint32_t packed[8][4];                     // per slot: 16 int8 codes or 8 bf16 values
            if (live) {
                // all of the chunk's input words first (one wait per box), refill the stages right away, then compute:
                // the groups of four channels below carry no barrier between them and overlap freely
                constexpr int HB = (C::CCH < 8) ? C::CCH : 8;     // channels loaded ahead
#pragma unroll
                for (int hb = 0; hb < C::CCH / HB; ++hb) {
                    RawPatch rawp[HB];
#pragma unroll
                    for (int bx = hb * (HB / C::CB); bx < (hb + 1) * (HB / C::CB); ++bx) {
                        const int stage = (m + bx) % C::S;
                        ok = ok && ring.wait(stage, (uint32_t)((m + bx) / C::S) & 1u);
#pragma unroll
                        for (int d = 0; d < C::CB; ++d) ring.read_raw(stage, d, rawp[bx * C::CB + d - hb * HB]);   // channels beyond Cin arrive as zeros
                    }
                    __syncwarp();
                    if (lane == 0) {
#pragma unroll
                        for (int bx = hb * (HB / C::CB); bx < (hb + 1) * (HB / C::CB); ++bx)
                            if (m + bx + C::S < my_boxes) ring.issue(&tmx, (m + bx) % C::S, x0, y0, box_c0(m + bx + C::S), n);
                    }
#pragma unroll
                    for (int gg = 0; gg < HB / 4; ++gg) {
                        const int g = hb * (HB / 4) + gg;
                        float p[4][2][4], o[4][8];
#pragma unroll
                        for (int d = 0; d < 4; ++d) unpack_patch<T>(rawp[gg * 4 + d], p[d]);
                        haar_fwd_lanes_raw<L, 4>(p, o, lane);
                        uint32_t code[4][8];
#pragma unroll
                        for (int d = 0; d < 4; ++d) {
#pragma unroll
                            for (int s = 0; s < 8; s += 2) {
                                float2 v = mul2(make_float2(o[d][s], o[d][s + 1]), make_float2(mul[s], mul[s + 1]));
                                // int8: the low byte of (v + 1.5*2^23) is the two's complement code of rint(v).  The sum is
                                // written as fma(v, 1, 1.5*2^23): the product above keeps its own rounding (a packed add right
                                // after the packed product gets contracted into one fused operation, which changes half-way codes).
                                // clamping before the rounding is the same as after it: the bounds are integers
                                if (CLAMP && clamp) { v.x = fminf(fmaxf(v.x, -qmax), qmax); v.y = fminf(fmaxf(v.y, -qmax), qmax); }
                                if (I8) v = __ffma2_rn(v, make_float2(1.0f, 1.0f), make_float2(fz::MAGIC, fz::MAGIC));
                                code[d][s] = __float_as_uint(v.x);
                                code[d][s + 1] = __float_as_uint(v.y);
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
                }
                m += C::BPC;
            }
            if (ks >= pr.na) {                         // the tensor core must be done with the buffer's previous K step
                ok = ok && tc::mbar_wait(tc::smem_u32(&ctl->empty_a[buf]), (uint32_t)(ks / pr.na - 1) & 1u, abort_flag);
                tc::fence_after();
            }
            if (live) {
#pragma unroll
                for (int s = 0; s < 8; ++s) {
                    uint8_t* dst = sA + (size_t)buf * KSTEP_BYTES + ((size_t)jj * ROWS + s * 128 + t * 32 + lane) * 16;
                    *reinterpret_cast<uint4*>(dst) = make_uint4(packed[s][0], packed[s][1], packed[s][2], packed[s][3]);
                    if (pr.xq_tap && rk[s] >= 0)
                        *reinterpret_cast<uint4*>(pr.xq_tap + ((size_t)n * pr.k + rk[s]) * krow + (size_t)j * 16) =
                            make_uint4(packed[s][0], packed[s][1], packed[s][2], packed[s][3]);
                }
            } else {
#pragma unroll
                for (int s = 0; s < 8; ++s)
                    *reinterpret_cast<uint4*>(sA + (size_t)buf * KSTEP_BYTES + ((size_t)jj * ROWS + s * 128 + t * 32 + lane) * 16) =
                        make_uint4(0u, 0u, 0u, 0u);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(tc::smem_u32(&ctl->full_a[buf]));
        }

        // ---- phase 3: accumulators -> dequantize -> inverse transform -> y ---------------------------------
        T* yout = static_cast<T*>(pr.y);
        const T* res = static_cast<const T*>(pr.residual);
        const bool coarse6 = L == 3 && ((lane / TT::CG) & 1) == 0;     // slot 6 holds a level-3 coefficient
        // NEXT: the norm chain of the next layer's input.  Output channels leave in groups of eight that alternate between
        // the two warps of a tile; the partial sums (one fused multiply-add per channel, ascending channel order, as the
        // first pass builds them) and the running maxima travel with a token from the warp of group G to the warp of G + 1.
        float2 nsum[4];
        float nmax[8];
        int tok_seen = 0;
        const int last_group = (pr.Cout - 1) >> 3;
#pragma unroll
        for (int i = 0; i < 4; ++i) nsum[i] = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int i = 0; i < 8; ++i) nmax[i] = 0.0f;
        for (int c = 0; c < pr.nn && ok; ++c) {
            const int tb = c % pr.nbuf;
            ok = tc::mbar_wait(tc::smem_u32(&ctl->ready[tb]), (uint32_t)(c / pr.nbuf) & 1u, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
            if (!ok) break;
            tc::fence_after();
            const int n0 = c * pr.nchunk, cur = min(min(pr.nchunk, pr.npad - n0), o_cnt);
            for (int g = q; g * 8 < cur; g += WPT) {
                const int o0 = o_lo + n0 + g * 8;      // first output channel of the group
                if (!live || o0 >= pr.Cout) continue;
                uint32_t r[8][8];                      // [slot][channel]
                const uint32_t taddr = tmem + ((uint32_t)(t * 32) << 16) + (uint32_t)(tb * 8 * pr.nchunk + g * 8);
#pragma unroll
                for (int s = 0; s < 8; ++s) fz::tmem_ld8_nowait(taddr + (uint32_t)(s * pr.nchunk), r[s]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (pr.acc_tap) {
#pragma unroll
                    for (int s = 0; s < 8; ++s) {
                        if (rk[s] >= 0) {
#pragma unroll
                            for (int jn = 0; jn < 8; ++jn)
                                if (o0 + jn < pr.Cout) pr.acc_tap[((size_t)n * pr.k + rk[s]) * pr.Cout + o0 + jn] = (int32_t)r[s][jn];
                        }
                    }
                }
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    float sl[4][8], p[4][2][4];
#pragma unroll
                    for (int d = 0; d < 4; ++d) {
                        const int o = o0 + hh * 4 + d;
                        // dequantize straight into the pre-scaled slots of haar_inv_lanes_raw: acc * (scale * 2^-level)
                        float sc = 1.0f;
                        if (I8) sc = sscale[o];
                        const float s1 = __fmul_rn(sc, 0.5f), s2 = __fmul_rn(sc, 0.25f);
                        const float s6 = (L == 1) ? s1 : (coarse6 ? __fmul_rn(sc, 0.125f) : s2), s7 = (L == 1) ? s1 : s2;
#pragma unroll
                        for (int s = 0; s < 8; ++s) {
                            const float f = I8 ? __int2float_rn((int)r[s][hh * 4 + d]) : __uint_as_float(r[s][hh * 4 + d]);
                            sl[d][s] = __fmul_rn(f, s < 6 ? s1 : (s == 6 ? s6 : s7));
                        }
                    }
                    haar_inv_lanes_raw<L, 4>(sl, p, lane);
#pragma unroll
                    for (int d = 0; d < 4; ++d) {
                        const int o = o0 + hh * 4 + d;
                        if (o < pr.Cout) {
                            const size_t plane = ((size_t)n * pr.Cout + o) * P;
                            if (RES && res) fz::add_residual<T, true>(res + plane, pr.W, lp, p[d]);
                            if (RELU && pr.relu) fz::relu_patch(p[d]);
                            store_patch<T, true>(yout + plane, pr.W, lp, p[d]);
                        }
                    }
                    if (NEXT && pr.nx.nrm2) {
                        // what the next layer reads is the stored value: round to the activation type first.  Channels
                        // beyond Cout have zero accumulators and get neither residual nor store: they add nothing.
                        if (sizeof(T) == 2) {
#pragma unroll
                            for (int d = 0; d < 4; ++d)
#pragma unroll
                                for (int a = 0; a < 2; ++a)
#pragma unroll
                                    for (int b = 0; b < 4; ++b) p[d][a][b] = __bfloat162float(__float2bfloat16_rn(p[d][a][b]));
                        }
                        float o2[4][8];
                        haar_fwd_lanes_raw<L, 4>(p, o2, lane);
                        const int G = o0 >> 3;
                        if (hh == 0 && G > 0) {            // partial sums and maxima of the channels before this group
                            ok = ok && tc::mbar_wait(tc::smem_u32(&ctl->tok[t][q]), (uint32_t)tok_seen & 1u, abort_flag);
                            ++tok_seen;
                            const float4* tk = stok + ((size_t)(t * 2 + q) * 4) * 32;
                            const float4 a0 = tk[lane], a1 = tk[32 + lane], m0 = tk[64 + lane], m1 = tk[96 + lane];
                            nsum[0] = make_float2(a0.x, a0.y); nsum[1] = make_float2(a0.z, a0.w);
                            nsum[2] = make_float2(a1.x, a1.y); nsum[3] = make_float2(a1.z, a1.w);
                            nmax[0] = m0.x; nmax[1] = m0.y; nmax[2] = m0.z; nmax[3] = m0.w;
                            nmax[4] = m1.x; nmax[5] = m1.y; nmax[6] = m1.z; nmax[7] = m1.w;
                        }
#pragma unroll
                        for (int d = 0; d < 4; ++d) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 v = make_float2(o2[d][2 * i], o2[d][2 * i + 1]);
                                nsum[i] = __ffma2_rn(v, v, nsum[i]);
                            }
#pragma unroll
                            for (int s = 0; s < 8; ++s) nmax[s] = fmaxf(nmax[s], fabsf(o2[d][s]));
                        }
                        if (hh == 1) {
                            if (G < last_group) {          // hand over to the warp of the next group
                                float4* tk = stok + ((size_t)(t * 2 + (q ^ 1)) * 4) * 32;
                                tk[lane] = make_float4(nsum[0].x, nsum[0].y, nsum[1].x, nsum[1].y);
                                tk[32 + lane] = make_float4(nsum[2].x, nsum[2].y, nsum[3].x, nsum[3].y);
                                tk[64 + lane] = make_float4(nmax[0], nmax[1], nmax[2], nmax[3]);
                                tk[96 + lane] = make_float4(nmax[4], nmax[5], nmax[6], nmax[7]);
                                __syncwarp();
                                if (lane == 0) tc::mbar_arrive(tc::smem_u32(&ctl->tok[t][q ^ 1]));
                            } else if (ok) {               // last group: these are the next layer's norms of this tile
                                float sc2[8], nacc[8], am[8];
                                slot_scales<L>(lane, false, sc2);
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    nacc[2 * i] = __fmul_rn(nsum[i].x, __fmul_rn(sc2[2 * i], sc2[2 * i]));
                                    nacc[2 * i + 1] = __fmul_rn(nsum[i].y, __fmul_rn(sc2[2 * i + 1], sc2[2 * i + 1]));
                                }
#pragma unroll
                                for (int s = 0; s < 8; ++s) am[s] = __fmul_rn(nmax[s], fabsf(sc2[s]));
                                store_slots<L, true>(pr.nx.nrm2 + (size_t)n * P, lp, nacc);
                                store_slots<L, true>(pr.nx.amaxpos + (size_t)n * P, lp, am);
                                uint32_t* h = pr.nx.hist1 + (size_t)n * 3 * 2048;      // zero norms are not counted
#pragma unroll
                                for (int s = 0; s < 8; ++s) hist_add(h, norm_digit11(nacc[s]), lp.ok0 && nacc[s] != 0.0f);
                                if (lp.ok0) {
                                    uint32_t* f = pr.nx.fine + (size_t)n * 65536;
#pragma unroll
                                    for (int s = 0; s < 8; ++s)
                                        if (nacc[s] != 0.0f) atomicAdd(&f[norm_digit16(nacc[s])], 1u);
                                }
                            }
                        }
                    }
                }
            }
            tc::fence_before();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(tc::smem_u32(&ctl->tfree[tb]));
        }
    }

    // ---- tear-down ------------------------------------------------------------------------------------
    ok = __all_sync(0xFFFFFFFFu, ok ? 1 : 0) != 0;
    if (!ok) {
        *abort_flag = 1;
        if (lane == 0) atomicExch(pr.status, (int)WCC_ERR_TIMEOUT);
    }
    tc::fence_before();
    __syncthreads();
    if (*abort_flag) {                                 // give copies that were already issued time to land
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (is_mma) {
        tc::fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)pr.tmem_cols) : "memory");
    }
}

}  // namespace ft

// Host-side plan of the four-tile kernel: how the output channels are chunked, how many operand buffers and TMEM
// columns it takes, and whether the problem fits at all (ok).  Pure arithmetic: callers decide before anything is launched.
struct FtPlan { int npad, nchunk, nn, nbuf, na, tmem_cols; size_t smem; bool ok; };

static FtPlan ft_plan(const void* x, int esz, int W, int Cout, int kpad, int bits, bool next = false)
{
    constexpr int WPT = 2, S = 4;                     // as instantiated below (Cfg<T, I8, 2>::S)
    FtPlan p = {};
    const bool i8 = bits >= 2;
    const int es = i8 ? 1 : 2;
    if ((W % 4) != 0 || !tc::tma_ok_x(x, esz, W) || (kpad * es) % 32 != 0) return p;
    p.npad = ceil_div(Cout, 16) * 16;
    const int kchunks = kpad * es / 16, ksteps = kpad * es / 32;
    if (p.npad <= 64) { p.nchunk = p.npad; p.nn = 1; p.nbuf = 1; p.na = ksteps < 2 ? ksteps : 2; }
    else { p.nchunk = 32; p.nn = ceil_div(p.npad, 32); p.nbuf = 2; p.na = ksteps; }
    if (p.na > ft::MAX_NA) return p;
    p.tmem_cols = 32;
    while (p.tmem_cols < 8 * p.nchunk * p.nbuf) p.tmem_cols <<= 1;
    if (p.tmem_cols > 512) return p;
    const size_t ring_bytes = (size_t)ft::TILES * WPT * S * 4096;
    p.smem = 128 + (size_t)p.na * ft::KSTEP_BYTES + ring_bytes + (size_t)kchunks * p.npad * 16 +
             (size_t)ft::TILES * WPT * 8 * 8 + sizeof(ft::Ctl) + (size_t)p.npad * 4 + 64;
    if (next) p.smem += (size_t)ft::TILES * 2 * ft::TOKEN_BYTES + 16;
    p.ok = p.smem <= 227 * 1024;
    return p;
}

// Returns WCC_ERR_SHAPE when this kernel does not cover the problem (the caller then uses fused_pass2_kernel).
template <typename T, int L>
static wcc_status fused_tiles_dispatch(const void* x, const void* Wq, const int32_t* rank, const float* nrm2, const uint32_t* thr,
                                       const float* amax_kept, int bits, const float* scale_w, int N, int Cin, int Cout, int H,
                                       int W, int k, int kpad, void* y, void* xq_tap, int32_t* acc_tap, const FusedExtra& fx,
                                       cudaStream_t st, const ft::NextNorms* nx = nullptr)
{
    using TT = HaarTile<L>;
    constexpr int WPT = 2;
    static_assert(ft::Cfg<T, true, WPT>::S == 4 && ft::Cfg<T, false, WPT>::S == 4, "ft_plan assumes four boxes per ring");
    const bool i8 = bits >= 2;
    const FtPlan plan = ft_plan(x, (int)sizeof(T), W, Cout, kpad, bits, nx != nullptr);
    if (!plan.ok) return WCC_ERR_SHAPE;
    ft::Params pr = {};
    if (nx) pr.nx = *nx;
    pr.npad = plan.npad; pr.nchunk = plan.nchunk; pr.nn = plan.nn; pr.nbuf = plan.nbuf; pr.na = plan.na; pr.tmem_cols = plan.tmem_cols;
    const size_t smem = plan.smem;
    const long long tiles = (long long)N * ceil_div(W, TT::TW) * (H / TT::TH);
    if (tiles > 0x7FFFFFFFLL) return WCC_ERR_SHAPE;
    CUtensorMap tmx;
    if (!tc::make_map_x(&tmx, x, (int)sizeof(T), N, Cin, H, W, TT::TW, TT::TH, (sizeof(T) == 2) ? 8 : 4)) return WCC_ERR_CUDA;
    pr.Wq = static_cast<const uint8_t*>(Wq); pr.rank = rank; pr.nrm2 = nrm2; pr.thr = thr; pr.amax_kept = amax_kept;
    pr.scale_w = scale_w; pr.qmax = i8 ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    pr.N = N; pr.Cin = Cin; pr.Cout = Cout; pr.H = H; pr.W = W; pr.k = k; pr.kpad = kpad; pr.tiles_total = (int)tiles;
    pr.y = y; pr.xq_tap = static_cast<uint8_t*>(xq_tap); pr.acc_tap = acc_tap;
    pr.alpha = fx.alpha; pr.relu = fx.relu; pr.residual = fx.residual;
    WCC_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&pr.status), g_status));
    const unsigned groups = (unsigned)((tiles + ft::TILES - 1) / ft::TILES);
    // One CTA per SM at a time: the groups run in waves.  The groups of a last, partial wave are shared 4 or 2 ways by
    // output channels when that still fits one wave (the SMs would idle otherwise); the chain variant keeps whole
    // groups, its norm chain runs over all output channels of a tile.
    int dev = 0, sms = 0;
    WCC_CUDA_TRY(cudaGetDevice(&dev));
    WCC_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const unsigned rem = sms > 0 ? groups % (unsigned)sms : 0u;
    pr.parts = 1;
    if (plan.nn == 1 && !nx && rem > 0) {
        for (int parts = 4; parts >= 2; parts >>= 1)
            if (rem * (unsigned)parts <= (unsigned)sms && plan.npad % (16 * parts) == 0) { pr.parts = parts; break; }
    }
    pr.split_from = (pr.parts > 1) ? (int)(groups - rem) : (int)groups;
    const unsigned ctas = (unsigned)pr.split_from + (groups - (unsigned)pr.split_from) * (unsigned)pr.parts;
    auto launch = [&](auto kern, int threads) -> wcc_status {
        WCC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        kern<<<ctas, threads, smem, st>>>(tmx, pr);
        WCC_LAUNCH_CHECK();
        return WCC_OK;
    };
    const bool clampv = i8 && fx.alpha > 0.0f;
    const int want = (fx.relu ? 1 : 0) | (nx ? 2 : 0) | (clampv ? 4 : 0) | (fx.residual ? 8 : 0);
    const int have[5] = {1, 3, 5, 7, 15};              // after the plain variant, smallest first
    int mode = 0;
    if (want) {
        mode = 15;
        for (int i = 0; i < 5; ++i)
            if ((want & ~have[i]) == 0) { mode = have[i]; break; }
    }
    switch (mode) {
        case 1: if (i8) return launch(ft::fused_tiles_kernel<T, L, true, WPT, 1>, ft::Cfg<T, true, WPT>::THREADS);
                return launch(ft::fused_tiles_kernel<T, L, false, WPT, 1>, ft::Cfg<T, false, WPT>::THREADS);
        case 3: if (i8) return launch(ft::fused_tiles_kernel<T, L, true, WPT, 3>, ft::Cfg<T, true, WPT>::THREADS);
                return launch(ft::fused_tiles_kernel<T, L, false, WPT, 3>, ft::Cfg<T, false, WPT>::THREADS);
        case 5: return launch(ft::fused_tiles_kernel<T, L, true, WPT, 5>, ft::Cfg<T, true, WPT>::THREADS);
        case 7: return launch(ft::fused_tiles_kernel<T, L, true, WPT, 7>, ft::Cfg<T, true, WPT>::THREADS);
        case 15: if (i8) return launch(ft::fused_tiles_kernel<T, L, true, WPT, 15>, ft::Cfg<T, true, WPT>::THREADS);
                 return launch(ft::fused_tiles_kernel<T, L, false, WPT, 15>, ft::Cfg<T, false, WPT>::THREADS);
        default: break;
    }
    if (i8) return launch(ft::fused_tiles_kernel<T, L, true, WPT, 0>, ft::Cfg<T, true, WPT>::THREADS);
    return launch(ft::fused_tiles_kernel<T, L, false, WPT, 0>, ft::Cfg<T, false, WPT>::THREADS);
}

wcc_status launch_fused_tiles(const void* x, const void* Wq, const int32_t* rank, const float* nrm2, const uint32_t* thr,
                              const float* amax_kept, int bits, const float* scale_w, int N, int Cin, int Cout, int H, int W,
                              int L, int k, int kpad, wcc_dtype dt, void* y, void* xq_tap, int32_t* acc_tap, const FusedExtra& fx,
                              cudaStream_t st, const ft::NextNorms* nx = nullptr)
{
    if ((W % 4) != 0) return WCC_ERR_SHAPE;
#define WCC_FT(TY, LL) return fused_tiles_dispatch<TY, LL>(x, Wq, rank, nrm2, thr, amax_kept, bits, scale_w, N, Cin, Cout, H, W, k, kpad, y, xq_tap, acc_tap, fx, st, nx)
    if (dt == WCC_F32) { if (L == 1) WCC_FT(float, 1); if (L == 2) WCC_FT(float, 2); WCC_FT(float, 3); }
    if (L == 1) WCC_FT(__nv_bfloat16, 1);
    if (L == 2) WCC_FT(__nv_bfloat16, 2);
    WCC_FT(__nv_bfloat16, 3);
#undef WCC_FT
}

}  // namespace wcc

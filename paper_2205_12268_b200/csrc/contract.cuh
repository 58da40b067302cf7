// The pointwise (1x1) convolution on the compressed columns as a tensor-core contraction (step C of the
// WCC workflow; Alg. 1 "Y_wt = Conv(K_1x1, X[I])"):
//     acc[r][o] = sum_c Xq[r][c] * Wq[o][c],      r = kept position (row), o = output channel.
// Positions are the long dimension, so they map to the MMA M (tiles of 128 rows = 128 TMEM lanes); the output
// channels are the MMA N (tiles of up to 256, one instruction each); the input channels are K, streamed in 128-byte atoms.
//
// Blackwell path: operands are staged by TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into shared
// memory, one elected thread issues tcgen05.mma (kind::i8 with int32 accumulation, or kind::f16 on bf16 with
// fp32 accumulation) into a double-buffered TMEM accumulator, and four epilogue warps read it back with
// tcgen05.ld and store it.  Persistent CTAs walk the (row tile, column tile) pairs; the weights come from L2 every time.
// Every mbarrier wait is bounded: when one runs out the kernel raises WCC_ERR_TIMEOUT in the status word,
// lets the copies in flight land, frees its TMEM and returns.
#pragma once

#include "common.cuh"
#include "tma.cuh"

namespace wcc {
namespace tc {

constexpr int TILE_M = 128;                     // rows (kept positions) per tile = TMEM lanes
constexpr int TILE_N = 256;                     // output channels per tile (one instruction covers them)
constexpr int STAGES = 4;
constexpr int ATOM_BYTES = 128;                 // one swizzle row: 128 bytes of K
constexpr int A_ATOM_BYTES = TILE_M * ATOM_BYTES;
constexpr int B_ATOM_BYTES = TILE_N * ATOM_BYTES;
constexpr int STAGE_BYTES = A_ATOM_BYTES + B_ATOM_BYTES;      // 48 KB, a multiple of 1024 (swizzle alignment)
constexpr int TMEM_COLS = 2 * TILE_N;           // two accumulator buffers

// K-major operand tile, 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);                 // start, leading offset (unused)
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);                // stride 1024 B, version 1, SWIZZLE_128B
    return ((uint64_t)hi << 32) | lo;
}

template <bool I8>
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    if (I8)
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                     ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld8_nowait(uint32_t taddr, uint32_t (&r)[8])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

struct SmemCtl {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tfull[2];
    uint64_t tempty[2];
    uint32_t tmem_base;
    int abort_flag;
};

// 192 threads: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2-5 = epilogue.
// Persistent CTAs walk the (row tile, column tile) pairs; every pair streams its K range through a ring of stages, each
// holding one 128-byte K atom of the rows (128 x 128 B) and of the weights (TILE_N x 128 B), so any number of input
// channels and of output channels is covered: K is a loop, N is tiled by TILE_N.
template <bool I8>
__global__ void __launch_bounds__(192, 1)
contract_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                int M, int npad, int krow_bytes, int32_t* __restrict__ acc, int ldc, int* __restrict__ status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int katoms = (krow_bytes + ATOM_BYTES - 1) / ATOM_BYTES;
    SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem_raw + (base - raw) + (size_t)STAGES * STAGE_BYTES);
    volatile int* abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m_tiles = (M + TILE_M - 1) / TILE_M, n_tiles = (npad + TILE_N - 1) / TILE_N;
    const int items = m_tiles * n_tiles;                 // item = m_tile * n_tiles + n_tile: the column tiles of a row tile are neighbours
    const int elems_per_atom = I8 ? ATOM_BYTES : ATOM_BYTES / 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&ctl->tfull[b]), 1); mbar_init(smem_u32(&ctl->tempty[b]), 4); }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    bool failed = false;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;                                  // stages filled so far
            for (int w = blockIdx.x; w < items && !failed; w += gridDim.x) {
                const int mt = w / n_tiles, nt = w - mt * n_tiles;
                for (int a = 0; a < katoms; ++a, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                    if (!mbar_wait(smem_u32(&ctl->empty[s]), ph ^ 1u, abort_flag)) { failed = true; break; }
                    const uint32_t sA = base + (uint32_t)s * STAGE_BYTES, sB = sA + A_ATOM_BYTES;
                    mbar_expect_tx(smem_u32(&ctl->full[s]), (uint32_t)STAGE_BYTES);
                    tma_load_2d(sA, &tmA, a * elems_per_atom, mt * TILE_M, smem_u32(&ctl->full[s]));
                    tma_load_2d(sB, &tmB, a * elems_per_atom, nt * TILE_N, smem_u32(&ctl->full[s]));
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            int it = 0, item = 0;
            for (int w = blockIdx.x; w < items && !failed; w += gridDim.x, ++item) {
                const int nt = w % n_tiles;
                const int cur = min(TILE_N, npad - nt * TILE_N);
                // instruction descriptor: D format, A/B formats, N >> 3 at bit 17, M >> 4 at bit 24; K-major A and B
                const uint32_t idesc = (I8 ? (2u << 4) : (1u << 4)) | (1u << 7) | (1u << 10) |
                                       ((uint32_t)(cur >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
                const int buf = item & 1;
                const uint32_t bph = (uint32_t)(item >> 1) & 1u;
                if (!mbar_wait(smem_u32(&ctl->tempty[buf]), bph ^ 1u, abort_flag)) { failed = true; break; }
                fence_after();
                const uint32_t d = tmem_base + (uint32_t)(buf * TILE_N);
                uint32_t accumulate = 0;
                for (int a = 0; a < katoms; ++a, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                    if (!mbar_wait(smem_u32(&ctl->full[s]), ph, abort_flag)) { failed = true; break; }
                    fence_after();
                    const uint32_t sA = base + (uint32_t)s * STAGE_BYTES, sB = sA + A_ATOM_BYTES;
                    const int ksteps = min(4, (krow_bytes - a * ATOM_BYTES) / 32);
                    const uint64_t ad = smem_desc_sw128(sA), bd = smem_desc_sw128(sB);
                    for (int kk = 0; kk < ksteps; ++kk) {
                        mma_ss<I8>(d, ad + (uint64_t)(2 * kk), bd + (uint64_t)(2 * kk), idesc, accumulate);   // +32 bytes of K
                        accumulate = 1;
                    }
                    mma_commit(smem_u32(&ctl->empty[s]));
                }
                if (failed) break;
                mma_commit(smem_u32(&ctl->tfull[buf]));
            }
        }
        __syncwarp();
    } else {
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        int item = 0;
        for (int w = blockIdx.x; w < items; w += gridDim.x, ++item) {
            const int mt = w / n_tiles, nt = w - mt * n_tiles;
            const int n0 = nt * TILE_N, cur = min(TILE_N, npad - n0);
            const int buf = item & 1;
            const uint32_t bph = (uint32_t)(item >> 1) & 1u;
            int okw = mbar_wait(smem_u32(&ctl->tfull[buf]), bph, abort_flag) ? 1 : 0;
            okw = __all_sync(0xFFFFFFFFu, okw);
            if (!okw) { failed = true; break; }
            fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * TILE_N);
            const long long grow = (long long)mt * TILE_M + q * 32 + lane;
            int32_t* dst = acc + grow * ldc + n0;
            for (int c0 = 0; c0 < cur && n0 + c0 < ldc; c0 += 32) {       // 32 columns per wait: a 128-byte line per lane
                uint32_t r[4][8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (c0 + 8 * j < cur) {             // warp-uniform
                        tmem_ld8_nowait(taddr + (uint32_t)(c0 + 8 * j), r[j]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) r[j][i] = 0u;
                    }
                }
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (grow < M) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int c = c0 + 8 * j;
                        if (c < cur && n0 + c < ldc) {
                            *reinterpret_cast<uint4*>(dst + c) = make_uint4(r[j][0], r[j][1], r[j][2], r[j][3]);
                            if (n0 + c + 4 < ldc) *reinterpret_cast<uint4*>(dst + c + 4) = make_uint4(r[j][4], r[j][5], r[j][6], r[j][7]);
                        }
                    }
                }
            }
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->tempty[buf]));
        }
    }

    if (failed) {
        *abort_flag = 1;
        atomicExch(status, (int)WCC_ERR_TIMEOUT);
    }
    fence_before();
    __syncthreads();
    if (*abort_flag) {
        // give copies that were already issued time to land before the CTA's shared memory goes away
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// rows x row_elems matrix, row pitch = row_elems * elem size; box = 128 bytes of K x box_rows rows.
inline bool make_map(CUtensorMap* tm, const void* ptr, bool i8, uint64_t row_elems, uint64_t rows, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const uint32_t es = i8 ? 1 : 2;
    cuuint64_t dims[2] = {row_elems, rows};
    cuuint64_t strides[1] = {row_elems * es};
    cuuint32_t box[2] = {(cuuint32_t)(ATOM_BYTES / es), box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, i8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims,
              strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

wcc_status launch_contract(const void* Xq, const void* Wq, int M, int Cout, int kpad, int bits,
                           int32_t* acc, int ldc, cudaStream_t st)
{
    using namespace tc;
    const bool i8 = bits >= 2;
    const int krow_bytes = kpad * (i8 ? 1 : 2);
    const int npad = ceil_div(Cout, 16) * 16;
    if ((krow_bytes % 32) != 0) return WCC_ERR_SHAPE;

    CUtensorMap tmA, tmB;
    if (!make_map(&tmA, Xq, i8, (uint64_t)kpad, (uint64_t)M, TILE_M)) return WCC_ERR_CUDA;
    if (!make_map(&tmB, Wq, i8, (uint64_t)kpad, (uint64_t)Cout, TILE_N)) return WCC_ERR_CUDA;   // rows beyond Cout arrive as zeros

    const size_t smem = 1024 + (size_t)STAGES * STAGE_BYTES + sizeof(SmemCtl) + 16;
    static int sm_count[64] = {0};
    static bool attr_set[64][2] = {{false}};
    int dev = 0;
    WCC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return WCC_ERR_CUDA;
    if (!sm_count[dev]) WCC_CUDA_TRY(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
    if (!attr_set[dev][i8]) {
        if (i8) WCC_CUDA_TRY(cudaFuncSetAttribute(contract_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        else WCC_CUDA_TRY(cudaFuncSetAttribute(contract_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set[dev][i8] = true;
    }
    int* status = nullptr;
    WCC_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_status));
    const long long items = (long long)ceil_div(M, TILE_M) * ceil_div(npad, TILE_N);
    const int grid = (int)(items < sm_count[dev] ? items : sm_count[dev]);
    if (i8)
        contract_kernel<true><<<grid, 192, smem, st>>>(tmA, tmB, M, npad, krow_bytes, acc, ldc, status);
    else
        contract_kernel<false><<<grid, 192, smem, st>>>(tmA, tmB, M, npad, krow_bytes, acc, ldc, status);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

}  // namespace wcc

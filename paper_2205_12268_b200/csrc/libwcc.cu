// libwcc: C-ABI entry points (see include/wcc.h).  One translation unit: the kernels live in the *.cuh files.
#include "common.cuh"
#include "gather.cuh"
#include "haar.cuh"
#include "regather.cuh"
#include "select.cuh"
#include "contract.cuh"
#include "fused.cuh"
#include "fused_tiles.cuh"
#include "wavelet.cuh"

namespace wcc {

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static wcc_status check_plane_args(int N, int C, int H, int W, int L, wcc_dtype dt)
{
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0) return WCC_ERR_SHAPE;
    if (L < 1 || L > 3) return WCC_ERR_SHAPE;
    if ((H % (1 << L)) != 0 || (W % (1 << L)) != 0) return WCC_ERR_SHAPE;
    if ((long long)N * C * H * W > (1LL << 40)) return WCC_ERR_SHAPE;
    if ((long long)H * W > (1LL << 30)) return WCC_ERR_SHAPE;
    if (dt != WCC_F32 && dt != WCC_BF16) return WCC_ERR_DTYPE;
    return WCC_OK;
}

static wcc_status check_forward_args(int N, int Cin, int Cout, int H, int W, int L, int k, int bits, wcc_dtype dt)
{
    wcc_status s = check_plane_args(N, Cin, H, W, L, dt);
    if (s != WCC_OK) return s;
    if (Cout <= 0 || Cin > WCC_MAX_CHANNELS || Cout > WCC_MAX_CHANNELS) return WCC_ERR_SHAPE;
    if (k < 1 || (long long)k > (long long)H * W) return WCC_ERR_K;
    if (!(bits == 0 || (bits >= 2 && bits <= 8))) return WCC_ERR_BITS;
    if ((long long)N * k > (1LL << 30)) return WCC_ERR_SHAPE;
    return WCC_OK;
}

// Can one of the two fused second-pass kernels run this problem?  (x only enters through its alignment.)
static bool fused_fits(const void* x, int Cout, int W, int bits, wcc_dtype dt, int Cin)
{
    const int esz = (dt == WCC_BF16) ? 2 : 4, kpad = wcc_kpad(Cin, bits);
    return ft_plan(x, esz, W, Cout, kpad, bits).ok || fz_plan(esz, Cout, kpad, bits).ok;
}

// Can the staged contraction kernel run it?  (Mirrors launch_contract: K is a loop and N is tiled, so only the
// 32-byte granularity of a K step remains, which wcc_kpad guarantees.)
static bool staged_fits(int Cin, int Cout, int bits)
{
    (void)Cout;
    return (wcc_kpad(Cin, bits) * (bits >= 2 ? 1 : 2)) % 32 == 0;
}

struct FwdWs {
    float* coef; float* nrm2; float* amaxpos; int32_t* rank; int32_t* idx; void* sel; size_t sel_bytes;
    float* amax_kept; void* Xq; void* Wq; float* scale_w; int32_t* acc;
    int kpad, ldc, es;
    size_t total;
};

static FwdWs carve_forward_ws(void* ws, int N, int Cin, int Cout, int H, int W, int k, int bits)
{
    FwdWs f;
    const size_t P = (size_t)H * W, M = (size_t)N * k;
    f.kpad = wcc_kpad(Cin, bits);
    f.es = (bits == 0) ? 2 : 1;
    f.ldc = ceil_div(Cout, 4) * 4;
    size_t off = 0;
    char* b = static_cast<char*>(ws);
    auto take = [&](size_t bytes) { char* p = b ? b + off : nullptr; off += align_up(bytes, 256); return p; };
    f.coef = reinterpret_cast<float*>(take((size_t)N * Cin * P * 4));
    f.nrm2 = reinterpret_cast<float*>(take((size_t)N * P * 4));
    f.amaxpos = reinterpret_cast<float*>(take((size_t)N * P * 4));
    f.rank = reinterpret_cast<int32_t*>(take((size_t)N * P * 4));
    f.idx = reinterpret_cast<int32_t*>(take(M * 4));
    f.sel_bytes = select_ws_bytes(N, (int)P);
    f.sel = take(f.sel_bytes);
    f.amax_kept = b ? carve_select_ws(f.sel, N, (int)P).amax : nullptr;
    f.Xq = take(M * f.kpad * f.es);
    f.Wq = take((size_t)Cout * f.kpad * f.es);
    f.scale_w = reinterpret_cast<float*>(take((size_t)Cout * 4));
    f.acc = reinterpret_cast<int32_t*>(take(M * f.ldc * 4));
    f.total = off;
    return f;
}

// ---- scratch for wcc_select_topk_static ---------------------------------------------------------
// Lives in the device image of this library on every GPU that loads it.  In host code the name below is only a
// handle for the runtime; the device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_select_scratch[WCC_STATIC_SCRATCH_BYTES];

static wcc_status static_scratch_ptr(void** out)
{
    static void* ptr_of_device[64] = {nullptr};
    int dev = -1;
    WCC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return WCC_ERR_CUDA;
    if (!ptr_of_device[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return WCC_ERR_CUDA;
        }
        ptr_of_device[dev] = p;
    }
    *out = ptr_of_device[dev];
    return WCC_OK;
}

// ---- optional stage timing ------------------------------------------------------------------
static bool g_profile = false;
static cudaEvent_t g_ev[WCC_NUM_STAGES + 1] = {nullptr};
static bool g_ev_valid = false;

static wcc_status profile_mark(int i, cudaStream_t st)
{
    if (!g_profile) return WCC_OK;
    if (!g_ev[i]) WCC_CUDA_TRY(cudaEventCreate(&g_ev[i]));
    WCC_CUDA_TRY(cudaEventRecord(g_ev[i], st));
    if (i == WCC_NUM_STAGES) g_ev_valid = true;
    return WCC_OK;
}

// One warp waits on an mbarrier that nobody ever arrives on: the bounded wait runs out, the kernel records
// WCC_ERR_TIMEOUT in the status word and returns normally (no trap, no fault).
__global__ void wait_selftest_kernel(int* status)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        tc::mbar_init(tc::smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool ok = tc::mbar_wait(tc::smem_u32(&bar), 0u);
    if (!__all_sync(0xFFFFFFFFu, ok ? 1 : 0) && threadIdx.x == 0) atomicExch(status, (int)WCC_ERR_TIMEOUT);
}

__global__ void scale_tap_kernel(const float* amax_kept, float alpha, float qmax, float* out)
{
    *out = __fdiv_rn(alpha > 0.0f ? alpha : *amax_kept, qmax);
}

static wcc_status check_options(const wcc_options* o, int bits, const void* x, const void* y);
__global__ void set_word_kernel(float* dst, float v) { *dst = v; }

// dwk: NULL, or depthwise 3x3 kernels fp32 [Cin][3][3] applied to x before the transform (one fused pass).
static wcc_status staged_impl(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int W,
                               int L, int k, int bits, void* y, wcc_dtype dt, void* ws, size_t ws_bytes,
                               cudaStream_t st, const wcc_taps* taps, const wcc_options* opt = nullptr,
                               const float* dwk = nullptr)
{
    if (!x || !Wt || !y || !ws) return WCC_ERR_NULL;
    wcc_status s = check_forward_args(N, Cin, Cout, H, W, L, k, bits, dt);
    if (s != WCC_OK) return s;
    if ((s = check_options(opt, bits, x, y)) != WCC_OK) return s;
    if (opt && opt->Wq) return WCC_ERR_SHAPE;          // pre-quantized weights: fused path only
    if (!aligned16(x) || !aligned16(Wt) || !aligned16(y) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    if (!staged_fits(Cin, Cout, bits)) return WCC_ERR_SHAPE;          // decided before anything is launched
    const FwdWs f = carve_forward_ws(ws, N, Cin, Cout, H, W, k, bits);
    if (ws_bytes < f.total) return WCC_ERR_WORKSPACE;
    const int P = H * W, M = N * k;

    if ((s = profile_mark(0, st)) != WCC_OK) return s;
    // A: Haar transform + channel norms (and the per-position max |coef| the activation scale is taken from)
    s = dwk ? launch_dwconv_haar_fwd(x, dwk, N, Cin, H, W, L, dt, f.coef, f.nrm2, f.amaxpos, st)
            : launch_haar_fwd(x, N, Cin, H, W, L, dt, f.coef, f.nrm2, f.amaxpos, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(1, st)) != WCC_OK) return s;
    // B: joint shrinkage: kept index list, rank map, max |kept|
    s = launch_select(f.nrm2, N, P, k, f.idx, nullptr, f.rank, f.amaxpos, true, f.sel, f.sel_bytes, st);
    if (s != WCC_OK) return s;
    if (opt && opt->alpha > 0.0f && bits >= 2) {        // a given clipping parameter replaces the largest kept magnitude
        set_word_kernel<<<1, 1, 0, st>>>(f.amax_kept, opt->alpha);
        WCC_LAUNCH_CHECK();
    }
    if ((s = profile_mark(2, st)) != WCC_OK) return s;
    s = launch_weight_prep(Wt, Cout, Cin, f.kpad, (opt && opt->weight_bits && bits) ? opt->weight_bits : bits, f.Wq, f.scale_w, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(3, st)) != WCC_OK) return s;
    s = launch_gather_quant(f.coef, f.idx, f.amax_kept, N, Cin, P, k, f.kpad, bits, f.Xq, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(4, st)) != WCC_OK) return s;
    // C: pointwise convolution on the compressed columns
    s = launch_contract(f.Xq, f.Wq, M, Cout, f.kpad, bits, f.acc, f.ldc, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(5, st)) != WCC_OK) return s;
    // D + E: dequantize, zero-fill, inverse transform
    s = launch_scatter_inv(f.acc, f.ldc, bits == 0, f.rank, f.amax_kept, bits, f.scale_w, N, Cout, H, W, L, k, dt, y, st,
                           opt ? opt->residual : nullptr, opt ? opt->relu : 0);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(6, st)) != WCC_OK) return s;

    if (taps) {
        const cudaMemcpyKind dd = cudaMemcpyDeviceToDevice;
        if (taps->coef) WCC_CUDA_TRY(cudaMemcpyAsync(taps->coef, f.coef, (size_t)N * Cin * P * 4, dd, st));
        if (taps->nrm2) WCC_CUDA_TRY(cudaMemcpyAsync(taps->nrm2, f.nrm2, (size_t)N * P * 4, dd, st));
        if (taps->idx) WCC_CUDA_TRY(cudaMemcpyAsync(taps->idx, f.idx, (size_t)M * 4, dd, st));
        if (bits >= 2) {
            if (taps->Xq) WCC_CUDA_TRY(cudaMemcpyAsync(taps->Xq, f.Xq, (size_t)M * f.kpad, dd, st));
            if (taps->Wq) WCC_CUDA_TRY(cudaMemcpyAsync(taps->Wq, f.Wq, (size_t)Cout * f.kpad, dd, st));
            if (taps->scale_w) WCC_CUDA_TRY(cudaMemcpyAsync(taps->scale_w, f.scale_w, (size_t)Cout * 4, dd, st));
            if (taps->scale_a) {
                scale_tap_kernel<<<1, 1, 0, st>>>(f.amax_kept, 0.0f, (float)((1 << (bits - 1)) - 1), taps->scale_a);
                WCC_LAUNCH_CHECK();
            }
        } else if (taps->Xb) {
            WCC_CUDA_TRY(cudaMemcpyAsync(taps->Xb, f.Xq, (size_t)M * f.kpad * 2, dd, st));
        }
        if (taps->acc)
            WCC_CUDA_TRY(cudaMemcpy2DAsync(taps->acc, (size_t)Cout * 4, f.acc, (size_t)f.ldc * 4, (size_t)Cout * 4, M, dd, st));
    }
    return WCC_OK;
}

// ---- fused path ----------------------------------------------------------------------------------
struct FusedWs {
    float* nrm2; float* amaxpos; int32_t* rank; int32_t* idx; void* sel; size_t sel_bytes;
    uint32_t* fine; uint32_t* thr; size_t fine_bytes;
    float* amax_kept; void* Wq; float* scale_w;
    int kpad, es;
    size_t total;
};

static FusedWs carve_fused_ws(void* ws, int N, int Cin, int Cout, int H, int W, int k, int bits)
{
    FusedWs f;
    const size_t P = (size_t)H * W, M = (size_t)N * k;
    f.kpad = wcc_kpad(Cin, bits);
    f.es = (bits == 0) ? 2 : 1;
    size_t off = 0;
    char* b = static_cast<char*>(ws);
    auto take = [&](size_t bytes) { char* p = b ? b + off : nullptr; off += align_up(bytes, 256); return p; };
    f.nrm2 = reinterpret_cast<float*>(take((size_t)N * P * 4));
    f.amaxpos = reinterpret_cast<float*>(take((size_t)N * P * 4));
    f.rank = reinterpret_cast<int32_t*>(take((size_t)N * P * 4));
    f.idx = reinterpret_cast<int32_t*>(take(M * 4));
    f.thr = reinterpret_cast<uint32_t*>(take((size_t)N * 16));
    // the 16-bit histogram sits right before the select scratch, whose zeroed part comes first: one memset clears both
    f.fine_bytes = align_up((size_t)N * FINE_BINS * 4, 256);
    f.fine = reinterpret_cast<uint32_t*>(take(f.fine_bytes));
    f.sel_bytes = select_ws_bytes(N, (int)P);
    f.sel = take(f.sel_bytes);
    f.amax_kept = b ? carve_select_ws(f.sel, N, (int)P).amax : nullptr;
    f.Wq = take((size_t)Cout * f.kpad * f.es);
    f.scale_w = reinterpret_cast<float*>(take((size_t)Cout * 4));
    f.total = off;
    return f;
}

static wcc_status check_options(const wcc_options* o, int bits, const void* x, const void* y)
{
    (void)y;
    if (!o) return WCC_OK;
    if (o->weight_bits != 0 && (bits == 0 || o->weight_bits < 2 || o->weight_bits > 8)) return WCC_ERR_BITS;
    if (o->alpha != o->alpha || o->alpha > 3.0e38f) return WCC_ERR_SHAPE;      // NaN or infinite clipping parameter
    if ((o->Wq != nullptr) != (o->scale_w != nullptr)) return WCC_ERR_NULL;
    if (o->Wq && bits == 0) return WCC_ERR_BITS;                               // codes only exist on the quantized path
    if (!aligned16(o->residual) || !aligned16(o->Wq) || !aligned16(o->scale_w)) return WCC_ERR_ALIGN;
    (void)x;
    return WCC_OK;
}

// ---- many channels: two passes over x, the kept columns gathered from the second ---------------------------------
// Layers beyond one operand tile of the fused kernels.  Like the fused path, the first pass keeps only norms, maxima and
// histograms; the select writes index list and rank map; the kept columns are then transformed again and quantized
// straight into the compressed matrix (no coefficient map in memory), and the contraction over the kept columns, the
// scatter and the inverse transform follow as in the stage-by-stage pipeline.
struct WideWs {
    float* nrm2; float* amaxpos; int32_t* rank; int32_t* idx; uint32_t* thr; uint32_t* fine; size_t fine_bytes;
    void* sel; size_t sel_bytes; float* amax_kept; void* Xq; void* Wq; float* scale_w; int32_t* acc;
    int kpad, ldc, es;
    size_t total;
};

static WideWs carve_wide_ws(void* ws, int N, int Cin, int Cout, int H, int W, int k, int bits)
{
    WideWs f;
    const size_t P = (size_t)H * W, M = (size_t)N * k;
    f.kpad = wcc_kpad(Cin, bits);
    f.es = (bits == 0) ? 2 : 1;
    f.ldc = ceil_div(Cout, 4) * 4;
    size_t off = 0;
    char* b = static_cast<char*>(ws);
    auto take = [&](size_t bytes) { char* p = b ? b + off : nullptr; off += align_up(bytes, 256); return p; };
    f.nrm2 = reinterpret_cast<float*>(take((size_t)N * P * 4));
    f.amaxpos = reinterpret_cast<float*>(take((size_t)N * P * 4));
    f.rank = reinterpret_cast<int32_t*>(take((size_t)N * P * 4));
    f.idx = reinterpret_cast<int32_t*>(take(M * 4));
    f.thr = reinterpret_cast<uint32_t*>(take((size_t)N * 16));
    f.fine_bytes = align_up((size_t)N * FINE_BINS * 4, 256);       // right before the select scratch: one memset clears both
    f.fine = reinterpret_cast<uint32_t*>(take(f.fine_bytes));
    f.sel_bytes = select_ws_bytes(N, (int)P);
    f.sel = take(f.sel_bytes);
    f.amax_kept = b ? carve_select_ws(f.sel, N, (int)P).amax : nullptr;
    f.Xq = take(M * f.kpad * f.es);
    f.Wq = take((size_t)Cout * f.kpad * f.es);
    f.scale_w = reinterpret_cast<float*>(take((size_t)Cout * 4));
    f.acc = reinterpret_cast<int32_t*>(take(M * f.ldc * 4));
    f.total = off;
    return f;
}

// One cluster per image in the selection (it reads the first pass's histograms), vector loads of whole patches.
static bool wide_fits(const void* x, int Cin, int Cout, int H, int W, int bits, wcc_dtype dt)
{
    (void)x; (void)dt;
    return staged_fits(Cin, Cout, bits) && select_in_cluster(H * W) && (W % 4) == 0;
}

static wcc_status wide_impl(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int W,
                            int L, int k, int bits, void* y, wcc_dtype dt, void* ws, size_t ws_bytes,
                            cudaStream_t st, const wcc_taps* taps, const wcc_options* opt)
{
    const WideWs f = carve_wide_ws(ws, N, Cin, Cout, H, W, k, bits);
    if (ws_bytes < f.total) return WCC_ERR_WORKSPACE;
    const int P = H * W, M = N * k;
    wcc_status s;
    if ((s = profile_mark(0, st)) != WCC_OK) return s;
    const SelectWs sw = carve_select_ws(f.sel, N, P);
    WCC_CUDA_TRY(cudaMemsetAsync(f.fine, 0, f.fine_bytes + sw.zero_bytes, st));       // histograms, max |kept|, barrier counters
    NormsExtra ex = {};
    ex.hist1 = sw.hist;
    ex.fine = f.fine;
    const int wbits = (opt && opt->weight_bits && bits) ? opt->weight_bits : bits;
    ex.Wt = Wt; ex.Wq = f.Wq; ex.scale_w = f.scale_w; ex.Cout = Cout; ex.kpad = f.kpad; ex.bits = wbits;
    s = launch_haar_norms(x, N, Cin, H, W, L, dt, f.nrm2, f.amaxpos, ex, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(1, st)) != WCC_OK) return s;
    s = launch_select(f.nrm2, N, P, k, f.idx, nullptr, f.rank, f.amaxpos, true, f.sel, f.sel_bytes, st, true, f.fine, f.thr, true);
    if (s != WCC_OK) return s;
    if (opt && opt->alpha > 0.0f && bits >= 2) {        // a given clipping parameter replaces the largest kept magnitude
        set_word_kernel<<<1, 1, 0, st>>>(f.amax_kept, opt->alpha);
        WCC_LAUNCH_CHECK();
    }
    for (int i = 2; i <= 3; ++i)
        if ((s = profile_mark(i, st)) != WCC_OK) return s;
    s = launch_regather_quant(x, f.rank, f.amax_kept, N, Cin, H, W, L, k, f.kpad, bits, dt, f.Xq, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(4, st)) != WCC_OK) return s;
    s = launch_contract(f.Xq, f.Wq, M, Cout, f.kpad, bits, f.acc, f.ldc, st);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(5, st)) != WCC_OK) return s;
    s = launch_scatter_inv(f.acc, f.ldc, bits == 0, f.rank, f.amax_kept, bits, f.scale_w, N, Cout, H, W, L, k, dt, y, st,
                           opt ? opt->residual : nullptr, opt ? opt->relu : 0);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(6, st)) != WCC_OK) return s;
    if (taps) {
        const cudaMemcpyKind dd = cudaMemcpyDeviceToDevice;
        if (taps->nrm2) WCC_CUDA_TRY(cudaMemcpyAsync(taps->nrm2, f.nrm2, (size_t)N * P * 4, dd, st));
        if (taps->idx) WCC_CUDA_TRY(cudaMemcpyAsync(taps->idx, f.idx, (size_t)M * 4, dd, st));
        if (bits >= 2) {
            if (taps->Xq) WCC_CUDA_TRY(cudaMemcpyAsync(taps->Xq, f.Xq, (size_t)M * f.kpad, dd, st));
            if (taps->Wq) WCC_CUDA_TRY(cudaMemcpyAsync(taps->Wq, f.Wq, (size_t)Cout * f.kpad, dd, st));
            if (taps->scale_w) WCC_CUDA_TRY(cudaMemcpyAsync(taps->scale_w, f.scale_w, (size_t)Cout * 4, dd, st));
            if (taps->scale_a) {
                scale_tap_kernel<<<1, 1, 0, st>>>(f.amax_kept, 0.0f, (float)((1 << (bits - 1)) - 1), taps->scale_a);
                WCC_LAUNCH_CHECK();
            }
        } else if (taps->Xb) {
            WCC_CUDA_TRY(cudaMemcpyAsync(taps->Xb, f.Xq, (size_t)M * f.kpad * 2, dd, st));
        }
        if (taps->acc)
            WCC_CUDA_TRY(cudaMemcpy2DAsync(taps->acc, (size_t)Cout * 4, f.acc, (size_t)f.ldc * 4, (size_t)Cout * 4, M, dd, st));
    }
    return WCC_OK;
}

// Chain fusion hooks of forward_impl: norms_ready = the previous layer's second pass has already produced this layer's
// norms, per-position maxima and histograms in this workspace (no first pass; the weights are quantized by a launch of
// their own); next_ws = workspace of the next layer, whose first pass this layer's second pass performs.
struct ChainHooks { bool norms_ready; void* next_ws; int next_cout; };

// Can the second pass of layer (Cin -> Cout) also be the first pass of a next layer?  (The four-tile kernel with room
// for the tokens, one cluster per image in the selection.)
// It pays while the next layer's input is narrow: the extra transform and norm chain cost the second pass about 0.2 us
// per output channel on a 2 x 256 x 512 map (192 channels: +41 us against a 31 us first pass of its own; 32 channels:
// +12 us against 18 us), because the pass is bound by instruction issue, not by the bytes the fusion saves.
constexpr int CHAIN_FUSE_MAX_CHANNELS = 64;

static bool chain_fusable(const void* x, int Cin, int Cout, int H, int W, int bits, wcc_dtype dt)
{
    const int esz = (dt == WCC_BF16) ? 2 : 4;
    return Cout <= CHAIN_FUSE_MAX_CHANNELS && select_in_cluster(H * W) &&
           ft_plan(x, esz, W, Cout, wcc_kpad(Cin, bits), bits, true).ok;
}

static wcc_status forward_impl(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int W,
                               int L, int k, int bits, void* y, wcc_dtype dt, void* ws, size_t ws_bytes,
                               cudaStream_t st, const wcc_taps* taps, const wcc_options* opt = nullptr,
                               const ChainHooks* hooks = nullptr)
{
    const bool own_codes = opt && opt->Wq;             // weights arrive quantized: Wt is not read
    if (!x || (!Wt && !own_codes) || !y || !ws) return WCC_ERR_NULL;
    wcc_status s = check_forward_args(N, Cin, Cout, H, W, L, k, bits, dt);
    if (s != WCC_OK) return s;
    if ((s = check_options(opt, bits, x, y)) != WCC_OK) return s;
    if (!aligned16(x) || !aligned16(Wt) || !aligned16(y) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    if (taps && (!aligned16(taps->coef) || !aligned16(taps->Xq) || !aligned16(taps->Xb) || !aligned16(taps->acc)))
        return WCC_ERR_ALIGN;
    if (!fused_fits(x, Cout, W, bits, dt, Cin)) {      // decided before anything is launched: channel counts beyond one
        if (own_codes) return WCC_ERR_SHAPE;           // operand tile run stage by stage (the contraction there tiles K and N)
        if (wide_fits(x, Cin, Cout, H, W, bits, dt) && !(taps && taps->coef))
            return wide_impl(x, Wt, N, Cin, Cout, H, W, L, k, bits, y, dt, ws, ws_bytes, st, taps, opt);
        return staged_impl(x, Wt, N, Cin, Cout, H, W, L, k, bits, y, dt, ws, ws_bytes, st, taps, opt);
    }
    const FusedWs f = carve_fused_ws(ws, N, Cin, Cout, H, W, k, bits);
    if (ws_bytes < f.total) return WCC_ERR_WORKSPACE;
    const int P = H * W, M = N * k;

    if ((s = profile_mark(0, st)) != WCC_OK) return s;
    // first pass over x: transform in registers, keep only the channel norms and the per-position max |coef| (the
    // coefficient map is written only when a test asks for it).  The same launch fills round 1 of the select's
    // histogram and quantizes the weights in a few extra CTAs.
    const SelectWs sw = carve_select_ws(f.sel, N, P);
    const bool norms_ready = hooks && hooks->norms_ready;
    if (!norms_ready)
        WCC_CUDA_TRY(cudaMemsetAsync(f.fine, 0, f.fine_bytes + sw.zero_bytes, st));   // histograms, max |kept|, barrier counters
    if ((s = profile_mark(1, st)) != WCC_OK) return s;
    NormsExtra ex = {};
    ex.coef = taps ? taps->coef : nullptr;
    ex.hist1 = sw.hist;
    ex.fine = f.fine;
    const int wbits = (opt && opt->weight_bits && bits) ? opt->weight_bits : bits;
    if (!own_codes) { ex.Wt = Wt; ex.Wq = f.Wq; ex.scale_w = f.scale_w; ex.Cout = Cout; ex.kpad = f.kpad; ex.bits = wbits; }
    const void* Wq_use = own_codes ? static_cast<const void*>(opt->Wq) : f.Wq;
    const float* scale_w_use = own_codes ? opt->scale_w : f.scale_w;
    const FusedExtra fx = {opt ? opt->alpha : 0.0f, opt ? opt->relu : 0, opt ? opt->residual : nullptr};
    if (norms_ready) {
        if (!own_codes) {
            s = launch_weight_prep(Wt, Cout, Cin, f.kpad, wbits, f.Wq, f.scale_w, st);
            if (s != WCC_OK) return s;
        }
    } else {
        s = launch_haar_norms(x, N, Cin, H, W, L, dt, f.nrm2, f.amaxpos, ex, st);
        if (s != WCC_OK) return s;
    }
    if ((s = profile_mark(2, st)) != WCC_OK) return s;
    // joint shrinkage: index list, rank map, max |kept|
    s = launch_select(f.nrm2, N, P, k, f.idx, nullptr, f.rank, f.amaxpos, true, f.sel, f.sel_bytes, st, true,
                      f.fine, f.thr, taps != nullptr);
    if (s != WCC_OK) return s;
    if ((s = profile_mark(3, st)) != WCC_OK) return s;
    // second pass over x: transform, mask + quantize, tensor-core contraction, dequantize, inverse, store
    void* xq_tap = taps ? (bits >= 2 ? static_cast<void*>(taps->Xq) : taps->Xb) : nullptr;
    ft::NextNorms nx = {};
    const bool feeds_next = hooks && hooks->next_ws;
    if (feeds_next) {
        // the next layer's workspace (its input has Cout channels): clear its histograms, then let this layer's second
        // pass fill its norms, maxima and histograms
        const FusedWs g = carve_fused_ws(hooks->next_ws, N, Cout, hooks->next_cout, H, W, k, bits);
        const SelectWs gs = carve_select_ws(g.sel, N, P);
        WCC_CUDA_TRY(cudaMemsetAsync(g.fine, 0, g.fine_bytes + gs.zero_bytes, st));
        nx.nrm2 = g.nrm2; nx.amaxpos = g.amaxpos; nx.hist1 = gs.hist; nx.fine = g.fine;
    }
    s = launch_fused_tiles(x, Wq_use, f.rank, f.nrm2, f.thr, f.amax_kept, bits, scale_w_use, N, Cin, Cout, H, W, L, k, f.kpad, dt, y,
                           xq_tap, taps ? taps->acc : nullptr, fx, st, feeds_next ? &nx : nullptr);
    if (feeds_next && s != WCC_OK) return s == WCC_ERR_SHAPE ? WCC_ERR_CUDA : s;       // (chain_fusable said it fits)
    if (s == WCC_ERR_SHAPE)                            // shapes the four-tile kernel does not cover (nothing was launched)
        s = launch_fused_pass2(x, Wq_use, f.rank, f.nrm2, f.thr, f.amax_kept, bits, scale_w_use, N, Cin, Cout, H, W, L, k, f.kpad, dt, y,
                               xq_tap, taps ? taps->acc : nullptr, fx, st);
    if (s != WCC_OK) return s;
    for (int i = 4; i <= WCC_NUM_STAGES; ++i)
        if ((s = profile_mark(i, st)) != WCC_OK) return s;

    if (taps) {
        const cudaMemcpyKind dd = cudaMemcpyDeviceToDevice;
        if (taps->nrm2) WCC_CUDA_TRY(cudaMemcpyAsync(taps->nrm2, f.nrm2, (size_t)N * P * 4, dd, st));
        if (taps->idx) WCC_CUDA_TRY(cudaMemcpyAsync(taps->idx, f.idx, (size_t)M * 4, dd, st));
        if (bits >= 2) {
            if (taps->Wq) WCC_CUDA_TRY(cudaMemcpyAsync(taps->Wq, Wq_use, (size_t)Cout * f.kpad, dd, st));
            if (taps->scale_w) WCC_CUDA_TRY(cudaMemcpyAsync(taps->scale_w, scale_w_use, (size_t)Cout * 4, dd, st));
            if (taps->scale_a) {
                scale_tap_kernel<<<1, 1, 0, st>>>(f.amax_kept, fx.alpha, (float)((1 << (bits - 1)) - 1), taps->scale_a);
                WCC_LAUNCH_CHECK();
            }
        }
    }
    return WCC_OK;
}

// ---- kept set as a bitmap ---------------------------------------------------------------------------
// bit p % 32 of word p / 32 of image n is set when position p is kept (rank map >= 0)
__global__ void __launch_bounds__(256)
rank_to_bitmap_kernel(const int32_t* __restrict__ rank, int N, int P, int words, uint32_t* __restrict__ bitmap)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;          // one thread per position, padded to words * 32
    const long long per = (long long)words * 32;
    if (i >= (long long)N * per) return;                                            // (whole warps leave together)
    const int n = (int)(i / per), p = (int)(i - (long long)n * per);
    const bool kept = p < P && rank[(size_t)n * P + p] >= 0;
    const unsigned m = __ballot_sync(0xFFFFFFFFu, kept);
    if ((threadIdx.x & 31) == 0) bitmap[(size_t)n * words + (p >> 5)] = m;
}

struct BitmapWs { int32_t* rank; int32_t* idx; void* sel; size_t sel_bytes; size_t total; };

static BitmapWs carve_bitmap_ws(void* ws, int N, int P, int k)
{
    BitmapWs b = {};
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off += align_up(bytes, 256); return p; };
    b.rank = reinterpret_cast<int32_t*>(take((size_t)N * P * 4));
    b.idx = reinterpret_cast<int32_t*>(take((size_t)N * k * 4));
    b.sel_bytes = select_ws_bytes(N, P);
    b.sel = take(b.sel_bytes);
    b.total = off;
    return b;
}

// ---- maps whose sides are no multiples of 2^levels: zero padding at the bottom and on the right -------------------
template <typename E>
__global__ void __launch_bounds__(256)
pad_planes_kernel(const E* __restrict__ src, long long planes, int H, int W, int Hp, int Wp, E* __restrict__ dst)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= planes * Hp * Wp) return;
    const int c = (int)(i % Wp);
    const long long t = i / Wp;
    const int r = (int)(t % Hp);
    const long long pl = t / Hp;
    dst[i] = (r < H && c < W) ? src[(pl * H + r) * W + c] : E(0);
}
template <typename E>
__global__ void __launch_bounds__(256)
crop_planes_kernel(const E* __restrict__ src, long long planes, int H, int W, int Hp, int Wp, E* __restrict__ dst)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= planes * H * W) return;
    const int c = (int)(i % W);
    const long long t = i / W;
    const int r = (int)(t % H);
    const long long pl = t / H;
    dst[i] = src[(pl * Hp + r) * Wp + c];
}

struct PaddedWs { void* xp; void* yp; void* inner; size_t inner_bytes; size_t total; int Hp, Wp; };

static PaddedWs carve_padded_ws(void* ws, int N, int Cin, int Cout, int H, int W, int L, int k, int bits, wcc_dtype dt)
{
    PaddedWs p = {};
    const int unit = 1 << L;
    p.Hp = ceil_div(H, unit) * unit;
    p.Wp = ceil_div(W, unit) * unit;
    const size_t es = (dt == WCC_BF16) ? 2 : 4;
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) { char* q = base ? base + off : nullptr; off += align_up(bytes, 256); return q; };
    p.xp = take((size_t)N * Cin * p.Hp * p.Wp * es);
    p.yp = take((size_t)N * Cout * p.Hp * p.Wp * es);
    p.inner_bytes = wcc_workspace_bytes(N, Cin, Cout, p.Hp, p.Wp, L, k, bits, dt);
    p.inner = take(p.inner_bytes);
    p.total = p.inner_bytes ? off : 0;
    return p;
}

// ---- other wavelets -----------------------------------------------------------------------------------
static wcc_status check_filters(const float* lo, const float* hi, int taps)
{
    if (!lo || !hi) return WCC_ERR_NULL;
    if (taps < 2 || taps > wv::MAX_TAPS || (taps & 1)) return WCC_ERR_SHAPE;
    return WCC_OK;
}

struct WaveletWs { FwdWs f; float* scratch_in; float* ywt; float* scratch_out; size_t total; };

static WaveletWs carve_wavelet_ws(void* ws, int N, int Cin, int Cout, int H, int W, int k, int bits)
{
    WaveletWs w = {};
    w.f = carve_forward_ws(ws, N, Cin, Cout, H, W, k, bits);
    const size_t P = (size_t)H * W;
    char* base = static_cast<char*>(ws);
    size_t off = w.f.total;
    auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off += align_up(bytes, 256); return p; };
    w.scratch_in = reinterpret_cast<float*>(take((size_t)N * Cin * P * 4));
    w.ywt = reinterpret_cast<float*>(take((size_t)N * Cout * P * 4));
    w.scratch_out = reinterpret_cast<float*>(take((size_t)N * Cout * P * 4));
    w.total = off;
    return w;
}

// ---- inverted residual block -------------------------------------------------------------------------
struct BlockWs { void* u; void* layer_ws; size_t layer_ws_bytes; size_t total; };

static BlockWs carve_block_ws(void* ws, int N, int C, int E, int H, int W, int L, int k, int bits, wcc_dtype dt)
{
    BlockWs b = {};
    const size_t es = (dt == WCC_BF16) ? 2 : 4;
    const size_t w1 = wcc_workspace_bytes(N, C, E, H, W, L, k, bits, dt);
    const size_t w3 = wcc_staged_workspace_bytes(N, E, C, H, W, L, k, bits, dt);
    if (w1 == 0 || w3 == 0) return b;
    char* base = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = base ? base + off : nullptr; off += align_up(bytes, 256); return p; };
    b.u = take((size_t)N * E * H * W * es);
    b.layer_ws_bytes = w1 > w3 ? w1 : w3;
    b.layer_ws = take(b.layer_ws_bytes);
    b.total = off;
    return b;
}

// ---- chain of layers -------------------------------------------------------------------------------
struct ChainWs { void* act[2]; void* layer_ws[2]; size_t layer_ws_bytes; size_t total; };

static wcc_status chain_shapes_ok(const wcc_chain_layer* layers, int n_layers)
{
    if (!layers) return WCC_ERR_NULL;
    if (n_layers < 1 || n_layers > 4096) return WCC_ERR_SHAPE;
    for (int i = 0; i + 1 < n_layers; ++i)
        if (layers[i].Cout != layers[i + 1].Cin) return WCC_ERR_SHAPE;
    return WCC_OK;
}

static ChainWs carve_chain_ws(void* ws, const wcc_chain_layer* layers, int n_layers, int N, int H, int W, int L, int k, int bits,
                              wcc_dtype dt)
{
    ChainWs c = {};
    const size_t es = (dt == WCC_BF16) ? 2 : 4, P = (size_t)H * W;
    size_t act = 0, lw = 0;
    for (int i = 0; i < n_layers; ++i) {
        if (i + 1 < n_layers) { const size_t b = (size_t)N * layers[i].Cout * P * es; if (b > act) act = b; }
        const size_t b = wcc_workspace_bytes(N, layers[i].Cin, layers[i].Cout, H, W, L, k, bits, dt);
        if (b == 0) { c.total = 0; return c; }
        if (b > lw) lw = b;
    }
    char* b = static_cast<char*>(ws);
    size_t off = 0;
    auto take = [&](size_t bytes) { char* p = b ? b + off : nullptr; off += align_up(bytes, 256); return p; };
    c.act[0] = take(act);
    c.act[1] = take(act);
    c.layer_ws_bytes = lw;
    c.layer_ws[0] = take(lw);                          // consecutive layers alternate: a fused second pass writes the next
    c.layer_ws[1] = take(lw);                          // layer's norms while it still reads its own
    c.total = off;
    return c;
}

}  // namespace wcc

using namespace wcc;

extern "C" {

int wcc_kpad(int Cin, int bits)
{
    if (Cin <= 0) return 0;
    return (bits == 0) ? ceil_div(Cin, 16) * 16 : ceil_div(Cin, 32) * 32;
}

size_t wcc_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt)
{
    if (check_forward_args(N, Cin, Cout, H, Wd, levels, k, bits, dt) != WCC_OK) return 0;
    if (!fused_fits(nullptr, Cout, Wd, bits, dt, Cin)) {                       // these shapes run around the tiled contraction
        if (!staged_fits(Cin, Cout, bits)) return 0;
        const size_t a = carve_forward_ws(nullptr, N, Cin, Cout, H, Wd, k, bits).total;
        const size_t b = carve_wide_ws(nullptr, N, Cin, Cout, H, Wd, k, bits).total;
        return a > b ? a : b;
    }
    return carve_fused_ws(nullptr, N, Cin, Cout, H, Wd, k, bits).total;
}

size_t wcc_staged_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt)
{
    if (check_forward_args(N, Cin, Cout, H, Wd, levels, k, bits, dt) != WCC_OK) return 0;
    if (!staged_fits(Cin, Cout, bits)) return 0;
    return carve_forward_ws(nullptr, N, Cin, Cout, H, Wd, k, bits).total;
}

size_t wcc_select_workspace_bytes(int N, int P)
{
    if (N <= 0 || P <= 0) return 0;
    return select_ws_bytes(N, P);
}

wcc_status wcc_haar_fwd(const void* x, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                        float* coef, float* nrm2, void* stream)
{
    if (!x || !coef) return WCC_ERR_NULL;
    wcc_status s = check_plane_args(N, C, H, Wd, levels, dt);
    if (s != WCC_OK) return s;
    if (!aligned16(x) || !aligned16(coef) || !aligned16(nrm2)) return WCC_ERR_ALIGN;
    return launch_haar_fwd(x, N, C, H, Wd, levels, dt, coef, nrm2, nullptr, static_cast<cudaStream_t>(stream));
}

wcc_status wcc_haar_inv(const float* coef, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                        void* x_out, void* stream)
{
    if (!coef || !x_out) return WCC_ERR_NULL;
    wcc_status s = check_plane_args(N, C, H, Wd, levels, dt);
    if (s != WCC_OK) return s;
    if (!aligned16(coef) || !aligned16(x_out)) return WCC_ERR_ALIGN;
    return launch_haar_inv(coef, N, C, H, Wd, levels, dt, x_out, static_cast<cudaStream_t>(stream));
}

wcc_status wcc_select_topk(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau,
                           void* ws, size_t ws_bytes, void* stream)
{
    if (!nrm2 || !idx || !ws) return WCC_ERR_NULL;
    if (N <= 0 || P <= 0 || N > 65535 || P > (1 << 30)) return WCC_ERR_SHAPE;
    if (k < 1 || k > P) return WCC_ERR_K;
    if (!aligned16(nrm2) || !aligned16(idx) || !aligned16(ws)) return WCC_ERR_ALIGN;
    if (ws_bytes < select_ws_bytes(N, P)) return WCC_ERR_WORKSPACE;
    return launch_select(nrm2, N, P, k, idx, tau, nullptr, nullptr, false, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

wcc_status wcc_select_topk_static(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau, void* stream)
{
    if (!nrm2 || !idx) return WCC_ERR_NULL;
    if (N <= 0 || P <= 0 || N > 65535 || P > (1 << 30)) return WCC_ERR_SHAPE;
    if (k < 1 || k > P) return WCC_ERR_K;
    if (!aligned16(nrm2) || !aligned16(idx)) return WCC_ERR_ALIGN;
    const size_t need = select_ws_bytes(N, P);
    if (need > (size_t)WCC_STATIC_SCRATCH_BYTES) return WCC_ERR_WORKSPACE;     // beyond the built-in scratch
    void* scratch = nullptr;
    wcc_status s = static_scratch_ptr(&scratch);                               // first call per device: address lookup
    if (s != WCC_OK) return s;
    // launch_select zeroes the histograms it accumulates into; everything else in the scratch is written before it is read
    return launch_select(nrm2, N, P, k, idx, tau, nullptr, nullptr, false, scratch, need, static_cast<cudaStream_t>(stream));
}

wcc_status wcc_forward(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                       int levels, int k, int bits, void* y, wcc_dtype dt,
                       void* ws, size_t ws_bytes, void* stream)
{
    return forward_impl(x, Wt, N, Cin, Cout, H, Wd, levels, k, bits, y, dt, ws, ws_bytes,
                        static_cast<cudaStream_t>(stream), nullptr);
}

wcc_status wcc_forward_ex(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                          int levels, int k, int bits, void* y, wcc_dtype dt,
                          void* ws, size_t ws_bytes, void* stream, const wcc_options* opt, const wcc_taps* taps)
{
    return forward_impl(x, Wt, N, Cin, Cout, H, Wd, levels, k, bits, y, dt, ws, ws_bytes,
                        static_cast<cudaStream_t>(stream), taps, opt);
}

wcc_status wcc_dwconv_haar_fwd(const void* u, const float* Wdw, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                               float* coef, float* nrm2, void* stream)
{
    if (!u || !Wdw || !coef) return WCC_ERR_NULL;
    wcc_status s = check_plane_args(N, C, H, Wd, levels, dt);
    if (s != WCC_OK) return s;
    if (!aligned16(u) || !aligned16(Wdw) || !aligned16(coef) || !aligned16(nrm2)) return WCC_ERR_ALIGN;
    return launch_dwconv_haar_fwd(u, Wdw, N, C, H, Wd, levels, dt, coef, nrm2, nullptr, static_cast<cudaStream_t>(stream));
}

size_t wcc_block_workspace_bytes(int N, int C, int E, int H, int Wd, int levels, int k, int bits, wcc_dtype dt)
{
    if (check_forward_args(N, C, E, H, Wd, levels, k, bits, dt) != WCC_OK) return 0;
    return carve_block_ws(nullptr, N, C, E, H, Wd, levels, k, bits, dt).total;
}

wcc_status wcc_block_forward(const void* x, const float* W1, const float* Wdw, const float* W3, int N, int C, int E,
                             int H, int Wd, int levels, int k, int bits, void* y, wcc_dtype dt,
                             void* ws, size_t ws_bytes, void* stream)
{
    if (!x || !W1 || !Wdw || !W3 || !y || !ws) return WCC_ERR_NULL;
    wcc_status s = check_forward_args(N, C, E, H, Wd, levels, k, bits, dt);
    if (s != WCC_OK) return s;
    if ((s = check_forward_args(N, E, C, H, Wd, levels, k, bits, dt)) != WCC_OK) return s;
    if (!aligned16(x) || !aligned16(W1) || !aligned16(Wdw) || !aligned16(W3) || !aligned16(y) ||
        (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    const BlockWs b = carve_block_ws(ws, N, C, E, H, Wd, levels, k, bits, dt);
    if (b.total == 0) return WCC_ERR_SHAPE;
    if (ws_bytes < b.total) return WCC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // u = WCC(W1, x): C -> E channels
    s = forward_impl(x, W1, N, C, E, H, Wd, levels, k, bits, b.u, dt, b.layer_ws, b.layer_ws_bytes, st, nullptr);
    if (s != WCC_OK) return s;
    // y = x + WCC(W3, dw3x3(u)): the depthwise convolution is fused with the second layer's transform
    wcc_options o = {};
    o.residual = x;
    return staged_impl(b.u, W3, N, E, C, H, Wd, levels, k, bits, y, dt, b.layer_ws, b.layer_ws_bytes, st, nullptr, &o, Wdw);
}

wcc_status wcc_dwt_fwd(const void* x, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                       const float* dec_lo, const float* dec_hi, int taps, float* coef, float* nrm2,
                       void* ws, size_t ws_bytes, void* stream)
{
    if (!x || !coef || !ws) return WCC_ERR_NULL;
    wcc_status s = check_plane_args(N, C, H, Wd, levels, dt);
    if (s != WCC_OK) return s;
    if ((s = check_filters(dec_lo, dec_hi, taps)) != WCC_OK) return s;
    if (!aligned16(x) || !aligned16(coef) || !aligned16(nrm2) || !aligned16(ws)) return WCC_ERR_ALIGN;
    const size_t need = (size_t)N * C * H * Wd * 4;
    if (ws_bytes < need) return WCC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const wv::TapProducts tp = wv::tap_products(dec_lo, dec_hi, taps);
    s = launch_dwt_fwd(x, (long long)N * C, H, Wd, levels, dt, tp, coef, static_cast<float*>(ws), st);
    if (s != WCC_OK) return s;
    if (nrm2) {
        const long long P = (long long)H * Wd;
        if ((s = launch_coef_norms(coef, N, C, P, nrm2, nullptr, st)) != WCC_OK) return s;
    }
    return WCC_OK;
}

wcc_status wcc_dwt_inv(const float* coef, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                       const float* rec_lo, const float* rec_hi, int taps, void* x_out,
                       void* ws, size_t ws_bytes, void* stream)
{
    if (!coef || !x_out || !ws) return WCC_ERR_NULL;
    wcc_status s = check_plane_args(N, C, H, Wd, levels, dt);
    if (s != WCC_OK) return s;
    if ((s = check_filters(rec_lo, rec_hi, taps)) != WCC_OK) return s;
    if (!aligned16(coef) || !aligned16(x_out) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    const size_t plane_bytes = align_up((size_t)N * C * H * Wd * 4, 256);
    if (ws_bytes < 2 * plane_bytes) return WCC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* work = static_cast<float*>(ws);
    float* scratch = reinterpret_cast<float*>(static_cast<char*>(ws) + plane_bytes);
    WCC_CUDA_TRY(cudaMemcpyAsync(work, coef, (size_t)N * C * H * Wd * 4, cudaMemcpyDeviceToDevice, st));
    const wv::TapProducts tp = wv::tap_products(rec_lo, rec_hi, taps);
    return launch_dwt_inv(work, (long long)N * C, H, Wd, levels, dt, tp, x_out, scratch, st);
}

size_t wcc_wavelet_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt)
{
    if (check_forward_args(N, Cin, Cout, H, Wd, levels, k, bits, dt) != WCC_OK || !staged_fits(Cin, Cout, bits)) return 0;
    return carve_wavelet_ws(nullptr, N, Cin, Cout, H, Wd, k, bits).total;
}

wcc_status wcc_forward_wavelet(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                               int levels, int k, int bits, const float* dec_lo, const float* dec_hi,
                               const float* rec_lo, const float* rec_hi, int taps, void* y, wcc_dtype dt,
                               void* ws, size_t ws_bytes, void* stream, const wcc_taps* tp_out)
{
    if (!x || !Wt || !y || !ws) return WCC_ERR_NULL;
    wcc_status s = check_forward_args(N, Cin, Cout, H, Wd, levels, k, bits, dt);
    if (s != WCC_OK) return s;
    if ((s = check_filters(dec_lo, dec_hi, taps)) != WCC_OK) return s;
    if ((s = check_filters(rec_lo, rec_hi, taps)) != WCC_OK) return s;
    if (!aligned16(x) || !aligned16(Wt) || !aligned16(y) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    if (!staged_fits(Cin, Cout, bits)) return WCC_ERR_SHAPE;
    const WaveletWs w = carve_wavelet_ws(ws, N, Cin, Cout, H, Wd, k, bits);
    if (ws_bytes < w.total) return WCC_ERR_WORKSPACE;
    const FwdWs& f = w.f;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long P = (long long)H * Wd;
    const int M = N * k;
    // A: the transform with the given decomposition filters, then norms and per-position maxima
    s = launch_dwt_fwd(x, (long long)N * Cin, H, Wd, levels, dt, wv::tap_products(dec_lo, dec_hi, taps), f.coef, w.scratch_in, st);
    if (s != WCC_OK) return s;
    if ((s = launch_coef_norms(f.coef, N, Cin, P, f.nrm2, f.amaxpos, st)) != WCC_OK) return s;
    // B, C: as for Haar
    s = launch_select(f.nrm2, N, (int)P, k, f.idx, nullptr, f.rank, f.amaxpos, true, f.sel, f.sel_bytes, st);
    if (s != WCC_OK) return s;
    if ((s = launch_weight_prep(Wt, Cout, Cin, f.kpad, bits, f.Wq, f.scale_w, st)) != WCC_OK) return s;
    if ((s = launch_gather_quant(f.coef, f.idx, f.amax_kept, N, Cin, (int)P, k, f.kpad, bits, f.Xq, st)) != WCC_OK) return s;
    if ((s = launch_contract(f.Xq, f.Wq, M, Cout, f.kpad, bits, f.acc, f.ldc, st)) != WCC_OK) return s;
    // D: dequantize into the zero map; E: the synthesis with the reconstruction filters
    WCC_CUDA_TRY(cudaMemsetAsync(w.ywt, 0, (size_t)N * Cout * P * 4, st));
    const long long items = (long long)M * Cout;
    const float qmax = (bits >= 2) ? (float)((1 << (bits - 1)) - 1) : 1.0f;
    if (bits == 0)
        wv::scatter_coef_kernel<true><<<(unsigned)((items + 255) / 256), 256, 0, st>>>(f.acc, f.ldc, f.idx, f.amax_kept, qmax, f.scale_w, N, Cout, P, k, w.ywt);
    else
        wv::scatter_coef_kernel<false><<<(unsigned)((items + 255) / 256), 256, 0, st>>>(f.acc, f.ldc, f.idx, f.amax_kept, qmax, f.scale_w, N, Cout, P, k, w.ywt);
    WCC_LAUNCH_CHECK();
    s = launch_dwt_inv(w.ywt, (long long)N * Cout, H, Wd, levels, dt, wv::tap_products(rec_lo, rec_hi, taps), y, w.scratch_out, st);
    if (s != WCC_OK) return s;
    if (tp_out) {
        const cudaMemcpyKind dd = cudaMemcpyDeviceToDevice;
        if (tp_out->coef) WCC_CUDA_TRY(cudaMemcpyAsync(tp_out->coef, f.coef, (size_t)N * Cin * P * 4, dd, st));
        if (tp_out->nrm2) WCC_CUDA_TRY(cudaMemcpyAsync(tp_out->nrm2, f.nrm2, (size_t)N * P * 4, dd, st));
        if (tp_out->idx) WCC_CUDA_TRY(cudaMemcpyAsync(tp_out->idx, f.idx, (size_t)M * 4, dd, st));
        if (bits >= 2 && tp_out->Xq) WCC_CUDA_TRY(cudaMemcpyAsync(tp_out->Xq, f.Xq, (size_t)M * f.kpad, dd, st));
        if (tp_out->acc)
            WCC_CUDA_TRY(cudaMemcpy2DAsync(tp_out->acc, (size_t)Cout * 4, f.acc, (size_t)f.ldc * 4, (size_t)Cout * 4, M, dd, st));
    }
    return WCC_OK;
}

size_t wcc_select_bitmap_workspace_bytes(int N, int P, int k)
{
    if (N <= 0 || P <= 0 || k < 1 || k > P) return 0;
    return carve_bitmap_ws(nullptr, N, P, k).total;
}

wcc_status wcc_select_topk_bitmap(const float* nrm2, int N, int P, int k, uint32_t* bitmap, float* tau,
                                  void* ws, size_t ws_bytes, void* stream)
{
    if (!nrm2 || !bitmap || !ws) return WCC_ERR_NULL;
    if (N <= 0 || P <= 0 || N > 65535 || P > (1 << 30)) return WCC_ERR_SHAPE;
    if (k < 1 || k > P) return WCC_ERR_K;
    if (!aligned16(nrm2) || !aligned16(bitmap) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    const BitmapWs b = carve_bitmap_ws(ws, N, P, k);
    if (ws_bytes < b.total) return WCC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    wcc_status s = launch_select(nrm2, N, P, k, b.idx, tau, b.rank, nullptr, false, b.sel, b.sel_bytes, st);
    if (s != WCC_OK) return s;
    const int words = ceil_div(P, 32);
    const long long threads = (long long)N * words * 32;
    rank_to_bitmap_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(b.rank, N, P, words, bitmap);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

size_t wcc_padded_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt)
{
    if (N <= 0 || Cin <= 0 || Cout <= 0 || H <= 0 || Wd <= 0 || levels < 1 || levels > 3) return 0;
    return carve_padded_ws(nullptr, N, Cin, Cout, H, Wd, levels, k, bits, dt).total;
}

wcc_status wcc_forward_padded(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                              int levels, int k, int bits, void* y, wcc_dtype dt,
                              void* ws, size_t ws_bytes, void* stream)
{
    if (!x || !Wt || !y || !ws) return WCC_ERR_NULL;
    if (N <= 0 || Cin <= 0 || Cout <= 0 || H <= 0 || Wd <= 0 || levels < 1 || levels > 3) return WCC_ERR_SHAPE;
    if (dt != WCC_F32 && dt != WCC_BF16) return WCC_ERR_DTYPE;
    if (!aligned16(x) || !aligned16(Wt) || !aligned16(y) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return WCC_ERR_ALIGN;
    const PaddedWs p = carve_padded_ws(ws, N, Cin, Cout, H, Wd, levels, k, bits, dt);
    wcc_status s = check_forward_args(N, Cin, Cout, p.Hp, p.Wp, levels, k, bits, dt);       // k counts padded positions
    if (s != WCC_OK) return s;
    if (p.total == 0) return WCC_ERR_SHAPE;
    if (ws_bytes < p.total) return WCC_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (p.Hp == H && p.Wp == Wd)                       // nothing to pad: the plain layer
        return forward_impl(x, Wt, N, Cin, Cout, H, Wd, levels, k, bits, y, dt, p.inner, p.inner_bytes, st, nullptr);
    const long long in_planes = (long long)N * Cin, out_planes = (long long)N * Cout;
    const long long n_in = in_planes * p.Hp * p.Wp, n_out = out_planes * H * Wd;
    if (dt == WCC_BF16)
        pad_planes_kernel<uint16_t><<<(unsigned)((n_in + 255) / 256), 256, 0, st>>>(static_cast<const uint16_t*>(x), in_planes, H, Wd, p.Hp, p.Wp, static_cast<uint16_t*>(p.xp));
    else
        pad_planes_kernel<uint32_t><<<(unsigned)((n_in + 255) / 256), 256, 0, st>>>(static_cast<const uint32_t*>(x), in_planes, H, Wd, p.Hp, p.Wp, static_cast<uint32_t*>(p.xp));
    WCC_LAUNCH_CHECK();
    s = forward_impl(p.xp, Wt, N, Cin, Cout, p.Hp, p.Wp, levels, k, bits, p.yp, dt, p.inner, p.inner_bytes, st, nullptr);
    if (s != WCC_OK) return s;
    if (dt == WCC_BF16)
        crop_planes_kernel<uint16_t><<<(unsigned)((n_out + 255) / 256), 256, 0, st>>>(static_cast<const uint16_t*>(p.yp), out_planes, H, Wd, p.Hp, p.Wp, static_cast<uint16_t*>(y));
    else
        crop_planes_kernel<uint32_t><<<(unsigned)((n_out + 255) / 256), 256, 0, st>>>(static_cast<const uint32_t*>(p.yp), out_planes, H, Wd, p.Hp, p.Wp, static_cast<uint32_t*>(y));
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

size_t wcc_chain_workspace_bytes(const wcc_chain_layer* layers, int n_layers, int N, int H, int Wd, int levels, int k,
                                 int bits, wcc_dtype dt)
{
    if (chain_shapes_ok(layers, n_layers) != WCC_OK) return 0;
    return carve_chain_ws(nullptr, layers, n_layers, N, H, Wd, levels, k, bits, dt).total;
}

wcc_status wcc_chain_forward(const void* x, const wcc_chain_layer* layers, int n_layers, int N, int H, int Wd,
                             int levels, int k, int bits, void* y, wcc_dtype dt, void* ws, size_t ws_bytes, void* stream)
{
    if (!x || !y || !ws) return WCC_ERR_NULL;
    wcc_status s = chain_shapes_ok(layers, n_layers);
    if (s != WCC_OK) return s;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return WCC_ERR_ALIGN;
    // every layer's arguments are checked before the first one is launched
    for (int i = 0; i < n_layers; ++i) {
        if (!layers[i].Wt) return WCC_ERR_NULL;
        if ((s = check_forward_args(N, layers[i].Cin, layers[i].Cout, H, Wd, levels, k, bits, dt)) != WCC_OK) return s;
        if (!aligned16(layers[i].Wt)) return WCC_ERR_ALIGN;
        if (layers[i].alpha != layers[i].alpha || layers[i].alpha > 3.0e38f) return WCC_ERR_SHAPE;
    }
    const ChainWs c = carve_chain_ws(ws, layers, n_layers, N, H, Wd, levels, k, bits, dt);
    if (c.total == 0) return WCC_ERR_SHAPE;
    if (ws_bytes < c.total) return WCC_ERR_WORKSPACE;
    // Layer i's second pass doubles as layer i+1's first pass (inverse transform, ReLU and the next forward transform
    // on the same tile while it is in registers) wherever both layers run the four-tile kernel.
    const void* in = x;
    bool norms_ready = false;
    for (int i = 0; i < n_layers; ++i) {
        void* out = (i + 1 == n_layers) ? y : c.act[i & 1];
        wcc_options o = {};
        o.alpha = layers[i].alpha;
        o.relu = layers[i].relu;
        const bool this_fused = fused_fits(in, layers[i].Cout, Wd, bits, dt, layers[i].Cin);
        const bool feed = this_fused && i + 1 < n_layers && chain_fusable(in, layers[i].Cin, layers[i].Cout, H, Wd, bits, dt) &&
                          fused_fits(out, layers[i + 1].Cout, Wd, bits, dt, layers[i + 1].Cin) &&
                          tc::tma_ok_x(out, dt == WCC_BF16 ? 2 : 4, Wd);
        const ChainHooks hooks = {norms_ready, feed ? c.layer_ws[(i + 1) & 1] : nullptr, feed ? layers[i + 1].Cout : 0};
        s = forward_impl(in, layers[i].Wt, N, layers[i].Cin, layers[i].Cout, H, Wd, levels, k, bits, out, dt,
                         c.layer_ws[i & 1], c.layer_ws_bytes, static_cast<cudaStream_t>(stream), nullptr, &o, &hooks);
        if (s != WCC_OK) return s;
        norms_ready = feed;
        in = out;
    }
    return WCC_OK;
}

wcc_status wcc_forward_staged(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                              int levels, int k, int bits, void* y, wcc_dtype dt,
                              void* ws, size_t ws_bytes, void* stream, const wcc_taps* taps)
{
    return staged_impl(x, Wt, N, Cin, Cout, H, Wd, levels, k, bits, y, dt, ws, ws_bytes,
                       static_cast<cudaStream_t>(stream), taps);
}

wcc_status wcc_forward_debug(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                             int levels, int k, int bits, void* y, wcc_dtype dt,
                             void* ws, size_t ws_bytes, void* stream, const wcc_taps* taps)
{
    return forward_impl(x, Wt, N, Cin, Cout, H, Wd, levels, k, bits, y, dt, ws, ws_bytes,
                        static_cast<cudaStream_t>(stream), taps);
}

wcc_status wcc_last_status(void* stream)
{
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return WCC_ERR_CUDA;
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_status, sizeof(int)) != cudaSuccess) return WCC_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_status, &zero, sizeof(int)) != cudaSuccess) return WCC_ERR_CUDA;
    }
    return static_cast<wcc_status>(v);
}

wcc_status wcc_debug_set_wait_limit(unsigned polls)
{
    const uint32_t v = polls ? (uint32_t)polls : tc::WAIT_LIMIT_DEFAULT;
    if (cudaMemcpyToSymbol(tc::c_wait_limit, &v, sizeof(v)) != cudaSuccess) return WCC_ERR_CUDA;
    return WCC_OK;
}

wcc_status wcc_debug_wait_selftest(void* stream)
{
    int* status = nullptr;
    WCC_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_status));
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status);
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

wcc_status wcc_profile_enable(int on)
{
    g_profile = on != 0;
    if (!g_profile) g_ev_valid = false;
    return WCC_OK;
}

wcc_status wcc_profile_read(float* ms)
{
    if (!ms) return WCC_ERR_NULL;
    if (!g_ev_valid) return WCC_ERR_CUDA;
    if (cudaEventSynchronize(g_ev[WCC_NUM_STAGES]) != cudaSuccess) return WCC_ERR_CUDA;
    for (int i = 0; i < WCC_NUM_STAGES; ++i)
        if (cudaEventElapsedTime(&ms[i], g_ev[i], g_ev[i + 1]) != cudaSuccess) return WCC_ERR_CUDA;
    return WCC_OK;
}

unsigned long long wcc_kernel_launches(void) { return g_launches; }

const char* wcc_status_str(wcc_status s)
{
    switch (s) {
        case WCC_OK: return "ok";
        case WCC_ERR_NULL: return "null pointer";
        case WCC_ERR_SHAPE: return "bad shape";
        case WCC_ERR_K: return "k out of range";
        case WCC_ERR_BITS: return "bits not in {0, 2..8}";
        case WCC_ERR_DTYPE: return "unknown dtype";
        case WCC_ERR_ALIGN: return "misaligned pointer";
        case WCC_ERR_WORKSPACE: return "workspace too small";
        case WCC_ERR_CUDA: return "CUDA error";
        case WCC_ERR_TIMEOUT: return "device wait timed out";
        case WCC_ERR_NONFINITE: return "non-finite input";
    }
    return "unknown status";
}

}  // extern "C"

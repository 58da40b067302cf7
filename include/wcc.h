/*
 * wcc.h -- C ABI of libwcc: the forward pass of one Wavelet Compressed Convolution (WCC) layer
 * on an NVIDIA B200 (sm_100a).
 *
 *     WCC(K, x) = H^T T^T K_1x1 T H x                                   (Eq. 9, Alg. 1)
 *
 * H is the multi-level per-channel 2-D Haar transform (Eq. 3-6), T keeps the k wavelet-domain
 * positions of largest feature norm across channels, the same positions for every channel
 * (Eq. 7 and Sec. 4 "Joint hard shrinkage"), K_1x1 is the pointwise convolution applied to the kept
 * columns only, T^T zero-fills and H^T is the inverse transform (Eq. 4).  The kept columns and the
 * weights are quantized with the signed symmetric scheme of Eq. 1-2 (8 bits).
 *
 * Conventions, valid for every entry point unless it says otherwise:
 *  - Every data pointer is a DEVICE pointer owned by the caller, 16-byte aligned.  The library
 *    allocates no device memory; scratch space is passed in (`ws`, sized by wcc_workspace_bytes).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue
 *    work; they never synchronise and never throw.  Errors the host can see (bad shape, null or
 *    misaligned pointer, small workspace) are returned before anything is launched.
 *  - Tensors are dense, row-major: activations [N][C][H][Wd], weights [Cout][Cin].
 *  - Wavelet-domain maps use the quadrant layout inside each H x Wd plane: level l works on the
 *    top-left (H/2^(l-1)) x (Wd/2^(l-1)) corner and leaves y1 (low-pass) top-left, y2 (difference
 *    along the width) top-right, y3 (difference along the height) bottom-left, y4 bottom-right.
 *    A "position" p = row * Wd + col indexes this layout; P = H * Wd.
 *  - levels is 1, 2 or 3 (the paper uses 3); H and Wd must be multiples of 2^levels.
 *  - Cin, Cout <= WCC_MAX_CHANNELS.  wcc_forward runs its fused two-pass kernels while the operands of one tile group
 *    fit one SM's shared memory and tensor memory (up to 256 channels on the quantized path) and otherwise the
 *    stage-by-stage pipeline of wcc_forward_staged, whose contraction tiles K and N; wcc_workspace_bytes accounts for it.
 *  - There is no CPU fallback: the library is built for sm_100a only.
 */
#ifndef WCC_H_
#define WCC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    WCC_OK = 0,
    WCC_ERR_NULL = 1,        /* a required pointer is NULL */
    WCC_ERR_SHAPE = 2,       /* non-positive dims, H or Wd not a multiple of 2^levels, levels/channels out of range */
    WCC_ERR_K = 3,           /* k < 1 or k > H*Wd */
    WCC_ERR_BITS = 4,        /* bits not in {0, 2..8} */
    WCC_ERR_DTYPE = 5,       /* unknown wcc_dtype */
    WCC_ERR_ALIGN = 6,       /* a pointer is not 16-byte aligned */
    WCC_ERR_WORKSPACE = 7,   /* ws_bytes smaller than wcc_workspace_bytes(...) */
    WCC_ERR_CUDA = 8,        /* a CUDA runtime call or launch failed */
    WCC_ERR_TIMEOUT = 9,     /* a bounded device-side wait ran out (reported by wcc_last_status) */
    WCC_ERR_NONFINITE = 10   /* reserved */
} wcc_status;

typedef enum { WCC_F32 = 0, WCC_BF16 = 1 } wcc_dtype;   /* element type of activations x and y */
#define WCC_MAX_CHANNELS 8192

/* Scratch bytes wcc_forward / wcc_forward_debug need for these arguments (0 on invalid arguments). */
size_t wcc_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt);
/* Scratch bytes wcc_forward_staged needs (it materialises the coefficient map, the compressed matrix and the accumulators). */
size_t wcc_staged_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt);

/* Scratch bytes wcc_select_topk needs. */
size_t wcc_select_workspace_bytes(int N, int P);

/*
 * Forward Haar transform, all levels, of every (n, c) plane (Eq. 3, 5, 6), and in the same pass the
 * per-position l2 norm over the channels (Alg. 1, norm step).
 *   x     in : [N][C][H][Wd] of dt
 *   coef  out: fp32 [N][C][H][Wd], quadrant layout.  Arithmetic is fp32: per 2x2 block a,b / c,d:
 *              s0=a+b d0=a-b s1=c+d d1=c-d; y1=(s0+s1)/2 y2=(d0+d1)/2 y3=(s0-s1)/2 y4=(d0-d1)/2.
 *   nrm2  out: fp32 [N][P] squared l2 norm over channels, one fused multiply-add per channel in
 *              ascending channel order; NULL to skip.
 */
wcc_status wcc_haar_fwd(const void* x, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                        float* coef, float* nrm2, void* stream);

/*
 * Inverse Haar transform (Eq. 4: the transposed convolution, coarsest level first).
 *   coef  in : fp32 [N][C][H][Wd], quadrant layout
 *   x_out out: [N][C][H][Wd] of dt (bf16: round to nearest even)
 * Per quadruple: t0=y1+y3 t1=y1-y3 u0=y2+y4 u1=y2-y4; a=(t0+u0)/2 b=(t0-u0)/2 c=(t1+u1)/2 d=(t1-u1)/2.
 */
wcc_status wcc_haar_inv(const float* coef, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                        void* x_out, void* stream);

/*
 * Joint shrinkage T (Eq. 7; Alg. 1, index-set step): for each image the k = ceil(gamma * H * Wd)
 * positions of largest norm.  Ties at the k-th value go to the lowest position.  -0 ranks equal to +0;
 * the order of NaNs is unspecified.
 *   nrm2 in : fp32 [N][P]
 *   idx  out: int32 [N][k], ascending within each image
 *   tau  out: fp32 [N], the k-th largest norm of each image; NULL to skip
 *   ws       : scratch of at least wcc_select_workspace_bytes(N, P) bytes
 */
wcc_status wcc_select_topk(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * The same selection reported as a bitmap instead of an index list (Sec. 4 lets the shared index set be kept as "a
 * single index list or a bit-map"; one bit per position serves all channels): bit (p % 32) of word p / 32 of image n
 * is set when position p is kept.
 *   bitmap out: uint32 [N][ceil(P / 32)]; bits beyond P are zero
 *   ws        : scratch of at least wcc_select_bitmap_workspace_bytes(N, P, k) bytes, 256-byte aligned
 */
size_t wcc_select_bitmap_workspace_bytes(int N, int P, int k);
wcc_status wcc_select_topk_bitmap(const float* nrm2, int N, int P, int k, uint32_t* bitmap, float* tau,
                                  void* ws, size_t ws_bytes, void* stream);

/*
 * wcc_select_topk without a scratch argument (the paper has no counterpart: this is a packaging variant).
 * For callers that have no way to obtain scratch memory: code that runs where cudaMalloc must not be called
 * (a latency-critical loop in which the allocator's implicit device synchronisation is unacceptable, or a host
 * that has handed all device memory to a pool the caller cannot reach) and that receives only its input and
 * output pointers.  The scratch is a fixed array inside the library's device image, WCC_STATIC_SCRATCH_BYTES
 * large; every GPU that loads the library holds that much memory until the process exits.
 *  - Same arguments, results and error codes as wcc_select_topk; additionally returns WCC_ERR_WORKSPACE when
 *    wcc_select_workspace_bytes(N, P) exceeds WCC_STATIC_SCRATCH_BYTES (about 24 KB per image: N = 32 images do not fit).
 *  - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *  - The first call on each device looks up the array's device address (with that device current); make that
 *    first call before starting any stream capture.
 *  - All calls on a device share the one array, and it keeps the previous call's contents; the entry point
 *    clears the parts that must start at zero.  Two calls whose kernels overlap on the GPU (different streams
 *    without ordering) race on it: order them.
 */
#define WCC_STATIC_SCRATCH_BYTES (512 * 1024)
wcc_status wcc_select_topk_static(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau, void* stream);

/*
 * The whole layer (Eq. 9 in the order of Alg. 1).
 *   x   in : [N][Cin][H][Wd] of dt          Wt in: fp32 [Cout][Cin] (no bias)
 *   k      : kept positions per image (ceil(gamma * H * Wd))
 *   bits   : 8 (or 2..7, a smaller grid on the same int8 path): kept columns quantized with one scale
 *            for the whole call, scale_a = max|kept| / qmax, qmax = 2^(bits-1)-1, code =
 *            clamp(rint(v * (qmax / max|kept|))); weights with one scale per output channel; int8 x int8
 *            -> int32 contraction on tensor cores; y_wt = acc * (scale_a * scale_w[o]).
 *            0: no quantization; columns and weights rounded to bf16, fp32 accumulation.
 *   y   out: [N][Cout][H][Wd] of dt; must not overlap x
 *   ws     : scratch of at least wcc_workspace_bytes(...) bytes, 256-byte aligned; contents undefined afterwards
 * Execution: three launches, two passes over x around the selection.  Pass 1 transforms x in registers and keeps
 * only the channel norms, the per-position max |coefficient| and two histograms of the norms' leading bits below the sign (it
 * also quantizes the weights); the selection finds the threshold norm, max|kept| and, only if ties at the threshold
 * are kept in part, the rank of every position; pass 2 transforms x again, zeroes the dropped positions, quantizes
 * into shared memory, runs the contraction on tensor cores, dequantizes, applies the inverse transform and stores y.
 * The results are those of the step-by-step definition above (same integers, same fp32 operation order).
 */
wcc_status wcc_forward(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                       int levels, int k, int bits, void* y, wcc_dtype dt,
                       void* ws, size_t ws_bytes, void* stream);

/*
 * Intermediate results of wcc_forward for tests; any member may be NULL.  Row r = n * k + j is the
 * j-th kept position of image n.  Rows of Xq / Xb are padded to kpad = wcc_kpad(Cin, bits) elements,
 * the padding is zero.
 */
typedef struct wcc_taps {
    float*   coef;      /* fp32 [N][Cin][P] */
    float*   nrm2;      /* fp32 [N][P] */
    int32_t* idx;       /* int32 [N][k] */
    int8_t*  Xq;        /* int8 [N*k][kpad]           (bits >= 2) */
    void*    Xb;        /* bf16 [N*k][kpad]           (bits == 0) */
    float*   scale_a;   /* fp32 [1]                   (bits >= 2) */
    int8_t*  Wq;        /* int8 [Cout][kpad]          (bits >= 2) */
    float*   scale_w;   /* fp32 [Cout]                (bits >= 2) */
    int32_t* acc;       /* int32 [N*k][Cout] (bits >= 2) or fp32 bit patterns of the products (bits == 0) */
} wcc_taps;

int wcc_kpad(int Cin, int bits);

/*
 * wcc_forward with the requested intermediates written out by the same kernels (the transform kernel also stores
 * the coefficient map, the fused kernel also stores the codes and accumulators of the kept rows).
 * Tap pointers must be 16-byte aligned.
 */
wcc_status wcc_forward_debug(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                             int levels, int k, int bits, void* y, wcc_dtype dt,
                             void* ws, size_t ws_bytes, void* stream, const wcc_taps* taps);

/*
 * The layer on maps whose sides are no multiples of 2^levels (the paper's segmentation networks have 513 x 1025 maps,
 * App. C; it does not say how they are transformed).  Reading taken here: the map is zero-padded at the bottom and on
 * the right to the next multiples Hp, Wp of 2^levels, the layer runs on the padded map, and the output is cropped
 * back to H x Wd.  k counts kept positions of the PADDED map (1 <= k <= Hp * Wp).  With everything kept and no
 * quantization the result is still the dense 1x1 convolution of x: zero padding commutes with a pointwise convolution
 * that has no bias.  ws: at least wcc_padded_workspace_bytes(...) bytes (padded input and output plus the layer's own
 * workspace).  Sizes that need no padding run wcc_forward directly.
 */
size_t wcc_padded_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt);
wcc_status wcc_forward_padded(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                              int levels, int k, int bits, void* y, wcc_dtype dt,
                              void* ws, size_t ws_bytes, void* stream);

/*
 * Options of the layer beyond Alg. 1, as a network built from WCC layers uses them.  A zeroed structure (or NULL)
 * means wcc_forward.
 *   alpha        > 0: the clipping parameter of the activation quantizer (Eq. 2; per layer, Sec. 4 -- in the paper it is
 *                learned, here it is an argument): codes = clamp(rint(v * (qmax / alpha)), -qmax, qmax), scale_a =
 *                alpha / qmax, so kept coefficients beyond +-alpha saturate.  <= 0: the largest kept magnitude of this
 *                call, as in wcc_forward.  Ignored when bits == 0.
 *   weight_bits  0: as `bits`; 2..8: bits of the weight codes (Tables 1-2 run 4-bit weights with 8-bit activations).
 *   relu         non-zero: y = max(., 0), applied last before rounding to dt (the non-linearity between chained layers).
 *   residual     NULL, or a DEVICE map [N][Cout][H][Wd] of dt added to the layer's output before the ReLU: the skip
 *                connection of the inverted residual block (Eq. 13); one fp32 addition per element.  May be y itself.
 *   Wq, scale_w  NULL, or the weights already quantized (DEVICE): int8 [Cout][wcc_kpad(Cin, bits)], rows zero padded,
 *                and fp32 [Cout] scales (what taps Wq / scale_w return).  Static weights need quantizing only once;
 *                Wt is then not read and may be NULL.  Only with bits >= 2.
 */
typedef struct wcc_options {
    float alpha;
    int weight_bits;
    int relu;
    const void* residual;
    const int8_t* Wq;
    const float* scale_w;
} wcc_options;

/* wcc_forward with options (opt may be NULL) and optional taps (may be NULL).  Same workspace as wcc_forward. */
wcc_status wcc_forward_ex(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                          int levels, int k, int bits, void* y, wcc_dtype dt,
                          void* ws, size_t ws_bytes, void* stream, const wcc_options* opt, const wcc_taps* taps);

/*
 * Other wavelets than Haar (App. F compares db2, db3, coif1, bior1.3, bior2.2, sym4 under the same layer): a generic
 * two-channel filter bank.  Filters are HOST arrays of `taps` floats (taps even, 2..8; shorter filters are zero padded
 * by the caller), in this indexing: one 2-D level on the low-pass corner (hc x wc) is the stride-2 cross-correlation
 *     band[i][j] = sum_{tr, tc} f_row[tr] * f_col[tc] * x[(2i + tr - c0) mod hc][(2j + tc - c0) mod wc],  c0 = taps/2 - 1
 * with periodic extension (the transformed map keeps the size of the input; the paper does not name the extension),
 * bands placed like Haar's: (lo, lo) top-left, (lo along the height, hi along the width) top-right, (hi, lo)
 * bottom-left, (hi, hi) bottom-right.  The inverse is the adjoint structure with the reconstruction filters (equal to
 * the decomposition filters for an orthogonal wavelet).  fp32, one fused multiply-add per tap in row-major tap order.
 * [1, 1]/sqrt 2 and [1, -1]/sqrt 2 give Eq. 3 up to rounding.  Plain kernels: this is the ablation, not the hot path.
 *   wcc_dwt_fwd        x [N][C][H][Wd] of dt -> coef fp32 (quadrant layout), nrm2 fp32 [N][P] or NULL;
 *                      ws: at least N*C*H*Wd*4 bytes
 *   wcc_dwt_inv        coef -> x_out of dt; ws: at least 2 * align256(N*C*H*Wd*4) bytes
 *   wcc_forward_wavelet  the layer of Alg. 1 stage by stage with these transforms (selection, quantization and the
 *                      tensor-core contraction as in wcc_forward_staged); taps may be NULL (coef, nrm2, idx, Xq, acc are
 *                      served); ws: at least wcc_wavelet_workspace_bytes(...) bytes, 256-byte aligned
 */
wcc_status wcc_dwt_fwd(const void* x, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                       const float* dec_lo, const float* dec_hi, int taps, float* coef, float* nrm2,
                       void* ws, size_t ws_bytes, void* stream);
wcc_status wcc_dwt_inv(const float* coef, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                       const float* rec_lo, const float* rec_hi, int taps, void* x_out,
                       void* ws, size_t ws_bytes, void* stream);
size_t wcc_wavelet_workspace_bytes(int N, int Cin, int Cout, int H, int Wd, int levels, int k, int bits, wcc_dtype dt);
wcc_status wcc_forward_wavelet(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                               int levels, int k, int bits, const float* dec_lo, const float* dec_hi,
                               const float* rec_lo, const float* rec_hi, int taps, void* y, wcc_dtype dt,
                               void* ws, size_t ws_bytes, void* stream, const wcc_taps* tp_out);

/*
 * Depthwise 3x3 convolution fused with the forward transform (App. H, "a kernel for a fused depthwise convolution and
 * Haar transform": both are separable per channel, so the convolution's output never goes to memory).
 *   u    in : [N][C][H][Wd] of dt           Wdw in: fp32 [C][3][3], stride 1, zero padding 1, no bias, cross-correlation
 *   coef out: fp32 [N][C][H][Wd] = forward transform of dw3x3(u), quadrant layout; nrm2 out: fp32 [N][P] or NULL
 * Per pixel one fused multiply-add per tap in row-major tap order from +0; then exactly wcc_haar_fwd's arithmetic.
 */
wcc_status wcc_dwconv_haar_fwd(const void* u, const float* Wdw, int N, int C, int H, int Wd, int levels, wcc_dtype dt,
                               float* coef, float* nrm2, void* stream);

/*
 * The inverted residual block of Eq. 13 with both pointwise convolutions as WCC layers and no non-linearities:
 *     y = x + WCC(W3, dw3x3(Wdw, WCC(W1, x)))
 *   x, y: [N][C][H][Wd] of dt      W1: fp32 [E][C]      Wdw: fp32 [E][3][3]      W3: fp32 [C][E]      (E: expanded channels)
 * The expanded map u = WCC(W1, x) is stored in dt in the workspace; the depthwise convolution feeds the second layer's
 * transform in fp32 without going to memory; the skip connection is added after the second layer's inverse transform.
 * Same levels, k and bits for both layers.  ws: at least wcc_block_workspace_bytes(...) bytes.
 */
size_t wcc_block_workspace_bytes(int N, int C, int E, int H, int Wd, int levels, int k, int bits, wcc_dtype dt);
wcc_status wcc_block_forward(const void* x, const float* W1, const float* Wdw, const float* W3, int N, int C, int E,
                             int H, int Wd, int levels, int k, int bits, void* y, wcc_dtype dt,
                             void* ws, size_t ws_bytes, void* stream);

/*
 * A chain of pointwise WCC layers on one feature map (e.g. the 32 -> 192 -> 32 ... stacks of an inverted-residual
 * network): layer i maps the output of layer i-1 with Wt [Cout][Cin]; Cin of a layer must equal Cout of the one before.
 * `layers` is a HOST array (read during the call only); Wt are DEVICE pointers.  relu / alpha as in wcc_options.
 * Same levels, k and bits for every layer.  Intermediate maps live in the workspace (two buffers of the largest one).
 * All arguments of all layers are checked before the first launch.
 */
typedef struct wcc_chain_layer {
    const float* Wt;
    int Cin, Cout;
    float alpha;
    int relu;
} wcc_chain_layer;
size_t wcc_chain_workspace_bytes(const wcc_chain_layer* layers, int n_layers, int N, int H, int Wd, int levels, int k,
                                 int bits, wcc_dtype dt);
wcc_status wcc_chain_forward(const void* x, const wcc_chain_layer* layers, int n_layers, int N, int H, int Wd,
                             int levels, int k, int bits, void* y, wcc_dtype dt, void* ws, size_t ws_bytes, void* stream);

/*
 * The same layer as wcc_forward computed stage by stage with every intermediate in memory (Alg. 1 literally):
 * transform + norms -> select -> gather + quantize -> tensor-core contraction on the compressed matrix ->
 * dequantize + scatter + inverse.  Same results as wcc_forward; used to measure the stages one by one and as a
 * cross-check.  ws: at least wcc_staged_workspace_bytes(...) bytes.  taps may be NULL.
 */
wcc_status wcc_forward_staged(const void* x, const float* Wt, int N, int Cin, int Cout, int H, int Wd,
                              int levels, int k, int bits, void* y, wcc_dtype dt,
                              void* ws, size_t ws_bytes, void* stream, const wcc_taps* taps);

/*
 * Synchronises `stream` and returns the device-side status word of the calling thread's current device:
 * WCC_OK, or WCC_ERR_TIMEOUT if a bounded wait inside a kernel gave up (the output of that call is then
 * undefined).  Reading clears the word.
 */
wcc_status wcc_last_status(void* stream);

const char* wcc_status_str(wcc_status s);

/*
 * Test hooks for the device-side timeout contract (no counterpart in the paper).  Every wait inside a kernel (on an
 * mbarrier of a TMA ring, of the tensor-core pipeline, on the arrival counter of the cooperative select) polls a
 * bounded number of times, then the kernel records WCC_ERR_TIMEOUT, lets its copies in flight land, frees its TMEM
 * and returns; nothing traps or faults.
 *   wcc_debug_set_wait_limit  sets the number of polls (each suspends for up to about a microsecond) on the current
 *                             device; 0 restores the default (2,000,000).  Synchronous.
 *   wcc_debug_wait_selftest   enqueues one warp that waits on a barrier nobody arrives on; with a small limit it
 *                             returns within a millisecond and wcc_last_status then reports WCC_ERR_TIMEOUT.
 */
wcc_status wcc_debug_set_wait_limit(unsigned polls);
wcc_status wcc_debug_wait_selftest(void* stream);

/*
 * Measurement helpers (no counterpart in the paper).  With profiling on, wcc_forward records CUDA events on its
 * stream around each stage; wcc_profile_read waits for the last recorded call and writes, to the HOST array ms, the
 * milliseconds of, for wcc_forward_staged: 0 Haar transform + norms, 1 top-k select + compaction, 2 weight
 * quantization, 3 gather + quantize, 4 tensor-core contraction, 5 dequantize + scatter + inverse Haar; for wcc_forward:
 * 0 clearing of the select's histograms (a memset node), 1 pass 1 (transform + norms, select histograms, weight
 * quantization), 2 select, 3 fused pass 2, 4 and 5 zero.
 * Off by default; not thread-safe.
 */
#define WCC_NUM_STAGES 6
wcc_status wcc_profile_enable(int on);
wcc_status wcc_profile_read(float* ms);
/* Number of kernels this library has launched in this process so far (memset nodes not counted). */
unsigned long long wcc_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* WCC_H_ */

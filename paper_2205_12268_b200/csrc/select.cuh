// Joint shrinkage: per image, the k positions of largest norm (Alg. 1; Eq. 7 with the joint rule).
//
// Radix select on the order-preserving 32-bit key of the fp32 norm, most significant digit first, in three
// rounds of 11 + 11 + 10 bits.  Each round is one kernel: every CTA histograms the digit of the keys of its
// chunk that match the prefix found so far (shared-memory histogram, then one global atomic per non-empty
// bin); the next kernel finds, redundantly in every CTA, the bin that holds the k-th largest key.  After
// the third round the threshold key tau and the number of keys equal to tau that must be kept are known.
// Two more kernels do an ordered stream compaction (chunk counts, then a block scan) so that idx comes out
// ascending and ties go to the lowest position.  Results are deterministic: no output depends on the order
// in which atomics land.
#pragma once

#include "common.cuh"

namespace wcc {

constexpr int SEL_THREADS = 256;
constexpr int SEL_KPT = 8;                           // keys per thread
constexpr int SEL_CHUNK = SEL_THREADS * SEL_KPT;     // keys per CTA
constexpr int SEL_BINS = 2048;

// per-image state words
enum { ST_B1 = 0, ST_K1 = 1, ST_B2 = 2, ST_K2 = 3, ST_TAU = 4, ST_NEED_EQ = 5, ST_WORDS = 8 };

struct SelectWs {
    uint32_t* hist;     // [N][3][SEL_BINS]
    float* amax;        // [1] largest |coef| over the kept positions (float bits, merged by integer atomicMax)
    uint32_t* bar;      // [N] arrival counters of the per-image barriers of the single-kernel select
    uint32_t* state;    // [N][ST_WORDS]
    uint32_t* chunkcnt; // [N][chunks][2]
    size_t zero_bytes;  // hist + amax + bar are contiguous and cleared by one memset
    int chunks;
};

inline size_t select_ws_bytes(int N, int P)
{
    const size_t chunks = (size_t)ceil_div(P, SEL_CHUNK);
    return align_up((size_t)N * 3 * SEL_BINS * 4, 256) + align_up(64 + (size_t)N * 4, 256) +
           align_up((size_t)N * ST_WORDS * 4, 256) + align_up((size_t)N * chunks * 2 * 4, 256);
}

inline SelectWs carve_select_ws(void* ws, int N, int P)
{
    SelectWs s;
    char* p = static_cast<char*>(ws);
    s.chunks = ceil_div(P, SEL_CHUNK);
    s.hist = reinterpret_cast<uint32_t*>(p);
    p += align_up((size_t)N * 3 * SEL_BINS * 4, 256);
    s.amax = reinterpret_cast<float*>(p);
    s.bar = reinterpret_cast<uint32_t*>(p + 64);
    p += align_up(64 + (size_t)N * 4, 256);
    s.zero_bytes = (size_t)(p - static_cast<char*>(ws));
    s.state = reinterpret_cast<uint32_t*>(p);
    p += align_up((size_t)N * ST_WORDS * 4, 256);
    s.chunkcnt = reinterpret_cast<uint32_t*>(p);
    return s;
}

// Block-wide exclusive scan of one value per thread (256 threads); returns the exclusive prefix, total in *total.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* warp_sums, uint32_t* total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) warp_sums[w] = inc;
    __syncthreads();
    if (w == 0) {
        uint32_t s = (lane < SEL_THREADS / 32) ? warp_sums[lane] : 0u;
        uint32_t si = s;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, si, d);
            if (lane >= d) si += t;
        }
        if (lane < SEL_THREADS / 32) warp_sums[lane] = si - s;     // exclusive warp offsets
        if (lane == SEL_THREADS / 32 - 1) warp_sums[SEL_THREADS / 32] = si;
    }
    __syncthreads();
    const uint32_t res = warp_sums[w] + inc - v;
    *total = warp_sums[SEL_THREADS / 32];
    __syncthreads();
    return res;
}

// Among nbins counts h[] (nbins = 8 * 256 or 4 * 256), find the bin b holding the krem-th key counted from
// the top bin downwards; *above = number of keys in bins > b.  Every thread returns the same values.
template <int NBINS>
__device__ __forceinline__ void find_bin(const uint32_t* __restrict__ h, uint32_t krem, uint32_t* sh_scan,
                                         uint32_t* sh_res, uint32_t& bin, uint32_t& above)
{
    constexpr int PER = NBINS / SEL_THREADS;
    const int top = NBINS - 1 - (int)threadIdx.x * PER;      // this thread covers bins top, top-1, ..., top-PER+1
    uint32_t c[PER], sum = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) { c[i] = __ldcg(&h[top - i]); sum += c[i]; }
    uint32_t total;
    uint32_t before = block_exclusive_scan(sum, sh_scan, &total);
    if (before < krem && krem <= before + sum) {
        uint32_t a = before;
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            if (a < krem && krem <= a + c[i]) { sh_res[0] = (uint32_t)(top - i); sh_res[1] = a; }
            a += c[i];
        }
    }
    __syncthreads();
    bin = sh_res[0];
    above = sh_res[1];
    __syncthreads();
}

__device__ __forceinline__ void load_keys(const float* __restrict__ v, int P, int base, uint32_t (&key)[SEL_KPT], bool (&ok)[SEL_KPT])
{
    if (base + SEL_KPT <= P && (P % 4) == 0) {
        const float4 a = *reinterpret_cast<const float4*>(v + base);
        const float4 b = *reinterpret_cast<const float4*>(v + base + 4);
        key[0] = float_key(a.x); key[1] = float_key(a.y); key[2] = float_key(a.z); key[3] = float_key(a.w);
        key[4] = float_key(b.x); key[5] = float_key(b.y); key[6] = float_key(b.z); key[7] = float_key(b.w);
#pragma unroll
        for (int i = 0; i < SEL_KPT; ++i) ok[i] = true;
    } else {
#pragma unroll
        for (int i = 0; i < SEL_KPT; ++i) {
            ok[i] = base + i < P;
            key[i] = ok[i] ? float_key(v[base + i]) : 0u;
        }
    }
}

// Round R in {1, 2, 3}: resolve the digit of round R-1 (if any), then histogram digit R of matching keys.
template <int R>
__global__ void __launch_bounds__(SEL_THREADS)
select_hist_kernel(const float* __restrict__ nrm2, int P, int k, uint32_t* __restrict__ hist, uint32_t* __restrict__ state)
{
    __shared__ uint32_t sh[SEL_BINS];
    __shared__ uint32_t sh_scan[SEL_THREADS / 32 + 1];
    __shared__ uint32_t sh_res[2];
    const int n = blockIdx.y;
    uint32_t* hn = hist + (size_t)n * 3 * SEL_BINS;
    uint32_t* stn = state + (size_t)n * ST_WORDS;

    uint32_t prefix = 0;        // digits found so far, right-aligned
    if (R == 2) {
        uint32_t b1, above;
        find_bin<SEL_BINS>(hn, (uint32_t)k, sh_scan, sh_res, b1, above);
        prefix = b1;
        if (blockIdx.x == 0 && threadIdx.x == 0) { stn[ST_B1] = b1; stn[ST_K1] = (uint32_t)k - above; }
    } else if (R == 3) {
        const uint32_t b1 = stn[ST_B1], k1 = stn[ST_K1];
        uint32_t b2, above;
        find_bin<SEL_BINS>(hn + SEL_BINS, k1, sh_scan, sh_res, b2, above);
        prefix = (b1 << 11) | b2;
        if (blockIdx.x == 0 && threadIdx.x == 0) { stn[ST_B2] = b2; stn[ST_K2] = k1 - above; }
    }
    for (int i = threadIdx.x; i < SEL_BINS; i += SEL_THREADS) sh[i] = 0u;
    __syncthreads();

    uint32_t key[SEL_KPT];
    bool ok[SEL_KPT];
    load_keys(nrm2 + (size_t)n * P, P, blockIdx.x * SEL_CHUNK + threadIdx.x * SEL_KPT, key, ok);
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
        if (!ok[i]) continue;
        if (R == 1) atomicAdd(&sh[key[i] >> 21], 1u);
        if (R == 2 && (key[i] >> 21) == prefix) atomicAdd(&sh[(key[i] >> 10) & 0x7FFu], 1u);
        if (R == 3 && (key[i] >> 10) == prefix) atomicAdd(&sh[key[i] & 0x3FFu], 1u);
    }
    __syncthreads();
    uint32_t* out = hn + (R - 1) * SEL_BINS;
    for (int i = threadIdx.x; i < SEL_BINS; i += SEL_THREADS) {
        const uint32_t c = sh[i];
        if (c) atomicAdd(&out[i], c);
    }
}

// Resolve the last digit; count, per chunk, the keys above and equal to the threshold.
__global__ void __launch_bounds__(SEL_THREADS)
select_count_kernel(const float* __restrict__ nrm2, int P, uint32_t* __restrict__ hist, uint32_t* __restrict__ state,
                    uint32_t* __restrict__ chunkcnt, float* __restrict__ tau)
{
    __shared__ uint32_t sh_scan[SEL_THREADS / 32 + 1];
    __shared__ uint32_t sh_res[2];
    __shared__ uint32_t sh_cnt[2];
    const int n = blockIdx.y;
    uint32_t* hn = hist + (size_t)n * 3 * SEL_BINS;
    uint32_t* stn = state + (size_t)n * ST_WORDS;
    const uint32_t prefix = (stn[ST_B1] << 11) | stn[ST_B2], k2 = stn[ST_K2];
    uint32_t b3, above;
    find_bin<1024>(hn + 2 * SEL_BINS, k2, sh_scan, sh_res, b3, above);
    const uint32_t tkey = (prefix << 10) | b3;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        stn[ST_TAU] = tkey;
        stn[ST_NEED_EQ] = k2 - above;        // how many keys equal to tau are kept (lowest positions first)
        if (tau) tau[n] = key_float(tkey);
    }
    if (threadIdx.x < 2) sh_cnt[threadIdx.x] = 0u;
    __syncthreads();
    uint32_t key[SEL_KPT];
    bool ok[SEL_KPT];
    load_keys(nrm2 + (size_t)n * P, P, blockIdx.x * SEL_CHUNK + threadIdx.x * SEL_KPT, key, ok);
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
        if (!ok[i]) continue;
        gt += key[i] > tkey;
        eq += key[i] == tkey;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        gt += __shfl_xor_sync(0xFFFFFFFFu, gt, d);
        eq += __shfl_xor_sync(0xFFFFFFFFu, eq, d);
    }
    if ((threadIdx.x & 31) == 0) { atomicAdd(&sh_cnt[0], gt); atomicAdd(&sh_cnt[1], eq); }
    __syncthreads();
    if (threadIdx.x < 2) chunkcnt[((size_t)n * gridDim.x + blockIdx.x) * 2 + threadIdx.x] = sh_cnt[threadIdx.x];
}

// Ordered compaction: idx (ascending), rank map, and the largest |coef| over the kept positions.
__global__ void __launch_bounds__(SEL_THREADS)
select_compact_kernel(const float* __restrict__ nrm2, int P, int k, const uint32_t* __restrict__ state,
                      const uint32_t* __restrict__ chunkcnt, int32_t* __restrict__ idx, int32_t* __restrict__ rank,
                      const float* __restrict__ amaxpos, float* __restrict__ amax_kept)
{
    __shared__ uint32_t sh_scan[SEL_THREADS / 32 + 1];
    __shared__ uint32_t sh_base[2];
    __shared__ uint32_t sh_amax;
    const int n = blockIdx.y;
    const uint32_t* stn = state + (size_t)n * ST_WORDS;
    const uint32_t tkey = stn[ST_TAU], need_eq = stn[ST_NEED_EQ];

    // keys above / equal to tau in the chunks before this one
    if (threadIdx.x < 2) sh_base[threadIdx.x] = 0u;
    if (threadIdx.x == 0) sh_amax = 0u;
    __syncthreads();
    {
        uint32_t g = 0, e = 0;
        const uint32_t* cc = chunkcnt + (size_t)n * gridDim.x * 2;
        for (int c = threadIdx.x; c < (int)blockIdx.x; c += SEL_THREADS) { g += cc[2 * c]; e += cc[2 * c + 1]; }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            g += __shfl_xor_sync(0xFFFFFFFFu, g, d);
            e += __shfl_xor_sync(0xFFFFFFFFu, e, d);
        }
        if ((threadIdx.x & 31) == 0 && (g | e)) { atomicAdd(&sh_base[0], g); atomicAdd(&sh_base[1], e); }
    }
    __syncthreads();
    const uint32_t base_gt = sh_base[0], base_eq = sh_base[1];

    uint32_t key[SEL_KPT];
    bool ok[SEL_KPT];
    const int base = blockIdx.x * SEL_CHUNK + threadIdx.x * SEL_KPT;
    load_keys(nrm2 + (size_t)n * P, P, base, key, ok);
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
        if (!ok[i]) continue;
        gt += key[i] > tkey;
        eq += key[i] == tkey;
    }
    uint32_t tot;
    uint32_t gt_before = base_gt + block_exclusive_scan(gt, sh_scan, &tot);
    uint32_t eq_before = base_eq + block_exclusive_scan(eq, sh_scan, &tot);

    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
        if (!ok[i]) continue;
        const bool is_gt = key[i] > tkey, is_eq = key[i] == tkey;
        const bool keep = is_gt || (is_eq && eq_before < need_eq);
        const uint32_t pos = gt_before + min(eq_before, need_eq);
        if (keep) {
            idx[(size_t)n * k + pos] = base + i;
            if (amaxpos) amax = fmaxf(amax, amaxpos[(size_t)n * P + base + i]);
        }
        if (rank) rank[(size_t)n * P + base + i] = keep ? (int32_t)pos : -1;
        gt_before += is_gt;
        eq_before += is_eq;
    }
    if (amax_kept) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if ((threadIdx.x & 31) == 0) atomicMax(&sh_amax, __float_as_uint(amax));
        __syncthreads();
        if (threadIdx.x == 0 && sh_amax) atomicMax(reinterpret_cast<uint32_t*>(amax_kept), sh_amax);
    }
}


// ---- the same select as ONE cooperative kernel -------------------------------------------------------
// All phases in one launch; the CTAs of an image meet at per-image barriers (an arrival counter in global memory,
// a bounded spin).  The launch is cooperative, so every CTA is resident and the barriers can complete.  The keys
// stay in registers across the phases.
constexpr uint32_t SEL_SPIN_LIMIT = 4000000u;

__device__ __forceinline__ bool image_barrier(uint32_t* counter, uint32_t target)
{
    __shared__ int sh_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        int ok = 0;
        for (uint32_t it = 0; it < SEL_SPIN_LIMIT; ++it) {
            if (*reinterpret_cast<volatile uint32_t*>(counter) >= target) { ok = 1; break; }
            __nanosleep(40);
        }
        __threadfence();
        sh_ok = ok;
    }
    __syncthreads();
    return sh_ok != 0;
}

template <int NBINS>
__device__ __forceinline__ void flush_hist(uint32_t* sh, uint32_t* __restrict__ out)
{
    __syncthreads();
    for (int i = threadIdx.x; i < NBINS; i += SEL_THREADS) {
        const uint32_t c = sh[i];
        if (c) atomicAdd(&out[i], c);
        sh[i] = 0u;
    }
}

__global__ void __launch_bounds__(SEL_THREADS)
select_coop_kernel(const float* __restrict__ nrm2, int P, int k, uint32_t* __restrict__ hist, uint32_t* __restrict__ bar,
                   uint32_t* __restrict__ chunkcnt, int32_t* __restrict__ idx, float* __restrict__ tau,
                   int32_t* __restrict__ rank, const float* __restrict__ amaxpos, float* __restrict__ amax_kept,
                   int* __restrict__ status)
{
    __shared__ uint32_t sh[SEL_BINS];
    __shared__ uint32_t sh_scan[SEL_THREADS / 32 + 1];
    __shared__ uint32_t sh_res[2];
    __shared__ uint32_t sh_base[2];
    __shared__ uint32_t sh_amax;
    const int n = blockIdx.y;
    const uint32_t chunks = gridDim.x;
    uint32_t* hn = hist + (size_t)n * 3 * SEL_BINS;
    uint32_t* barn = bar + n;

    uint32_t key[SEL_KPT];
    bool okk[SEL_KPT];
    const int base = blockIdx.x * SEL_CHUNK + threadIdx.x * SEL_KPT;
    load_keys(nrm2 + (size_t)n * P, P, base, key, okk);
    for (int i = threadIdx.x; i < SEL_BINS; i += SEL_THREADS) sh[i] = 0u;
    if (threadIdx.x < 2) sh_base[threadIdx.x] = 0u;
    if (threadIdx.x == 0) sh_amax = 0u;
    __syncthreads();

    // round 1
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i)
        if (okk[i]) atomicAdd(&sh[key[i] >> 21], 1u);
    flush_hist<SEL_BINS>(sh, hn);
    bool good = image_barrier(barn, chunks);
    // round 2
    uint32_t b1, above;
    find_bin<SEL_BINS>(hn, (uint32_t)k, sh_scan, sh_res, b1, above);
    const uint32_t k1 = (uint32_t)k - above;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i)
        if (okk[i] && (key[i] >> 21) == b1) atomicAdd(&sh[(key[i] >> 10) & 0x7FFu], 1u);
    flush_hist<SEL_BINS>(sh, hn + SEL_BINS);
    good = image_barrier(barn, 2 * chunks) && good;
    // round 3
    uint32_t b2;
    find_bin<SEL_BINS>(hn + SEL_BINS, k1, sh_scan, sh_res, b2, above);
    const uint32_t k2 = k1 - above;
    const uint32_t prefix = (b1 << 11) | b2;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i)
        if (okk[i] && (key[i] >> 10) == prefix) atomicAdd(&sh[key[i] & 0x3FFu], 1u);
    flush_hist<1024>(sh, hn + 2 * SEL_BINS);
    good = image_barrier(barn, 3 * chunks) && good;
    // threshold, chunk counts
    uint32_t b3;
    find_bin<1024>(hn + 2 * SEL_BINS, k2, sh_scan, sh_res, b3, above);
    const uint32_t tkey = (prefix << 10) | b3, need_eq = k2 - above;
    if (tau && blockIdx.x == 0 && threadIdx.x == 0) tau[n] = key_float(tkey);
    uint32_t gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
        if (!okk[i]) continue;
        gt += key[i] > tkey;
        eq += key[i] == tkey;
    }
    uint32_t tot_gt, tot_eq;
    const uint32_t gt_local = block_exclusive_scan(gt, sh_scan, &tot_gt);
    const uint32_t eq_local = block_exclusive_scan(eq, sh_scan, &tot_eq);
    uint32_t* cc = chunkcnt + (size_t)n * chunks * 2;
    if (threadIdx.x == 0) { cc[2 * blockIdx.x] = tot_gt; cc[2 * blockIdx.x + 1] = tot_eq; }
    good = image_barrier(barn, 4 * chunks) && good;
    // ordered compaction
    {
        uint32_t g = 0, e = 0;
        for (int c = threadIdx.x; c < (int)blockIdx.x; c += SEL_THREADS) {
            g += __ldcg(&cc[2 * c]);
            e += __ldcg(&cc[2 * c + 1]);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            g += __shfl_xor_sync(0xFFFFFFFFu, g, d);
            e += __shfl_xor_sync(0xFFFFFFFFu, e, d);
        }
        if ((threadIdx.x & 31) == 0 && (g | e)) { atomicAdd(&sh_base[0], g); atomicAdd(&sh_base[1], e); }
    }
    __syncthreads();
    uint32_t gt_before = sh_base[0] + gt_local, eq_before = sh_base[1] + eq_local;
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) {
        if (!okk[i]) continue;
        const bool is_gt = key[i] > tkey, is_eq = key[i] == tkey;
        const bool keep = is_gt || (is_eq && eq_before < need_eq);
        const uint32_t pos = gt_before + min(eq_before, need_eq);
        if (keep) {
            idx[(size_t)n * k + pos] = base + i;
            if (amaxpos) amax = fmaxf(amax, amaxpos[(size_t)n * P + base + i]);
        }
        if (rank) rank[(size_t)n * P + base + i] = keep ? (int32_t)pos : -1;
        gt_before += is_gt;
        eq_before += is_eq;
    }
    if (amax_kept) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if ((threadIdx.x & 31) == 0) atomicMax(&sh_amax, __float_as_uint(amax));
        __syncthreads();
        if (threadIdx.x == 0 && sh_amax) atomicMax(reinterpret_cast<uint32_t*>(amax_kept), sh_amax);
    }
    if (!good && threadIdx.x == 0) atomicExch(status, (int)WCC_ERR_TIMEOUT);
}

wcc_status launch_select(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau,
                         int32_t* rank, const float* amaxpos, bool want_amax,
                         void* ws, size_t ws_bytes, cudaStream_t st)
{
    if (ws_bytes < select_ws_bytes(N, P)) return WCC_ERR_WORKSPACE;
    const SelectWs s = carve_select_ws(ws, N, P);
    float* amax_kept = want_amax ? s.amax : nullptr;
    WCC_CUDA_TRY(cudaMemsetAsync(s.hist, 0, s.zero_bytes, st));
    const dim3 grid(s.chunks, N);

    // one cooperative kernel when every CTA can be resident at once, else one kernel per phase
    static int coop_cap[64] = {0};          // per device: 0 unknown, -1 unsupported, else max resident CTAs
    int dev = 0;
    WCC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && coop_cap[dev] == 0) {
        int coop = 0, sms = 0, per_sm = 0;
        WCC_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
        WCC_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        WCC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, select_coop_kernel, SEL_THREADS, 0));
        coop_cap[dev] = (coop && per_sm > 0) ? sms * per_sm : -1;
    }
    const long long ctas = (long long)s.chunks * N;
    if (dev >= 0 && dev < 64 && coop_cap[dev] > 0 && ctas <= coop_cap[dev]) {
        int* status = nullptr;
        WCC_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_status));
        uint32_t* hist = s.hist; uint32_t* bar = s.bar; uint32_t* chunkcnt = s.chunkcnt;
        void* args[] = {(void*)&nrm2, (void*)&P, (void*)&k, (void*)&hist, (void*)&bar, (void*)&chunkcnt, (void*)&idx,
                        (void*)&tau, (void*)&rank, (void*)&amaxpos, (void*)&amax_kept, (void*)&status};
        WCC_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(select_coop_kernel), grid, dim3(SEL_THREADS), args, 0, st));
        WCC_LAUNCH_CHECK();
        return WCC_OK;
    }
    select_hist_kernel<1><<<grid, SEL_THREADS, 0, st>>>(nrm2, P, k, s.hist, s.state);
    select_hist_kernel<2><<<grid, SEL_THREADS, 0, st>>>(nrm2, P, k, s.hist, s.state);
    select_hist_kernel<3><<<grid, SEL_THREADS, 0, st>>>(nrm2, P, k, s.hist, s.state);
    select_count_kernel<<<grid, SEL_THREADS, 0, st>>>(nrm2, P, s.hist, s.state, s.chunkcnt, tau);
    select_compact_kernel<<<grid, SEL_THREADS, 0, st>>>(nrm2, P, k, s.state, s.chunkcnt, idx, rank, amaxpos, amax_kept);
    g_launches += 4;
    WCC_LAUNCH_CHECK();
    return WCC_OK;
}

}  // namespace wcc

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

#include <cooperative_groups.h>

#include "common.cuh"
#include "tma.cuh"

namespace wcc {
namespace cg = cooperative_groups;

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
        if (R == 1) hist_add(sh, key[i] >> 21, ok[i]);
        if (R == 2) hist_add(sh, (key[i] >> 10) & 0x7FFu, ok[i] && (key[i] >> 21) == prefix);
        if (R == 3) hist_add(sh, key[i] & 0x3FFu, ok[i] && (key[i] >> 10) == prefix);
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

__device__ __forceinline__ bool image_barrier(uint32_t* counter, uint32_t target)
{
    __shared__ int sh_ok;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1u);
        int ok = 0;
        const uint32_t limit = 2u * tc::c_wait_limit;               // polls of >= 40 ns
        for (uint32_t it = 0; it < limit; ++it) {
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
    for (int i = 0; i < SEL_KPT; ++i) hist_add(sh, key[i] >> 21, okk[i]);
    flush_hist<SEL_BINS>(sh, hn);
    // A barrier that ran out leaves the histograms incomplete: report it and leave at once (the decision is uniform
    // over the block), so that nothing is derived from them and no index is written.
    auto give_up = [&]() { if (threadIdx.x == 0) atomicExch(status, (int)WCC_ERR_TIMEOUT); };
    if (!image_barrier(barn, chunks)) { give_up(); return; }
    // round 2
    uint32_t b1, above;
    find_bin<SEL_BINS>(hn, (uint32_t)k, sh_scan, sh_res, b1, above);
    const uint32_t k1 = (uint32_t)k - above;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) hist_add(sh, (key[i] >> 10) & 0x7FFu, okk[i] && (key[i] >> 21) == b1);
    flush_hist<SEL_BINS>(sh, hn + SEL_BINS);
    if (!image_barrier(barn, 2 * chunks)) { give_up(); return; }
    // round 3
    uint32_t b2;
    find_bin<SEL_BINS>(hn + SEL_BINS, k1, sh_scan, sh_res, b2, above);
    const uint32_t k2 = k1 - above;
    const uint32_t prefix = (b1 << 11) | b2;
#pragma unroll
    for (int i = 0; i < SEL_KPT; ++i) hist_add(sh, key[i] & 0x3FFu, okk[i] && (key[i] >> 10) == prefix);
    flush_hist<1024>(sh, hn + 2 * SEL_BINS);
    if (!image_barrier(barn, 3 * chunks)) { give_up(); return; }
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
    if (!image_barrier(barn, 4 * chunks)) { give_up(); return; }
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
        if (keep && pos < (uint32_t)k) {
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

// ---- the select as one thread-block cluster per image -------------------------------------------------
// Up to 8 CTAs of 1024 threads form one cluster per image (P <= 131072 keys, at most 16 per thread, held in
// registers).  Each CTA histograms its keys in shared memory; the histograms are combined through distributed
// shared memory (every CTA sums one slice of the bins over all CTAs, then all CTAs read the slice totals and the
// slice that holds the k-th key), and the phases are separated by hardware cluster barriers: no global-memory
// round trips, no spinning, no scratch memory.
constexpr int CL_THREADS = 1024;
constexpr int CL_MAXKPT = 16;
constexpr int CL_MAXCS = 16;          // 8 is the portable cluster size; 16 needs the non-portable opt-in
constexpr int CL_CAND_CTA = 512;     // candidate slots per CTA
constexpr int CL_CAND_MAX = 1024;    // most candidates ranked by brute force; beyond that: histogram rounds
constexpr int FINE_BINS = 65536;     // histogram of the 16 bits below the sign of every norm, filled by the producer of the norms

struct ClusterSmem {
    uint32_t hist[SEL_BINS];
    uint32_t slice[SEL_BINS];       // sums over all CTAs of this CTA's slice of bins
    uint32_t warp_sums[CL_THREADS / 32 + 1];
    uint32_t slice_total;
    uint32_t cnt[2];                // keys above / equal to the threshold in this CTA
    uint32_t res[3];                // found bin, keys above it, keys in it
    uint32_t tot[CL_MAXCS];
    uint32_t amax;
    uint32_t ncand;                 // candidates of this CTA (keys in the 16-bit bin that holds the threshold)
    uint32_t cand[CL_CAND_CTA];
    __align__(16) uint32_t all[CL_CAND_MAX];      // candidates of the whole cluster
    uint32_t thr[3];                // threshold key, ties to keep, ties in total
};

// exclusive scan over the threads of the block (256, 512 or 1024); every thread also gets the total
__device__ __forceinline__ uint32_t block_scan_1024(uint32_t v, uint32_t* warp_sums, uint32_t* total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) warp_sums[w] = inc;
    __syncthreads();
    if (w == 0) {
        const uint32_t s = (lane < nw) ? warp_sums[lane] : 0u;
        uint32_t si = s;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, si, d);
            if (lane >= d) si += t;
        }
        if (lane < nw) warp_sums[lane] = si - s;
        if (lane == 31) warp_sums[32] = si;
    }
    __syncthreads();
    const uint32_t res = warp_sums[w] + inc - v;
    *total = warp_sums[32];
    __syncthreads();
    return res;
}

// After every CTA has filled sm.hist: find the bin holding the krem-th key from the top over the whole cluster.
// nbins = 2048 or 1024.  Contains two cluster barriers.  Every thread of every CTA returns the same (bin, above).
__device__ __forceinline__ void cluster_find_bin(cg::cluster_group& cluster, ClusterSmem& sm, int cs, int crank, int nbins,
                                                 uint32_t krem, uint32_t& bin, uint32_t& above)
{
    const int B = nbins / cs;                        // bins per slice: 128 .. 2048
    cluster.sync();                                  // all local histograms complete
    uint32_t mine = 0;
    for (int t = threadIdx.x; t < B; t += blockDim.x) {
        uint32_t sum = 0;
        for (int r = 0; r < cs; ++r) sum += cluster.map_shared_rank(sm.hist, r)[crank * B + t];
        sm.slice[t] = sum;
        mine += sum;
    }
    uint32_t total;
    block_scan_1024(mine, sm.warp_sums, &total);
    if (threadIdx.x == 0) sm.slice_total = total;
    cluster.sync();                                  // all slices and slice totals complete
    if (threadIdx.x < cs) sm.tot[threadIdx.x] = *cluster.map_shared_rank(&sm.slice_total, threadIdx.x);
    __syncthreads();
    uint32_t above_slices = 0;
    int target = 0;
    for (int r = cs - 1; r >= 0; --r) {              // slices from the top bins downwards
        const uint32_t t = sm.tot[r];
        if (krem <= above_slices + t) { target = r; break; }
        above_slices += t;
    }
    const uint32_t kin = krem - above_slices;        // rank inside the target slice, from its top bin
    const uint32_t* rs = cluster.map_shared_rank(sm.slice, target);
    // thread t covers the `per` bins (B-1 - t*per) downwards of the slice (per <= 8)
    const int per = (B + (int)blockDim.x - 1) / (int)blockDim.x;
    const int top = B - 1 - (int)threadIdx.x * per;
    uint32_t c[8], mysum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        c[i] = (i < per && top - i >= 0) ? rs[top - i] : 0u;
        mysum += c[i];
    }
    uint32_t tot2;
    const uint32_t before = block_scan_1024(mysum, sm.warp_sums, &tot2);
    if (before < kin && kin <= before + mysum) {
        uint32_t a = before;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (a < kin && kin <= a + c[i]) { sm.res[0] = (uint32_t)(target * B + top - i); sm.res[1] = above_slices + a; sm.res[2] = c[i]; }
            a += c[i];
        }
    }
    __syncthreads();
    bin = sm.res[0];
    above = sm.res[1];
    __syncthreads();
}


// Find the bin of a complete 2048-bin histogram in global memory that holds the krem-th key from the top; block of
// 256, 512 or 1024 threads, every thread returns the same values.
__device__ __forceinline__ void block_find_bin_2048(const uint32_t* __restrict__ h, uint32_t krem, ClusterSmem& sm,
                                                    uint32_t& bin, uint32_t& above, uint32_t& tot)
{
    const int per = SEL_BINS / (int)blockDim.x;            // 8, 4 or 2
    const int top = SEL_BINS - 1 - (int)threadIdx.x * per;
    uint32_t c[8], mysum = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        c[i] = (i < per) ? __ldcg(&h[top - i]) : 0u;
        mysum += c[i];
    }
    const uint32_t before = block_scan_1024(mysum, sm.warp_sums, &tot);
    if (before < krem && krem <= before + mysum) {
        uint32_t a = before;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (a < krem && krem <= a + c[i]) { sm.res[0] = (uint32_t)(top - i); sm.res[1] = a; sm.res[2] = c[i]; }
            a += c[i];
        }
    }
    __syncthreads();
    bin = sm.res[0];
    above = sm.res[1];
    __syncthreads();
}

// hist1 ([N][3][2048], round 1 first) and fine ([N][65536]) are optional histograms of the 11 and 16 bits below the sign
// of every norm (norm_digit11 / norm_digit16: norms are never negative) that the producer of the norms filled; with both, the threshold is usually found without any histogram round:
// the 16-bit bin that holds the k-th key contains few keys, which the cluster gathers and ranks directly.
// idx and rank are written only when asked for (want_rank) or when the threshold's ties are kept only in part
// (then the order of positions matters); otherwise consumers compare keys with thr[n] = {threshold key, ties
// kept, use_rank flag, number of candidate keys that were ranked (diagnostic)}.
// MAXKPT: key registers per thread (16, or 4 for the launches that spread an image over enough threads).
template <int MAXKPT>
__global__ void __launch_bounds__(CL_THREADS, 1)
select_cluster_kernel(const float* __restrict__ nrm2, int P, int k, int kpt, int32_t* __restrict__ idx, float* __restrict__ tau,
                      int32_t* __restrict__ rank, const float* __restrict__ amaxpos, float* __restrict__ amax_kept,
                      const uint32_t* __restrict__ hist1, const uint32_t* __restrict__ fine, uint32_t* __restrict__ thr,
                      int want_rank)
{
    __shared__ ClusterSmem sm;
    cg::cluster_group cluster = cg::this_cluster();
    const int cs = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
    const int n = blockIdx.y;
    const float* v = nrm2 + (size_t)n * P;
    const int base = (crank * (int)blockDim.x + (int)threadIdx.x) * kpt;  // kpt consecutive keys per thread
    const int lane = threadIdx.x & 31;

    uint32_t key[MAXKPT];
#pragma unroll
    for (int i = 0; i < MAXKPT; ++i) key[i] = (i < kpt && base + i < P) ? float_key(v[base + i]) : 0u;
    auto valid = [&](int i) { return i < kpt && base + i < P; };
    // few keys per thread: the per-position maxima are fetched together with the keys, so that the pass over the kept
    // positions at the end waits for no further load
    constexpr bool PRE = MAXKPT <= 4;
    float pre[PRE ? MAXKPT : 1];
    if (PRE) {
#pragma unroll
        for (int i = 0; i < MAXKPT; ++i) pre[PRE ? i : 0] = (amaxpos && valid(i)) ? amaxpos[(size_t)n * P + base + i] : 0.0f;
    }

    for (int i = threadIdx.x; i < SEL_BINS; i += blockDim.x) sm.hist[i] = 0u;
    if (threadIdx.x == 0) { sm.amax = 0u; sm.ncand = 0u; sm.thr[0] = 0xFFFFFFFFu; sm.thr[1] = 0u; sm.thr[2] = 0u; }   // thr: keep nothing
                                                       // unless a candidate is found (histograms that do not match the keys)
    __syncthreads();

    uint32_t tkey = 0, need_eq = 0, total_eq = 0, ranked = 0;    // ranked: candidates counted through (diagnostic)
    bool found = false;
    // The supplied histograms count the non-zero norms only; the zeros are the positions they leave out and rank
    // below everything else.  More kept positions than non-zero norms: the threshold is zero.
    bool zero_thr = false;
    uint32_t b1h = 0, aboveh = 0;
    if (hist1 && fine) {
        // the 11-bit bin of the threshold
        uint32_t nonzero;
        if (threadIdx.x == 0) { sm.res[0] = 0u; sm.res[1] = 0u; sm.res[2] = 0u; }      // (a barrier follows inside)
        block_find_bin_2048(hist1 + (size_t)n * 3 * SEL_BINS, (uint32_t)k, sm, b1h, aboveh, nonzero);
        zero_thr = (uint32_t)k > nonzero;              // the same in every CTA of the cluster
        if (zero_thr) {
            tkey = 0x80000000u;                        // key of +0
            need_eq = (uint32_t)k - nonzero;
            total_eq = (uint32_t)P - nonzero;
            found = true;
        }
    }
    if (hist1 && fine && !zero_thr) {
        // the 16-bit bin inside the 11-bit bin (32 fine bins, one per lane of warp 0, top bin in lane 0)
        const uint32_t b1 = b1h, above = aboveh;
        const uint32_t k1 = (uint32_t)k - above;
        if (threadIdx.x < 32) {
            const uint32_t f = __ldcg(&fine[(size_t)n * FINE_BINS + (b1 << 5) + 31u - (uint32_t)lane]);
            uint32_t inc = f;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc += t;
            }
            const uint32_t before = inc - f;
            if (before < k1 && k1 <= inc) { sm.res[0] = (b1 << 5) + 31u - (uint32_t)lane; sm.res[1] = before; sm.res[2] = f; }
        }
        __syncthreads();
        const uint32_t prefix16 = sm.res[0], k16 = k1 - sm.res[1];
        __syncthreads();
        // collect this CTA's candidates
#pragma unroll
        for (int i = 0; i < MAXKPT; ++i) {
            if (i >= kpt) break;
            const bool c = valid(i) && ((key[i] >> 15) & 0xFFFFu) == prefix16;
            const unsigned m = __ballot_sync(0xFFFFFFFFu, c);
            if (m) {
                uint32_t off = 0;
                if (lane == 0) off = atomicAdd(&sm.ncand, (uint32_t)__popc(m));
                off = __shfl_sync(0xFFFFFFFFu, off, 0);
                const uint32_t slot = off + (uint32_t)__popc(m & ((1u << lane) - 1u));
                if (c && slot < CL_CAND_CTA) sm.cand[slot] = key[i];
            }
        }
        cluster.sync();
        if (threadIdx.x < cs) sm.tot[threadIdx.x] = *cluster.map_shared_rank(&sm.ncand, threadIdx.x);
        __syncthreads();
        uint32_t M = 0;
        bool overflow = false;
        for (int r = 0; r < cs; ++r) { overflow = overflow || sm.tot[r] > CL_CAND_CTA; M += sm.tot[r]; }
        overflow = overflow || M > CL_CAND_MAX;
        if (!overflow) {
            // one remote load per thread, all in flight together (rank after rank would expose every rank's latency)
            for (uint32_t g = threadIdx.x; g < M; g += blockDim.x) {
                uint32_t pre = 0;
                int r = 0;
                while (g >= pre + sm.tot[r]) { pre += sm.tot[r]; ++r; }
                sm.all[g] = cluster.map_shared_rank(sm.cand, r)[g - pre];
            }
            __syncthreads();
            // the k16-th largest candidate, by counting (M is small)
            for (uint32_t i = threadIdx.x; i < M; i += blockDim.x) {
                const uint32_t ci = sm.all[i];
                uint32_t g = 0, e = 0;
                const uint4* all4 = reinterpret_cast<const uint4*>(sm.all);
                for (uint32_t j4 = 0; j4 < M / 4; ++j4) {        // four candidates per shared-memory load
                    const uint4 c = all4[j4];
                    g += (c.x > ci) + (c.y > ci) + (c.z > ci) + (c.w > ci);
                    e += (c.x == ci) + (c.y == ci) + (c.z == ci) + (c.w == ci);
                }
                for (uint32_t j = M & ~3u; j < M; ++j) { const uint32_t cj = sm.all[j]; g += cj > ci; e += cj == ci; }
                if (g < k16 && k16 <= g + e) { sm.thr[0] = ci; sm.thr[1] = k16 - g; sm.thr[2] = e; }   // equal keys write equal values
            }
            __syncthreads();
            tkey = sm.thr[0]; need_eq = sm.thr[1]; total_eq = sm.thr[2];
            ranked = M;
            found = true;
        }
    }
    if (!found) {
        // round 1: top 11 bits (only the bin search when the producer of the norms histogrammed them).  The producer's
        // digits start below the sign bit (norm_digit11), so with its histogram the rounds run on the keys shifted left
        // by one: 11 + 11 + 9 bits and a zero; the threshold is shifted back at the end.
        uint32_t b1, above;
        const bool shifted = hist1 != nullptr;
        if (shifted) {
#pragma unroll
            for (int i = 0; i < MAXKPT; ++i) key[i] <<= 1;
        }
        if (hist1) {
            uint32_t nonzero;
            block_find_bin_2048(hist1 + (size_t)n * 3 * SEL_BINS, (uint32_t)k, sm, b1, above, nonzero);
        } else {
#pragma unroll
            for (int i = 0; i < MAXKPT; ++i)
                if (i < kpt) hist_add(sm.hist, key[i] >> 21, valid(i));
            cluster_find_bin(cluster, sm, cs, crank, SEL_BINS, (uint32_t)k, b1, above);
            for (int i = threadIdx.x; i < SEL_BINS; i += blockDim.x) sm.hist[i] = 0u;
            __syncthreads();
        }
        const uint32_t k1 = (uint32_t)k - above;
        // round 2: next 11 bits of the keys that match
#pragma unroll
        for (int i = 0; i < MAXKPT; ++i)     // plain atomics: these digits are mantissa bits, spread over the bins
            if (valid(i) && (key[i] >> 21) == b1) atomicAdd(&sm.hist[(key[i] >> 10) & 0x7FFu], 1u);
        uint32_t b2;
        cluster_find_bin(cluster, sm, cs, crank, SEL_BINS, k1, b2, above);
        const uint32_t k2 = k1 - above;
        const uint32_t prefix = (b1 << 11) | b2;
        // round 3: last 10 bits
        for (int i = threadIdx.x; i < SEL_BINS; i += blockDim.x) sm.hist[i] = 0u;
        __syncthreads();
#pragma unroll
        for (int i = 0; i < MAXKPT; ++i)
            if (valid(i) && (key[i] >> 10) == prefix) atomicAdd(&sm.hist[key[i] & 0x3FFu], 1u);
        uint32_t b3;
        cluster_find_bin(cluster, sm, cs, crank, 1024, k2, b3, above);
        tkey = (prefix << 10) | b3;
        need_eq = k2 - above;
        total_eq = sm.res[2];
        if (shifted) {                                 // back to whole keys (every norm has the sign bit of +0 and above)
            tkey = (tkey >> 1) | 0x80000000u;
#pragma unroll
            for (int i = 0; i < MAXKPT; ++i) key[i] = (key[i] >> 1) | 0x80000000u;
        }
    }
    if (tau && crank == 0 && threadIdx.x == 0) tau[n] = key_float(tkey);

    // Ties kept in part need the order of positions, except ties at zero: a position whose norm is zero holds only zero
    // coefficients, so keeping more of them than asked changes nothing downstream (consumers that get the threshold
    // alone keep every position with key >= threshold).
    const bool ordered = want_rank || (need_eq < total_eq && !zero_thr);       // uniform over the cluster
    float amax = 0.0f;
    // Nobody may leave while a neighbour can still read its shared memory.  When no further exchange follows, every CTA
    // signals here that it is done reading and only waits for the others at the very end (the wait is hidden behind the
    // pass over the kept positions).
    if (!ordered) cluster.barrier_arrive();
    if (!ordered) {
        // every key >= threshold is kept; nobody needs the order
        if (amaxpos) {
#pragma unroll
            for (int i = 0; i < MAXKPT; ++i)
                if (valid(i) && key[i] >= tkey) amax = fmaxf(amax, PRE ? pre[PRE ? i : 0] : amaxpos[(size_t)n * P + base + i]);
        }
    } else {
        // ordered compaction: ascending idx, rank map, ties to the lowest positions
        uint32_t gt = 0, eq = 0;
#pragma unroll
        for (int i = 0; i < MAXKPT; ++i) {
            if (!valid(i)) continue;
            gt += key[i] > tkey;
            eq += key[i] == tkey;
        }
        uint32_t tot_gt, tot_eq;
        uint32_t gt_before = block_scan_1024(gt, sm.warp_sums, &tot_gt);
        uint32_t eq_before = block_scan_1024(eq, sm.warp_sums, &tot_eq);
        if (threadIdx.x == 0) { sm.cnt[0] = tot_gt; sm.cnt[1] = tot_eq; }
        cluster.sync();
        for (int r = 0; r < crank; ++r) {
            const uint32_t* c = cluster.map_shared_rank(sm.cnt, r);
            gt_before += c[0];
            eq_before += c[1];
        }
#pragma unroll
        for (int i = 0; i < MAXKPT; ++i) {
            if (!valid(i)) continue;
            const bool is_gt = key[i] > tkey, is_eq = key[i] == tkey;
            const bool keep = is_gt || (is_eq && eq_before < need_eq);
            const uint32_t pos = gt_before + min(eq_before, need_eq);
            if (keep) {
                if (idx) idx[(size_t)n * k + pos] = base + i;
                if (amaxpos) amax = fmaxf(amax, PRE ? pre[PRE ? i : 0] : amaxpos[(size_t)n * P + base + i]);
            }
            if (rank) rank[(size_t)n * P + base + i] = keep ? (int32_t)pos : -1;
            gt_before += is_gt;
            eq_before += is_eq;
        }
    }
    if (thr && crank == 0 && threadIdx.x == 0) {
        thr[n * 4 + 0] = tkey;
        thr[n * 4 + 1] = need_eq;
        thr[n * 4 + 2] = ordered ? 1u : 0u;
        thr[n * 4 + 3] = ranked;
    }
    if (amax_kept) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        if (lane == 0) atomicMax(&sm.amax, __float_as_uint(amax));
        __syncthreads();
        if (threadIdx.x == 0 && sm.amax) atomicMax(reinterpret_cast<uint32_t*>(amax_kept), sm.amax);
    }
    if (!ordered) cluster.barrier_wait();
    else cluster.sync();                             // nobody leaves while a neighbour may still read its shared memory
}

__global__ void thr_use_rank_kernel(uint32_t* thr, int N)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n < N) { thr[n * 4 + 0] = 0u; thr[n * 4 + 1] = 0u; thr[n * 4 + 2] = 1u; }
}

// One cluster per image holds up to this many positions in registers (the path that uses a producer's histograms).
inline bool select_in_cluster(int P) { return P <= 8 * CL_THREADS * CL_MAXKPT; }

// hist1_ready: the caller has already cleared the zero region of the workspace (carve_select_ws(...).hist,
// zero_bytes) and filled round 1 of the histogram (norm_digit11 of every non-zero norm) before this call.
// fine / thr: see select_cluster_kernel; want_rank: idx (if non-NULL) and rank must be written even when the
// threshold alone would do.  Without thr the rank map and idx are always written.
wcc_status launch_select(const float* nrm2, int N, int P, int k, int32_t* idx, float* tau,
                         int32_t* rank, const float* amaxpos, bool want_amax,
                         void* ws, size_t ws_bytes, cudaStream_t st, bool hist1_ready,
                         const uint32_t* fine, uint32_t* thr, bool want_rank)
{
    if (ws_bytes < select_ws_bytes(N, P)) return WCC_ERR_WORKSPACE;
    const SelectWs s = carve_select_ws(ws, N, P);
    float* amax_kept = want_amax ? s.amax : nullptr;
    // one cluster per image while its keys fit in the registers of 8 x 1024 threads
    // clusters of 16 CTAs (opt-in) for images beyond 64 K positions, when the device schedules them
    static int max_cs[64] = {0};
    int devc = 0;
    WCC_CUDA_TRY(cudaGetDevice(&devc));
    if (devc >= 0 && devc < 64 && max_cs[devc] == 0) {
        max_cs[devc] = 8;
        if (cudaFuncSetAttribute(select_cluster_kernel<CL_MAXKPT>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
            cudaFuncSetAttribute(select_cluster_kernel<4>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3(16, 1);
            q.blockDim = dim3(CL_THREADS);
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = 16; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
            q.attrs = qa; q.numAttrs = 1;
            int nclusters = 0;
            if (cudaOccupancyMaxActiveClusters(&nclusters, select_cluster_kernel<CL_MAXKPT>, &q) == cudaSuccess && nclusters > 0) max_cs[devc] = 16;
        }
        (void)cudaGetLastError();
    }
    const int cs_cap = (devc >= 0 && devc < 64) ? max_cs[devc] : 8;
    if (select_in_cluster(P)) {
        // as many CTAs per image as useful, then as few threads as hold the keys (<= 16 each): the per-thread cost of
        // the scans and barriers is fixed, so fewer, busier threads finish sooner
        int cs = 1;
        while (cs < 8 && cs * 512 < P) cs <<= 1;
        if (cs == 8 && cs_cap == 16 && P > 65536) cs = 16;
        int threads = 256;
        const int kpt_goal = hist1_ready ? 4 : CL_MAXKPT;               // few keys per thread when no scans are needed
        while (threads < CL_THREADS && (long long)cs * threads * kpt_goal < P) threads <<= 1;
        const int kpt = ceil_div(P, cs * threads);
        if (amax_kept && !hist1_ready) WCC_CUDA_TRY(cudaMemsetAsync(amax_kept, 0, sizeof(float), st));
        const uint32_t* hist1 = hist1_ready ? s.hist : nullptr;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(cs, N);
        cfg.blockDim = dim3(threads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const uint32_t* fine_use = hist1_ready ? fine : (const uint32_t*)nullptr;
        const int wr = (want_rank || !thr) ? 1 : 0;
        if (kpt <= 4)                                  // few keys per thread: the instantiation with four key registers
            WCC_CUDA_TRY(cudaLaunchKernelEx(&cfg, select_cluster_kernel<4>, nrm2, P, k, kpt, idx, tau, rank, amaxpos, amax_kept, hist1,
                                            fine_use, thr, wr));
        else
            WCC_CUDA_TRY(cudaLaunchKernelEx(&cfg, select_cluster_kernel<CL_MAXKPT>, nrm2, P, k, kpt, idx, tau, rank, amaxpos, amax_kept,
                                            hist1, fine_use, thr, wr));
        WCC_LAUNCH_CHECK();
        return WCC_OK;
    }
    if (thr) {                                        // these paths always write idx and the rank map
        thr_use_rank_kernel<<<ceil_div(N, 128), 128, 0, st>>>(thr, N);
        ++g_launches;
    }
    // (histograms supplied by the caller are not used by these paths: they start from a clean slate)
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

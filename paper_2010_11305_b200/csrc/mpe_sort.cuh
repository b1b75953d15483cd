// Segmented stable LSD radix sort and device-wide prefix sums.
//
// The batch's indices arrive grouped by table, so sorting "by (table, row)"
// (Section 5.1: sort the row indices of the mini-batch, then merge duplicates)
// only has to order the rows inside each table's segment.  Every pass sorts by
// an 8-bit digit with per-(table, digit, tile) counters, so one pass over the
// whole array sorts all segments at once and never moves a key out of its
// segment.  No kernel here waits on another block: a pass is histogram ->
// prefix sum -> scatter, three ordinary launches.  A tile is 4096 elements:
// 16 per thread, ranked by warp (match on the digit, warp-private counters),
// reordered through shared memory so that global writes are runs.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mpe {

#ifndef MPE_SORT_ITEMS
#define MPE_SORT_ITEMS 16      // keys per thread of the scatter kernel (even)
#endif
#ifndef MPE_SORT_MINB
#define MPE_SORT_MINB 4        // resident blocks per SM the scatter kernel is compiled for
#endif
constexpr int SORT_THREADS = 256;
constexpr int SORT_ITEMS = MPE_SORT_ITEMS;
constexpr int SORT_TILE = SORT_THREADS * SORT_ITEMS;   // keys per block
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 16;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

// ---- block-wide exclusive prefix sum of one value per thread -----------------
template <int THREADS>
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* total, uint32_t* smem /*[THREADS/32 + 1]*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffU, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < THREADS / 32 ? smem[lane] : 0;
        uint32_t winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t n = __shfl_up_sync(0xffffffffU, winc, o);
            if (lane >= o) winc += n;
        }
        if (lane < THREADS / 32) smem[lane] = winc - w;
        if (lane == THREADS / 32 - 1) smem[THREADS / 32] = winc;
    }
    __syncthreads();
    const uint32_t r = smem[warp] + inc - v;
    *total = smem[THREADS / 32];
    __syncthreads();
    return r;
}

// ---- segment -> tile bookkeeping ----------------------------------------------
// tile_base[t] = number of SORT_TILE-sized tiles of segments 0..t-1; tile_base[T] = total.
// A non-zero *skip (the step was abandoned) yields zero tiles, which turns the whole sort into a no-op.
__global__ void k_tile_setup(const int32_t* __restrict__ seg_start, int T, int32_t* __restrict__ tile_base,
                             uint32_t* __restrict__ hist_len, const uint32_t* __restrict__ skip) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const bool off = *skip != 0;
        int32_t acc = 0;
        for (int t = 0; t < T; ++t) {
            tile_base[t] = acc;
            int32_t len = off ? 0 : seg_start[t + 1] - seg_start[t];
            acc += (len + SORT_TILE - 1) / SORT_TILE;
        }
        tile_base[T] = acc;
        *hist_len = (uint32_t)acc * 256u;
    }
}

__device__ __forceinline__ int find_segment(const int32_t* __restrict__ base, int T, int32_t v) {
    // largest t in [0,T) with base[t] <= v  (base non-decreasing, base[0] <= v < base[T])
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (base[mid] <= v) lo = mid; else hi = mid;
    }
    return lo;
}

// ---- pass 1 of 3: per-(table, digit, tile) counts ------------------------------
// PAIRS: the keys are the .x members of (key, payload) records (every pass but the first)
template <bool PAIRS>
__global__ void __launch_bounds__(SORT_THREADS)
k_sort_hist(const uint32_t* __restrict__ keys, const int32_t* __restrict__ seg_start, const int32_t* __restrict__ tile_base,
            int T, int shift, uint32_t* __restrict__ hist) {
    // one warp per tile: its own 256 counters, eight key loads in flight per lane, no block-wide barrier
    constexpr int WARPS = SORT_THREADS / 32;
    constexpr int STRIDE = PAIRS ? 2 : 1;
    __shared__ uint32_t cnt[WARPS][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ntiles = tile_base[T];
    for (int tile = blockIdx.x * WARPS + warp; tile < ntiles; tile += gridDim.x * WARPS) {
        const int t = find_segment(tile_base, T, tile);
        const int local = tile - tile_base[t];
        const int nt = tile_base[t + 1] - tile_base[t];
        const int32_t start = seg_start[t] + local * SORT_TILE;
        const int32_t end = min(start + SORT_TILE, seg_start[t + 1]);
#pragma unroll
        for (int i = 0; i < 8; ++i) cnt[warp][i * 32 + lane] = 0;
        __syncwarp();
        for (int32_t i0 = start + lane; i0 < end; i0 += 32 * 8) {
            uint32_t k[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) k[q] = i0 + 32 * q < end ? keys[(size_t)(i0 + 32 * q) * STRIDE] : 0u;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (i0 + 32 * q < end) atomicAdd(&cnt[warp][(k[q] >> shift) & 255u], 1u);
        }
        __syncwarp();
        uint32_t* out = hist + (size_t)256 * tile_base[t] + local;
#pragma unroll
        for (int i = 0; i < 8; ++i) out[(size_t)(i * 32 + lane) * nt] = cnt[warp][i * 32 + lane];
        __syncwarp();
    }
}

// ---- pass 3 of 3: stable scatter ------------------------------------------------
// Between passes an element travels as one 8-byte (key, payload) record, so a pass reads and writes it with one
// instruction each and a digit's run of a tile is one contiguous piece of memory.
// FIRST: the input is the bare key array and the payload is the element's position.
// LAST: the output is split into the sorted keys and the sorted payloads (out_keys / out_vals), which is what the
// kernels after the sort read.
template <bool FIRST, bool LAST>
__global__ void __launch_bounds__(SORT_THREADS, MPE_SORT_MINB)
k_sort_scatter(const uint32_t* __restrict__ keys_in, const uint2* __restrict__ pairs_in, uint2* __restrict__ pairs_out,
               uint32_t* __restrict__ out_keys, uint32_t* __restrict__ out_vals,
               const int32_t* __restrict__ seg_start, const int32_t* __restrict__ tile_base, int T, int shift,
               const uint32_t* __restrict__ hist_scanned) {
    constexpr int WARPS = SORT_THREADS / 32;
    __shared__ uint32_t wcnt[WARPS][256];      // per-warp digit counters, then tile-local position of the warp's first key of each digit
    __shared__ uint32_t goff[256];             // first global position of each digit of this tile minus its tile-local start
    __shared__ uint2 skv[SORT_TILE];
    __shared__ uint32_t scan_tmp[SORT_THREADS / 32 + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const int ntiles = tile_base[T];
    volatile uint32_t* myc = wcnt[warp];
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int t = find_segment(tile_base, T, tile);
        const int local = tile - tile_base[t];
        const int nt = tile_base[t + 1] - tile_base[t];
        const int32_t start = seg_start[t] + local * SORT_TILE;
        const int32_t count = min(SORT_TILE, seg_start[t + 1] - start);
        // warp w owns elements [w*32*ITEMS, (w+1)*32*ITEMS) of the tile, item i of lane l is w*32*ITEMS + i*32 + l,
        // so "item order, then lane order" is the original order
        uint32_t key[SORT_ITEMS], val[SORT_ITEMS];
        const int e0 = warp * (32 * SORT_ITEMS) + lane;
        if (e0 - lane + 32 * SORT_ITEMS <= count) {                    // the warp's whole share is inside the tile
#pragma unroll
            for (int i = 0; i < SORT_ITEMS; ++i) {
                const int e = e0 + i * 32;
                if (FIRST) { key[i] = keys_in[start + e]; val[i] = (uint32_t)(start + e); }
                else { const uint2 kv = pairs_in[start + e]; key[i] = kv.x; val[i] = kv.y; }
            }
        } else {
#pragma unroll
            for (int i = 0; i < SORT_ITEMS; ++i) {
                const int e = e0 + i * 32;
                key[i] = 0xffffffffU; val[i] = 0u;                     // padding: digit 255 in every pass, behind every real key
                if (e < count) {
                    if (FIRST) { key[i] = keys_in[start + e]; val[i] = (uint32_t)(start + e); }
                    else { const uint2 kv = pairs_in[start + e]; key[i] = kv.x; val[i] = kv.y; }
                }
            }
        }
        const uint32_t gb = hist_scanned[(size_t)256 * tile_base[t] + (size_t)threadIdx.x * nt + local];   // digit threadIdx.x
#pragma unroll
        for (int i = 0; i < 8; ++i) wcnt[warp][i * 32 + lane] = 0;
        __syncwarp();
        // stable rank among the warp's keys of the same digit: the counters are the warp's own, so the first lane of each
        // group of equal digits updates them with plain loads and stores
        uint32_t rank[SORT_ITEMS / 2];
#pragma unroll
        for (int i = 0; i < SORT_ITEMS; ++i) {
            const uint32_t dg = (key[i] >> shift) & 255u;
            const uint32_t peers = __match_any_sync(0xffffffffU, dg);
            const int leader = __ffs(peers) - 1;
            uint32_t before = 0;
            if (lane == leader) { before = myc[dg]; myc[dg] = before + (uint32_t)__popc(peers); }
            before = __shfl_sync(0xffffffffU, before, leader);
            const uint32_t r = before + (uint32_t)__popc(peers & lt);
            if (i & 1) rank[i >> 1] |= r << 16; else rank[i >> 1] = r;
            __syncwarp();
        }
        __syncthreads();
        // digit d (= threadIdx.x): exclusive sum over warps, then over digits
        uint32_t tot = 0;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) tot += wcnt[w][threadIdx.x];
        uint32_t all;
        const uint32_t ds = block_exclusive_scan<SORT_THREADS>(tot, &all, scan_tmp);
        uint32_t run = ds;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {                                      // tile-local position of warp w's first key with this digit
            const uint32_t c = wcnt[w][threadIdx.x];
            wcnt[w][threadIdx.x] = run;
            run += c;
        }
        goff[threadIdx.x] = gb - ds;                                           // global position = goff + tile-local position
        __syncthreads();
#pragma unroll
        for (int i = 0; i < SORT_ITEMS; ++i) {
            const uint32_t dg = (key[i] >> shift) & 255u;
            const uint32_t r = (i & 1) ? rank[i >> 1] >> 16 : rank[i >> 1] & 0xffffu;
            skv[wcnt[warp][dg] + r] = make_uint2(key[i], val[i]);
        }
        __syncthreads();
        // padding keys follow every real key of the tile, so positions [0,count) are real
        for (int j = threadIdx.x; j < count; j += SORT_THREADS) {
            const uint2 kv = skv[j];
            const uint32_t dst = goff[(kv.x >> shift) & 255u] + (uint32_t)j;
            if (LAST) { out_keys[dst] = kv.x; out_vals[dst] = kv.y; }
            else pairs_out[dst] = kv;
        }
        __syncthreads();
    }
}

// ---- device-wide exclusive prefix sum over uint32 (length read from device memory) ------------
__global__ void __launch_bounds__(SCAN_THREADS)
k_scan_reduce(const uint32_t* __restrict__ in, const uint32_t* __restrict__ n_ptr, uint32_t* __restrict__ block_sums) {
    __shared__ uint32_t tmp[SCAN_THREADS / 32 + 1];
    const uint32_t n = *n_ptr;
    const uint32_t nblk = (n + SCAN_TILE - 1) / SCAN_TILE;
    for (uint32_t b = blockIdx.x; b < nblk; b += gridDim.x) {
        uint32_t s = 0;
        const uint32_t base = b * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
#pragma unroll
        for (int i = 0; i < SCAN_ITEMS; ++i) if (base + i < n) s += in[base + i];
        uint32_t total;
        block_exclusive_scan<SCAN_THREADS>(s, &total, tmp);
        if (threadIdx.x == 0) block_sums[b] = total;
    }
}

// one small block (it has to fit next to whatever else is resident): exclusive scan of block_sums[0..nblk) in place;
// the grand total goes to *total_out
constexpr int BSUM_THREADS = 256;
__global__ void __launch_bounds__(BSUM_THREADS)
k_scan_block_sums(uint32_t* __restrict__ block_sums, const uint32_t* __restrict__ n_ptr, uint32_t tile,
                  uint32_t* __restrict__ total_out) {
    __shared__ uint32_t tmp[BSUM_THREADS / 32 + 1];
    const uint32_t n = *n_ptr;
    const uint32_t nblk = (n + tile - 1) / tile;
    uint32_t carry = 0;
    for (uint32_t base = 0; base < nblk; base += BSUM_THREADS * 4) {
        const uint32_t i = base + threadIdx.x * 4;
        uint32_t v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = i + q < nblk ? block_sums[i + q] : 0;
        uint32_t total;
        uint32_t ex = carry + block_exclusive_scan<BSUM_THREADS>(v[0] + v[1] + v[2] + v[3], &total, tmp);
#pragma unroll
        for (int q = 0; q < 4; ++q) { if (i + q < nblk) block_sums[i + q] = ex; ex += v[q]; }
        carry += total;
    }
    if (threadIdx.x == 0 && total_out) *total_out = carry;
}

__global__ void __launch_bounds__(SCAN_THREADS)
k_scan_apply(uint32_t* __restrict__ data, const uint32_t* __restrict__ n_ptr, const uint32_t* __restrict__ block_sums) {
    __shared__ uint32_t tmp[SCAN_THREADS / 32 + 1];
    const uint32_t n = *n_ptr;
    const uint32_t nblk = (n + SCAN_TILE - 1) / SCAN_TILE;
    for (uint32_t b = blockIdx.x; b < nblk; b += gridDim.x) {
        uint32_t v[SCAN_ITEMS];
        uint32_t s = 0;
        const uint32_t base = b * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
#pragma unroll
        for (int i = 0; i < SCAN_ITEMS; ++i) { v[i] = base + i < n ? data[base + i] : 0; s += v[i]; }
        uint32_t total;
        uint32_t ex = block_exclusive_scan<SCAN_THREADS>(s, &total, tmp) + block_sums[b];
#pragma unroll
        for (int i = 0; i < SCAN_ITEMS; ++i) { if (base + i < n) data[base + i] = ex; ex += v[i]; }
    }
}

// short arrays: the whole exclusive scan in one block and one launch (in place)
constexpr int SCAN1_THREADS = 512;
constexpr int SCAN1_ITEMS = 8;
constexpr int64_t SCAN1_MAX = 32768;
__global__ void __launch_bounds__(SCAN1_THREADS)
k_scan_single(uint32_t* __restrict__ data, const uint32_t* __restrict__ n_ptr) {
    __shared__ uint32_t tmp[SCAN1_THREADS / 32 + 1];
    const uint32_t n = *n_ptr;
    uint32_t carry = 0;
    for (uint32_t base = 0; base < n; base += SCAN1_THREADS * SCAN1_ITEMS) {
        const uint32_t i = base + threadIdx.x * SCAN1_ITEMS;
        uint32_t v[SCAN1_ITEMS], sum = 0;
#pragma unroll
        for (int q = 0; q < SCAN1_ITEMS; ++q) { v[q] = i + q < n ? data[i + q] : 0; sum += v[q]; }
        uint32_t total;
        uint32_t ex = carry + block_exclusive_scan<SCAN1_THREADS>(sum, &total, tmp);
#pragma unroll
        for (int q = 0; q < SCAN1_ITEMS; ++q) { if (i + q < n) data[i + q] = ex; ex += v[q]; }
        carry += total;
    }
}

}  // namespace mpe

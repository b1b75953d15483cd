// Segmented stable LSD radix sort and device-wide prefix sums.
//
// The batch's indices arrive grouped by table, so sorting "by (table, row)"
// (Section 5.1: sort the row indices of the mini-batch, then merge duplicates)
// only has to order the rows inside each table's segment.  Every pass sorts by
// an 8-bit digit with per-(table, digit, tile) counters, so one pass over the
// whole array sorts all segments at once and never moves a key out of its
// segment.  No kernel here waits on another block: a pass is histogram ->
// offsets (one block per table) -> scatter, three ordinary launches.  A tile is 4096 elements:
// 16 per thread, ranked by warp (match on the digit, warp-private counters),
// reordered through shared memory so that global writes are runs.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mpe {

#ifndef MPE_SORT_MINB
#define MPE_SORT_MINB 4        // resident blocks per SM the scatter kernel is compiled for
#endif
constexpr int SORT_THREADS = 256;
// Keys per thread of the scatter kernel, hence keys per tile: 16 (4096-key tiles) for large batches, where the fixed cost
// of a tile is spread over more keys and a digit's run is longer; 8 (2048-key tiles) for batches so small that larger
// tiles would leave SMs without a tile.  The tile size of a sort travels as an argument.
constexpr int SORT_ITEMS_LARGE = 16, SORT_ITEMS_SMALL = 8;
constexpr int SORT_TILE_MAX = SORT_THREADS * SORT_ITEMS_LARGE;
__host__ __device__ constexpr int sort_tile(bool small) { return SORT_THREADS * (small ? SORT_ITEMS_SMALL : SORT_ITEMS_LARGE); }
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
// tile_base[t] = number of tiles (of `tile` keys) of segments 0..t-1; tile_base[T] = total.  Called by one warp whose
// lanes all take part; `off` (the step was abandoned) yields zero tiles, which turns the whole sort into a no-op.
__device__ __forceinline__ void warp_tile_bases(const int32_t* seg_start, int T, int32_t* tile_base, bool off, int tile) {
    const int lane = threadIdx.x & 31;
    int32_t run = 0;
    for (int t0 = 0; t0 < T; t0 += 32) {
        const int t = t0 + lane;
        const int32_t len = (t < T && !off) ? seg_start[t + 1] - seg_start[t] : 0;
        const int32_t c = (len + tile - 1) / tile;
        int32_t inc = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int32_t v = __shfl_up_sync(0xffffffffU, inc, o); if (lane >= o) inc += v; }
        if (t < T) tile_base[t] = run + inc - c;
        run += __shfl_sync(0xffffffffU, inc, 31);
    }
    if (lane == 0) tile_base[T] = run;
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
            int T, int shift, uint32_t* __restrict__ hist, int tile_keys) {
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
        const int32_t start = seg_start[t] + local * tile_keys;
        const int32_t end = min(start + tile_keys, seg_start[t + 1]);
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

// ---- pass 2 of 3: counts -> first global position of every (table, digit, tile) ----------------
// One block per table.  The counts of table t sit as 256 rows (one per digit value) of nt tiles; the first key of
// (digit d, tile j) goes to  seg_start[t] + (all keys of the table with a smaller digit) + (keys with digit d in the
// tiles before j).  A warp takes rows d = warp, warp + 32, ...: an exclusive prefix sum along the row, the row totals
// to shared memory, then the prefix sum over the 256 totals, then the rows again to add their base.
constexpr int OFFS_THREADS = 1024;
constexpr int OFFS_SMALL_NT = 32;        // up to this many tiles in a table: one thread per digit value
__global__ void __launch_bounds__(OFFS_THREADS)
k_sort_offsets(uint32_t* __restrict__ hist, const int32_t* __restrict__ seg_start, const int32_t* __restrict__ tile_base, int T) {
    __shared__ uint32_t total[256];
    __shared__ uint32_t scan_tmp[OFFS_THREADS / 32 + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int t = blockIdx.x; t < T; t += gridDim.x) {
        const int nt = tile_base[t + 1] - tile_base[t];
        if (nt == 0) continue;                                   // block-uniform
        uint32_t* __restrict__ rows = hist + (size_t)256 * tile_base[t];
        if (nt <= OFFS_SMALL_NT) {
            // few tiles: one thread per digit value walks its row (eight loads in flight at a time)
            uint32_t* __restrict__ row = rows + (size_t)threadIdx.x * nt;
            uint32_t sum = 0;
            if (threadIdx.x < 256) {
                for (int j0 = 0; j0 < nt; j0 += 8) {
                    uint32_t v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) v[q] = j0 + q < nt ? row[j0 + q] : 0u;
#pragma unroll
                    for (int q = 0; q < 8; ++q) { if (j0 + q < nt) row[j0 + q] = sum; sum += v[q]; }
                }
            }
            uint32_t all;
            const uint32_t base = block_exclusive_scan<OFFS_THREADS>(threadIdx.x < 256 ? sum : 0u, &all, scan_tmp) + (uint32_t)seg_start[t];
            if (threadIdx.x < 256) {
                for (int j0 = 0; j0 < nt; j0 += 8) {
                    uint32_t v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) v[q] = j0 + q < nt ? row[j0 + q] : 0u;
#pragma unroll
                    for (int q = 0; q < 8; ++q) if (j0 + q < nt) row[j0 + q] = v[q] + base;
                }
            }
            continue;
        }
        for (int d = warp; d < 256; d += OFFS_THREADS / 32) {
            uint32_t* __restrict__ row = rows + (size_t)d * nt;
            uint32_t carry = 0;
            for (int j0 = 0; j0 < nt; j0 += 32) {
                const uint32_t v = j0 + lane < nt ? row[j0 + lane] : 0u;
                uint32_t inc = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const uint32_t n = __shfl_up_sync(0xffffffffU, inc, o); if (lane >= o) inc += n; }
                if (j0 + lane < nt) row[j0 + lane] = carry + inc - v;
                carry += __shfl_sync(0xffffffffU, inc, 31);
            }
            if (lane == 0) total[d] = carry;
        }
        __syncthreads();
        uint32_t all;
        const uint32_t mine = threadIdx.x < 256 ? total[threadIdx.x] : 0u;
        const uint32_t ex = block_exclusive_scan<OFFS_THREADS>(mine, &all, scan_tmp);
        if (threadIdx.x < 256) total[threadIdx.x] = ex + (uint32_t)seg_start[t];
        __syncthreads();
        for (int d = warp; d < 256; d += OFFS_THREADS / 32) {
            uint32_t* __restrict__ row = rows + (size_t)d * nt;
            const uint32_t base = total[d];
            for (int j = lane; j < nt; j += 32) row[j] += base;
        }
        __syncthreads();
    }
}

// ---- pass 3 of 3: stable scatter ------------------------------------------------
// Between passes an element travels as one 8-byte (key, payload) record, so a pass reads and writes it with one
// instruction each and a digit's run of a tile is one contiguous piece of memory.
// FIRST: the input is the bare key array and the payload is the element's position.
// LAST: the output is split into the sorted keys and the sorted payloads (out_keys / out_vals), which is what the
// kernels after the sort read.
template <bool FIRST, bool LAST, int SORT_ITEMS>
__global__ void __launch_bounds__(SORT_THREADS, MPE_SORT_MINB)
k_sort_scatter(const uint32_t* __restrict__ keys_in, const uint2* __restrict__ pairs_in, uint2* __restrict__ pairs_out,
               uint32_t* __restrict__ out_keys, uint32_t* __restrict__ out_vals,
               const int32_t* __restrict__ seg_start, const int32_t* __restrict__ tile_base, int T, int shift,
               const uint32_t* __restrict__ hist_scanned) {
    constexpr int WARPS = SORT_THREADS / 32;
    constexpr int SORT_TILE = SORT_THREADS * SORT_ITEMS;
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

// ---- prefix sum over per-block counts (the compactions of the step: distinct rows, admission candidates) ----
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

}  // namespace mpe

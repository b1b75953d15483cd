// Segmented stable LSD radix sort, and what a single-pass kernel needs to order its tiles.
//
// The batch's indices arrive grouped by table, so sorting "by (table, row)"
// (Section 5.1: sort the row indices of the mini-batch, then merge duplicates)
// only has to order the rows inside each table's segment.  Every pass sorts by
// an 8-bit digit with per-(table, digit, tile) counters, so one pass over the
// whole array sorts all segments at once and never moves a key out of its
// segment.  One kernel counts the digits of all passes; then a pass is one
// kernel whose tiles learn their output positions from the tiles before them
// (bounded look-back over per-tile words).  A tile is 4096 or 2048 elements:
// 16 or 8 per thread, ranked by warp (match on the digit, warp-private counters),
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

// ---- what one tile tells the tiles behind it ------------------------------------------------
// A pass hands its tiles out in order (a ticket counter), so a tile's predecessors are always held by blocks that are
// running.  For each of the 256 digit values a tile publishes one 8-byte word: first how many of its keys have that digit
// (an "aggregate"), later where its successor's keys of that digit begin (a "prefix").  A tile finds where its own keys
// begin by walking back over its predecessors' words, adding aggregates until it meets a prefix.  The words carry a tag
// that changes with every pass, so the array is never cleared: a word with another tag is simply not there yet.
// Every wait is bounded: a tile that gives up poisons what it publishes, the tiles behind it write nothing, and the
// step is abandoned with a sticky error.
constexpr int SORT_MAX_PASSES = 4;
struct SortCtl {
    uint32_t seq;        // passes completed on this workspace; pass tags are seq + 1
    uint32_t ticket;     // next tile to hand out; the block that draws the last ticket of a pass puts it back to 0
    uint32_t timeout;    // sticky: look-backs that gave up
    uint32_t done;       // blocks that have finished the current pass
};
constexpr uint32_t SORT_TAG_MASK = 0x3fffffffU;
constexpr unsigned long long SORT_PREFIX = 1ULL << 32, SORT_POISON = 1ULL << 33;
constexpr int SORT_LOOK = 4;                  // predecessors' words a look-back fetches at a time
constexpr int SORT_POLL_LIMIT = 1 << 22;      // polls of one word before a look-back gives up (about a second)
__device__ __forceinline__ unsigned long long sort_word(uint32_t tag, unsigned long long flags, uint32_t value) {
    return ((unsigned long long)tag << 34) | flags | value;
}
__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// Hands the calling block its next tile (all threads call); false when none is left.
// Tickets are drawn when the block is ready for the tile, never ahead of time: the tiles behind a ticket wait for its tile.
__device__ __forceinline__ bool draw_tile(SortCtl* ctl, uint32_t ntiles, uint32_t* s_turn /* [2], shared */, uint32_t* tile, uint32_t* tag) {
    __syncthreads();
    if (threadIdx.x == 0) { s_turn[0] = atomicAdd(&ctl->ticket, 1u); s_turn[1] = (ctl->seq + 1u) & SORT_TAG_MASK; }
    __syncthreads();
    *tile = s_turn[0]; *tag = s_turn[1];
    return *tile < ntiles;
}
// After its last draw: true in exactly one block of the grid, the last one to get here.  Every other block's writes are
// visible to that block (through L2: read them with __ldcg), which ends the pass with close_pass() when it is done.
__device__ __forceinline__ bool last_block_of_pass(SortCtl* ctl, uint32_t* s_turn) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_turn[0] = atomicAdd(&ctl->done, 1u);
    __syncthreads();
    return s_turn[0] == gridDim.x - 1u;
}
__device__ __forceinline__ void close_pass(SortCtl* ctl, uint32_t tag) {
    if (threadIdx.x == 0) { ctl->ticket = 0; ctl->done = 0; ctl->seq = tag; }
}

// One word per tile (the compactions).  tile_publish (one thread): how many items the tile holds, as soon as it is known.
// tile_look_back (one whole warp, any time later): the sum of `total` over the tiles before `tile`, reading 32 predecessors'
// words at a time; it leaves the tile's prefix in its word.
__device__ __forceinline__ void tile_publish(unsigned long long* words, uint32_t tile, uint32_t total, uint32_t tag) {
    st_relaxed_u64(words + tile, sort_word(tag, tile == 0 ? SORT_PREFIX : 0ULL, total));
}
__device__ __forceinline__ uint32_t tile_look_back(unsigned long long* words, uint32_t tile, uint32_t total, uint32_t tag, bool* poison,
                                                   int poll_limit = SORT_POLL_LIMIT) {
    const int lane = threadIdx.x & 31;
    uint32_t sum = 0;
    bool bad = false;
    if (tile > 0) {
        for (int64_t base = (int64_t)tile - 1;; base -= 32) {
            const int64_t j = base - lane;
            unsigned long long v = sort_word(tag, SORT_PREFIX, 0);            // before the first tile: nothing
            if (j >= 0) {
                v = ld_relaxed_u64(words + j);
                for (int polls = 0; (uint32_t)(v >> 34) != tag; v = ld_relaxed_u64(words + j)) {
                    if (++polls > poll_limit) { v = SORT_PREFIX | SORT_POISON; break; }
                    if (polls > 32) __nanosleep(200);
                }
            }
            const uint32_t pm = __ballot_sync(0xffffffffU, (v & SORT_PREFIX) != 0);
            const int stop = pm ? __ffs(pm) - 1 : 31;                          // nearest predecessor that knows its prefix
            sum += __reduce_add_sync(0xffffffffU, lane <= stop ? (uint32_t)v : 0u);
            bad |= __any_sync(0xffffffffU, lane <= stop && (v & SORT_POISON) != 0);
            if (pm) break;
        }
        if (lane == 0) st_relaxed_u64(words + tile, sort_word(tag, SORT_PREFIX | (bad ? SORT_POISON : 0ULL), sum + total));
    }
    *poison = bad;
    return sum;
}

// Sum of what the `left` tiles before the one that owns `word` hold of this thread's digit, plus where the first of them
// begins: walks back over their words until it meets a prefix.
__device__ __forceinline__ uint32_t sort_look_back(const unsigned long long* word, int left, uint32_t tag, bool* poison) {
    uint32_t sum = 0;
    bool bad = false;
    const unsigned long long* q = word - 256;
    for (bool done = false; !done;) {
        // several predecessors' words are fetched at once and then read in order, nearest first
        unsigned long long v[SORT_LOOK];
#pragma unroll
        for (int u = 0; u < SORT_LOOK; ++u) v[u] = u < left ? ld_relaxed_u64(q - 256 * u) : 0ULL;
#pragma unroll
        for (int u = 0; u < SORT_LOOK; ++u) {
            if (done) break;
            for (int polls = 0; (uint32_t)(v[u] >> 34) != tag; v[u] = ld_relaxed_u64(q - 256 * u)) {
                if (++polls > SORT_POLL_LIMIT) { v[u] = SORT_PREFIX | SORT_POISON; break; }
                if (polls > 32) __nanosleep(200);
            }
            sum += (uint32_t)v[u];
            bad |= (v[u] & SORT_POISON) != 0;
            done = (v[u] & SORT_PREFIX) != 0;
        }
        q -= 256 * SORT_LOOK; left -= SORT_LOOK;
    }
    *poison = bad;
    return sum;
}

// ---- before the passes: how many keys of each table have each digit value, for every pass at once ----
// The counts do not depend on the order of the keys, so one read of the unsorted keys serves all passes.
// ghist[t][pass][digit] must be zero on entry; the pass that uses a row of it clears it again, and a pass that finds the
// step abandoned clears all of its rows.
// PAIRS: the keys are the .x members of (key, payload) records
template <bool PAIRS>
__global__ void __launch_bounds__(SORT_THREADS)
k_sort_digits(const uint32_t* __restrict__ keys, const int32_t* __restrict__ seg_start, const int32_t* __restrict__ tile_base,
              int T, int passes, uint32_t* __restrict__ ghist, int tile_keys, int split) {
    // one warp per piece of a tile (`split` pieces per tile: whole tiles in large steps, where the cost of emptying the
    // counters wants many keys to spread over; quarters in small steps, where whole tiles would leave most SMs idle):
    // its own counters, eight key loads in flight per lane, no block-wide barrier
    constexpr int WARPS = SORT_THREADS / 32;
    constexpr int STRIDE = PAIRS ? 2 : 1;
    __shared__ uint32_t cnt[WARPS][SORT_MAX_PASSES * 256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int npieces = tile_base[T] * split;
    const int piece_keys = tile_keys / split;
    for (int piece = blockIdx.x * WARPS + warp; piece < npieces; piece += gridDim.x * WARPS) {
        const int tile = piece / split;
        const int t = find_segment(tile_base, T, tile);
        const int local = tile - tile_base[t];
        const int32_t start = seg_start[t] + local * tile_keys + (piece - tile * split) * piece_keys;
        const int32_t end = min(start + piece_keys, seg_start[t + 1]);
        if (start >= end) continue;                    // warp-uniform: the table's last tile is not full
        for (int i = lane; i < passes * 256; i += 32) cnt[warp][i] = 0;
        __syncwarp();
        for (int32_t i0 = start + lane; i0 < end; i0 += 32 * 8) {
            uint32_t k[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) k[q] = i0 + 32 * q < end ? keys[(size_t)(i0 + 32 * q) * STRIDE] : 0u;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (i0 + 32 * q < end)
                    for (int p = 0; p < passes; ++p) atomicAdd(&cnt[warp][p * 256 + ((k[q] >> (8 * p)) & 255u)], 1u);
        }
        __syncwarp();
        uint32_t* out = ghist + (size_t)t * (SORT_MAX_PASSES * 256);
        for (int i = lane; i < passes * 256; i += 32) {
            const uint32_t c = cnt[warp][i];
            if (c) atomicAdd(out + i, c);
        }
        __syncwarp();
    }
}

// ---- one pass: stable scatter ---------------------------------------------------
// Between passes an element travels as one 8-byte (key, payload) record, so a pass reads and writes it with one
// instruction each and a digit's run of a tile is one contiguous piece of memory.
// FIRST: the input is the bare key array and the payload is the element's position.
// LAST: the output is split into the sorted keys and the sorted payloads (out_keys / out_vals), which is what the
// kernels after the sort read.
template <bool FIRST, bool LAST, int SORT_ITEMS>
__global__ void __launch_bounds__(SORT_THREADS, MPE_SORT_MINB)
k_sort_scatter(const uint32_t* __restrict__ keys_in, const uint2* __restrict__ pairs_in, uint2* __restrict__ pairs_out,
               uint32_t* __restrict__ out_keys, uint32_t* __restrict__ out_vals,
               const int32_t* __restrict__ seg_start, const int32_t* __restrict__ tile_base, int T, int pass,
               uint32_t* __restrict__ ghist, unsigned long long* __restrict__ status, SortCtl* __restrict__ ctl,
               uint32_t* __restrict__ abort_flag) {
    constexpr int WARPS = SORT_THREADS / 32;
    constexpr int SORT_TILE = SORT_THREADS * SORT_ITEMS;
    __shared__ uint32_t wcnt[WARPS][256];      // per-warp digit counters, then tile-local position of the warp's first key of each digit
    __shared__ uint32_t goff[256];             // first global position of each digit of this tile minus its tile-local start
    __shared__ uint2 skv[SORT_TILE];
    __shared__ uint32_t scan_tmp[SORT_THREADS / 32 + 1];
    __shared__ uint32_t s_ticket[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t lt = (1u << lane) - 1u;
    const bool off = *abort_flag != 0;          // the step was abandoned before this pass: nothing to sort
    const int ntiles = off ? 0 : tile_base[T];
    const int shift = 8 * pass;
    volatile uint32_t* myc = wcnt[warp];
    for (;;) {
        uint32_t ticket, tag;
        if (!draw_tile(ctl, (uint32_t)ntiles, s_ticket, &ticket, &tag)) {
            // every block draws one ticket too many; the block that draws the last of those ends the pass
            if (ticket == (uint32_t)ntiles + gridDim.x - 1u) {
                if (off)            // the digit counts of this pass were never used: they must not meet the next step's
                    for (int i = threadIdx.x; i < T * 256; i += SORT_THREADS) ghist[((size_t)(i >> 8) * SORT_MAX_PASSES + pass) * 256 + (i & 255)] = 0;
                close_pass(ctl, tag);
            }
            break;
        }
        const int tile = (int)ticket;
        const int t = find_segment(tile_base, T, tile);
        const int local = tile - tile_base[t];
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
        // tell the tiles behind this one how many keys of digit d it holds, as early as possible
        unsigned long long* word = status + (size_t)tile * 256 + threadIdx.x;
        if (local != 0) st_relaxed_u64(word, sort_word(tag, 0, tot));
        uint32_t all;
        const uint32_t ds = block_exclusive_scan<SORT_THREADS>(tot, &all, scan_tmp);
        uint32_t run = ds;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) {                                      // tile-local position of warp w's first key with this digit
            const uint32_t c = wcnt[w][threadIdx.x];
            wcnt[w][threadIdx.x] = run;
            run += c;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < SORT_ITEMS; ++i) {
            const uint32_t dg = (key[i] >> shift) & 255u;
            const uint32_t r = (i & 1) ? rank[i >> 1] >> 16 : rank[i >> 1] & 0xffffu;
            skv[wcnt[warp][dg] + r] = make_uint2(key[i], val[i]);
        }
        // where this tile's keys of digit d begin in the output (the tile is in order in shared memory by now, so the
        // waiting is done with nothing else left to do)
        uint32_t gb;
        bool poison = false;
        if (local == 0) {
            // first tile of its table: the table's start plus its keys with a smaller digit
            uint32_t* g = ghist + ((size_t)t * SORT_MAX_PASSES + pass) * 256 + threadIdx.x;
            const uint32_t mine = *g;
            *g = 0;
            gb = (uint32_t)seg_start[t] + block_exclusive_scan<SORT_THREADS>(mine, &all, scan_tmp);
        } else {
            gb = sort_look_back(word, local, tag, &poison);
        }
        st_relaxed_u64(word, sort_word(tag, SORT_PREFIX | (poison ? SORT_POISON : 0ULL), gb + tot));
        goff[threadIdx.x] = gb - ds;                                           // global position = goff + tile-local position
        if (__syncthreads_or(poison)) {                                        // a look-back gave up: write nothing, abandon the step
            if (threadIdx.x == 0) { atomicAdd(&ctl->timeout, 1u); *abort_flag = 1; }
            continue;
        }
        // padding keys follow every real key of the tile, so positions [0,count) are real
        for (int j = threadIdx.x; j < count; j += SORT_THREADS) {
            const uint2 kv = skv[j];
            const uint32_t dst = goff[(kv.x >> shift) & 255u] + (uint32_t)j;
            if (LAST) { out_keys[dst] = kv.x; out_vals[dst] = kv.y; }
            else pairs_out[dst] = kv;
        }
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

// ---- self-check of the bounded wait ----------------------------------------------------------
// One warp plays tile 1 of a pass whose tile 0 belongs to nobody, with the wait cut to a few thousand polls (about a
// millisecond): the look-back has to give up and say so.  The pass number moves on afterwards, so the word it leaves
// can never be taken for one of a real pass.
__global__ void k_selftest_look_back(unsigned long long* words, SortCtl* ctl) {
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    const uint32_t tag = (ctl->seq + 1u) & SORT_TAG_MASK;
    bool poison = false;
    tile_look_back(words, 1u, 0u, tag, &poison, 4096);
    if (threadIdx.x == 0) {
        if (poison) atomicAdd(&ctl->timeout, 1u);
        ctl->seq = tag;
    }
}

}  // namespace mpe

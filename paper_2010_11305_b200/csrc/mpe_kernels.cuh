// Kernels of the training step.  Naming follows the paper: T = low-precision
// table, C = FP32 cache, I_C = tags, PV = priority values, I_U = distinct rows
// of the batch (Section 3, Algorithm 2, Section 5.1).
#pragma once
#include "mpe_device.cuh"
#include "mpe_sort.cuh"

namespace mpe {

constexpr int HOT_SPAN = 1024;        // occurrences covered by one multi-block gradient task (two tree levels)
constexpr int HOT_MIN = 256;          // rows with more occurrences than this take the multi-block path
// A step with few distinct rows has few warps' worth of work in k_update, and its duration is that of the warp with the
// longest rows: there the multi-block path starts earlier.
constexpr int HOT_MIN_SMALL = 64;
constexpr int HOT_SMALL_U = 131072;   // "few": at most this many distinct rows
// upper bound of the number of hot rows, and of their tasks, in a step of L indices (either threshold)
__host__ __device__ constexpr int64_t hot_capacity(int64_t L) {
    return (L / HOT_MIN_SMALL < HOT_SMALL_U ? L / HOT_MIN_SMALL : HOT_SMALL_U) + L / HOT_MIN + L / HOT_SPAN + 4;
}
constexpr int ERR_INDEX = 0, ERR_OFFSETS = 1;

struct TableDev {
    int64_t row_base;    // first row of this table in the concatenated store
    int64_t set_base;    // first set of this table in the concatenated cache
    int32_t N;           // rows
    int32_t n_sets;      // cache sets (0 = no cache)
    uint32_t salt;       // of the set hash
    int32_t pad;
};

struct Counters {
    uint32_t L;            // indices in this batch
    uint32_t U;            // distinct (table,row) pairs incl. one pseudo row per table that had bad indices
    uint32_t unused0, unused1;
    uint32_t hot_rows;
    uint32_t hot_tasks;
    uint32_t abort;        // offsets were inconsistent: every later kernel of the step returns at once
    uint32_t deferred;     // newcomers that wait for the write-back of an updated row
    uint32_t n_heads;      // cache sets that have miss candidates in this step
    uint32_t upd_next;     // next block of 32 distinct rows to hand to a warp of k_update
    uint32_t n_cand;       // candidates for admission in this step
    unsigned long long dropped;      // out-of-range indices in this batch
    unsigned long long hot_occ;      // indices that belong to hot rows
    unsigned long long err[2];       // sticky: ERR_INDEX, ERR_OFFSETS
};

struct State {
    int T, dim, lanes, ways, policy, optimizer, bits;
    int rounding;          // how rows are down-converted while training: 1 stochastic (default), 0 nearest-even
    uint64_t seed;
    float eps;
    const TableDev* tables;
    uint8_t* codes;        // [sum N][dim*bits/8]
    float2* sb;            // [sum N] (scale, bias)
    uint32_t* cnt;         // LFU: [sum N]
    float* G;              // Adagrad: [sum N]
    float* slab;           // [slots][dim]
    int32_t* tags;         // [slots], -1 empty
    uint32_t* ts;          // [slots] priority value of the resident row: LRU time stamp, or a copy of its LFU count
    uint32_t* hit_epoch;   // [slots] forward call in which the slot was last hit
    int32_t* hit_k;        // [slots] unique-row index of that hit
    uint32_t* floor;       // [sets] a lower bound of the lowest priority value among the set's residents (0: none known)
    unsigned long long* stats;   // [T][8]
};

// What changes from call to call.  It lives in device memory so that a captured CUDA graph of the step stays valid:
// the kernels read it, one tiny kernel at the head of the graph writes it.
// Destination of the pooled vectors when the tables are partitioned over several GPUs (Section 1: model parallelism
// with no replication): sample b belongs to rank b / B_local, whose buffer is [B_local][T_global * dim].
constexpr int MAX_RANKS = 72;
struct Route {
    float* out[MAX_RANKS];
    int32_t B_local, T_global, t_base, n_ranks;
};

struct StepArgs {
    const int32_t* indices; const int32_t* offsets; float* out; const float* grad;
    int32_t B; uint32_t L; uint32_t epoch; float lr;
    unsigned long long step;
    const Route* route;      // null: out is one [B][T * dim] array on this GPU
};

struct Work {
    Counters* ctr;
    StepArgs* args;
    int32_t *table_start, *tile_base, *ustart, *ctile_base;   // [T+1]
    int32_t* bag_of;       // [L] bag of every index position
    uint32_t* kidx;        // [L] unique-row index of the i-th sorted element
    int32_t* occ_loc;      // [L] by position: cache slot, LOC_MISS or LOC_INVALID
    int32_t* occ_b;        // [L] by sorted order: sample of the element; sign bit: last occurrence of its row
    int32_t *uniq_row, *uniq_t, *seg, *loc, *final_loc, *victim, *hot_base, *uset;   // per unique row
    int32_t* task_k;       // [hot tasks]
    int32_t* hot_k;        // [hot rows]
    uint32_t* cand_key;    // [distinct rows] large steps: the row's set if it is a candidate for admission, else the table's number of sets
    int32_t* cand_cnt;     // [T] candidates of each table (counted by k_priority, cleared once the candidates' segments are known)
    int32_t* cstart;       // [T+1] where each table's candidates begin in the compacted candidate list
    int32_t* defer_k;      // [deferred newcomers]
    int32_t* heads;        // [sets with candidates] position of the set's first candidate in the set-sorted list
    float* partial;        // [hot tasks][dim]
    int32_t sort_tile;     // keys per tile of the sorts of this workspace
};

// ---------------------------------------------------------------------------------------------
// step prologue
// ---------------------------------------------------------------------------------------------
__global__ void k_set_route(Route* dst, Route r) {
    for (int g = threadIdx.x; g < MAX_RANKS; g += blockDim.x) dst->out[g] = r.out[g];
    if (threadIdx.x == 0) { dst->B_local = r.B_local; dst->T_global = r.T_global; dst->t_base = r.t_base; dst->n_ranks = r.n_ranks; }
}
__global__ void k_set_args_backward(StepArgs* a, const float* grad, float lr, unsigned long long step) {
    a->grad = grad; a->lr = lr; a->step = step;
}

// one warp: resets the step's counters and reads where each table's bags begin (the offsets of bags 0, B, 2B, ...), 32
// tables at a time so that the loads overlap; offsets that do not start at 0, end at L or grow abandon the step
// In a replayed step this is the graph's first kernel and the one whose parameters change from call to call: it passes the
// forward's arguments on to the kernels behind it through the block in device memory.
template <bool IND>
__global__ void k_prelude(Work w, int T, StepArgs av) {
    const StepArgs a = av;
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    if (IND && lane == 0) {
        StepArgs* d = w.args;
        d->indices = a.indices; d->offsets = a.offsets; d->out = a.out; d->B = a.B; d->L = a.L; d->epoch = a.epoch; d->route = a.route;
    }
    const int32_t* __restrict__ offsets = a.offsets;
    const int B = a.B;
    const uint32_t L = a.L;
    Counters* c = w.ctr;
    if (lane == 0) {
        c->L = L; c->U = 0; c->hot_rows = 0; c->hot_tasks = 0; c->abort = 0; c->dropped = 0; c->hot_occ = 0; c->deferred = 0; c->n_heads = 0; c->upd_next = 0;
    }
    bool bad = false;
    for (int t0 = 0; t0 <= T; t0 += 32) {
        const int t = t0 + lane;
        if (t <= T) {
            const int32_t v = offsets[(int64_t)t * B];
            const int32_t before = t > 0 ? offsets[(int64_t)(t - 1) * B] : 0;
            if (v < before || v < 0 || v > (int32_t)L || (t == 0 && v != 0) || (t == T && v != (int32_t)L)) bad = true;
            w.table_start[t] = v;
        }
    }
    bad = __any_sync(0xffffffffU, bad);
    if (bad) {                                   // nothing downstream may trust the offsets: every table is empty
        for (int t = lane; t <= T; t += 32) w.table_start[t] = t == T ? (int32_t)L : 0;
        if (lane == 0) { c->abort = 1; atomicAdd(&c->err[ERR_OFFSETS], 1ULL); }
    }
    __syncwarp();
    warp_tile_bases(w.table_start, T, w.tile_base, bad, w.sort_tile);     // the sort's tiles, table by table
}

// keys for the sort: the row id, or N_t for an id outside [0, N_t); eight lanes per bag, four bags per warp
template <bool IND>
__global__ void __launch_bounds__(256)
k_make_keys(State s, Work w, uint32_t* __restrict__ keys, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    const int32_t* __restrict__ indices = a.indices;
    const int32_t* __restrict__ offsets = a.offsets;
    const int B = a.B;
    const int sub = threadIdx.x & 7;
    const int64_t nbags = (int64_t)s.T * B;
    const int64_t ng = (int64_t)gridDim.x * (blockDim.x >> 3);
    const int32_t L = (int32_t)w.ctr->L;
    int64_t bag = (int64_t)blockIdx.x * (blockDim.x >> 3) + (threadIdx.x >> 3);
    int t = (int)(bag / B);
    int64_t b = bag - (int64_t)t * B;
    unsigned long long bad = 0;
    for (; bag < nbags; bag += ng) {
        const int32_t lo = offsets[bag], hi = offsets[bag + 1];
        if (lo < 0 || hi < lo || hi > L) {
            if (sub == 0) { w.ctr->abort = 1; atomicAdd(&w.ctr->err[ERR_OFFSETS], 1ULL); }
        } else {
            const int32_t N = s.tables[t].N;
            for (int32_t p = lo + sub; p < hi; p += 8) {
                const int32_t r = indices[p];
                const bool ok = r >= 0 && r < N;
                keys[p] = ok ? (uint32_t)r : (uint32_t)N;
                w.bag_of[p] = (int32_t)bag;
                bad += !ok;
            }
        }
        b += ng;
        while (b >= B) { b -= B; ++t; }
    }
    if (bad) { atomicAdd(&w.ctr->dropped, bad); atomicAdd(&w.ctr->err[ERR_INDEX], bad); }
}

// ---------------------------------------------------------------------------------------------
// distinct rows of the sorted batch (I_U), multiplicities, element -> distinct-row map
// ---------------------------------------------------------------------------------------------
// Small steps (the ones replayed from a graph, where every launch counts), one pass: a tile of the sorted batch flags the first element of every run of equal (table, row), learns how many
// distinct rows the tiles before it hold (look-back over one word per tile), and writes its part of the lists.  The block
// that ends the pass fills in where each table's distinct rows begin.
__global__ void __launch_bounds__(SCAN_THREADS)
k_unique(Work w, int T, const uint32_t* __restrict__ skey, unsigned long long* __restrict__ words, SortCtl* __restrict__ ctl) {
    __shared__ uint32_t tmp[SCAN_THREADS / 32 + 1];
    __shared__ uint32_t s_turn[2];
    __shared__ uint32_t s_prefix[2];
    const bool off = w.ctr->abort != 0;                 // an abandoned step has no tiles
    const uint32_t n = off ? 0u : w.ctr->L;
    const uint32_t nblk = (n + SCAN_TILE - 1) / SCAN_TILE;
    uint32_t b, tag;
    while (draw_tile(ctl, nblk, s_turn, &b, &tag)) {
        const uint32_t base = b * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
        uint32_t flag[SCAN_ITEMS];
        int tcur[SCAN_ITEMS];
        uint32_t sum = 0;
        uint32_t keyv[SCAN_ITEMS];
        if (base < n) {
            int t = find_segment(w.table_start, T, (int32_t)base);
            while (w.table_start[t + 1] <= (int32_t)base) ++t;     // skip empty tables that start here
            uint32_t prev = base > 0 ? skey[base - 1] : 0;
            if (base + SCAN_ITEMS <= n) {                           // 16 keys as four 16-byte loads
#pragma unroll
                for (int i = 0; i < SCAN_ITEMS; i += 4) {
                    const uint4 v = *reinterpret_cast<const uint4*>(skey + base + i);
                    keyv[i] = v.x; keyv[i + 1] = v.y; keyv[i + 2] = v.z; keyv[i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < SCAN_ITEMS; ++i) keyv[i] = base + i < n ? skey[base + i] : 0;
            }
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; ++i) {
                const uint32_t e = base + i;
                flag[i] = 0; tcur[i] = t;
                if (e < n) {
                    while (w.table_start[t + 1] <= (int32_t)e) ++t;
                    tcur[i] = t;
                    const uint32_t k = keyv[i];
                    flag[i] = (e == (uint32_t)w.table_start[t] || k != prev) ? 1u : 0u;
                    prev = k;
                    sum += flag[i];
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; ++i) { flag[i] = 0; tcur[i] = 0; keyv[i] = 0; }
        }
        uint32_t total;
        uint32_t ex = block_exclusive_scan<SCAN_THREADS>(sum, &total, tmp);
        if (threadIdx.x < 32) {
            if (threadIdx.x == 0) tile_publish(words, b, total, tag);
            bool poison;
            const uint32_t before = tile_look_back(words, b, total, tag, &poison);
            if (threadIdx.x == 0) { s_prefix[0] = before; s_prefix[1] = poison; }
        }
        __syncthreads();
        if (s_prefix[1]) {                                         // a look-back gave up: write nothing, abandon the step
            if (threadIdx.x == 0) { atomicAdd(&ctl->timeout, 1u); w.ctr->abort = 1; }
            continue;
        }
        ex += s_prefix[0];
        if (b == nblk - 1 && threadIdx.x == 0) w.ctr->U = s_prefix[0] + total;
        uint32_t kout[SCAN_ITEMS];
#pragma unroll
        for (int i = 0; i < SCAN_ITEMS; ++i) {
            const uint32_t e = base + i;
            ex += flag[i];
            kout[i] = ex - 1;
            if (e < n && flag[i]) { w.uniq_row[kout[i]] = (int32_t)keyv[i]; w.uniq_t[kout[i]] = tcur[i]; w.seg[kout[i]] = (int32_t)e; }
        }
        if (base + SCAN_ITEMS <= n) {
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; i += 4)
                *reinterpret_cast<uint4*>(w.kidx + base + i) = make_uint4(kout[i], kout[i + 1], kout[i + 2], kout[i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; ++i) if (base + i < n) w.kidx[base + i] = kout[i];
        }
    }
    if (last_block_of_pass(ctl, s_turn)) {
        // every tile is done and its results are visible: where each table's distinct rows begin, and the end mark
        if (!off && !__ldcg(&w.ctr->abort)) {
            const uint32_t U = __ldcg(&w.ctr->U);
            for (int t = threadIdx.x; t <= T; t += blockDim.x) {
                const int32_t s0 = w.table_start[t];
                w.ustart[t] = (uint32_t)s0 < n ? (int32_t)__ldcg(w.kidx + s0) : (int32_t)U;
            }
            if (threadIdx.x == 0) w.seg[U] = (int32_t)n;
        }
        close_pass(ctl, tag);
    }
}

// Large steps: the same in two passes over the sorted batch with a prefix sum over the tiles' counts between them
// (count, k_scan_block_sums, write), and one small kernel for the tables' starts; nothing waits for anything there.
template <bool WRITE>
__global__ void __launch_bounds__(SCAN_THREADS)
k_unique_pass(Work w, int T, const uint32_t* __restrict__ skey, uint32_t* __restrict__ block_sums) {
    __shared__ uint32_t tmp[SCAN_THREADS / 32 + 1];
    if (w.ctr->abort) return;
    const uint32_t n = w.ctr->L;
    const uint32_t nblk = (n + SCAN_TILE - 1) / SCAN_TILE;
    for (uint32_t b = blockIdx.x; b < nblk; b += gridDim.x) {
        const uint32_t base = b * SCAN_TILE + threadIdx.x * SCAN_ITEMS;
        uint32_t flag[SCAN_ITEMS];
        int tcur[SCAN_ITEMS];
        uint32_t sum = 0;
        uint32_t keyv[SCAN_ITEMS];
        if (base < n) {
            int t = find_segment(w.table_start, T, (int32_t)base);
            while (w.table_start[t + 1] <= (int32_t)base) ++t;     // skip empty tables that start here
            uint32_t prev = base > 0 ? skey[base - 1] : 0;
            if (base + SCAN_ITEMS <= n) {                           // 16 keys as four 16-byte loads
#pragma unroll
                for (int i = 0; i < SCAN_ITEMS; i += 4) {
                    const uint4 v = *reinterpret_cast<const uint4*>(skey + base + i);
                    keyv[i] = v.x; keyv[i + 1] = v.y; keyv[i + 2] = v.z; keyv[i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int i = 0; i < SCAN_ITEMS; ++i) keyv[i] = base + i < n ? skey[base + i] : 0;
            }
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; ++i) {
                const uint32_t e = base + i;
                flag[i] = 0; tcur[i] = t;
                if (e < n) {
                    while (w.table_start[t + 1] <= (int32_t)e) ++t;
                    tcur[i] = t;
                    const uint32_t k = keyv[i];
                    flag[i] = (e == (uint32_t)w.table_start[t] || k != prev) ? 1u : 0u;
                    prev = k;
                    sum += flag[i];
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; ++i) { flag[i] = 0; tcur[i] = 0; keyv[i] = 0; }
        }
        uint32_t total;
        uint32_t ex = block_exclusive_scan<SCAN_THREADS>(sum, &total, tmp);
        if (!WRITE) {
            if (threadIdx.x == 0) block_sums[b] = total;
        } else {
            ex += block_sums[b];
            uint32_t kout[SCAN_ITEMS];
#pragma unroll
            for (int i = 0; i < SCAN_ITEMS; ++i) {
                const uint32_t e = base + i;
                ex += flag[i];
                kout[i] = ex - 1;
                if (e < n && flag[i]) { w.uniq_row[kout[i]] = (int32_t)keyv[i]; w.uniq_t[kout[i]] = tcur[i]; w.seg[kout[i]] = (int32_t)e; }
            }
            if (base + SCAN_ITEMS <= n) {
#pragma unroll
                for (int i = 0; i < SCAN_ITEMS; i += 4)
                    *reinterpret_cast<uint4*>(w.kidx + base + i) = make_uint4(kout[i], kout[i + 1], kout[i + 2], kout[i + 3]);
            } else {
#pragma unroll
                for (int i = 0; i < SCAN_ITEMS; ++i) if (base + i < n) w.kidx[base + i] = kout[i];
            }
        }
    }
}

__global__ void k_ustart(Work w, int T) {
    if (w.ctr->abort) return;
    const uint32_t L = w.ctr->L, U = w.ctr->U;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t <= T; t += gridDim.x * blockDim.x) {
        const int32_t s = w.table_start[t];
        w.ustart[t] = (uint32_t)s < L ? (int32_t)w.kidx[s] : (int32_t)U;
        if (t == 0) w.seg[U] = (int32_t)L;
    }
}

// ---------------------------------------------------------------------------------------------
// cache tag lookup: one lane per distinct row, which reads the `ways` tags of the row's set (Section 3 "Cache Structure")
// ---------------------------------------------------------------------------------------------
template <bool IND>
__global__ void __launch_bounds__(256)
k_probe(State s, Work w, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    const uint32_t epoch = a.epoch;
    if (w.ctr->abort) return;
    const int ways = s.ways;
    const int lane = threadIdx.x & 31;
    const int64_t U = w.ctr->U;
    const uint32_t hot_min = U <= HOT_SMALL_U ? (uint32_t)HOT_MIN_SMALL : (uint32_t)HOT_MIN;
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t k0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32; k0 < U; k0 += nwarps * 32) {
        const int64_t k = k0 + lane;
        int32_t row = 0, set = 0, gset = -1;         // gset: index of the row's set in the concatenated cache, -1 = no probe
        int myloc = LOC_MISS;
        if (k < U) {
            const TableDev tb = s.tables[w.uniq_t[k]];
            row = w.uniq_row[k];
            if (row >= tb.N) myloc = LOC_INVALID;
            else if (tb.n_sets > 0) { set = set_of((uint32_t)row, tb.salt, tb.n_sets); gset = (int32_t)(tb.set_base + set); }
        }
        // every lane compares its own row with the tags of the row's set (contiguous: `ways` INT32, read 16 bytes at a
        // time with all loads in flight before any comparison); a set holds a row at most once
        if (gset >= 0) {
            const int32_t* __restrict__ tg = s.tags + (int64_t)gset * ways;
            int mw = -1;
            if (ways >= 4) {
                for (int w0 = 0; w0 < ways; w0 += 32) {
                    int4 t4[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        t4[j] = w0 + 4 * j < ways ? *reinterpret_cast<const int4*>(tg + w0 + 4 * j) : make_int4(-1, -1, -1, -1);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (t4[j].x == row) mw = w0 + 4 * j;
                        if (t4[j].y == row) mw = w0 + 4 * j + 1;
                        if (t4[j].z == row) mw = w0 + 4 * j + 2;
                        if (t4[j].w == row) mw = w0 + 4 * j + 3;
                    }
                }
            } else {
                for (int w0 = 0; w0 < ways; ++w0) if (tg[w0] == row) mw = w0;
            }
            if (mw >= 0) {
                const int64_t slot = (int64_t)gset * ways + mw;
                myloc = (int)slot;
                s.hit_epoch[slot] = epoch; s.hit_k[slot] = (int32_t)k;
            }
        }
        if (k < U) {
            w.loc[k] = myloc; w.final_loc[k] = myloc; w.uset[k] = set;
            // rows with very many occurrences get their gradient summed by whole blocks, HOT_SPAN occurrences per task
            int hb = -1;
            const uint32_t mult = (uint32_t)(w.seg[k + 1] - w.seg[k]);
            if (myloc != LOC_INVALID && mult > hot_min) {
                const uint32_t nt = (mult + HOT_SPAN - 1) / HOT_SPAN;
                hb = (int)atomicAdd(&w.ctr->hot_tasks, nt);
                w.hot_k[atomicAdd(&w.ctr->hot_rows, 1u)] = (int32_t)k;
                atomicAdd(&w.ctr->hot_occ, (unsigned long long)mult);
                for (uint32_t j = 0; j < nt; ++j) w.task_k[hb + j] = (int32_t)k;
            }
            w.hot_base[k] = hb;
        }
    }
}

// per sorted element: where its row lives (by index position) and which sample it belongs to
template <bool IND>
__global__ void __launch_bounds__(256)
k_broadcast(State s, Work w, const uint32_t* __restrict__ spos, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    if (w.ctr->abort) return;
    const int B = a.B;
    const int64_t L = w.ctr->L;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < L; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t k = w.kidx[i];
        const uint32_t p = spos[i];
        w.occ_loc[p] = w.loc[k];
        // the sign bit marks the last occurrence of a distinct row (sample ids are below 2^31)
        const bool last = i + 1 >= L || w.kidx[i + 1] != k;
        w.occ_b[i] = (w.bag_of[p] - w.uniq_t[k] * B) | (last ? (int32_t)0x80000000 : 0);
    }
}

// ---------------------------------------------------------------------------------------------
// forward: fetch + sum-pool, one group of LANES = dim/4 lanes per bag (Section 3 fetch; Algorithm 1
// up-conversion).  The group reads LANES (slot, row id) pairs with one coalesced load, hands them
// round with shuffles, and keeps up to eight row loads in flight; rows are added in index order.
// ---------------------------------------------------------------------------------------------
template <int BITS, bool RO>
__device__ __forceinline__ float4 fetch4(const State& s, const TableDev& tb, int32_t row, int loc, int sub) {
    if (loc >= 0) {
        const float4* src = reinterpret_cast<const float4*>(s.slab + (int64_t)loc * s.dim) + sub;
        return RO ? __ldg(src) : *src;
    }
    return dequant4<BITS, RO>(s.codes, s.sb, tb.row_base + row, s.dim, sub);
}

template <int BITS, int LANES, bool IND>
__global__ void __launch_bounds__(256)
k_pool(State s, Work w, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    const int32_t* __restrict__ indices = a.indices;
    const int32_t* __restrict__ offsets = a.offsets;
    float* __restrict__ out = a.out;
    const int B = a.B;
    constexpr int NB = LANES < 4 ? LANES : 4;        // rows per batch; two batches are in flight
    constexpr int dim = 4 * LANES;
    const int sub = threadIdx.x & (LANES - 1);
    const int gbase = (threadIdx.x & 31) & ~(LANES - 1);
    const uint32_t gmask = group_mask(LANES);
    const int64_t nbags = (int64_t)s.T * B;
    const int64_t gpb = blockDim.x / LANES, ng = gpb * gridDim.x;
    const bool abort = w.ctr->abort != 0;
    const char* slab_col = reinterpret_cast<const char*>(s.slab) + 16 * sub;
    int64_t bag = blockIdx.x * gpb + threadIdx.x / LANES;
    int t = (int)(bag / B);
    int64_t b = bag - (int64_t)t * B;
    // (slot, row id) of the first LANES indices of a bag, one per lane; fetched one bag ahead
    int32_t lo = 0, hi = 0; int wloc = LOC_INVALID; int32_t wrow = 0;
    auto open_bag = [&](int64_t bg) {
        wloc = LOC_INVALID;
        if (bg < nbags && !abort) {
            lo = offsets[bg]; hi = offsets[bg + 1];
            if (lo + sub < hi) { wloc = w.occ_loc[lo + sub]; wrow = indices[lo + sub]; }
        } else { lo = hi = 0; }
    };
    open_bag(bag);
    for (; bag < nbags; bag += ng) {
        const int64_t row_base = s.tables[t].row_base;
        const int32_t clo = lo, chi = hi;
        int myloc = wloc; int32_t myrow = wrow;
        open_bag(bag + ng);                           // the next bag's first window is on its way while this one is pooled
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        // one row: cache resident -> the FP32 row; uncached -> up-convert the codes; out of range -> +0 (never changes the sum)
        auto fetch = [&](int src_lane) {
            const int lc = __shfl_sync(gmask, myloc, gbase + src_lane);
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lc >= 0) {
                x = __ldg(reinterpret_cast<const float4*>(slab_col + (size_t)(uint32_t)lc * (size_t)(dim * 4)));
            } else if (lc == LOC_MISS) {
                const int32_t rw = __shfl_sync(gmask, myrow, gbase + src_lane);
                x = dequant4<BITS, true>(s.codes, s.sb, row_base + rw, dim, sub);
            }
            return x;
        };
        auto fetch_hit = [&](int src_lane) {          // the row is known to be cache resident
            const uint32_t lc = (uint32_t)__shfl_sync(gmask, myloc, gbase + src_lane);
            return __ldg(reinterpret_cast<const float4*>(slab_col + (size_t)lc * (size_t)(dim * 4)));
        };
        for (int32_t p0 = clo; p0 < chi; p0 += LANES) {
            if (p0 > clo) {                           // later windows of a long bag
                myloc = LOC_INVALID;
                if (p0 + sub < chi) { myloc = w.occ_loc[p0 + sub]; myrow = indices[p0 + sub]; }
            }
            const int n = min(LANES, chi - p0);
            const uint32_t hits = (__ballot_sync(gmask, myloc >= 0) & gmask) >> gbase;    // bit u: row u of the window is cached
            constexpr uint32_t FULL = (1u << NB) - 1u;
            float4 xa[NB], xb[NB];
            if ((hits & FULL) == FULL) {
#pragma unroll
                for (int u = 0; u < NB; ++u) xa[u] = fetch_hit(u);
            } else {
#pragma unroll
                for (int u = 0; u < NB; ++u) xa[u] = fetch(u);
            }
            for (int u0 = 0; u0 < n; u0 += 2 * NB) {  // rows are added in index order
                if (u0 + NB < n) {
                    if (((hits >> (u0 + NB)) & FULL) == FULL) {
#pragma unroll
                        for (int u = 0; u < NB; ++u) xb[u] = fetch_hit(u0 + NB + u);
                    } else {
#pragma unroll
                        for (int u = 0; u < NB; ++u) xb[u] = fetch((u0 + NB + u) & (LANES - 1));
                    }
                }
#pragma unroll
                for (int u = 0; u < NB; ++u) acc = add4(acc, xa[u]);
                if (u0 + NB < n) {
                    if (u0 + 2 * NB < n) {
                        if (((hits >> (u0 + 2 * NB)) & FULL) == FULL) {
#pragma unroll
                            for (int u = 0; u < NB; ++u) xa[u] = fetch_hit(u0 + 2 * NB + u);
                        } else {
#pragma unroll
                            for (int u = 0; u < NB; ++u) xa[u] = fetch((u0 + 2 * NB + u) & (LANES - 1));
                        }
                    }
#pragma unroll
                    for (int u = 0; u < NB; ++u) acc = add4(acc, xb[u]);
                }
            }
        }
        float* dst = out + (b * s.T + t) * dim;
        if (a.route) {                                // the owner of sample b gets the vector, straight into its buffer
            const Route* __restrict__ r = a.route;
            const int g = (int)(b / r->B_local);
            dst = r->out[g] + ((b - (int64_t)g * r->B_local) * r->T_global + r->t_base + t) * dim;
        }
        __stcs(reinterpret_cast<float4*>(dst) + sub, acc);      // written once, read by somebody else: not worth a place in L2
        b += ng;
        while (b >= B) { b -= B; ++t; }
    }
}

// ---------------------------------------------------------------------------------------------
// backward 1: new priority value of every row of I_U (Section 3 "Cache Replacement Policy"), candidate keys, counters
// ---------------------------------------------------------------------------------------------
constexpr int PRI_Q = 4;                 // independent rows per thread: the counter updates are random accesses
constexpr int PRI_CHUNK = PRI_Q * 256;   // rows per block and round

// The rows that may be admitted (few, once the caches are warm) are to become a list of (set, distinct-row index)
// records in the order of the distinct rows (table, then row id).
// Small steps (the ones replayed from a graph, where every launch counts): the list leaves this kernel.  A chunk learns
// how many candidates the chunks before it hold by look-back over one word per chunk, and the block that ends the pass
// turns the per-table candidate counts into the segments and tiles of the sort by set that follows.
// Large steps: this kernel leaves each row's candidate key and each chunk's number of candidates, and three small kernels
// (prefix sum, k_cand_write, k_cand_starts) make the list -- waiting for the chunks before costs more there than
// reading the keys again.
// pairs == nullptr: no table has a cache, no list.
template <bool IND>
__global__ void __launch_bounds__(256, IND ? 2 : 3)
k_priority(State s, Work w, uint2* __restrict__ pairs, unsigned long long* __restrict__ words, SortCtl* __restrict__ ctl,
           uint32_t* __restrict__ block_sums, StepArgs av) {
    constexpr bool FUSED = IND;
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    __shared__ uint32_t wcand[8][PRI_Q];        // candidates per warp and round
    __shared__ uint32_t s_turn[2];
    __shared__ uint32_t s_prefix[2];
    __shared__ uint2 stash[2][PRI_CHUNK];       // the candidates of this chunk and of the one before, in row order
    const bool off = w.ctr->abort != 0;         // an abandoned step has no chunks
    const uint32_t step = (uint32_t)a.step;
    constexpr int Q = PRI_Q;
    const int64_t U = off ? 0 : w.ctr->U;
    const uint32_t nchunk = (uint32_t)((U + PRI_CHUNK - 1) / PRI_CHUNK);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // A chunk's candidates wait in shared memory while the block works on its next chunk, and go out once that is done:
    // by then the chunks before it have said how many candidates they hold, so the look-back finds its answer at once.
    bool have_prev = false; uint32_t prev_chunk = 0, prev_total = 0; int buf = 0;
    auto write_out = [&](uint32_t chunk_id, uint32_t total, int b) {
        if (warp == 0) {
            bool poison;
            const uint32_t before = tile_look_back(words, chunk_id, total, s_turn[1], &poison);
            if (lane == 0) { s_prefix[0] = before; s_prefix[1] = poison; }
        }
        __syncthreads();
        if (s_prefix[1]) {                                         // a look-back gave up: write nothing, abandon the step
            if (threadIdx.x == 0) { atomicAdd(&ctl->timeout, 1u); w.ctr->abort = 1; }
        } else {
            for (uint32_t j = threadIdx.x; j < total; j += 256) pairs[s_prefix[0] + j] = stash[b][j];
        }
    };
    uint32_t chunk = blockIdx.x, tag = 0;
    // a block takes PRI_CHUNK consecutive rows at a time, thread i the rows i, i + 256, i + 512, i + 768 of them
    for (;; chunk += gridDim.x) {
        if (FUSED) { if (!draw_tile(ctl, nchunk, s_turn, &chunk, &tag)) break; }
        else if (chunk >= nchunk) break;
        const int64_t c0 = (int64_t)chunk * PRI_CHUNK;
        int t[Q], loc[Q]; int32_t row[Q]; uint32_t mult[Q], old[Q]; int64_t rb[Q], sbase[Q]; int32_t nsets[Q];
        uint32_t ckey[Q]; uint32_t cmask = 0;
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int64_t k = c0 + q * 256 + threadIdx.x;
            t[q] = -1;
            if (k < U) { t[q] = w.uniq_t[k]; row[q] = w.uniq_row[k]; loc[q] = w.loc[k]; mult[q] = (uint32_t)(w.seg[k + 1] - w.seg[k]); }
        }
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            old[q] = 0;
            if (t[q] >= 0) {
                const TableDev tb = s.tables[t[q]];
                rb[q] = tb.row_base; nsets[q] = tb.n_sets; sbase[q] = tb.set_base;
                if (s.policy == 1 && loc[q] != LOC_INVALID) old[q] = s.cnt[rb[q] + row[q]];
            }
        }
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int64_t k = c0 + q * 256 + threadIdx.x;
            unsigned long long m = 0, hitm = 0, uh = 0, un = 0, byp = 0, cand = 0;
            ckey[q] = t[q] >= 0 ? (uint32_t)nsets[q] : 0u;           // large steps: "not a candidate"
            if (t[q] >= 0 && loc[q] != LOC_INVALID) {
                m = mult[q]; un = 1;
                uint32_t pv = step;                      // the priority value the row has from now on
                if (s.policy == 1) {                     // LFU: access count of the row, saturating
                    pv = old[q] + mult[q] < old[q] ? 0xffffffffU : old[q] + mult[q];
                    s.cnt[rb[q] + row[q]] = pv;
                }
                // the cached row's priority value, kept per slot: the LRU time stamp, or a copy of the LFU count (so
                // that the policy kernel reads one line per set instead of one counter per resident row)
                if (loc[q] >= 0) s.ts[loc[q]] = pv;
                if (loc[q] >= 0) { hitm = mult[q]; uh = 1; }
                else if (nsets[q] > 0) {
                    // The lowest priority value in a set never falls (counts and time stamps only grow, a replacement
                    // puts a larger value in the place of the lowest, no way is ever emptied), so a row that does not
                    // beat a bound recorded earlier is bypassed whatever happens in this step (Algorithm 2's test).
                    const int32_t set = w.uset[k];
                    const bool always = s.ways == 1 && s.policy == 0;
                    if (!always && pv <= s.floor[sbase[q] + set]) byp = 1;
                    else { ckey[q] = (uint32_t)set; cand = 1; cmask |= 1u << q; }
                }
            }
            // counters: one atomic per warp when the warp sits inside one table
            if (c0 + q * 256 + (threadIdx.x & ~31) >= U) continue;           // warp-uniform: nothing left for this q
            const int t0 = __shfl_sync(0xffffffffU, t[q], 0);
            const bool same = __all_sync(0xffffffffU, t[q] == t0 || t[q] < 0);
            if (same && t0 >= 0) {
                for (int o = 16; o > 0; o >>= 1) {
                    m += __shfl_xor_sync(0xffffffffU, m, o); hitm += __shfl_xor_sync(0xffffffffU, hitm, o);
                    uh += __shfl_xor_sync(0xffffffffU, uh, o); un += __shfl_xor_sync(0xffffffffU, un, o);
                    byp += __shfl_xor_sync(0xffffffffU, byp, o); cand += __shfl_xor_sync(0xffffffffU, cand, o);
                }
                if (lane == 0) {
                    unsigned long long* st = s.stats + (int64_t)t0 * 8;
                    atomicAdd(st + 0, m); atomicAdd(st + 1, hitm); atomicAdd(st + 2, un); atomicAdd(st + 3, uh);
                    if (byp) atomicAdd(st + 6, byp);
                    if (cand) atomicAdd(&w.cand_cnt[t0], (int32_t)cand);
                }
            } else if (t[q] >= 0) {
                unsigned long long* st = s.stats + (int64_t)t[q] * 8;
                atomicAdd(st + 0, m); atomicAdd(st + 1, hitm); atomicAdd(st + 2, un); atomicAdd(st + 3, uh);
                if (byp) atomicAdd(st + 6, byp);
                if (cand) atomicAdd(&w.cand_cnt[t[q]], 1);
            }
        }
        if (!pairs) continue;
        if constexpr (!FUSED) {
            // large steps: the keys and the chunk's number of candidates, for the kernels that make the list
#pragma unroll
            for (int q = 0; q < Q; ++q) if (t[q] >= 0) w.cand_key[c0 + q * 256 + threadIdx.x] = ckey[q];
            const uint32_t nc = (uint32_t)__syncthreads_count(cmask & 1u) + (uint32_t)__syncthreads_count(cmask & 2u) +
                                (uint32_t)__syncthreads_count(cmask & 4u) + (uint32_t)__syncthreads_count(cmask & 8u);
            if (threadIdx.x == 0) block_sums[chunk] = nc;
        } else {
        // the chunk's candidates in row order: round q's rows come before round q + 1's, a warp's before the next warp's
        uint32_t below[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const uint32_t bq = __ballot_sync(0xffffffffU, (cmask >> q) & 1u);
            below[q] = (uint32_t)__popc(bq & ((1u << lane) - 1u));
            if (lane == 0) wcand[warp][q] = (uint32_t)__popc(bq);
        }
        __syncthreads();
        uint32_t total = 0, mine[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            mine[q] = total + below[q];
#pragma unroll
            for (int v = 0; v < 8; ++v) { const uint32_t c = wcand[v][q]; total += c; if (v < warp) mine[q] += c; }
        }
        if (threadIdx.x == 0) tile_publish(words, chunk, total, tag);
#pragma unroll
        for (int q = 0; q < Q; ++q)
            if ((cmask >> q) & 1u) stash[buf][mine[q]] = make_uint2(ckey[q], (uint32_t)(c0 + q * 256 + threadIdx.x));
        if (have_prev) write_out(prev_chunk, prev_total, buf ^ 1);
        have_prev = true; prev_chunk = chunk; prev_total = total; buf ^= 1;
        }
    }
    if constexpr (FUSED) {
    if (have_prev) { __syncthreads(); write_out(prev_chunk, prev_total, buf ^ 1); }
    if (last_block_of_pass(ctl, s_turn)) {
        // every chunk is done and the per-table candidate counts are complete: where each table's candidates begin in
        // the list, and the tiles of the sort by set (one warp; the counts are cleared for the next step)
        if (pairs && warp == 0) {
            const bool dead = off || __ldcg(&w.ctr->abort) != 0;
            const int T = s.T;
            int32_t run = 0;
            for (int t0 = 0; t0 < T; t0 += 32) {
                const int tt = t0 + lane;
                const int32_t c = tt < T ? __ldcg(w.cand_cnt + tt) : 0;
                int32_t inc = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int32_t v = __shfl_up_sync(0xffffffffU, inc, o); if (lane >= o) inc += v; }
                if (tt < T) { w.cstart[tt] = run + inc - c; w.cand_cnt[tt] = 0; }
                run += __shfl_sync(0xffffffffU, inc, 31);
            }
            if (lane == 0) { w.cstart[T] = dead ? 0 : run; w.ctr->n_cand = dead ? 0u : (uint32_t)run; }
            __syncwarp();
            warp_tile_bases(w.cstart, T, w.ctile_base, dead, w.sort_tile);
        }
        close_pass(ctl, tag);
    }
    }
}

// The candidates for admission, in the order of the distinct rows (table, then row id), as (set, distinct-row index)
// records: block_sums holds the exclusive prefix of the per-chunk counts.
__global__ void __launch_bounds__(256)
k_cand_write(State s, Work w, const uint32_t* __restrict__ block_sums, uint2* __restrict__ pairs) {
    __shared__ uint32_t tmp[256 / 32 + 1];
    if (w.ctr->abort) return;
    const int64_t U = w.ctr->U;
    const uint32_t* __restrict__ ckey = w.cand_key;
    for (int64_t c0 = (int64_t)blockIdx.x * PRI_CHUNK; c0 < U; c0 += (int64_t)gridDim.x * PRI_CHUNK) {
        const int64_t k0 = c0 + 4 * threadIdx.x;             // four consecutive rows per thread
        uint32_t key[4]; bool is[4]; uint32_t n = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            is[i] = false; key[i] = 0;
            if (k0 + i < U) {
                key[i] = ckey[k0 + i];
                is[i] = key[i] < (uint32_t)s.tables[w.uniq_t[k0 + i]].n_sets;
            }
            n += is[i];
        }
        uint32_t total;
        uint32_t pos = block_exclusive_scan<256>(n, &total, tmp) + block_sums[c0 / PRI_CHUNK];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (is[i]) pairs[pos++] = make_uint2(key[i], (uint32_t)(k0 + i));
    }
}

// where each table's candidates begin (one warp; the per-table counts are cleared for the next step)
__global__ void k_cand_starts(Work w, int T) {
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    int32_t run = 0;
    for (int t0 = 0; t0 < T; t0 += 32) {
        const int t = t0 + lane;
        const int32_t c = t < T ? w.cand_cnt[t] : 0;
        int32_t inc = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int32_t v = __shfl_up_sync(0xffffffffU, inc, o); if (lane >= o) inc += v; }
        if (t < T) { w.cstart[t] = run + inc - c; w.cand_cnt[t] = 0; }
        run += __shfl_sync(0xffffffffU, inc, 31);
    }
    if (lane == 0) w.cstart[T] = w.ctr->abort ? 0 : run;
    __syncwarp();
    warp_tile_bases(w.cstart, T, w.ctile_base, w.ctr->abort != 0, w.sort_tile);     // the tiles of the sort by set
}

// ---------------------------------------------------------------------------------------------
// backward 2: admission / eviction, integer only.  One group of `ways` lanes walks the miss
// candidates of one set in ascending row id (Algorithm 2's admission test: a candidate whose priority value does
// not exceed the lowest one among the residents bypasses, otherwise it takes that resident's place).  Lane w holds way w of the set; the candidates are fetched `ways`
// at a time (one per lane) and handed round with shuffles.  No row value is read or written here.
// ---------------------------------------------------------------------------------------------
constexpr int VICTIM_NONE = -1;       // the way was empty, or the displaced row writes itself back
constexpr int VICTIM_DEFER = -2;      // the displaced row was hit in this step: the newcomer waits for its write-back

// the first candidate of every set that has any (the set-sorted list is grouped by table, then set)
__global__ void k_policy_heads(State s, Work w, const uint32_t* __restrict__ ckey) {
    if (w.ctr->abort) return;
    const int64_t U = w.cstart[s.T];                           // candidates, sorted by (table, set), row ids ascending inside a set
    const int64_t U32 = (U + 31) & ~31LL;
    const int lane = threadIdx.x & 31;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < U32; j += (int64_t)gridDim.x * blockDim.x) {
        bool head = false;
        if (j < U) {
            const uint32_t key = ckey[j];
            const int t = find_segment(w.cstart, s.T, (int32_t)j);
            head = j == w.cstart[t] || ckey[j - 1] != key;
        }
        const uint32_t m = __ballot_sync(0xffffffffU, head);
        uint32_t base = 0;
        if (lane == 0 && m) base = atomicAdd(&w.ctr->n_heads, (uint32_t)__popc(m));
        base = __shfl_sync(0xffffffffU, base, 0);
        if (head) w.heads[base + __popc(m & ((1u << lane) - 1u))] = (int32_t)j;
    }
}

template <bool IND>
__global__ void __launch_bounds__(256)
k_policy(State s, Work w, const uint32_t* __restrict__ ckey, const uint32_t* __restrict__ cval, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    if (w.ctr->abort) return;
    const uint32_t step = (uint32_t)a.step, epoch = a.epoch;
    const int ways = s.ways;
    const int lane = threadIdx.x & 31, way = lane & (ways - 1), gbase = lane & ~(ways - 1);
    const uint32_t gmask = group_mask(ways);
    const int64_t nheads = w.ctr->n_heads;
    const int64_t gpb = blockDim.x / ways, ng = gpb * gridDim.x;
    for (int64_t hi = blockIdx.x * gpb + threadIdx.x / ways; hi < nheads; hi += ng) {
        const int64_t j = w.heads[hi];
        const uint32_t key = ckey[j];
        const int t = find_segment(w.cstart, s.T, (int32_t)j);
        const TableDev tb = s.tables[t];
        const int64_t slot = (tb.set_base + key) * ways + way;
        int32_t tag = s.tags[slot];
        uint32_t pri = 0;
        if (tag >= 0) pri = s.ts[slot];
        int32_t cand = -1, vict = VICTIM_NONE;
        uint32_t n_admit = 0, n_evict = 0, n_bypass = 0;
        const int64_t jend = w.cstart[t + 1];
        for (int64_t jj0 = j;; jj0 += ways) {
            const int64_t jj = jj0 + way;
            const bool valid = jj < jend && ckey[jj] == key;
            int32_t ckk = 0, crow = 0; uint32_t cpv = step;
            if (valid) {
                ckk = (int32_t)cval[jj];
                crow = w.uniq_row[ckk];
                if (s.policy == 1) cpv = s.cnt[tb.row_base + crow];
            }
            const int n = __popc(__ballot_sync(gmask, valid) & gmask);   // the valid lanes are a prefix of the group
            // Between two replacements the set does not change, so every candidate that cannot beat the current
            // minimum bypasses at once; only the candidates that replace are walked one by one.
            int u = 0;
            while (u < n) {
                // empty ways rank below every priority; ties go to the lowest way
                const uint32_t empties = __ballot_sync(gmask, tag < 0) & gmask;
                int jw; bool jempty; uint32_t jpri = 0;
                if (empties) { jw = __ffs(empties) - 1 - gbase; jempty = true; }
                else {
                    jpri = __reduce_min_sync(gmask, pri);
                    jw = __ffs(__ballot_sync(gmask, pri == jpri) & gmask) - 1 - gbase;
                    jempty = false;
                }
                // lane `way` holds candidate number `way` of this batch
                const bool always = ways == 1 && s.policy == 0;                 // direct-mapped LRU never compares
                const bool would = valid && way >= u && (jempty || always || cpv > jpri);
                const uint32_t wm = (__ballot_sync(gmask, would) & gmask) >> gbase;
                if (wm == 0) { n_bypass += (uint32_t)(n - u); break; }
                const int f = __ffs(wm) - 1;                                    // the first candidate that replaces
                n_bypass += (uint32_t)(f - u);
                const int32_t kk = __shfl_sync(gmask, ckk, gbase + f);
                const int32_t row = __shfl_sync(gmask, crow, gbase + f);
                const uint32_t pv = __shfl_sync(gmask, cpv, gbase + f);
                ++n_admit;
                if (!jempty) ++n_evict;
                if (way == jw) {
                    if (tag >= 0 && cand < 0) {
                        // a row that was resident when the step began leaves the cache
                        if (s.hit_epoch[slot] == epoch) { w.final_loc[s.hit_k[slot]] = LOC_MISS; vict = VICTIM_DEFER; }
                        else vict = tag;
                    }
                    tag = row; pri = pv; cand = kk;
                }
                u = f + 1;
            }
            if (n < ways) break;
        }
        {   // what the set's lowest priority value is now bounds it from below for good
            const bool any_empty = (__ballot_sync(gmask, tag < 0) & gmask) != 0;
            const uint32_t low = __reduce_min_sync(gmask, tag < 0 ? 0u : pri);
            if (way == 0) s.floor[tb.set_base + key] = any_empty ? 0u : low;
        }
        if (cand >= 0) {
            s.tags[slot] = tag;
            s.ts[slot] = pri;                            // the newcomer's priority value (LRU: this step)
            w.final_loc[cand] = (int32_t)slot;
            w.victim[cand] = vict;
            if (vict == VICTIM_DEFER) w.defer_k[atomicAdd(&w.ctr->deferred, 1u)] = cand;
        }
        if (way == 0) {
            unsigned long long* st = s.stats + (int64_t)t * 8;
            if (n_admit) atomicAdd(st + 4, (unsigned long long)n_admit);
            if (n_evict) atomicAdd(st + 5, (unsigned long long)n_evict);
            if (n_bypass) atomicAdd(st + 6, (unsigned long long)n_bypass);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// backward 3: merged gradient of one distinct row (Section 5.1), radix-32 tree over index positions
// ---------------------------------------------------------------------------------------------
// up to 32 consecutive occurrences, added left to right; the group reads LANES sample ids at a time.
// gcol points at the group's lane-th float4 of column block t; stride_bytes is the size of one sample's row of grad_out.
template <int LANES>
__device__ __forceinline__ float4 sum_chunk(const int32_t* __restrict__ occ_b, const char* __restrict__ gcol, uint32_t stride_bytes,
                                            int32_t first, int len, uint32_t gmask, int gbase, int sub) {
    constexpr int NB = LANES < 8 ? LANES : 8;
    float4 acc;
    if (LANES == 32 && len == 32) {       // a full chunk handled by a whole warp: no bounds to check, 8 rows in flight
        const uint32_t myb = (uint32_t)occ_b[first + sub] & 0x7fffffffU;
        float4 va[4], vb[4];
        auto row = [&](int u) { return __ldg(reinterpret_cast<const float4*>(gcol + (size_t)__shfl_sync(0xffffffffU, myb, u) * stride_bytes)); };
#pragma unroll
        for (int u = 0; u < 4; ++u) va[u] = row(u);
#pragma unroll
        for (int u = 0; u < 4; ++u) vb[u] = row(4 + u);
        acc = va[0];
#pragma unroll
        for (int u = 1; u < 4; ++u) acc = add4(acc, va[u]);
#pragma unroll
        for (int g = 1; g < 4; ++g) {
#pragma unroll
            for (int u = 0; u < 4; ++u) va[u] = row(8 * g + u);
#pragma unroll
            for (int u = 0; u < 4; ++u) acc = add4(acc, vb[u]);
#pragma unroll
            for (int u = 0; u < 4; ++u) vb[u] = row(8 * g + 4 + u);
#pragma unroll
            for (int u = 0; u < 4; ++u) acc = add4(acc, va[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc = add4(acc, vb[u]);
        return acc;
    }
    acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int j0 = 0; j0 < len; j0 += LANES) {
        const int n = min(LANES, len - j0);
        const uint32_t myb = sub < n ? (uint32_t)occ_b[first + j0 + sub] & 0x7fffffffU : 0u;
        for (int u0 = 0; u0 < n; u0 += NB) {
            float4 v[NB];
#pragma unroll
            for (int u = 0; u < NB; ++u) {
                const uint32_t b = __shfl_sync(gmask, myb, gbase + u0 + u);
                if (u0 + u < n) v[u] = __ldg(reinterpret_cast<const float4*>(gcol + (size_t)b * stride_bytes));
            }
#pragma unroll
            for (int u = 0; u < NB; ++u)
                if (u0 + u < n) acc = (j0 + u0 + u == 0) ? v[u] : add4(acc, v[u]);
        }
    }
    return acc;
}

// LEVEL 0 adds up to 32 terms left to right; LEVEL l adds up to 32 results of LEVEL l-1
template <int LEVEL, class Term>
__device__ __forceinline__ float4 tree_reduce(const Term& term, int64_t first, int64_t n) {
    if constexpr (LEVEL == 0) {
        float4 acc = term(first);
        for (int64_t j = 1; j < n; ++j) acc = add4(acc, term(first + j));
        return acc;
    } else {
        int64_t span = 32;
        for (int l = 1; l < LEVEL; ++l) span *= 32;
        float4 acc = tree_reduce<LEVEL - 1>(term, first, n < span ? n : span);
        for (int64_t c = span; c < n; c += span)
            acc = add4(acc, tree_reduce<LEVEL - 1>(term, first + c, n - c < span ? n - c : span));
        return acc;
    }
}

// rows with more than HOT_SPAN occurrences: one block per HOT_SPAN occurrences computes two tree levels
// (8 groups of LANES lanes share the 32 chunks of a task)
template <int LANES, bool IND>
__global__ void __launch_bounds__(8 * LANES, LANES == 32 ? 3 : 1)
k_hot_partial(State s, Work w, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    extern __shared__ float chunk_sums[];     // [32][dim]
    if (w.ctr->abort) return;
    const float* __restrict__ grad = a.grad;
    const int dim = s.dim;
    const int sub = threadIdx.x & (LANES - 1), grp = threadIdx.x / LANES, ngrp = blockDim.x / LANES;
    const int gbase = (threadIdx.x & 31) & ~(LANES - 1);
    const uint32_t gmask = group_mask(LANES);
    const uint32_t ntask = w.ctr->hot_tasks;
    const uint32_t stride_bytes = (uint32_t)s.T * (uint32_t)dim * 4u;
    for (uint32_t task = blockIdx.x; task < ntask; task += gridDim.x) {
        const int32_t k = w.task_k[task];
        const int32_t j = (int32_t)task - w.hot_base[k];
        const int32_t first = w.seg[k] + j * HOT_SPAN;
        const int32_t n = min(HOT_SPAN, w.seg[k + 1] - first);
        const int nchunk = (n + 31) >> 5;
        const char* gcol = reinterpret_cast<const char*>(grad + (int64_t)w.uniq_t[k] * dim + 4 * sub);
        for (int c = grp; c < nchunk; c += ngrp) {
            const float4 v = sum_chunk<LANES>(w.occ_b, gcol, stride_bytes, first + 32 * c, min(32, n - 32 * c), gmask, gbase, sub);
            reinterpret_cast<float4*>(chunk_sums + c * dim)[sub] = v;
        }
        __syncthreads();
        if (grp == 0) {
            float4 acc = reinterpret_cast<const float4*>(chunk_sums)[sub];
            for (int c = 1; c < nchunk; ++c) acc = add4(acc, reinterpret_cast<const float4*>(chunk_sums + c * dim)[sub]);
            reinterpret_cast<float4*>(w.partial + (int64_t)task * dim)[sub] = acc;
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// backward 4: update(T, C, i, x) for one distinct row whose merged gradient g is known
// ---------------------------------------------------------------------------------------------
template <int BITS, int LANES>
__device__ __forceinline__ void apply_update(const State& s, const TableDev& tb, int t, int32_t row, int loc, int floc,
                                             int32_t victim, float4 g, float4 x, float lr, uint64_t step, int sub, uint32_t gmask) {
    const int dim = 4 * LANES;
    const int64_t grow = tb.row_base + row;
    float mult = lr;                                         // SGD: x <- x - lr * g
    if (s.optimizer == 1) {                                  // row-wise Adagrad
        float a = __fmul_rn(g.x, g.x);
        a = __fmaf_rn(g.y, g.y, a); a = __fmaf_rn(g.z, g.z, a); a = __fmaf_rn(g.w, g.w, a);
#pragma unroll
        for (int o = LANES >> 1; o > 0; o >>= 1) a = __fadd_rn(a, __shfl_xor_sync(gmask, a, o));
        const float Gold = s.G[grow];
        __syncwarp(gmask);                                   // every lane has read G before lane 0 replaces it
        const float Gn = __fadd_rn(Gold, __fmul_rn(a, __fdiv_rn(1.0f, (float)dim)));
        if (sub == 0) s.G[grow] = Gn;
        mult = __fdiv_rn(lr, __fadd_rn(__fsqrt_rn(Gn), s.eps));
    }
    const float4 xn = fma4(-mult, g, x);
    if (floc >= 0) {
        float4* dst = reinterpret_cast<float4*>(s.slab + (int64_t)floc * dim) + sub;
        if (loc < 0 && victim >= 0)     // the row this newcomer displaces is down-converted and placed back in T
            quantize_store<BITS>(*dst, s.codes, s.sb, tb.row_base + victim, dim, sub, LANES,
                                rowkey(s.seed, DOMAIN_SR, (uint32_t)t, (uint32_t)victim, step), s.rounding != 0);
        *dst = xn;                      // cached rows keep full precision, a newcomer enters verbatim
    } else {
        quantize_store<BITS>(xn, s.codes, s.sb, grow, dim, sub, LANES,
                            rowkey(s.seed, DOMAIN_SR, (uint32_t)t, (uint32_t)row, step), s.rounding != 0);
    }
}

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

struct RawRow { float4 f; uint2 q; float2 sb; };

constexpr int UPD_WARPS = 4;     // warps per block of k_update
constexpr int UPD_NB = 4;        // gradient rows per batch of asynchronous copies
constexpr int UPD_DEPTH = 2;     // batches in flight per group
constexpr int UPD_SMALL_U = 524288;   // at most this many distinct rows: blocks of 8 rows instead of 32
constexpr int UPD_SMEM = UPD_WARPS * (UPD_DEPTH * UPD_NB * 32 * 16 + 32 * 3 * 16);

// Every distinct row that is not on the multi-block path, except newcomers that wait for a write-back.  A warp stages the
// bookkeeping of 32 consecutive rows in shared memory, one row per lane (coalesced loads; the per-row scalar work --
// addresses, the stochastic-rounding key -- is done there once, 32 rows at a time).  The distinct rows of a block are
// consecutive in the sorted batch, so the gradient rows they need are one contiguous run of the sorted occurrence list
// (broken only where a row is not this kernel's, or where the table changes).  Each group of LANES lanes walks such a
// run four occurrences at a time: a batch of asynchronous 16-byte copies brings four gradient rows into shared memory
// while the batch before it is added, and a row is finished (FP32 update, commit) the moment its last term has been added.

template <int BITS, int LANES, bool IND>
__global__ void __launch_bounds__(UPD_WARPS * 32, 8)
k_update(State s, Work w, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    extern __shared__ __align__(16) unsigned char upd_smem[];
    if (w.ctr->abort) return;
    const float* __restrict__ grad = a.grad;
    const float lr = a.lr;
    const uint64_t step = a.step;
    constexpr int dim = 4 * LANES, G = 32 / LANES, NB = LANES < UPD_NB ? LANES : UPD_NB, BPW = LANES / NB;
    constexpr int SLOTS = UPD_DEPTH * NB;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane & (LANES - 1), grp = lane / LANES, gbase = lane & ~(LANES - 1);
    const uint32_t gmask = group_mask(LANES);
    float4* ring = reinterpret_cast<float4*>(upd_smem) + ((warp * G + grp) * SLOTS) * LANES + sub;       // slot i: ring[i * LANES]
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    // per staged row: A = {loc, final loc, global row lo, hi}, B = {rounding key, occurrences, first occurrence, victim},
    // C = {victim's key, victim's global row lo, hi, gradient column}
    int4* recs = reinterpret_cast<int4*>(upd_smem + UPD_WARPS * UPD_DEPTH * UPD_NB * 32 * 16) + warp * 96;
    const int64_t U = w.ctr->U;
    // rows per hand-out and per group: 32 per warp when there is plenty of work; a step with few distinct rows is cut
    // finer, because there the kernel lasts as long as its longest chain of rows (each row ends in dependent loads)
    const int rpt = U > UPD_SMALL_U ? 32 : (G > 8 ? G : 8);
    const int rpg = rpt / G;
    const uint32_t stride_bytes = (uint32_t)s.T * (uint32_t)dim * 4u;
    const char* gcol = reinterpret_cast<const char*>(grad + 4 * sub);
    const float NZ = __int_as_float(0x80000000);          // -0: adding it changes no value, not even a zero's sign
    for (;;) {
        // blocks of 32 rows are handed out on demand: their cost varies with the rows' multiplicities
        uint32_t blk = 0;
        if (lane == 0) blk = atomicAdd(&w.ctr->upd_next, 1u);
        const int64_t k0 = (int64_t)__shfl_sync(0xffffffffU, blk, 0) * rpt;
        if (k0 >= U) break;
        const int64_t k = k0 + lane;
        bool skip = true; int myt = -1;
        if (lane < rpt && k < U) {
            const int32_t first = w.seg[k], row = w.uniq_row[k];
            const int loc = w.loc[k], floc = w.final_loc[k], hb = w.hot_base[k], victim = w.victim[k], t = w.uniq_t[k];
            myt = t;
            // pseudo rows, hot rows (own kernel) and newcomers that wait for a write-back are not ours
            const bool newcomer = loc < 0 && floc >= 0;
            skip = loc == LOC_INVALID || hb >= 0 || (newcomer && victim == VICTIM_DEFER);
            int4 A = make_int4(loc, floc, 0, 0), Bq = make_int4(0, w.seg[k + 1] - first, first, victim), C = make_int4(0, 0, 0, t * dim);
            if (!skip) {
                const int64_t rb = s.tables[t].row_base;
                const int64_t grow = rb + row;
                A.z = (int32_t)(uint32_t)grow; A.w = (int32_t)(grow >> 32);
                Bq.x = (int32_t)rowkey(s.seed, DOMAIN_SR, (uint32_t)t, (uint32_t)row, step);
                // pull this row's current value towards L2 now; it is needed when its gradient has been summed
                if (loc >= 0) {
                    const char* src = reinterpret_cast<const char*>(s.slab + (int64_t)loc * dim);
#pragma unroll
                    for (int o = 0; o < dim * 4; o += 128) prefetch_l2(src + o);
                } else {
                    prefetch_l2(s.codes + grow * (dim * BITS / 8));
                    if (BITS != 16) prefetch_l2(s.sb + grow);
                }
                if (newcomer && victim >= 0) {
                    const int64_t vrow = rb + victim;
                    C.x = (int32_t)rowkey(s.seed, DOMAIN_SR, (uint32_t)t, (uint32_t)victim, step);
                    C.y = (int32_t)(uint32_t)vrow; C.z = (int32_t)(vrow >> 32);
                    const char* src = reinterpret_cast<const char*>(s.slab + (int64_t)floc * dim);
#pragma unroll
                    for (int o = 0; o < dim * 4; o += 128) prefetch_l2(src + o);
                }
            }
            recs[lane * 3] = A; recs[lane * 3 + 1] = Bq; recs[lane * 3 + 2] = C;
        }
        const int tprev = __shfl_up_sync(0xffffffffU, myt, 1);
        const uint32_t skipmask = __ballot_sync(0xffffffffU, skip);                       // rows that are not ours (or past the end)
        const uint32_t stopmask = skipmask | __ballot_sync(0xffffffffU, lane > 0 && myt != tprev);   // a run ends before these rows
        __syncwarp();
        // this group's rows: rpg consecutive ones; their runs
        const int gr0 = grp * rpg, gr1 = gr0 + rpg;
        uint32_t avail = ~skipmask & (rpg == 32 ? 0xffffffffU : (((1U << rpg) - 1U) << gr0));
        while (avail) {
            const int rs = __ffs(avail) - 1;
            const uint32_t above = stopmask & (rs == 31 ? 0u : (0xfffffffeU << rs));
            int re = above ? __ffs(above) - 1 : 32;
            re = min(re, gr1);
            avail = re >= 32 ? 0u : (avail & (0xffffffffU << re));
            // the run's occurrences and gradient column
            const int4 Bs = recs[rs * 3 + 1], Be = recs[(re - 1) * 3 + 1];
            const int32_t os = Bs.z, oe = Be.z + Be.y;
            const char* src = gcol + (size_t)(uint32_t)recs[rs * 3 + 2].w * 4u;
            const int nbatch = (oe - os + NB - 1) / NB;
            uint32_t wb = 0, wlast = 0;                        // sample ids of LANES consecutive occurrences, one per lane; their row ends
            uint32_t pend = 0;                                 // row-end bits of the batches in flight, NB bits per batch
            auto issue = [&](int j) {                          // copies of batch j (none when j is past the end); always one group
                if (j < nbatch) {
                    const int jw = j % BPW;
                    if (jw == 0) {
                        const int32_t o = os + j * NB + sub;
                        const uint32_t raw = o < oe ? (uint32_t)w.occ_b[o] : 0u;
                        wlast = (__ballot_sync(gmask, (raw >> 31) != 0) & gmask) >> gbase;
                        wb = raw & 0x7fffffffU;
                    }
                    constexpr uint32_t BM = (1u << NB) - 1u;
                    const int f = (j % UPD_DEPTH) * NB;
                    pend = (pend & ~(BM << f)) | (((wlast >> (jw * NB)) & BM) << f);
                    const int32_t left = oe - (os + j * NB);
                    const uint32_t dst = ring_s + (uint32_t)(((j % UPD_DEPTH) * NB) * LANES * 16);
#pragma unroll
                    for (int u = 0; u < NB; ++u) {
                        const uint32_t b = __shfl_sync(gmask, wb, gbase + jw * NB + u);          // 0 (a valid sample) past the end
                        cp_async16_if(dst + (uint32_t)(u * LANES * 16), src + (size_t)b * stride_bytes, u < left);
                    }
                }
                cp_async_commit();
            };
            // current row: its records, its stored value, how many terms are still to come
            int r = rs;
            int4 A, Bq; RawRow xr;
            auto open_row = [&]() {
                A = recs[r * 3]; Bq = recs[r * 3 + 1];
                if (A.x >= 0) {
                    xr.f = reinterpret_cast<const float4*>(s.slab + (int64_t)A.x * dim)[sub];
                } else {
                    const int64_t grow = ((int64_t)A.w << 32) | (uint32_t)A.z;
                    if (BITS != 16) xr.sb = s.sb[grow];
                    xr.q = load_codes4<BITS, false>(s.codes, grow, dim, sub);
                }
            };
            open_row();
#pragma unroll
            for (int j = 0; j < UPD_DEPTH; ++j) issue(j);
            float4 chunkacc = make_float4(NZ, NZ, NZ, NZ), rowacc = chunkacc;
            int c = 0;                                         // terms of the current row added so far
            const int nocc = oe - os;
            for (int j = 0; j < nbatch; ++j) {
                if (j) issue(j - 1 + UPD_DEPTH);               // refill the slots just drained,
                cp_async_wait<UPD_DEPTH - 1>();                // then wait for this batch
                const uint32_t m = (pend >> ((j % UPD_DEPTH) * NB)) & ((1u << NB) - 1u);      // bit u: occurrence u ends its row
                const float4* slot = ring + ((j % UPD_DEPTH) * NB) * LANES;
                const int cnt = min(NB, nocc - j * NB);
                if (NB == 4 && m == 0 && cnt == 4 && (c & 31) <= 28) {
                    // four terms of one row and one chunk of 32 (the long rows are mostly made of these): no bookkeeping
                    chunkacc = add4(add4(add4(add4(chunkacc, slot[0]), slot[LANES]), slot[2 * LANES]), slot[3 * LANES]);
                    c += 4;
                    if ((c & 31) == 0) { rowacc = add4(rowacc, chunkacc); chunkacc = make_float4(NZ, NZ, NZ, NZ); }
                    continue;
                }
#pragma unroll 1
                for (int u = 0; u < cnt; ++u) {
                    chunkacc = add4(chunkacc, slot[u * LANES]);
                    ++c;
                    const bool last = (m >> u) & 1u;
                    if (last || (c & 31) == 0) {               // a finished chunk joins the sum of chunk sums
                        rowacc = add4(rowacc, chunkacc);
                        chunkacc = make_float4(NZ, NZ, NZ, NZ);
                    }
                    if (last) {
                        c = 0;
                        const int loc = A.x, floc = A.y;
                        float4 x = xr.f;
                        if (loc < 0) x = decode4<BITS>(xr.q, xr.sb);
                        const int64_t grow = ((int64_t)A.w << 32) | (uint32_t)A.z;
                        float mult = lr;                                         // SGD: x <- x - lr * g
                        if (s.optimizer == 1) {                                  // row-wise Adagrad
                            float q = __fmul_rn(rowacc.x, rowacc.x);
                            q = __fmaf_rn(rowacc.y, rowacc.y, q); q = __fmaf_rn(rowacc.z, rowacc.z, q); q = __fmaf_rn(rowacc.w, rowacc.w, q);
#pragma unroll
                            for (int o = LANES >> 1; o > 0; o >>= 1) q = __fadd_rn(q, __shfl_xor_sync(gmask, q, o));
                            const float Gold = s.G[grow];
                            __syncwarp(gmask);                                   // every lane has read G before lane 0 replaces it
                            const float Gn = __fadd_rn(Gold, __fmul_rn(q, __fdiv_rn(1.0f, (float)dim)));
                            if (sub == 0) s.G[grow] = Gn;
                            mult = __fdiv_rn(lr, __fadd_rn(__fsqrt_rn(Gn), s.eps));
                        }
                        const float4 xn = fma4(-mult, rowacc, x);
                        if (floc >= 0) {
                            float4* dst = reinterpret_cast<float4*>(s.slab + (int64_t)floc * dim) + sub;
                            if (loc < 0 && Bq.w >= 0) {          // the row this newcomer displaces is down-converted and placed back in T
                                const int4 C = recs[r * 3 + 2];
                                const int64_t vrow = ((int64_t)C.z << 32) | (uint32_t)C.y;
                                quantize_store<BITS>(*dst, s.codes, s.sb, vrow, dim, sub, LANES, (uint32_t)C.x, s.rounding != 0);
                            }
                            *dst = xn;                           // cached rows keep full precision, a newcomer enters verbatim
                        } else {
                            quantize_store<BITS>(xn, s.codes, s.sb, grow, dim, sub, LANES, (uint32_t)Bq.x, s.rounding != 0);
                        }
                        rowacc = make_float4(NZ, NZ, NZ, NZ);
                        if (++r < re) open_row();
                    }
                }
            }
            cp_async_wait<0>();
        }
        __syncwarp();                                          // the records are rewritten by the next block
    }
}

// Rows named by a list: the hot rows (gradient from the partial sums of k_hot_partial), and, in a
// second launch, the newcomers whose slot had to be vacated by a row that was itself updated.
template <int BITS, int LANES, bool IND>
__global__ void __launch_bounds__(256)
k_update_list(State s, Work w, const int32_t* __restrict__ list, const uint32_t* __restrict__ count, int deferred_pass, StepArgs av) {
    StepArgs a = av; if (IND) a = *w.args;      // replayed from a graph: the arguments come from device memory
    if (w.ctr->abort) return;
    const float* __restrict__ grad = a.grad;
    const float lr = a.lr;
    const uint64_t step = a.step;
    constexpr int dim = 4 * LANES;
    const int lane = threadIdx.x & 31;
    const int sub = lane & (LANES - 1), gbase = lane & ~(LANES - 1);
    const uint32_t gmask = group_mask(LANES);
    const int64_t n = *count;
    const int64_t gpb = blockDim.x / LANES, ng = gpb * gridDim.x;
    const uint32_t stride_bytes = (uint32_t)s.T * (uint32_t)dim * 4u;
    for (int64_t i = blockIdx.x * gpb + threadIdx.x / LANES; i < n; i += ng) {
        const int32_t k = list[i];
        const int loc = w.loc[k], floc = w.final_loc[k];
        if (loc == LOC_INVALID) continue;
        int32_t victim = (loc < 0 && floc >= 0) ? w.victim[k] : VICTIM_NONE;
        if (!deferred_pass && victim == VICTIM_DEFER) continue;          // comes back in the deferred pass
        const int t = w.uniq_t[k];
        const int32_t row = w.uniq_row[k];
        const TableDev tb = s.tables[t];
        const int32_t first = w.seg[k], m = w.seg[k + 1] - first;
        const char* gcol = reinterpret_cast<const char*>(grad + (int64_t)t * dim + 4 * sub);
        const float4 x = fetch4<BITS, false>(s, tb, row, loc, sub);
        float4 g;
        const int hb = w.hot_base[k];
        if (hb < 0) {
            g = sum_chunk<LANES>(w.occ_b, gcol, stride_bytes, first, min(32, m), gmask, gbase, sub);
            for (int32_t c = 32; c < m; c += 32)
                g = add4(g, sum_chunk<LANES>(w.occ_b, gcol, stride_bytes, first + c, min(32, m - c), gmask, gbase, sub));
        } else {
            const float* part = w.partial + (int64_t)hb * dim + 4 * sub;
            auto term = [&](int64_t j) { return *reinterpret_cast<const float4*>(part + j * dim); };
            g = tree_reduce<4>(term, 0, (m + HOT_SPAN - 1) / HOT_SPAN);
        }
        apply_update<BITS, LANES>(s, tb, t, row, loc, floc, victim, g, x, lr, step, sub, gmask);
    }
}

// ---------------------------------------------------------------------------------------------
// create / flush / export
// ---------------------------------------------------------------------------------------------
template <int BITS>
__global__ void k_init_table(State s, int t, float lo, float hi) {
    const int lanes = s.lanes;
    const int sub = threadIdx.x & (lanes - 1);
    const TableDev tb = s.tables[t];
    const int64_t gpb = blockDim.x / lanes, ng = gpb * gridDim.x;
    const float width = __fsub_rn(hi, lo);
    for (int64_t row = blockIdx.x * gpb + threadIdx.x / lanes; row < tb.N; row += ng) {
        const uint32_t key = rowkey(s.seed, DOMAIN_INIT, (uint32_t)t, (uint32_t)row, 0);
        float4 x;
        x.x = __fmaf_rn(uniform01(key, 4 * sub + 0), width, lo);
        x.y = __fmaf_rn(uniform01(key, 4 * sub + 1), width, lo);
        x.z = __fmaf_rn(uniform01(key, 4 * sub + 2), width, lo);
        x.w = __fmaf_rn(uniform01(key, 4 * sub + 3), width, lo);
        quantize_store<BITS>(x, s.codes, s.sb, tb.row_base + row, s.dim, sub, lanes, 0u, false);
    }
}

// every resident row of every table is down-converted into the low-precision table (and stays resident): one group of
// lanes per cache slot of the concatenated cache; the slot's table is found by bisection over the tables' first sets
template <int BITS>
__global__ void __launch_bounds__(256)
k_flush(State s, int64_t total_slots, uint64_t step) {
    const int lanes = s.lanes;
    const int sub = threadIdx.x & (lanes - 1);
    const int64_t gpb = blockDim.x / lanes, ng = gpb * gridDim.x;
    constexpr int Q = 4;                           // slots per group and round: their loads are in flight together
    for (int64_t slot0 = blockIdx.x * gpb + threadIdx.x / lanes; slot0 < total_slots; slot0 += Q * ng) {
        int32_t tag[Q]; float4 x[Q];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            const int64_t slot = slot0 + q * ng;
            tag[q] = slot < total_slots ? s.tags[slot] : -1;
        }
#pragma unroll
        for (int q = 0; q < Q; ++q)
            if (tag[q] >= 0) x[q] = reinterpret_cast<const float4*>(s.slab + (slot0 + q * ng) * s.dim)[sub];
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            if (tag[q] < 0) continue;
            const int64_t set = (slot0 + q * ng) / s.ways;
            int lo = 0, hi = s.T;                  // largest t with tables[t].set_base <= set (tables without a cache share a base)
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (s.tables[mid].set_base <= set) lo = mid; else hi = mid;
            }
            const int t = lo;
            quantize_store<BITS>(x[q], s.codes, s.sb, s.tables[t].row_base + tag[q], s.dim, sub, lanes,
                                 rowkey(s.seed, DOMAIN_FLUSH, (uint32_t)t, (uint32_t)tag[q], step), s.rounding != 0);
        }
    }
}

__global__ void k_gather_rows(State s, int t, const int64_t* __restrict__ rows, int64_t n, int code_bytes,
                              uint8_t* __restrict__ codes, float* __restrict__ scale, float* __restrict__ bias,
                              uint32_t* __restrict__ cnt, float* __restrict__ G) {
    const TableDev tb = s.tables[t];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = rows[i];
        if (r < 0 || r >= tb.N) continue;
        const int64_t g = tb.row_base + r;
        if (codes) {
            for (int c = 0; c < code_bytes; ++c) codes[i * code_bytes + c] = s.codes[g * code_bytes + c];
            scale[i] = s.sb ? s.sb[g].x : 1.0f; bias[i] = s.sb ? s.sb[g].y : 0.0f;
        }
        if (cnt) cnt[i] = s.cnt ? s.cnt[g] : 0u;
        if (G) G[i] = s.G ? s.G[g] : 0.0f;
    }
}

// The reverse exchange before backward: this rank's columns of every rank's [B_local][T_global * dim] gradient buffer are
// pulled into one local [B][T * dim] array (plain loads from the owners' memory, 16 bytes per thread).
__global__ void __launch_bounds__(256)
k_gather_grad(const Route* __restrict__ r, float* __restrict__ dst, int64_t B, int T, int dim) {
    const int64_t row4 = (int64_t)T * dim / 4;
    const int64_t total = B * row4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t b = i / row4, c = i - b * row4;
        const int g = (int)(b / r->B_local);
        const float4* src = reinterpret_cast<const float4*>(r->out[g] + ((b - (int64_t)g * r->B_local) * r->T_global + r->t_base) * dim);
        reinterpret_cast<float4*>(dst)[i] = src[c];
    }
}

__global__ void k_fill_i32(int32_t* p, int64_t n, int32_t v) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) p[i] = v;
}

}  // namespace mpe

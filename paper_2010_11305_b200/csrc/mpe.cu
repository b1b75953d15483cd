// Host side of the C ABI declared in include/mpe.h: state, workspace, and the
// kernel sequence of one training step.  Nothing here computes on the host;
// every step of the path runs in the kernels of mpe_kernels.cuh.
#include "../../include/mpe.h"
#include "mpe_kernels.cuh"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <type_traits>
#include <vector>

using namespace mpe;

namespace {

struct ProfRec { int name; cudaEvent_t a, b; };

}  // namespace

struct mpe_handle {
    int device = 0, num_sms = 148;
    bool table_on_host = false;
    int T = 0, dim = 0, bits = 0, ways = 0, policy = 0, optimizer = 0, code_bytes = 0;
    float eps = 0, lo = 0, hi = 0;
    uint64_t seed = 0;
    std::vector<TableDev> tables;
    int64_t total_rows = 0, total_sets = 0, total_slots = 0;
    int32_t max_rows = 0, max_sets = 0;
    State st{};
    Work wk{};
    TableDev* d_tables = nullptr;
    // workspace
    int64_t cap_L = 0, cap_bags = 0;
    uint64_t ws_bytes = 0;                  // bytes of the per-step workspace
    uint32_t *sortA = nullptr, *sortB = nullptr;   // two buffers of 2 * sort_n words: (key, payload) records, or keys | payloads
    int64_t sort_n = 0;
    uint32_t *ghist = nullptr, *block_sums = nullptr;      // the sort's per-table digit counts; candidates per chunk of distinct rows (large steps)
    unsigned long long* sort_status = nullptr;             // the sort's per-tile words
    SortCtl* sort_ctl = nullptr;
    uint64_t sort_passes_bound = 0;                        // no more than this many sort passes have run on either workspace
    std::vector<void*> ws_allocs;
    cudaEvent_t ev_free = nullptr;          // recorded behind the last kernel that uses this workspace
    // A second workspace, allocated on the first mpe_prepare: the next batch is sorted and de-duplicated there while the
    // kernels of the current step still run.  `alt` holds exactly the members above that belong to a workspace.
    struct WsSet {
        Work wk{};
        uint32_t *sortA = nullptr, *sortB = nullptr, *ghist = nullptr, *block_sums = nullptr;
        unsigned long long* sort_status = nullptr; SortCtl* sort_ctl = nullptr;
        int64_t sort_n = 0;
        const uint32_t *skey = nullptr, *spos = nullptr;
        std::vector<void*> allocs;
        cudaEvent_t ev_free = nullptr;
        uint64_t bytes = 0;
    } alt;
    bool prepared = false;                  // `alt` holds a sorted batch that the next forward may take over
    StepArgs prep_args{};                   // ... of these inputs
    cudaEvent_t ev_prep = nullptr;
    cudaStream_t prep = nullptr;            // mpe_step_host_submit prepares on this stream
    // staging for mpe_step_host / mpe_step_host_submit: two slots, so that the copies of one step run next to the kernels of another
    struct HostSlot {
        int32_t *idx = nullptr, *off = nullptr; float *grad = nullptr, *out = nullptr;
        cudaEvent_t ev_idx = nullptr, ev_grad = nullptr, ev_fwd = nullptr, ev_done = nullptr, ev_down = nullptr;
        bool used = false;
    } slot[2];
    int64_t sh_cap_L = 0, sh_cap_off = 0, sh_cap_out = 0;
    uint64_t submitted = 0;
    // step state
    cudaStream_t stream = nullptr;
    cudaStream_t side = nullptr;            // runs the hot rows' partial sums next to the policy kernels
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;   // mpe_step_host: host<->device copies next to the kernels
    bool have_forward = false;
    bool fwd_replayed = false;              // the pending forward ran as a graph replay, so the device copy of its arguments is current
    int64_t last_step = 0;
    uint64_t steps = 0;
    uint32_t epoch = 0;
    int32_t B = 0; int64_t L = 0;
    const uint32_t *skey = nullptr, *spos = nullptr;
    StepArgs args{};                        // the current call's arguments (passed by value when launching directly)
    Route* d_route = nullptr;               // destinations of the pooled vectors when the tables are spread over several GPUs
    // CUDA graphs of the two halves of a step (small batches are launch-latency bound)
    bool graphs_enabled = true;
    cudaStream_t cap = nullptr;             // stream the step is captured on
    cudaGraph_t g_fwd = nullptr, g_bwd = nullptr;
    cudaGraphExec_t x_fwd = nullptr, x_bwd = nullptr;
    cudaGraphNode_t n_fwd = nullptr, n_bwd = nullptr;      // the nodes that write the per-call arguments
    uint64_t k_fwd = 0, k_bwd = 0;                         // kernel nodes per graph
    // instrumentation
    uint64_t launches = 0;
    bool profiling = false;
    std::vector<std::string> prof_names;
    std::vector<ProfRec> prof_recs;
    std::vector<cudaEvent_t> event_pool;
    int last_cuda_error = 0;
    std::map<const void*, int> resident;    // blocks per SM, per kernel
};

namespace {

struct DeviceGuard {
    int prev = 0;
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

#define CK(h, expr) do { cudaError_t e_ = (expr); if (e_ != cudaSuccess) { (h)->last_cuda_error = (int)e_; return e_ == cudaErrorMemoryAllocation ? MPE_ERR_NOMEM : MPE_ERR_CUDA; } } while (0)

cudaEvent_t get_event(mpe_handle* h) {
    if (!h->event_pool.empty()) { cudaEvent_t e = h->event_pool.back(); h->event_pool.pop_back(); return e; }
    cudaEvent_t e; cudaEventCreate(&e); return e;
}

int prof_name(mpe_handle* h, const char* name) {
    for (size_t i = 0; i < h->prof_names.size(); ++i) if (h->prof_names[i] == name) return (int)i;
    h->prof_names.push_back(name);
    return (int)h->prof_names.size() - 1;
}

struct LaunchScope {
    mpe_handle* h; cudaStream_t st; ProfRec rec{};
    LaunchScope(mpe_handle* h_, const char* name, cudaStream_t st_) : h(h_), st(st_) {
        ++h->launches;
        if (h->profiling) { rec.name = prof_name(h, name); rec.a = get_event(h); rec.b = get_event(h); cudaEventRecord(rec.a, st); }
    }
    ~LaunchScope() { if (h->profiling) { cudaEventRecord(rec.b, st); h->prof_recs.push_back(rec); } }
};

#define LAUNCH_ON(h, st, name, kern, grid, block, smem, ...) \
    do { LaunchScope ls_(h, name, st); kern<<<(grid), (block), (smem), (st)>>>(__VA_ARGS__); } while (0)
#define LAUNCH(h, name, kern, grid, block, smem, ...) LAUNCH_ON(h, (h)->stream, name, kern, grid, block, smem, __VA_ARGS__)

int grid_for(const mpe_handle* h, int64_t work_items, int64_t items_per_block, int blocks_per_sm) {
    int64_t need = (work_items + items_per_block - 1) / items_per_block;
    int64_t cap = (int64_t)h->num_sms * blocks_per_sm;
    return (int)std::max<int64_t>(1, std::min(need, cap));
}

// how many blocks of a kernel fit on one SM at a time (asked once per kernel): grids of the kernels that loop over their
// work are sized as whole waves of resident blocks, so that no kernel ends with a wave that fills a fraction of the GPU
template <class K>
int resident_blocks(mpe_handle* h, K kernel, int threads, size_t smem) {
    const void* key = reinterpret_cast<const void*>(kernel);
    auto it = h->resident.find(key);
    if (it != h->resident.end()) return it->second;
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem) != cudaSuccess || n < 1) { cudaGetLastError(); n = 1; }
    h->resident[key] = n;
    return n;
}

int bits_for(uint32_t v) { int b = 1; while (b < 32 && (v >> b) != 0) ++b; return b; }

template <class T>
int dmalloc(mpe_handle* h, T** p, int64_t n, std::vector<void*>* track) {
    *p = nullptr;
    cudaError_t e = cudaMalloc((void**)p, (size_t)std::max<int64_t>(n, 1) * sizeof(T));
    if (e != cudaSuccess) { h->last_cuda_error = (int)e; return MPE_ERR_NOMEM; }
    if (track) track->push_back(*p);
    return MPE_OK;
}

void drop_graphs(mpe_handle* h) {
    if (h->x_fwd) cudaGraphExecDestroy(h->x_fwd);
    if (h->x_bwd) cudaGraphExecDestroy(h->x_bwd);
    if (h->g_fwd) cudaGraphDestroy(h->g_fwd);
    if (h->g_bwd) cudaGraphDestroy(h->g_bwd);
    h->x_fwd = h->x_bwd = nullptr; h->g_fwd = h->g_bwd = nullptr; h->n_fwd = h->n_bwd = nullptr;
}

// the current workspace and the other one change places
void swap_sets(mpe_handle* h) {
    std::swap(h->wk, h->alt.wk);
    std::swap(h->sortA, h->alt.sortA); std::swap(h->sortB, h->alt.sortB);
    std::swap(h->ghist, h->alt.ghist); std::swap(h->block_sums, h->alt.block_sums);
    std::swap(h->sort_status, h->alt.sort_status); std::swap(h->sort_ctl, h->alt.sort_ctl);
    std::swap(h->sort_n, h->alt.sort_n);
    std::swap(h->skey, h->alt.skey); std::swap(h->spos, h->alt.spos);
    std::swap(h->ws_allocs, h->alt.allocs);
    std::swap(h->ev_free, h->alt.ev_free);
    std::swap(h->ws_bytes, h->alt.bytes);
}

void free_set(mpe_handle* h) {
    for (void* p : h->ws_allocs) cudaFree(p);
    h->ws_allocs.clear();
    h->wk = Work{};
    h->ws_bytes = 0;
}

void free_workspace(mpe_handle* h) {
    drop_graphs(h);                       // they hold the workspace's addresses
    free_set(h);
    swap_sets(h); free_set(h); swap_sets(h);
    h->prepared = false;
    h->cap_L = 0; h->cap_bags = 0;
}

// Steps this small are bound by launch latency (they are replayed from CUDA graphs); above it the launches hide behind the kernels.
constexpr int64_t GRAPH_MAX_INDICES = 4 << 20;

int alloc_set(mpe_handle* h, int64_t L, int64_t bags);

int64_t sort_max_tiles(const mpe_handle* h, int64_t L) {
    const int tile = sort_tile(L <= GRAPH_MAX_INDICES);
    return (L + tile - 1) / tile + h->T + 1;
}

// The sort's per-tile words carry a 30-bit pass number.  Long before it can come round to a value that old words still
// hold (hundreds of millions of steps), everything is brought to rest once and the words and the counter start over.
int renew_sort_tags(mpe_handle* h) {
    CK(h, cudaDeviceSynchronize());
    for (int set = 0; set < 2; ++set) {
        if (h->sort_status) {
            CK(h, cudaMemset(h->sort_status, 0, sizeof(unsigned long long) * 256 * sort_max_tiles(h, h->cap_L)));
            CK(h, cudaMemset(h->sort_ctl, 0, sizeof(SortCtl)));
        }
        swap_sets(h);
    }
    h->sort_passes_bound = 0;
    return MPE_OK;
}

int alloc_workspace(mpe_handle* h, int64_t L, int64_t bags) {
    free_workspace(h);
    int rc = alloc_set(h, L, bags);
    if (rc != MPE_OK) return rc;
    h->cap_L = L; h->cap_bags = bags;
    return MPE_OK;
}

int alloc_set(mpe_handle* h, int64_t L, int64_t bags) {
    // everything a step needs between its first and last kernel, sized for L indices
    (void)bags;
    free_set(h);
    auto* tr = &h->ws_allocs;
    const int T = h->T;
    const int64_t n = L + 1;
    // arrays with one entry per distinct row: there are at most as many distinct rows as indices, and at most as many
    // as the tables have rows (plus one pseudo row per table that collects its out-of-range ids)
    const int64_t nu = std::min<int64_t>(L, h->total_rows + T) + 2;
    Work& w = h->wk;
    int rc = MPE_OK;
    h->ws_bytes = 0;
#define A(ptr, count) do { if ((rc = dmalloc(h, &(ptr), (count), tr)) != MPE_OK) return rc; \
                           h->ws_bytes += (uint64_t)std::max<int64_t>((count), 1) * sizeof(*(ptr)); } while (0)
    // the sort's two buffers; the second sort (miss candidates by cache set) runs in backward, when the first sort's
    // results have been consumed, and uses the same two
    h->sort_n = (n + 3) & ~int64_t(3);
    A(h->sortA, 2 * h->sort_n); A(h->sortB, 2 * h->sort_n);
    // small batches (the ones that are replayed from a graph) get small tiles, so that every SM has one
    w.sort_tile = sort_tile(L <= GRAPH_MAX_INDICES);
    const int64_t max_tiles = sort_max_tiles(h, L);
    A(h->sort_status, 256 * max_tiles); A(h->ghist, (int64_t)T * SORT_MAX_PASSES * 256); A(h->sort_ctl, 1);
    // the sort keeps these consistent by itself from one pass to the next; they start from zero
    CK(h, cudaMemset(h->sort_status, 0, sizeof(unsigned long long) * 256 * max_tiles));
    CK(h, cudaMemset(h->ghist, 0, sizeof(uint32_t) * T * SORT_MAX_PASSES * 256));
    CK(h, cudaMemset(h->sort_ctl, 0, sizeof(SortCtl)));
    A(h->block_sums, n / std::min<int64_t>(SCAN_TILE, PRI_CHUNK) + 2);
    A(w.ctr, 1); A(w.args, 1);
    A(w.table_start, T + 1); A(w.tile_base, T + 1); A(w.ustart, T + 1); A(w.ctile_base, T + 1);
    A(w.bag_of, n); A(w.kidx, n); A(w.occ_loc, n); A(w.occ_b, n);
    A(w.uniq_row, nu); A(w.uniq_t, nu); A(w.seg, nu + 1); A(w.loc, nu); A(w.final_loc, nu);
    A(w.hot_base, nu); A(w.uset, nu); A(w.cand_key, nu); A(w.cand_cnt, T); A(w.cstart, T + 1);
    CK(h, cudaMemset(w.cand_cnt, 0, sizeof(int32_t) * T));
    // written and read by backward only, at most one entry per distinct row: they take the place of per-index arrays
    // that only forward uses
    w.victim = w.bag_of; w.defer_k = reinterpret_cast<int32_t*>(w.kidx); w.heads = w.occ_loc;
    const int64_t max_tasks = hot_capacity(L);
    A(w.task_k, max_tasks); A(w.partial, max_tasks * h->dim); A(w.hot_k, max_tasks);
#undef A
    CK(h, cudaMemset(w.ctr, 0, sizeof(Counters)));
    return MPE_OK;
}

// The sort's memory: two buffers of 2 * n words each.  The keys to sort are expected in the first n words of B
// (sort_input()); between passes the elements are (key, payload) records that alternate between A and B; the last
// pass leaves the sorted keys in the first n words and the sorted payloads in the second n words of its buffer.
struct SortBufs { uint32_t *A, *B; int64_t n; uint32_t* ghist; unsigned long long* status; SortCtl* ctl; uint32_t* abort_flag; int tile; };
uint32_t* sort_input(const SortBufs& b) { return b.B; }

// stable sort of every segment [seg_start[t], seg_start[t+1]) by the low `key_bits` bits of the key, the payload being
// the element's position before the sort; *skey / *sval receive where the sorted keys / payloads are
// tile_base: the segments' tile bookkeeping (warp_tile_bases), filled by the kernel that produced seg_start
void seg_sort(mpe_handle* h, const SortBufs& b, const int32_t* seg_start, const int32_t* tile_base,
              int key_bits, int64_t n_upper, const uint32_t** skey, const uint32_t** sval, bool input_pairs = false) {
    const int T = h->T;
    const int64_t max_tiles = (n_upper + b.tile - 1) / b.tile + T;
    const int passes = (key_bits + 7) / 8;
    const int split = b.tile == sort_tile(true) ? 4 : 1;         // pieces of a tile the digit count hands to its warps
    const int gh = grid_for(h, max_tiles * split, SORT_THREADS / 32, 4);
    if (input_pairs) LAUNCH(h, "sort_digits", k_sort_digits<true>, gh, SORT_THREADS, 0, (const uint32_t*)b.B, seg_start, tile_base, T, passes, b.ghist, b.tile, split);
    else LAUNCH(h, "sort_digits", k_sort_digits<false>, gh, SORT_THREADS, 0, (const uint32_t*)b.B, seg_start, tile_base, T, passes, b.ghist, b.tile, split);
    for (int p = 0; p < passes; ++p) {
        const bool first = p == 0 && !input_pairs, last = p == passes - 1;    // input_pairs: B holds (key, payload) records already
        uint32_t* src = (p & 1) ? b.A : b.B;                      // pass p reads B and writes A when p is even, the other way round when odd
        uint32_t* dst = (p & 1) ? b.B : b.A;
        const uint32_t* kin = src; const uint2* pin = reinterpret_cast<const uint2*>(src);
        uint2* pout = reinterpret_cast<uint2*>(dst); uint32_t* ok = dst; uint32_t* ov = dst + b.n;
        // tiles are handed out by ticket, so the grid only has to be large enough to fill the GPU
#define SCATTER(F, L) do { \
        if (b.tile == sort_tile(true)) { \
            auto kern = k_sort_scatter<F, L, SORT_ITEMS_SMALL>; \
            LAUNCH(h, "sort_scatter", kern, grid_for(h, max_tiles, 1, resident_blocks(h, kern, SORT_THREADS, 0)), SORT_THREADS, 0, kin, pin, pout, ok, ov, \
                   seg_start, tile_base, T, p, b.ghist, b.status, b.ctl, b.abort_flag); \
        } else { \
            auto kern = k_sort_scatter<F, L, SORT_ITEMS_LARGE>; \
            LAUNCH(h, "sort_scatter", kern, grid_for(h, max_tiles, 1, resident_blocks(h, kern, SORT_THREADS, 0)), SORT_THREADS, 0, kin, pin, pout, ok, ov, \
                   seg_start, tile_base, T, p, b.ghist, b.status, b.ctl, b.abort_flag); \
        } } while (0)
        if (first && last) SCATTER(true, true);
        else if (first) SCATTER(true, false);
        else if (last) SCATTER(false, true);
        else SCATTER(false, false);
#undef SCATTER
        if (last) { *skey = dst; *sval = dst + b.n; }
    }
}

// call f(integral_constant<BITS>, integral_constant<LANES>) for the handle's code width and lanes per row
template <class F>
void dispatch(int bits, int lanes, F&& f) {
#ifdef MPE_ONLY_BITS        // development builds: one code width and one row width only (much shorter compile)
    (void)bits; (void)lanes;
    f(std::integral_constant<int, MPE_ONLY_BITS>{}, std::integral_constant<int, MPE_ONLY_LANES>{});
    return;
#endif
    auto by_lanes = [&](auto bc) {
        switch (lanes) {
            case 1: f(bc, std::integral_constant<int, 1>{}); break;
            case 2: f(bc, std::integral_constant<int, 2>{}); break;
            case 4: f(bc, std::integral_constant<int, 4>{}); break;
            case 8: f(bc, std::integral_constant<int, 8>{}); break;
            case 16: f(bc, std::integral_constant<int, 16>{}); break;
            default: f(bc, std::integral_constant<int, 32>{}); break;
        }
    };
    if (bits == 8) by_lanes(std::integral_constant<int, 8>{});
    else if (bits == 4) by_lanes(std::integral_constant<int, 4>{});
    else if (bits == 2) by_lanes(std::integral_constant<int, 2>{});
    else by_lanes(std::integral_constant<int, 16>{});
}

int check_launch(mpe_handle* h) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { h->last_cuda_error = (int)e; return MPE_ERR_CUDA; }
    return MPE_OK;
}

}  // namespace

extern "C" {

const char* mpe_error_string(int code) {
    switch (code) {
        case MPE_OK: return "ok";
        case MPE_ERR_ARG: return "bad argument";
        case MPE_ERR_UNSUPPORTED: return "unsupported configuration";
        case MPE_ERR_CUDA: return "CUDA runtime error";
        case MPE_ERR_SEQUENCE: return "call out of sequence";
        case MPE_ERR_INDEX: return "row index out of range";
        case MPE_ERR_OFFSETS: return "inconsistent offsets";
        case MPE_ERR_NOMEM: return "out of memory";
        case MPE_ERR_TOO_LARGE: return "batch larger than the fixed scratch of mpe_forward_static";
        case MPE_ERR_TIMEOUT: return "a bounded wait between thread blocks ran out";
        default: return "unknown error";
    }
}

int mpe_create(mpe_handle** out, const mpe_table_spec* tables, int32_t num_tables, int32_t bits,
               double cache_fraction, int32_t ways, int32_t policy, int32_t optimizer, float eps,
               float init_lo, float init_hi, uint64_t seed, int32_t device) {
    return mpe_create_placed(out, tables, num_tables, bits, cache_fraction, ways, policy, optimizer, eps, init_lo, init_hi, seed,
                             device, MPE_TABLE_DEVICE);
}

int mpe_create_placed(mpe_handle** out, const mpe_table_spec* tables, int32_t num_tables, int32_t bits,
                      double cache_fraction, int32_t ways, int32_t policy, int32_t optimizer, float eps,
                      float init_lo, float init_hi, uint64_t seed, int32_t device, int32_t table_placement) {
    if (!out || !tables || num_tables < 1) return MPE_ERR_ARG;
    if (table_placement != MPE_TABLE_DEVICE && table_placement != MPE_TABLE_HOST) return MPE_ERR_ARG;
    *out = nullptr;
    if (!(cache_fraction >= 0.0 && cache_fraction <= 1.0)) return MPE_ERR_ARG;
    if (policy != MPE_LRU && policy != MPE_LFU) return MPE_ERR_ARG;
    if (optimizer != MPE_SGD && optimizer != MPE_ROWWISE_ADAGRAD) return MPE_ERR_ARG;
    if (bits != 8 && bits != 4 && bits != 2 && bits != 16) return MPE_ERR_UNSUPPORTED;
    if (ways == 0) ways = 32;
    if (ways < 1 || ways > 32 || (ways & (ways - 1))) return MPE_ERR_UNSUPPORTED;
    const int dim = tables[0].dim;
    if (dim < 4 || dim > 128 || (dim & (dim - 1))) return MPE_ERR_UNSUPPORTED;
    for (int t = 0; t < num_tables; ++t) {
        if (tables[t].dim != dim) return MPE_ERR_UNSUPPORTED;
        if (tables[t].num_rows < 1 || tables[t].num_rows > 0x7ffffffeLL) return MPE_ERR_ARG;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return MPE_ERR_CUDA;

    mpe_handle* h = new mpe_handle();
    h->device = device;
    h->table_on_host = table_placement == MPE_TABLE_HOST;
    DeviceGuard guard(device);
    cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, device);
    if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h->cap, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h->prep, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_free, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_prep, cudaEventDisableTiming) != cudaSuccess ||
        false) { delete h; return MPE_ERR_CUDA; }
    for (auto& sl : h->slot)
        for (cudaEvent_t* e : {&sl.ev_idx, &sl.ev_grad, &sl.ev_fwd, &sl.ev_done, &sl.ev_down})
            if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) { delete h; return MPE_ERR_CUDA; }
    h->T = num_tables; h->dim = dim; h->bits = bits; h->ways = ways; h->policy = policy; h->optimizer = optimizer;
    h->code_bytes = dim * bits / 8; h->eps = eps; h->lo = init_lo; h->hi = init_hi; h->seed = seed;
    h->tables.resize(num_tables);
    for (int t = 0; t < num_tables; ++t) {
        TableDev& tb = h->tables[t];
        tb.row_base = h->total_rows; tb.set_base = h->total_sets;
        tb.N = (int32_t)tables[t].num_rows;
        int64_t n = 0;
        if (cache_fraction > 0.0) {
            const int64_t cache_rows = (int64_t)std::floor(cache_fraction * (double)tables[t].num_rows + 1e-6);
            n = std::max<int64_t>(1, cache_rows / ways);
        }
        tb.n_sets = (int32_t)n;
        tb.salt = table_salt(seed, (uint32_t)t);
        tb.pad = 0;
        h->total_rows += tb.N; h->total_sets += n;
        h->max_rows = std::max(h->max_rows, tb.N); h->max_sets = std::max(h->max_sets, tb.n_sets);
    }
    h->total_slots = h->total_sets * ways;
    // slots are int32; one sample's row of the pooled output must stay below 4 GiB (32-bit byte strides in the kernels)
    if (h->total_slots > 0x7fffffffLL || (int64_t)num_tables * dim > 0x0fffffffLL) { delete h; return MPE_ERR_UNSUPPORTED; }

    State& s = h->st;
    s.T = num_tables; s.dim = dim; s.lanes = dim / 4; s.ways = ways; s.policy = policy; s.optimizer = optimizer;
    s.bits = bits; s.seed = seed; s.eps = eps; s.rounding = 1;
    int rc = MPE_OK;
    auto fail = [&](int code) { mpe_destroy(h); return code; };
    if ((rc = dmalloc(h, &h->d_tables, num_tables, nullptr)) != MPE_OK) return fail(rc);
    s.tables = h->d_tables;
    if (h->table_on_host) {
        // capacity tiering: the low-precision table stays in pinned host memory and is read and written in place over
        // the host link; the FP32 cache, tags, counters and optimizer state stay in HBM
        if (cudaHostAlloc((void**)&s.codes, (size_t)h->total_rows * h->code_bytes, cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess)
            return fail(MPE_ERR_NOMEM);
        if (bits != 16 && cudaHostAlloc((void**)&s.sb, (size_t)h->total_rows * sizeof(float2), cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess)
            return fail(MPE_ERR_NOMEM);
    } else {
        if ((rc = dmalloc(h, &s.codes, h->total_rows * h->code_bytes, nullptr)) != MPE_OK) return fail(rc);
        if (bits != 16 && (rc = dmalloc(h, &s.sb, h->total_rows, nullptr)) != MPE_OK) return fail(rc);   // an FP16 table has no scale/bias
    }
    if (policy == MPE_LFU && (rc = dmalloc(h, &s.cnt, h->total_rows, nullptr)) != MPE_OK) return fail(rc);
    if (optimizer == MPE_ROWWISE_ADAGRAD && (rc = dmalloc(h, &s.G, h->total_rows, nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.slab, h->total_slots * dim, nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.tags, h->total_slots, nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.ts, h->total_slots, nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.hit_epoch, h->total_slots, nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.hit_k, h->total_slots, nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.floor, std::max<int64_t>(1, h->total_sets), nullptr)) != MPE_OK) return fail(rc);
    if ((rc = dmalloc(h, &s.stats, (int64_t)num_tables * 8, nullptr)) != MPE_OK) return fail(rc);
#define CKC(expr) do { cudaError_t e_ = (expr); if (e_ != cudaSuccess) { h->last_cuda_error = (int)e_; return fail(MPE_ERR_CUDA); } } while (0)
    CKC(cudaMemcpy(h->d_tables, h->tables.data(), sizeof(TableDev) * num_tables, cudaMemcpyHostToDevice));
    if (s.cnt) CKC(cudaMemset(s.cnt, 0, sizeof(uint32_t) * h->total_rows));
    if (s.G) CKC(cudaMemset(s.G, 0, sizeof(float) * h->total_rows));
    CKC(cudaMemset(s.slab, 0, sizeof(float) * std::max<int64_t>(1, h->total_slots * dim)));
    if (s.ts) CKC(cudaMemset(s.ts, 0, sizeof(uint32_t) * std::max<int64_t>(1, h->total_slots)));
    CKC(cudaMemset(s.hit_epoch, 0, sizeof(uint32_t) * std::max<int64_t>(1, h->total_slots)));
    CKC(cudaMemset(s.floor, 0, sizeof(uint32_t) * std::max<int64_t>(1, h->total_sets)));
    CKC(cudaMemset(s.stats, 0, sizeof(unsigned long long) * 8 * num_tables));
    LAUNCH(h, "fill_tags", k_fill_i32, grid_for(h, h->total_slots, 256, 8), 256, 0, s.tags, h->total_slots, -1);
    for (int t = 0; t < num_tables; ++t) {
        const int g = grid_for(h, h->tables[t].N, 256 / s.lanes, 8);
        if (bits == 8) LAUNCH(h, "init_table", k_init_table<8>, g, 256, 0, s, t, init_lo, init_hi);
        else if (bits == 4) LAUNCH(h, "init_table", k_init_table<4>, g, 256, 0, s, t, init_lo, init_hi);
        else if (bits == 2) LAUNCH(h, "init_table", k_init_table<2>, g, 256, 0, s, t, init_lo, init_hi);
        else LAUNCH(h, "init_table", k_init_table<16>, g, 256, 0, s, t, init_lo, init_hi);
    }
    CKC(cudaGetLastError());
    CKC(cudaDeviceSynchronize());
#undef CKC
    *out = h;
    return MPE_OK;
}

int mpe_reserve(mpe_handle* h, int32_t max_batch, int64_t max_total_indices) {
    if (!h || max_batch < 0 || max_total_indices < 0 || max_total_indices > 0x7ffffff0LL) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    const int64_t bags = (int64_t)h->T * max_batch;
    if (max_total_indices <= h->cap_L && bags <= h->cap_bags && h->wk.ctr) return MPE_OK;
    if (h->have_forward) return MPE_ERR_SEQUENCE;     // a pending backward still needs the old workspace
    CK(h, cudaStreamSynchronize(h->stream));
    if (h->ev_prep) CK(h, cudaEventSynchronize(h->ev_prep));       // so does a batch that is being prepared
    return alloc_workspace(h, std::max(max_total_indices, h->cap_L), std::max(bags, h->cap_bags));
}

}  // extern "C"

namespace {

// Launch sizes follow L_grid / bags_grid (upper bounds: every kernel walks its range with a grid stride and reads the
// true sizes from device memory), so one captured graph serves every batch that fits the workspace.
// First half of forward, which needs the indices only (no table, cache or policy state): keys, sort, distinct rows.
void enqueue_index_chain(mpe_handle* h, int64_t L_grid, int64_t bags_grid, bool ind, const StepArgs& av) {
    const State& s = h->st;
    Work& w = h->wk;
    const int T = h->T;
    LAUNCH(h, "prelude", (ind ? k_prelude<true> : k_prelude<false>), 1, 32, 0, w, T, av);
    const SortBufs sb{h->sortA, h->sortB, h->sort_n, h->ghist, h->sort_status, h->sort_ctl, &h->wk.ctr->abort, h->wk.sort_tile};
    LAUNCH(h, "make_keys", (ind ? k_make_keys<true> : k_make_keys<false>), grid_for(h, bags_grid, 32, 8), 256, 0, s, w, sort_input(sb), av);
    // sort the row indices of the mini-batch (Section 5.1), table by table
    seg_sort(h, sb, w.table_start, w.tile_base, bits_for((uint32_t)h->max_rows), L_grid, &h->skey, &h->spos);
    // distinct rows
    const int gs = grid_for(h, L_grid, SCAN_TILE, 8);
    if (ind) {
        LAUNCH(h, "unique", k_unique, gs, SCAN_THREADS, 0, w, T, h->skey, h->sort_status, h->sort_ctl);
    } else {
        LAUNCH(h, "unique_count", k_unique_pass<false>, gs, SCAN_THREADS, 0, w, T, h->skey, h->block_sums);
        LAUNCH(h, "scan_block_sums", k_scan_block_sums, 1, BSUM_THREADS, 0, h->block_sums, (const uint32_t*)&w.ctr->L, (uint32_t)SCAN_TILE, &w.ctr->U);
        LAUNCH(h, "unique_write", k_unique_pass<true>, gs, SCAN_THREADS, 0, w, T, h->skey, h->block_sums);
        LAUNCH(h, "ustart", k_ustart, 1, 256, 0, w, T);
    }
}

// Second half: tag lookup, then fetch + pool.
void enqueue_lookup(mpe_handle* h, int64_t L_grid, int64_t bags_grid, bool ind, const StepArgs& av) {
    const State& s = h->st;
    Work& w = h->wk;
    LAUNCH(h, "probe", (ind ? k_probe<true> : k_probe<false>), grid_for(h, L_grid, 256, 8), 256, 0, s, w, av);
    LAUNCH(h, "broadcast", (ind ? k_broadcast<true> : k_broadcast<false>), grid_for(h, L_grid, 256, 8), 256, 0, s, w, h->spos, av);
    const int gp = grid_for(h, bags_grid, 256 / s.lanes, 8);
    dispatch(h->bits, s.lanes, [&](auto bc, auto lc) {
        constexpr int BITS = decltype(bc)::value, LANES = decltype(lc)::value;
        auto kern = ind ? k_pool<BITS, LANES, true> : k_pool<BITS, LANES, false>;
        LAUNCH(h, "pool", kern, gp, 256, 0, s, w, av);
    });
}

int enqueue_forward(mpe_handle* h, int64_t L_grid, int64_t bags_grid, bool ind) {
    const StepArgs av = h->args;
    enqueue_index_chain(h, L_grid, bags_grid, ind, av);
    enqueue_lookup(h, L_grid, bags_grid, ind, av);
    return check_launch(h);
}

int enqueue_backward(mpe_handle* h, int64_t L, bool ind) {
    const State& s = h->st;
    Work& w = h->wk;
    const StepArgs av = h->args;
    // the hot rows' partial gradient sums only need the sorted batch: they run on a second stream next to the
    // priority / candidate-sort / policy kernels, which leave most of the machine idle
    CK(h, cudaEventRecord(h->ev_fork, h->stream));
    CK(h, cudaStreamWaitEvent(h->side, h->ev_fork, 0));
    dispatch(h->bits, s.lanes, [&](auto bc, auto lc) {
        constexpr int LANES = decltype(lc)::value;
        auto hot = ind ? k_hot_partial<LANES, true> : k_hot_partial<LANES, false>;
        LAUNCH_ON(h, h->side, "hot_partial", hot, grid_for(h, hot_capacity(L), 1, 2), 8 * LANES, 32 * s.dim * sizeof(float), s, w, av);
    });
    CK(h, cudaEventRecord(h->ev_join, h->side));
    const SortBufs sb{h->sortA, h->sortB, h->sort_n, h->ghist, h->sort_status, h->sort_ctl, &h->wk.ctr->abort, h->wk.sort_tile};
    // new priority values; the rows that may be admitted (few, once the caches are warm) are gathered in row order ...
    LAUNCH(h, "priority", (ind ? k_priority<true> : k_priority<false>), grid_for(h, L, PRI_CHUNK, 8), 256, 0, s, w,
           h->max_sets > 0 ? reinterpret_cast<uint2*>(sb.B) : (uint2*)nullptr, h->sort_status, h->sort_ctl, h->block_sums, av);
    if (h->max_sets > 0) {
        if (!ind) {        // large steps: the list is made by three small kernels
            LAUNCH(h, "scan_block_sums", k_scan_block_sums, 1, BSUM_THREADS, 0, h->block_sums, (const uint32_t*)&w.ctr->U, (uint32_t)PRI_CHUNK, &w.ctr->n_cand);
            LAUNCH(h, "cand_write", k_cand_write, grid_for(h, L, PRI_CHUNK, 8), 256, 0, s, w, (const uint32_t*)h->block_sums, reinterpret_cast<uint2*>(sb.B));
            LAUNCH(h, "cand_starts", k_cand_starts, 1, 32, 0, w, h->T);
        }
        // ... and grouped by cache set, keeping ascending row id inside a set
        const uint32_t *ck = nullptr, *cv = nullptr;
        seg_sort(h, sb, w.cstart, w.ctile_base, bits_for((uint32_t)h->max_sets), L, &ck, &cv, true);
        LAUNCH(h, "policy_heads", k_policy_heads, grid_for(h, L, 256, 8), 256, 0, s, w, ck);
        auto pol = ind ? k_policy<true> : k_policy<false>;
        LAUNCH(h, "policy", pol, grid_for(h, std::min<int64_t>(L, h->total_sets), 256 / s.ways, resident_blocks(h, pol, 256, 0)), 256, 0, s, w, ck, cv, av);
    }
    const int gu = grid_for(h, (L + 7) / 8, UPD_WARPS, 8);
    const int gh = grid_for(h, hot_capacity(L), 256 / s.lanes, 4);
    dispatch(h->bits, s.lanes, [&](auto bc, auto lc) {
        constexpr int BITS = decltype(bc)::value, LANES = decltype(lc)::value;
        auto upd = ind ? k_update<BITS, LANES, true> : k_update<BITS, LANES, false>;
        auto lst = ind ? k_update_list<BITS, LANES, true> : k_update_list<BITS, LANES, false>;
        LAUNCH(h, "update", upd, gu, UPD_WARPS * 32, UPD_SMEM, s, w, av);
        cudaStreamWaitEvent(h->stream, h->ev_join, 0);
        LAUNCH(h, "update_hot", lst, gh, 256, 0, s, w, (const int32_t*)w.hot_k, (const uint32_t*)&w.ctr->hot_rows, 0, av);
        if (h->max_sets > 0)
            LAUNCH(h, "update_deferred", lst, gh, 256, 0, s, w, (const int32_t*)w.defer_k, (const uint32_t*)&w.ctr->deferred, 1, av);
    });
    return check_launch(h);
}


bool may_use_graph(mpe_handle* h) {
    if (!h->graphs_enabled || h->profiling || h->cap_L > GRAPH_MAX_INDICES) return false;
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(h->stream, &st) != cudaSuccess || st != cudaStreamCaptureStatusNone) return false;   // the caller captures: plain launches join his graph
    return true;
}

// Capture one half of the step (sized for the whole workspace) into a graph; `head` is the kernel that writes the arguments.
template <class Body>
int capture(mpe_handle* h, cudaGraph_t* graph, cudaGraphExec_t* exec, cudaGraphNode_t* args_node, uint64_t* kernels, const void* head,
            Body&& body) {
    cudaStream_t user = h->stream;
    const uint64_t launches_before = h->launches;
    h->stream = h->cap;
    cudaError_t e = cudaStreamBeginCapture(h->cap, cudaStreamCaptureModeThreadLocal);
    int rc = MPE_OK;
    if (e == cudaSuccess) {
        rc = body();
        e = cudaStreamEndCapture(h->cap, graph);
    }
    h->stream = user;
    h->launches = launches_before;
    if (e != cudaSuccess || rc != MPE_OK || !*graph) { h->last_cuda_error = (int)e; cudaGetLastError(); return rc != MPE_OK ? rc : MPE_ERR_CUDA; }
    CK(h, cudaGraphInstantiate(exec, *graph, 0));
    size_t n = 0;
    CK(h, cudaGraphGetNodes(*graph, nullptr, &n));
    std::vector<cudaGraphNode_t> nodes(n);
    CK(h, cudaGraphGetNodes(*graph, nodes.data(), &n));
    *args_node = nullptr; *kernels = 0;
    for (cudaGraphNode_t nd : nodes) {
        cudaGraphNodeType ty;
        CK(h, cudaGraphNodeGetType(nd, &ty));
        if (ty != cudaGraphNodeTypeKernel) continue;
        ++*kernels;
        cudaKernelNodeParams kp{};
        CK(h, cudaGraphKernelNodeGetParams(nd, &kp));
        if (kp.func == head) *args_node = nd;
    }
    return *args_node ? MPE_OK : MPE_ERR_CUDA;
}

// forward with the pooled vectors going either to d_out (route == nullptr) or to the buffers the route names
int forward_impl(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch,
                 int64_t total_indices, float* d_out, const Route* route) {
    h->have_forward = false;
    const int64_t bags = (int64_t)h->T * batch;
    if (total_indices > h->cap_L || bags > h->cap_bags || !h->wk.ctr) {
        int rc = mpe_reserve(h, batch, total_indices);
        if (rc != MPE_OK) return rc;
    }
    h->sort_passes_bound += 4 * SORT_MAX_PASSES;       // this step's two sorts, and those of a batch prepared meanwhile
    if (h->sort_passes_bound > SORT_TAG_MASK - 1024) { int rc = renew_sort_tags(h); if (rc != MPE_OK) return rc; }
    Work& w = h->wk;
    uint32_t L = (uint32_t)total_indices;
    h->B = batch; h->L = total_indices; ++h->epoch;
    h->args.indices = d_indices; h->args.offsets = d_offsets; h->args.out = d_out; h->args.B = batch; h->args.L = L; h->args.epoch = h->epoch;
    h->args.route = route;
    int rc = MPE_OK;
    if (may_use_graph(h)) {
        if (!h->x_fwd) {
            // the graph's first kernel, k_prelude, is the one whose parameters change from call to call
            rc = capture(h, &h->g_fwd, &h->x_fwd, &h->n_fwd, &h->k_fwd, (const void*)k_prelude<true>, [&]() {
                return enqueue_forward(h, h->cap_L, h->cap_bags, true);
            });
            if (rc != MPE_OK) { drop_graphs(h); h->graphs_enabled = false; }      // fall back to plain launches for good
        }
        if (rc == MPE_OK) {
            Work wv = w; int T = h->T; StepArgs av = h->args;
            void* params[] = {&wv, &T, &av};
            cudaKernelNodeParams kp{};
            kp.func = (void*)k_prelude<true>; kp.gridDim = dim3(1); kp.blockDim = dim3(32); kp.kernelParams = params;
            CK(h, cudaGraphExecKernelNodeSetParams(h->x_fwd, h->n_fwd, &kp));
            CK(h, cudaGraphLaunch(h->x_fwd, h->stream));
            h->launches += h->k_fwd;
            h->have_forward = true; h->fwd_replayed = true;
            return MPE_OK;
        }
    }
    if (h->prepared && h->prep_args.indices == d_indices && h->prep_args.offsets == d_offsets && h->prep_args.B == batch &&
        h->prep_args.L == L) {
        // the batch was sorted and de-duplicated ahead of time in the other workspace: it becomes the current one
        h->prepared = false;
        swap_sets(h);
        CK(h, cudaStreamWaitEvent(h->stream, h->ev_prep, 0));
        enqueue_lookup(h, total_indices, bags, false, h->args);
        rc = check_launch(h);
    } else {
        h->prepared = false;                 // whatever was prepared was for another batch
        rc = enqueue_forward(h, total_indices, bags, false);
    }
    if (rc != MPE_OK) return rc;
    if (h->ev_free) CK(h, cudaEventRecord(h->ev_free, h->stream));
    h->have_forward = true; h->fwd_replayed = false;
    return MPE_OK;
}

// see mpe_prepare in mpe.h
int prepare_impl(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch, int64_t total_indices,
                 cudaStream_t stream) {
    const int64_t bags = (int64_t)h->T * batch;
    h->prepared = false;
    // only what fits the reserved workspace, and only steps that are launched plainly (replayed steps are bound by launch
    // latency, not by their kernels): otherwise the forward simply does all of its work itself
    if (total_indices > h->cap_L || bags > h->cap_bags || !h->wk.ctr || may_use_graph(h)) return MPE_OK;
    if (!h->alt.wk.ctr) {                    // first use: the second workspace
        swap_sets(h);
        int rc = alloc_set(h, h->cap_L, h->cap_bags);
        if (rc == MPE_OK && !h->ev_free && cudaEventCreateWithFlags(&h->ev_free, cudaEventDisableTiming) != cudaSuccess) rc = MPE_ERR_CUDA;
        if (rc != MPE_OK) free_set(h);
        swap_sets(h);
        if (rc != MPE_OK) return rc;
    }
    StepArgs av{};
    av.indices = d_indices; av.offsets = d_offsets; av.B = batch; av.L = (uint32_t)total_indices;
    cudaStream_t user = h->stream;
    swap_sets(h);
    h->stream = stream;
    cudaError_t e = h->ev_free ? cudaStreamWaitEvent(stream, h->ev_free, 0) : cudaSuccess;   // the step that used this workspace last has finished
    if (e == cudaSuccess) {
        enqueue_index_chain(h, total_indices, bags, false, av);
        e = cudaEventRecord(h->ev_prep, stream);
    }
    int rc = check_launch(h);
    h->stream = user;
    swap_sets(h);
    if (e != cudaSuccess) { h->last_cuda_error = (int)e; return MPE_ERR_CUDA; }
    if (rc != MPE_OK) return rc;
    h->prepared = true;
    h->prep_args = av;
    return MPE_OK;
}

int check_route(const mpe_handle* h, const void* const* ptrs, int32_t n_ranks, int32_t tables_global, int32_t table_base, int32_t batch) {
    if (!ptrs || n_ranks < 1 || n_ranks > MAX_RANKS || batch < 0 || batch % n_ranks != 0) return MPE_ERR_ARG;
    if (table_base < 0 || tables_global < table_base + h->T) return MPE_ERR_ARG;
    for (int g = 0; g < n_ranks; ++g)
        if (!ptrs[g] || (reinterpret_cast<uintptr_t>(ptrs[g]) & 15)) return MPE_ERR_ARG;
    return MPE_OK;
}

// the route travels to the device as a kernel argument, so the caller's array may be reused at once
int send_route(mpe_handle* h, const void* const* ptrs, int32_t n_ranks, int32_t tables_global, int32_t table_base, int32_t batch) {
    if (!h->d_route) CK(h, cudaMalloc(&h->d_route, sizeof(Route)));
    Route r{};
    for (int g = 0; g < n_ranks; ++g) r.out[g] = const_cast<float*>(static_cast<const float*>(ptrs[g]));
    r.B_local = batch / n_ranks > 0 ? batch / n_ranks : 1; r.T_global = tables_global; r.t_base = table_base; r.n_ranks = n_ranks;
    LAUNCH(h, "set_route", k_set_route, 1, 128, 0, h->d_route, r);
    return MPE_OK;
}

}  // namespace

extern "C" {

int mpe_forward(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch,
                int64_t total_indices, float* d_out, void* cuda_stream) {
    if (!h || !d_offsets || batch < 0 || total_indices < 0 || total_indices > 0x7ffffff0LL) return MPE_ERR_ARG;
    if ((total_indices > 0 && !d_indices) || (batch > 0 && !d_out)) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (stream != h->stream) { CK(h, cudaStreamSynchronize(h->stream)); h->stream = stream; }
    return forward_impl(h, d_indices, d_offsets, batch, total_indices, d_out, nullptr);
}

int mpe_prepare(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch, int64_t total_indices,
                void* cuda_stream) {
    if (!h || !d_offsets || batch < 0 || total_indices < 0 || total_indices > 0x7ffffff0LL) return MPE_ERR_ARG;
    if (total_indices > 0 && !d_indices) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    return prepare_impl(h, d_indices, d_offsets, batch, total_indices, (cudaStream_t)cuda_stream);
}

int mpe_forward_routed(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch, int64_t total_indices,
                       float* const* out_ptrs, int32_t n_ranks, int32_t tables_global, int32_t table_base, void* cuda_stream) {
    if (!h || !d_offsets || batch < 0 || total_indices < 0 || total_indices > 0x7ffffff0LL) return MPE_ERR_ARG;
    if (total_indices > 0 && !d_indices) return MPE_ERR_ARG;
    int rc = check_route(h, reinterpret_cast<const void* const*>(out_ptrs), n_ranks, tables_global, table_base, batch);
    if (rc != MPE_OK) return rc;
    DeviceGuard guard(h->device);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (stream != h->stream) { CK(h, cudaStreamSynchronize(h->stream)); h->stream = stream; }
    rc = send_route(h, reinterpret_cast<const void* const*>(out_ptrs), n_ranks, tables_global, table_base, batch);
    if (rc != MPE_OK) return rc;
    return forward_impl(h, d_indices, d_offsets, batch, total_indices, nullptr, h->d_route);
}

int mpe_gather_grad(mpe_handle* h, const float* const* grad_ptrs, int32_t n_ranks, int32_t tables_global, int32_t table_base,
                    int32_t batch, float* d_grad_local, void* cuda_stream) {
    if (!h || (batch > 0 && !d_grad_local) || (reinterpret_cast<uintptr_t>(d_grad_local) & 15)) return MPE_ERR_ARG;
    int rc = check_route(h, reinterpret_cast<const void* const*>(grad_ptrs), n_ranks, tables_global, table_base, batch);
    if (rc != MPE_OK) return rc;
    DeviceGuard guard(h->device);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (stream != h->stream) { CK(h, cudaStreamSynchronize(h->stream)); h->stream = stream; }
    rc = send_route(h, reinterpret_cast<const void* const*>(grad_ptrs), n_ranks, tables_global, table_base, batch);
    if (rc != MPE_OK) return rc;
    const int64_t total4 = (int64_t)batch * h->T * h->dim / 4;
    if (total4 > 0)
        LAUNCH(h, "gather_grad", k_gather_grad, grid_for(h, total4, 256, 8), 256, 0, (const Route*)h->d_route, d_grad_local,
               (int64_t)batch, h->T, h->dim);
    return check_launch(h);
}

int mpe_peer_buffer_alloc(int32_t device, int64_t bytes, void** d_ptr, void* ipc_handle) {
    if (!d_ptr || !ipc_handle || bytes <= 0) return MPE_ERR_ARG;
    static_assert(sizeof(cudaIpcMemHandle_t) == MPE_IPC_HANDLE_BYTES, "handle size");
    DeviceGuard guard(device);
    void* p = nullptr;
    cudaError_t e = cudaMalloc(&p, (size_t)bytes);
    if (e != cudaSuccess) return e == cudaErrorMemoryAllocation ? MPE_ERR_NOMEM : MPE_ERR_CUDA;
    cudaIpcMemHandle_t hd;
    e = cudaIpcGetMemHandle(&hd, p);
    if (e != cudaSuccess) { cudaFree(p); return MPE_ERR_CUDA; }
    std::memcpy(ipc_handle, &hd, sizeof(hd));
    *d_ptr = p;
    return MPE_OK;
}

int mpe_peer_buffer_open(int32_t device, const void* ipc_handle, void** d_ptr) {
    if (!d_ptr || !ipc_handle) return MPE_ERR_ARG;
    DeviceGuard guard(device);
    cudaIpcMemHandle_t hd;
    std::memcpy(&hd, ipc_handle, sizeof(hd));
    void* p = nullptr;
    if (cudaIpcOpenMemHandle(&p, hd, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) return MPE_ERR_CUDA;
    *d_ptr = p;
    return MPE_OK;
}

int mpe_peer_buffer_close(int32_t device, void* d_ptr) {
    if (!d_ptr) return MPE_ERR_ARG;
    DeviceGuard guard(device);
    return cudaIpcCloseMemHandle(d_ptr) == cudaSuccess ? MPE_OK : MPE_ERR_CUDA;
}

int mpe_peer_buffer_free(int32_t device, void* d_ptr) {
    if (!d_ptr) return MPE_ERR_ARG;
    DeviceGuard guard(device);
    return cudaFree(d_ptr) == cudaSuccess ? MPE_OK : MPE_ERR_CUDA;
}

int mpe_backward(mpe_handle* h, const float* d_grad_out, float lr, int64_t step) {
    if (!h || (!d_grad_out && h->B > 0)) return MPE_ERR_ARG;
    if (!h->have_forward) return MPE_ERR_SEQUENCE;
    if (step < 1 || step > 0xffffffffLL) return MPE_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(d_grad_out) & 15) return MPE_ERR_ARG;   // rows are moved 16 bytes at a time
    if (step <= h->last_step) return MPE_ERR_SEQUENCE;
    DeviceGuard guard(h->device);
    Work& w = h->wk;
    unsigned long long ustep = (unsigned long long)step;
    h->args.grad = d_grad_out; h->args.lr = lr; h->args.step = ustep;
    int rc = MPE_OK;
    bool done = false;
    // the replayed kernels read the forward's arguments (indices, offsets, batch, epoch) from the device copy, which only
    // a replayed forward writes; after a plainly launched forward the backward is launched plainly too
    if (h->fwd_replayed && may_use_graph(h)) {
        if (!h->x_bwd) {
            rc = capture(h, &h->g_bwd, &h->x_bwd, &h->n_bwd, &h->k_bwd, (const void*)k_set_args_backward, [&]() {
                LAUNCH(h, "set_args", k_set_args_backward, 1, 1, 0, w.args, d_grad_out, lr, ustep);
                return enqueue_backward(h, h->cap_L, true);
            });
            if (rc != MPE_OK) { drop_graphs(h); h->graphs_enabled = false; }
        }
        if (rc == MPE_OK) {
            StepArgs* a = w.args;
            void* params[] = {&a, &d_grad_out, &lr, &ustep};
            cudaKernelNodeParams kp{};
            kp.func = (void*)k_set_args_backward; kp.gridDim = dim3(1); kp.blockDim = dim3(1); kp.kernelParams = params;
            CK(h, cudaGraphExecKernelNodeSetParams(h->x_bwd, h->n_bwd, &kp));
            CK(h, cudaGraphLaunch(h->x_bwd, h->stream));
            h->launches += h->k_bwd;
            done = true;
        }
    }
    if (!done) {
        rc = enqueue_backward(h, h->L, false);
        if (rc != MPE_OK) return rc;
    }
    if (h->ev_free) CK(h, cudaEventRecord(h->ev_free, h->stream));
    h->have_forward = false;
    h->last_step = step;
    ++h->steps;
    return MPE_OK;
}

int mpe_set_rounding(mpe_handle* h, int32_t mode) {
    if (!h || (mode != MPE_ROUND_NEAREST && mode != MPE_ROUND_STOCHASTIC)) return MPE_ERR_ARG;
    if (h->have_forward) return MPE_ERR_SEQUENCE;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    h->st.rounding = mode;
    drop_graphs(h);           // the captured kernels carry the old setting
    return MPE_OK;
}

int mpe_use_graphs(mpe_handle* h, int32_t enable) {
    if (!h) return MPE_ERR_ARG;
    if (h->have_forward) return MPE_ERR_SEQUENCE;      // both halves of a step are launched the same way
    h->graphs_enabled = enable != 0;
    return MPE_OK;
}

int mpe_step_host_submit(mpe_handle* h, const int32_t* h_indices, const int32_t* h_offsets, int32_t batch,
                         int64_t total_indices, const float* h_grad_out, float* h_out, float lr, int64_t step) {
    if (!h || !h_offsets || batch < 0 || total_indices < 0) return MPE_ERR_ARG;
    if ((total_indices > 0 && !h_indices) || (batch > 0 && (!h_grad_out || !h_out))) return MPE_ERR_ARG;
    if (h->have_forward) return MPE_ERR_SEQUENCE;
    if (step < 1 || step > 0xffffffffLL) return MPE_ERR_ARG;
    if (step <= h->last_step) return MPE_ERR_SEQUENCE;
    DeviceGuard guard(h->device);
    const int64_t noff = (int64_t)h->T * batch + 1, nout = (int64_t)batch * h->T * h->dim;
    // the workspace is sized here, before anything is enqueued (growing it waits for the stream)
    if (total_indices > h->cap_L || (int64_t)h->T * batch > h->cap_bags || !h->wk.ctr) {
        int rc = mpe_reserve(h, batch, total_indices);
        if (rc != MPE_OK) return rc;
    }
    if (total_indices > h->sh_cap_L || noff > h->sh_cap_off || nout > h->sh_cap_out) {
        // larger staging buffers: everything in flight has to finish first
        CK(h, cudaStreamSynchronize(h->stream)); CK(h, cudaStreamSynchronize(h->copy_in)); CK(h, cudaStreamSynchronize(h->copy_out));
        // sized like the workspace (mpe_reserve), so that a run of batches of slightly different sizes grows them once
        h->sh_cap_L = std::max({total_indices, h->sh_cap_L, h->cap_L});
        h->sh_cap_off = std::max({noff, h->sh_cap_off, h->cap_bags + 1});
        h->sh_cap_out = std::max({nout, h->sh_cap_out, h->cap_bags * (int64_t)h->dim});
        for (auto& sl : h->slot) {
            cudaFree(sl.idx); cudaFree(sl.off); cudaFree(sl.grad); cudaFree(sl.out);
            sl.idx = nullptr; sl.off = nullptr; sl.grad = nullptr; sl.out = nullptr; sl.used = false;
            int rc;
            if ((rc = dmalloc(h, &sl.idx, h->sh_cap_L, nullptr)) != MPE_OK) return rc;
            if ((rc = dmalloc(h, &sl.off, h->sh_cap_off, nullptr)) != MPE_OK) return rc;
            if ((rc = dmalloc(h, &sl.grad, h->sh_cap_out, nullptr)) != MPE_OK) return rc;
            if ((rc = dmalloc(h, &sl.out, h->sh_cap_out, nullptr)) != MPE_OK) return rc;
        }
    }
    // Three streams: uploads, kernels, downloads.  The slot's buffers are free again once the step that used them two
    // submissions ago has finished its kernels (inputs) and its download (output); the upload of this step therefore runs
    // while the previous step computes, and the previous step's download while this step's forward runs.
    mpe_handle::HostSlot& sl = h->slot[h->submitted & 1];
    cudaStream_t st = h->stream;
    if (sl.used) CK(h, cudaStreamWaitEvent(h->copy_in, sl.ev_done, 0));
    if (total_indices) CK(h, cudaMemcpyAsync(sl.idx, h_indices, sizeof(int32_t) * total_indices, cudaMemcpyHostToDevice, h->copy_in));
    CK(h, cudaMemcpyAsync(sl.off, h_offsets, sizeof(int32_t) * noff, cudaMemcpyHostToDevice, h->copy_in));
    CK(h, cudaEventRecord(sl.ev_idx, h->copy_in));
    if (nout) CK(h, cudaMemcpyAsync(sl.grad, h_grad_out, sizeof(float) * nout, cudaMemcpyHostToDevice, h->copy_in));
    CK(h, cudaEventRecord(sl.ev_grad, h->copy_in));
    // the part of forward that needs the indices only starts as soon as they have arrived, beside whatever the previous
    // step still has to do
    CK(h, cudaStreamWaitEvent(h->prep, sl.ev_idx, 0));
    int rc = prepare_impl(h, sl.idx, sl.off, batch, total_indices, h->prep);
    if (rc != MPE_OK) { cudaStreamSynchronize(h->copy_in); return rc; }
    CK(h, cudaStreamWaitEvent(st, sl.ev_idx, 0));
    if (sl.used) CK(h, cudaStreamWaitEvent(st, sl.ev_down, 0));           // the slot's previous output has left the device
    rc = mpe_forward(h, sl.idx, sl.off, batch, total_indices, sl.out, (void*)st);
    if (rc != MPE_OK) { cudaStreamSynchronize(h->copy_in); return rc; }
    CK(h, cudaEventRecord(sl.ev_fwd, st));
    CK(h, cudaStreamWaitEvent(h->copy_out, sl.ev_fwd, 0));
    if (nout) CK(h, cudaMemcpyAsync(h_out, sl.out, sizeof(float) * nout, cudaMemcpyDeviceToHost, h->copy_out));
    CK(h, cudaEventRecord(sl.ev_down, h->copy_out));
    CK(h, cudaStreamWaitEvent(st, sl.ev_grad, 0));
    rc = mpe_backward(h, sl.grad, lr, step);
    if (rc != MPE_OK) { cudaStreamSynchronize(h->copy_in); cudaStreamSynchronize(st); h->have_forward = false; return rc; }
    CK(h, cudaEventRecord(sl.ev_done, st));
    sl.used = true;
    ++h->submitted;
    return MPE_OK;
}

int mpe_step_host_wait(mpe_handle* h) {
    if (!h) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    cudaError_t e1 = cudaStreamSynchronize(h->copy_out), e2 = cudaStreamSynchronize(h->stream), e3 = cudaStreamSynchronize(h->copy_in);
    CK(h, e1); CK(h, e2); CK(h, e3);
    return MPE_OK;
}

int mpe_step_host(mpe_handle* h, const int32_t* h_indices, const int32_t* h_offsets, int32_t batch,
                  int64_t total_indices, const float* h_grad_out, float* h_out, float lr, int64_t step) {
    int rc = mpe_step_host_submit(h, h_indices, h_offsets, batch, total_indices, h_grad_out, h_out, lr, step);
    if (rc != MPE_OK) return rc;
    return mpe_step_host_wait(h);
}

int mpe_flush(mpe_handle* h) {
    if (!h) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    const State& s = h->st;
    if (h->total_slots > 0) {
        const int g = grid_for(h, h->total_slots, 256 / s.lanes, 8);
        if (h->bits == 8) LAUNCH(h, "flush", k_flush<8>, g, 256, 0, s, h->total_slots, (uint64_t)h->last_step);
        else if (h->bits == 4) LAUNCH(h, "flush", k_flush<4>, g, 256, 0, s, h->total_slots, (uint64_t)h->last_step);
        else if (h->bits == 2) LAUNCH(h, "flush", k_flush<2>, g, 256, 0, s, h->total_slots, (uint64_t)h->last_step);
        else LAUNCH(h, "flush", k_flush<16>, g, 256, 0, s, h->total_slots, (uint64_t)h->last_step);
    }
    return check_launch(h);
}

int mpe_destroy(mpe_handle* h) {
    if (!h) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    cudaStreamSynchronize(h->stream);
    if (h->side) { cudaStreamSynchronize(h->side); cudaStreamDestroy(h->side); }
    if (h->cap) cudaStreamDestroy(h->cap);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->prep) { cudaStreamSynchronize(h->prep); cudaStreamDestroy(h->prep); }
    for (cudaEvent_t e : {h->ev_free, h->alt.ev_free, h->ev_prep}) if (e) cudaEventDestroy(e);
    if (h->copy_in) { cudaStreamSynchronize(h->copy_in); cudaStreamDestroy(h->copy_in); }
    if (h->copy_out) { cudaStreamSynchronize(h->copy_out); cudaStreamDestroy(h->copy_out); }
    for (auto& sl : h->slot) {
        for (cudaEvent_t e : {sl.ev_idx, sl.ev_grad, sl.ev_fwd, sl.ev_done, sl.ev_down}) if (e) cudaEventDestroy(e);
        cudaFree(sl.idx); cudaFree(sl.off); cudaFree(sl.grad); cudaFree(sl.out);
    }
    free_workspace(h);
    State& s = h->st;
    if (h->table_on_host) { cudaFreeHost(s.codes); cudaFreeHost(s.sb); } else { cudaFree(s.codes); cudaFree(s.sb); }
    cudaFree(h->d_route);
    cudaFree(h->d_tables); cudaFree(s.cnt); cudaFree(s.G); cudaFree(s.slab);
    cudaFree(s.tags); cudaFree(s.ts); cudaFree(s.hit_epoch); cudaFree(s.hit_k); cudaFree(s.floor); cudaFree(s.stats);
    for (auto& r : h->prof_recs) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    for (auto e : h->event_pool) cudaEventDestroy(e);
    delete h;
    return MPE_OK;
}

int mpe_last_error(mpe_handle* h, int32_t* code, int64_t* detail) {
    if (!h || !code || !detail) return MPE_ERR_ARG;
    *code = MPE_OK; *detail = 0;
    if (!h->wk.ctr) return MPE_OK;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    Counters c;
    CK(h, cudaMemcpy(&c, h->wk.ctr, sizeof(c), cudaMemcpyDeviceToHost));
    CK(h, cudaMemset(&h->wk.ctr->err[0], 0, sizeof(c.err)));
    if (h->alt.wk.ctr && !h->prepared) {     // steps alternate between the two workspaces: conditions seen in either count
        Counters c2;                         // (a batch that is prepared but not yet taken over reports with its own step)
        CK(h, cudaMemcpy(&c2, h->alt.wk.ctr, sizeof(c2), cudaMemcpyDeviceToHost));
        CK(h, cudaMemset(&h->alt.wk.ctr->err[0], 0, sizeof(c2.err)));
        c.err[ERR_OFFSETS] += c2.err[ERR_OFFSETS]; c.err[ERR_INDEX] += c2.err[ERR_INDEX];
    }
    // a wait inside the sort that ran out (its step was abandoned) outranks the conditions of the inputs
    uint32_t timeouts = 0;
    for (SortCtl* ctl : {h->sort_ctl, h->prepared ? nullptr : h->alt.sort_ctl}) {
        if (!ctl) continue;
        SortCtl sc;
        CK(h, cudaMemcpy(&sc, ctl, sizeof(sc), cudaMemcpyDeviceToHost));
        if (sc.timeout) { timeouts += sc.timeout; CK(h, cudaMemset(&ctl->timeout, 0, sizeof(uint32_t))); }
    }
    if (timeouts) { *code = MPE_ERR_TIMEOUT; *detail = (int64_t)timeouts; }
    else if (c.err[ERR_OFFSETS]) { *code = MPE_ERR_OFFSETS; *detail = (int64_t)c.err[ERR_OFFSETS]; }
    else if (c.err[ERR_INDEX]) { *code = MPE_ERR_INDEX; *detail = (int64_t)c.err[ERR_INDEX]; }
    return MPE_OK;
}

int mpe_stats(mpe_handle* h, int32_t table, uint64_t* out8) {
    if (!h || !out8 || table < 0 || table >= h->T) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    CK(h, cudaMemcpy(out8, h->st.stats + (int64_t)table * 8, 8 * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    out8[7] = h->steps;
    return MPE_OK;
}

int mpe_memory_bytes(mpe_handle* h, uint64_t* out6) {
    if (!h || !out6) return MPE_ERR_ARG;
    const uint64_t N = (uint64_t)h->total_rows, slots = (uint64_t)h->total_slots, d = (uint64_t)h->dim;
    out6[0] = N * ((uint64_t)h->bits * d + (h->bits == 16 ? 0 : 64)) / 8;   // E x (bitwidth x D + 64) bits; FP16 has no scale/bias
    out6[1] = slots * 4 * d;                                         // 4 alpha n d bytes
    out6[2] = slots * 4;                                             // one INT32 tag per cached row
    uint64_t pv = 0;
    for (const TableDev& tb : h->tables)
        if (tb.n_sets > 0) pv += h->policy == MPE_LFU ? (uint64_t)tb.N * 4 : (uint64_t)tb.n_sets * h->ways * 4;
    out6[3] = pv;                                                    // INT32 counter per embedding row (LFU) / per cached row (LRU)
    out6[4] = h->optimizer == MPE_ROWWISE_ADAGRAD ? N * 4 : 0;
    out6[5] = N * 4 * d;
    return MPE_OK;
}

int mpe_selftest(mpe_handle* h, int32_t which) {
    if (!h) return MPE_ERR_ARG;
    if (!h->sort_ctl) return MPE_ERR_SEQUENCE;          // the workspace comes with mpe_reserve or the first forward
    DeviceGuard guard(h->device);
    if (which == MPE_SELFTEST_LOOK_BACK_TIMEOUT) {
        if (h->have_forward) return MPE_ERR_SEQUENCE;
        LAUNCH(h, "selftest", k_selftest_look_back, 1, 32, 0, h->sort_status, h->sort_ctl);
        ++h->sort_passes_bound;
        return check_launch(h);
    }
    if (which == MPE_SELFTEST_RENEW_TAGS) {
        h->sort_passes_bound = SORT_TAG_MASK;           // the next forward starts the pass numbers over
        return MPE_OK;
    }
    return MPE_ERR_ARG;
}

int mpe_workspace_bytes(mpe_handle* h, uint64_t* out2) {
    if (!h || !out2) return MPE_ERR_ARG;
    out2[0] = h->ws_bytes + h->alt.bytes;
    out2[1] = 2 * ((uint64_t)h->sh_cap_L * 4 + (uint64_t)h->sh_cap_off * 4 + 2 * (uint64_t)h->sh_cap_out * 4);
    return MPE_OK;
}

int mpe_cache_geometry(mpe_handle* h, int32_t table, int32_t* n_sets, int32_t* ways) {
    if (!h || table < 0 || table >= h->T || !n_sets || !ways) return MPE_ERR_ARG;
    *n_sets = h->tables[table].n_sets; *ways = h->ways;
    return MPE_OK;
}

int mpe_step_info(mpe_handle* h, int64_t* out6) {
    if (!h || !out6) return MPE_ERR_ARG;
    int64_t* out4 = out6;
    for (int i = 0; i < 6; ++i) out6[i] = 0;
    if (!h->wk.ctr) return MPE_OK;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    Counters c;
    CK(h, cudaMemcpy(&c, h->wk.ctr, sizeof(c), cudaMemcpyDeviceToHost));
    if (c.abort) return MPE_OK;
    std::vector<int32_t> us(h->T + 1), urow(1);
    out4[0] = (int64_t)c.L - (int64_t)c.dropped;
    // distinct rows: the sort puts each table's out-of-range ids into one pseudo row; leave those out
    int64_t pseudo = 0;
    if (c.dropped) {
        CK(h, cudaMemcpy(us.data(), h->wk.ustart, sizeof(int32_t) * (h->T + 1), cudaMemcpyDeviceToHost));
        for (int t = 0; t < h->T; ++t) {
            if (us[t + 1] == us[t]) continue;
            CK(h, cudaMemcpy(urow.data(), h->wk.uniq_row + us[t + 1] - 1, sizeof(int32_t), cudaMemcpyDeviceToHost));
            if (urow[0] >= h->tables[t].N) ++pseudo;
        }
    }
    out4[1] = (int64_t)c.U - pseudo;
    out4[2] = (int64_t)c.dropped;
    out4[3] = (int64_t)c.hot_rows;
    out6[4] = (int64_t)c.hot_occ;
    out6[5] = (int64_t)c.deferred;
    return MPE_OK;
}

int mpe_export_rows(mpe_handle* h, int32_t table, const int64_t* h_rows, int64_t n, uint8_t* h_codes,
                    float* h_scale, float* h_bias) {
    if (!h || table < 0 || table >= h->T || n < 0 || (n > 0 && (!h_rows || !h_codes || !h_scale || !h_bias))) return MPE_ERR_ARG;
    if (n == 0) return MPE_OK;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    int64_t* d_rows = nullptr; uint8_t* d_codes = nullptr; float *d_s = nullptr, *d_b = nullptr;
    int rc = MPE_OK;
    if ((rc = dmalloc(h, &d_rows, n, nullptr)) == MPE_OK && (rc = dmalloc(h, &d_codes, n * h->code_bytes, nullptr)) == MPE_OK &&
        (rc = dmalloc(h, &d_s, n, nullptr)) == MPE_OK && (rc = dmalloc(h, &d_b, n, nullptr)) == MPE_OK) {
        cudaMemcpy(d_rows, h_rows, sizeof(int64_t) * n, cudaMemcpyHostToDevice);
        cudaMemset(d_codes, 0, (size_t)n * h->code_bytes); cudaMemset(d_s, 0, sizeof(float) * n); cudaMemset(d_b, 0, sizeof(float) * n);
        LAUNCH(h, "gather_rows", k_gather_rows, grid_for(h, n, 256, 8), 256, 0, h->st, table, (const int64_t*)d_rows, n, h->code_bytes,
               d_codes, d_s, d_b, (uint32_t*)nullptr, (float*)nullptr);
        cudaMemcpy(h_codes, d_codes, (size_t)n * h->code_bytes, cudaMemcpyDeviceToHost);
        cudaMemcpy(h_scale, d_s, sizeof(float) * n, cudaMemcpyDeviceToHost);
        cudaMemcpy(h_bias, d_b, sizeof(float) * n, cudaMemcpyDeviceToHost);
        rc = check_launch(h);
    }
    cudaFree(d_rows); cudaFree(d_codes); cudaFree(d_s); cudaFree(d_b);
    return rc;
}

int mpe_export_cache(mpe_handle* h, int32_t table, int32_t* h_tags, float* h_rows, uint32_t* h_ts) {
    if (!h || table < 0 || table >= h->T) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    const TableDev& tb = h->tables[table];
    const int64_t nslot = (int64_t)tb.n_sets * h->ways, first = tb.set_base * h->ways;
    if (nslot == 0) return MPE_OK;
    if (h_tags) CK(h, cudaMemcpy(h_tags, h->st.tags + first, sizeof(int32_t) * nslot, cudaMemcpyDeviceToHost));
    if (h_rows) CK(h, cudaMemcpy(h_rows, h->st.slab + first * h->dim, sizeof(float) * nslot * h->dim, cudaMemcpyDeviceToHost));
    if (h_ts) {
        if (h->policy == MPE_LRU) CK(h, cudaMemcpy(h_ts, h->st.ts + first, sizeof(uint32_t) * nslot, cudaMemcpyDeviceToHost));
        else memset(h_ts, 0, sizeof(uint32_t) * nslot);      // under LFU the per-slot values are copies of the rows' counts
    }
    return MPE_OK;
}

int mpe_export_aux(mpe_handle* h, int32_t table, const int64_t* h_rows, int64_t n, uint32_t* h_cnt, float* h_adagrad) {
    if (!h || table < 0 || table >= h->T || n < 0 || (n > 0 && !h_rows)) return MPE_ERR_ARG;
    if (n == 0 || (!h_cnt && !h_adagrad)) return MPE_OK;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    int64_t* d_rows = nullptr; uint32_t* d_c = nullptr; float* d_g = nullptr;
    int rc = MPE_OK;
    if ((rc = dmalloc(h, &d_rows, n, nullptr)) == MPE_OK && (rc = dmalloc(h, &d_c, n, nullptr)) == MPE_OK &&
        (rc = dmalloc(h, &d_g, n, nullptr)) == MPE_OK) {
        cudaMemcpy(d_rows, h_rows, sizeof(int64_t) * n, cudaMemcpyHostToDevice);
        cudaMemset(d_c, 0, sizeof(uint32_t) * n); cudaMemset(d_g, 0, sizeof(float) * n);
        LAUNCH(h, "gather_rows", k_gather_rows, grid_for(h, n, 256, 8), 256, 0, h->st, table, (const int64_t*)d_rows, n, h->code_bytes,
               (uint8_t*)nullptr, (float*)nullptr, (float*)nullptr, d_c, d_g);
        if (h_cnt) cudaMemcpy(h_cnt, d_c, sizeof(uint32_t) * n, cudaMemcpyDeviceToHost);
        if (h_adagrad) cudaMemcpy(h_adagrad, d_g, sizeof(float) * n, cudaMemcpyDeviceToHost);
        rc = check_launch(h);
    }
    cudaFree(d_rows); cudaFree(d_c); cudaFree(d_g);
    return rc;
}

int mpe_kernel_launches(mpe_handle* h, uint64_t* count) {
    if (!h || !count) return MPE_ERR_ARG;
    *count = h->launches;
    return MPE_OK;
}

int mpe_profile(mpe_handle* h, int32_t enable) {
    if (!h) return MPE_ERR_ARG;
    if (h->have_forward) return MPE_ERR_SEQUENCE;      // both halves of a step are launched the same way
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    for (auto& r : h->prof_recs) { h->event_pool.push_back(r.a); h->event_pool.push_back(r.b); }
    h->prof_recs.clear();
    h->profiling = enable != 0;
    return MPE_OK;
}

int mpe_profile_read(mpe_handle* h, int32_t cap, char* names, double* ms, uint64_t* launches, int32_t* n) {
    if (!h || cap < 0 || !n || (cap > 0 && (!names || !ms || !launches))) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    CK(h, cudaStreamSynchronize(h->stream));
    std::vector<double> t(h->prof_names.size(), 0.0);
    std::vector<uint64_t> c(h->prof_names.size(), 0);
    for (auto& r : h->prof_recs) {
        float e = 0.f;
        cudaEventElapsedTime(&e, r.a, r.b);
        t[r.name] += e; c[r.name] += 1;
        h->event_pool.push_back(r.a); h->event_pool.push_back(r.b);
    }
    h->prof_recs.clear();
    int32_t k = 0;
    for (size_t i = 0; i < h->prof_names.size() && k < cap; ++i) {
        if (!c[i]) continue;
        std::memset(names + 32 * k, 0, 32);
        std::strncpy(names + 32 * k, h->prof_names[i].c_str(), 31);
        ms[k] = t[i]; launches[k] = c[i]; ++k;
    }
    *n = k;
    return MPE_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Evaluation forward whose whole per-step workspace is a fixed array inside the library image
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int64_t STATIC_MAX_INDICES = MPE_STATIC_MAX_INDICES;
constexpr int64_t STATIC_MAX_BAGS = MPE_STATIC_MAX_BAGS;
constexpr int STATIC_MAX_TABLES = MPE_STATIC_MAX_TABLES;
constexpr size_t align256(size_t v) { return (v + 255) & ~size_t(255); }
constexpr size_t STATIC_SCRATCH_BYTES =
    2 * align256(2 * (STATIC_MAX_INDICES + 4) * 4) + 12 * align256((STATIC_MAX_INDICES + 4) * 4) +                                 // keys, payloads, per-index and per-row maps
    align256(256 * ((STATIC_MAX_INDICES + sort_tile(true) - 1) / sort_tile(true) + STATIC_MAX_TABLES + 1) * 8) +   // the sort's per-tile words
    align256(STATIC_MAX_TABLES * SORT_MAX_PASSES * 256 * 4) + align256(sizeof(SortCtl)) +              // its per-table digit counts and its counters
    4 * align256((STATIC_MAX_TABLES + 1) * 4) +                                                        // per-table starts
    2 * align256(hot_capacity(STATIC_MAX_INDICES) * 4) +                                             // hot-row lists
    align256(sizeof(Counters)) + align256(sizeof(StepArgs));

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
unsigned char* g_scratch_addr[MAX_DEVICES] = {};     // device address of g_static_scratch, per device, filled on first use
uint64_t g_scratch_passes[MAX_DEVICES] = {};         // sort passes run in the array so far, per device (an upper bound)
std::mutex g_scratch_lock;                           // first calls from several host threads fill the table one at a time

struct Carver {
    unsigned char* p; size_t used = 0;
    template <class T> T* take(size_t count) { T* r = reinterpret_cast<T*>(p + used); used += align256(count * sizeof(T)); return r; }
};

}  // namespace

extern "C" int mpe_forward_static(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch,
                                  int64_t total_indices, float* d_out, void* cuda_stream) {
    if (!h || !d_offsets || batch < 0 || total_indices < 0) return MPE_ERR_ARG;
    if ((total_indices > 0 && !d_indices) || (batch > 0 && !d_out)) return MPE_ERR_ARG;
    const int64_t bags = (int64_t)h->T * batch;
    if (total_indices > STATIC_MAX_INDICES || bags > STATIC_MAX_BAGS || h->T > STATIC_MAX_TABLES) return MPE_ERR_TOO_LARGE;
    if (h->have_forward) return MPE_ERR_SEQUENCE;      // a training step is half done: its backward still needs the probe marks
    if (h->device < 0 || h->device >= MAX_DEVICES) return MPE_ERR_ARG;
    DeviceGuard guard(h->device);
    unsigned char* scratch = nullptr;
    bool renew_tags = false;          // the pass numbers in the sort's per-tile words are about to come round: start them over
    {
        std::lock_guard<std::mutex> lock(g_scratch_lock);
        if (!g_scratch_addr[h->device]) {
            // once per device, with that device current: ask the runtime where the array lives on this device
            void* addr = nullptr;
            CK(h, cudaGetSymbolAddress(&addr, g_static_scratch));
            g_scratch_addr[h->device] = static_cast<unsigned char*>(addr);
        }
        scratch = g_scratch_addr[h->device];
        g_scratch_passes[h->device] += SORT_MAX_PASSES;
        renew_tags = g_scratch_passes[h->device] > SORT_TAG_MASK - 1024;
        if (renew_tags) g_scratch_passes[h->device] = 0;
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (stream != h->stream) { CK(h, cudaStreamSynchronize(h->stream)); h->stream = stream; }

    // carve the step's arrays out of the scratch (same roles as the handle's own workspace)
    Carver c{scratch};
    const size_t n = (size_t)STATIC_MAX_INDICES + 4;
    uint32_t *sortA = c.take<uint32_t>(2 * n), *sortB = c.take<uint32_t>(2 * n);
    Work w{};
    w.bag_of = c.take<int32_t>(n); w.kidx = c.take<uint32_t>(n); w.occ_loc = c.take<int32_t>(n); w.occ_b = c.take<int32_t>(n);
    w.uniq_row = c.take<int32_t>(n); w.uniq_t = c.take<int32_t>(n); w.seg = c.take<int32_t>(n); w.loc = c.take<int32_t>(n);
    w.final_loc = c.take<int32_t>(n); w.uset = c.take<int32_t>(n); w.hot_base = c.take<int32_t>(n); w.victim = c.take<int32_t>(n);
    const size_t max_tiles = (STATIC_MAX_INDICES + sort_tile(true) - 1) / sort_tile(true) + STATIC_MAX_TABLES + 1;
    unsigned long long* sort_status = c.take<unsigned long long>(256 * max_tiles);
    uint32_t* ghist = c.take<uint32_t>((size_t)STATIC_MAX_TABLES * SORT_MAX_PASSES * 256);
    SortCtl* sort_ctl = c.take<SortCtl>(1);
    w.table_start = c.take<int32_t>(STATIC_MAX_TABLES + 1); w.tile_base = c.take<int32_t>(STATIC_MAX_TABLES + 1);
    w.ustart = c.take<int32_t>(STATIC_MAX_TABLES + 1); w.ctile_base = c.take<int32_t>(STATIC_MAX_TABLES + 1);
    w.hot_k = c.take<int32_t>(hot_capacity(STATIC_MAX_INDICES)); w.task_k = c.take<int32_t>(hot_capacity(STATIC_MAX_INDICES));
    w.ctr = c.take<Counters>(1);
    w.args = c.take<StepArgs>(1);
    if (c.used > STATIC_SCRATCH_BYTES) return MPE_ERR_ARG;      // cannot happen: the size formula above mirrors this list

    const State& s = h->st;
    const int T = h->T;
    const uint32_t L = (uint32_t)total_indices;
    ++h->epoch;
    // the array keeps whatever the previous call left: the counters are the only part that must start from zero
    CK(h, cudaMemsetAsync(w.ctr, 0, sizeof(Counters), stream));
    if (renew_tags) {
        CK(h, cudaMemsetAsync(sort_status, 0, sizeof(unsigned long long) * 256 * max_tiles, stream));
        CK(h, cudaMemsetAsync(sort_ctl, 0, sizeof(SortCtl), stream));
    }
    StepArgs av{};
    av.indices = d_indices; av.offsets = d_offsets; av.out = d_out; av.B = batch; av.L = L; av.epoch = h->epoch;
    w.sort_tile = sort_tile(true);
    const SortBufs sb{sortA, sortB, (int64_t)n, ghist, sort_status, sort_ctl, &w.ctr->abort, w.sort_tile};
    LAUNCH(h, "prelude", k_prelude<false>, 1, 32, 0, w, T, av);
    LAUNCH(h, "make_keys", k_make_keys<false>, grid_for(h, bags, 32, 8), 256, 0, s, w, sort_input(sb), av);
    // segmented radix sort, as in mpe_forward, on the carved buffers
    const uint32_t *skey = nullptr, *spos = nullptr;
    seg_sort(h, sb, w.table_start, w.tile_base, bits_for((uint32_t)h->max_rows), total_indices, &skey, &spos);
    const int gs = grid_for(h, total_indices, SCAN_TILE, 8);
    LAUNCH(h, "unique", k_unique, gs, SCAN_THREADS, 0, w, T, skey, sort_status, sort_ctl);
    LAUNCH(h, "probe", k_probe<false>, grid_for(h, total_indices, 256, 8), 256, 0, s, w, av);
    LAUNCH(h, "broadcast", k_broadcast<false>, grid_for(h, total_indices, 256, 8), 256, 0, s, w, spos, av);
    const int gp = grid_for(h, bags, 256 / s.lanes, 8);
    dispatch(h->bits, s.lanes, [&](auto bc, auto lc) {
        auto kern = k_pool<decltype(bc)::value, decltype(lc)::value, false>;
        LAUNCH(h, "pool", kern, gp, 256, 0, s, w, av);
    });
    return check_launch(h);
}

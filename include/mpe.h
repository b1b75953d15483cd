/*
 * mpe -- mixed-precision embedding tables behind an FP32 cache: the training
 * step of "Mixed-Precision Embedding using a Cache" on one B200 (sm_100a).
 *
 * Every table stores its rows row-wise quantized (INT8 or packed INT4 codes plus
 * an FP32 scale and bias per row; Section 3 "Precision", Appendix Eq. 3) and is
 * fronted by a set-associative cache of FP32 rows (Section 3 "Cache Structure")
 * managed by LRU or LFU priorities (Section 3 "Cache Replacement Policy",
 * Algorithm 2).  One training step = mpe_forward (fetch + sum-pool) followed by
 * mpe_backward (merge duplicate gradients, optimizer update in FP32, commit to
 * cache or stochastic-round back to the table, admission/eviction).
 *
 * C ABI, no exceptions.  Every function returns 0 (MPE_OK) or a negative
 * MPE_ERR_* code.  Pointers named d_* are device pointers on the handle's
 * device, h_* are host pointers.  The handle owns all table state and all
 * workspace; the caller owns every buffer it passes in, and device buffers need
 * to stay alive only until the stream work enqueued by that call has finished.
 * Calls on one handle must not overlap in time (no internal locking).
 */
#ifndef MPE_H
#define MPE_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mpe_handle mpe_handle;
typedef struct { int64_t num_rows; int32_t dim; } mpe_table_spec;

enum { MPE_LRU = 0, MPE_LFU = 1 };
enum { MPE_SGD = 0, MPE_ROWWISE_ADAGRAD = 1 };
enum { MPE_ROUND_NEAREST = 0, MPE_ROUND_STOCHASTIC = 1 };

enum {
    MPE_OK = 0,
    MPE_ERR_ARG = -1,          /* NULL pointer, negative size, value out of range */
    MPE_ERR_UNSUPPORTED = -2,  /* unequal dims, dim not a power of two in [4,128], bits not 16/8/4/2, ways not 2^k <= 32 */
    MPE_ERR_CUDA = -3,         /* a CUDA runtime call failed (detail = cudaError_t) */
    MPE_ERR_SEQUENCE = -4,     /* backward without a preceding forward, or step not strictly increasing */
    MPE_ERR_INDEX = -5,        /* device saw row ids outside [0, num_rows) (detail = how many); they were dropped */
    MPE_ERR_OFFSETS = -6,      /* device saw offsets that are not 0 = o[0] <= o[1] <= ... <= o[T*B] = total */
    MPE_ERR_NOMEM = -7,        /* allocation failed */
    MPE_ERR_TOO_LARGE = -8,    /* mpe_forward_static: the batch does not fit the fixed scratch */
    MPE_ERR_TIMEOUT = -9       /* a bounded wait between thread blocks of one kernel ran out (detail = how many); the step was abandoned */
};

/*
 * Create the tables, the caches and the policy state on `device`.
 *   tables[num_tables]  row count and dimension of each table; all dims must be equal
 *                       (a power of two in [4,128]); num_rows in [1, 2^31-2].
 *   bits                8, 4 or 2: width of the integer codes, ranges [0,255], [0,15], [0,3]; or 16: an IEEE FP16
 *                       table without scale/bias, rounded between the two FP16 neighbours (Section 3 "Precision").
 *   cache_fraction      in [0,1]; table t gets n_t = max(1, floor(cache_fraction*N_t + 1e-6) / ways) sets
 *                       of `ways` FP32 rows (Section 3 "Cache Structure"); 0 = no cache at all.
 *   ways                associativity alpha, a power of two <= 32; 0 selects 32 (Section 5.1).
 *   policy              MPE_LRU (timestamp of last access = step number, per cached row) or
 *                       MPE_LFU (access count per embedding row)  (Section 3 "Cache Replacement Policy").
 *   optimizer           MPE_SGD (x <- x - lr*g, Section 3) or MPE_ROWWISE_ADAGRAD
 *                       (G_row += mean(g^2); x <- x - lr/(sqrt(G_row)+eps)*g; Section 4.1 names a
 *                       sparse AdaGrad without a formula, this is the build's reading).
 *   init_lo, init_hi    rows start Uniform(init_lo, init_hi) drawn from a counter hash of
 *                       (seed, table, row, column) and are quantized with round-to-nearest-even;
 *                       the cache starts empty.
 * On success *out receives the handle.  Allocates device memory (cudaMalloc).
 */
int mpe_create(mpe_handle** out, const mpe_table_spec* tables, int32_t num_tables, int32_t bits,
               double cache_fraction, int32_t ways, int32_t policy, int32_t optimizer, float eps,
               float init_lo, float init_hi, uint64_t seed, int32_t device);

/* Same, with a choice of where the low-precision table lives.  MPE_TABLE_DEVICE keeps everything in HBM.
 * MPE_TABLE_HOST keeps the codes and (scale, bias) in pinned host memory that the kernels read and write in place
 * over the host link, while the FP32 cache and all policy and optimizer state stay in HBM: the arrangement of the
 * paper's speed experiment (Section 5.2), where a table too large for the device sits behind the cache.  Results
 * are bit-identical for both placements. */
enum { MPE_TABLE_DEVICE = 0, MPE_TABLE_HOST = 1 };
int mpe_create_placed(mpe_handle** out, const mpe_table_spec* tables, int32_t num_tables, int32_t bits,
                      double cache_fraction, int32_t ways, int32_t policy, int32_t optimizer, float eps,
                      float init_lo, float init_hi, uint64_t seed, int32_t device, int32_t table_placement);

/* Size the per-step workspace for batches of up to max_batch samples and max_total_indices
 * indices, so that later steps allocate nothing.  mpe_forward grows the workspace by itself
 * (a synchronising reallocation) when a larger batch arrives. */
int mpe_reserve(mpe_handle* h, int32_t max_batch, int64_t max_total_indices);

/*
 * Forward: x <- fetch(T, C, i) for every index, summed per bag (Section 3; multi-hot bags, Section 5.1).
 *   d_indices[total_indices]  table-local row ids, int32, table-major: bag (t,b) is
 *                             d_indices[d_offsets[t*batch+b] .. d_offsets[t*batch+b+1]).
 *   d_offsets[T*batch+1]      non-decreasing, first 0, last total_indices.
 *   d_out[batch][T*dim]       FP32, row-major; bag (t,b) lands in d_out[b][t*dim .. (t+1)*dim);
 *                             an empty bag gives zeros; rows are added in index order starting from +0.
 * The call sorts and de-duplicates the indices (Section 5.1), probes the cache tags, gathers FP32
 * rows on hits and dequantizes (q*scale+bias, Algorithm 1) on misses.  It reads but never changes
 * table, cache or policy state.  Work is enqueued on `cuda_stream` (a cudaStream_t; NULL = the
 * default stream) and the call returns without waiting.  Row ids outside [0, num_rows) contribute
 * nothing and raise the sticky MPE_ERR_INDEX.
 */
int mpe_forward(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch,
                int64_t total_indices, float* d_out, void* cuda_stream);

/*
 * Optional: start on the NEXT batch while the current step still runs.  The first part of a forward pass -- sorting the
 * indices and merging duplicates (Section 5.1) -- needs the indices only, not the tables, the cache or the policy state,
 * and its kernels leave most of the GPU idle.  mpe_prepare enqueues that part for the given batch on `cuda_stream`
 * (any stream on which the indices and offsets are ready; typically not the stream of the training step) into a second
 * workspace of the handle.  A later mpe_forward / mpe_forward_routed with the same d_indices, d_offsets, batch and
 * total_indices takes the result over (it waits for it on its own stream) and only looks up the tags and pools;
 * results are bit-identical with and without the call.  Layouts as in mpe_forward; the two buffers must stay
 * unchanged until that forward.  One batch can be prepared at a time; a forward with other arguments discards it.
 * The call does nothing (and returns MPE_OK) when the batch does not fit the workspace reserved with mpe_reserve, or
 * when steps of this size are replayed from a CUDA graph.  Do not prepare a batch whose forward will be issued while
 * the caller captures its stream into a graph (the hand-over is an event recorded outside that capture).
 * The first call allocates the second workspace
 * (cudaMalloc; as large as the first, see mpe_workspace_bytes).
 * Typical loop:  forward(k); prepare(k+1, other_stream); backward(k); forward(k+1); ...
 * It pays to give the training step's stream a higher priority than other_stream (cudaStreamCreateWithPriority):
 * the step's kernels then get the SMs first and the preparation fills the gaps (measured: 1.6 % of the step).
 */
int mpe_prepare(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch, int64_t total_indices,
                void* cuda_stream);

/* ---- Tables partitioned over several GPUs (Section 1: embeddings are placed model-parallel, with no replication) ----
 * Each rank owns some of the tables and sees the whole batch's indices for them; sample b of a batch of `batch` samples
 * belongs to rank b / (batch / n_ranks).  After the forward pass every rank needs the pooled vectors of ITS samples for ALL
 * tables (an all-to-all); before the backward pass every rank needs the gradients of ALL samples for ITS tables (the reverse).
 * The paper names the partitioning only; the exchange below is this library's.  The kernels of different ranks never
 * wait for one another: the caller orders them (a barrier between "all ranks have run forward" and "a rank reads its buffer").
 *
 * mpe_forward_routed: as mpe_forward, but the pooled vector of local table t and sample b is stored by the pooling kernel
 *   itself at out_ptrs[b / B_local] + ((b % B_local) * tables_global + table_base + t) * dim, B_local = batch / n_ranks.
 *   out_ptrs: HOST array of n_ranks DEVICE pointers (this GPU's own buffer and peers' buffers mapped into this process),
 *   each a float [B_local][tables_global * dim] array, 16-byte aligned; the array is read before the call returns.
 *   Errors: MPE_ERR_ARG when n_ranks is outside 1..72, batch is not a multiple of n_ranks, a pointer is null or unaligned,
 *   or table_base + (tables of this handle) exceeds tables_global; otherwise as mpe_forward.
 * mpe_gather_grad: d_grad_local[b][t][:] = grad_ptrs[b / B_local][(b % B_local)][table_base + t][:] for the handle's tables,
 *   plain loads from the owners' memory; d_grad_local is a DEVICE float [batch][tables * dim] array (caller-owned) that
 *   mpe_backward then takes.  Same pointer rules and errors as above.
 * mpe_peer_buffer_*: exchange buffers that other processes can map.  alloc: `bytes` of device memory on `device` plus the
 *   64-byte handle to send to the peers; open: map a peer's handle (enables peer access on first use); close: unmap;
 *   free: release an allocated buffer (after every peer has closed it).  Errors: MPE_ERR_ARG, MPE_ERR_NOMEM, MPE_ERR_CUDA. */
#define MPE_IPC_HANDLE_BYTES 64
int mpe_forward_routed(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch, int64_t total_indices,
                       float* const* out_ptrs, int32_t n_ranks, int32_t tables_global, int32_t table_base, void* cuda_stream);
int mpe_gather_grad(mpe_handle* h, const float* const* grad_ptrs, int32_t n_ranks, int32_t tables_global, int32_t table_base,
                    int32_t batch, float* d_grad_local, void* cuda_stream);
int mpe_peer_buffer_alloc(int32_t device, int64_t bytes, void** d_ptr, void* ipc_handle);
int mpe_peer_buffer_open(int32_t device, const void* ipc_handle, void** d_ptr);
int mpe_peer_buffer_close(int32_t device, void* d_ptr);
int mpe_peer_buffer_free(int32_t device, void* d_ptr);

/*
 * Backward of the preceding mpe_forward, on the same stream: update(T, C, i, x) for every distinct
 * row of the batch (Section 3, Algorithm 2).
 *   d_grad_out[batch][T*dim]  gradient of the loss w.r.t. d_out, FP32.
 *   lr                        learning rate.
 *   step                      1 <= step < 2^32, strictly increasing over the handle's life; it is the LRU
 *                             timestamp and part of the stochastic-rounding counter.
 * Gradients of duplicate rows are merged first (Section 5.1) in a fixed radix-32 tree over index
 * positions; priorities are updated; each row is updated once in FP32 from the value the forward
 * fetched; rows that are (or become) cache resident are written to the cache verbatim, all others
 * are re-quantized with stochastic rounding (Section 3 "Rounding"); an evicted row is down-converted
 * the same way.  Must follow exactly one mpe_forward (else MPE_ERR_SEQUENCE).  Returns without waiting.
 */
int mpe_backward(mpe_handle* h, const float* d_grad_out, float lr, int64_t step);

/* How update() down-converts a row into the low-precision table (Section 3 "Rounding"): MPE_ROUND_STOCHASTIC
 * (the default: one of the two neighbouring codes, with expectation equal to the value) or MPE_ROUND_NEAREST
 * (the closer code, ties to even).  Applies to mpe_backward and mpe_flush from the next call on; not allowed between
 * a forward and its backward (MPE_ERR_SEQUENCE).  Waits for the handle's stream. */
int mpe_set_rounding(mpe_handle* h, int32_t mode);

/* One whole step from HOST buffers: copies indices, offsets and grad_out to the device, runs
 * forward and backward, copies the pooled output back and waits for it.  Layouts as above.
 * Uses the stream of the last mpe_forward (default stream if none).  Equal to mpe_step_host_submit
 * followed by mpe_step_host_wait. */
int mpe_step_host(mpe_handle* h, const int32_t* h_indices, const int32_t* h_offsets, int32_t batch,
                  int64_t total_indices, const float* h_grad_out, float* h_out, float lr, int64_t step);

/* The same step without waiting, so that consecutive steps overlap on the host link: the call enqueues the
 * uploads, the kernels and the download of one step on three streams and returns.  The library keeps two sets
 * of device staging buffers; the upload of step k+1 runs while step k computes, and the download of step k
 * while step k+1 computes (the steps' kernels themselves run one after the other, in submission order, so the
 * results are those of mpe_step_host called in a loop).  Any number of steps may be submitted before waiting.
 *   h_indices, h_offsets, h_grad_out   must stay valid and unchanged until mpe_step_host_wait returns
 *                                      (pinned memory, or the copies do not overlap with anything);
 *   h_out                              holds the step's pooled output once mpe_step_host_wait has returned;
 *                                      give every step in flight its own buffer.
 * Errors: as mpe_forward / mpe_backward (argument and sequence errors are returned by the submit call;
 * nothing is enqueued then).  Growing the staging buffers or the workspace (first call, larger batch) waits
 * for everything in flight and reallocates; the staging buffers are sized for the batch at hand or for the
 * reservation made with mpe_reserve, whichever is larger, so reserve the largest batch first when batch sizes
 * vary.  mpe_step_host_wait waits for all submitted steps. */
int mpe_step_host_submit(mpe_handle* h, const int32_t* h_indices, const int32_t* h_offsets, int32_t batch,
                         int64_t total_indices, const float* h_grad_out, float* h_out, float lr, int64_t step);
int mpe_step_host_wait(mpe_handle* h);

/*
 * Evaluation forward that allocates nothing.  (The paper has no counterpart: this is an addition for
 * callers that are not allowed to allocate device memory when they call into the library -- code that
 * runs under a memory budget fixed at start-up, inside another framework's allocator that must see every
 * byte, or in a region where a synchronising cudaMalloc/cudaFree would stall concurrent streams.
 * mpe_forward sizes its workspace with cudaMalloc whenever a larger batch arrives; this entry point never
 * does.)
 *
 * Same inputs, outputs, layouts and result as mpe_forward -- the pooled FP32 sums of the bags, bit for bit
 * -- but every intermediate array of the step (sort keys and payloads, digit counts, per-tile words, the
 * distinct-row list and its maps) lives in ONE fixed array compiled into the library
 * (`static __device__`, about 2.5 MB; every GPU that loads the library holds it until the process exits).
 * Limits: total_indices <= MPE_STATIC_MAX_INDICES, num_tables * batch <= MPE_STATIC_MAX_BAGS,
 * num_tables <= MPE_STATIC_MAX_TABLES; a larger call returns MPE_ERR_TOO_LARGE and does nothing.
 * It calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * It is an evaluation forward: it never changes the tables, the cached rows, the tags or the priority values
 * (the only handle memory it writes are the per-slot marks "hit in forward call number e", which every forward
 * rewrites under a fresh call number before anything reads them) and cannot be followed by mpe_backward; calling it between the mpe_forward and mpe_backward of a training step returns
 * MPE_ERR_SEQUENCE.  Out-of-range row ids contribute nothing and inconsistent offsets give all-zero
 * output, as in mpe_forward, but this entry point does not record them for mpe_last_error.
 *
 * All calls, from every handle on that GPU, share the one array, and it keeps the previous call's
 * contents (the call clears the counters it needs at zero): two calls whose GPU work overlaps -- different
 * streams, or different handles -- race on it.  Issue them on one stream, or wait between them.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress); make that
 * first call outside any stream capture.  The look-up is guarded by a lock, so first calls may come from
 * several host threads (on different handles) at once.
 */
#define MPE_STATIC_MAX_INDICES 32768
#define MPE_STATIC_MAX_BAGS 32768
#define MPE_STATIC_MAX_TABLES 64
int mpe_forward_static(mpe_handle* h, const int32_t* d_indices, const int32_t* d_offsets, int32_t batch,
                       int64_t total_indices, float* d_out, void* cuda_stream);

/* Write every cache-resident row back into the low-precision table with stochastic rounding; rows
 * stay resident and unchanged.  Afterwards the table alone is a complete snapshot of the model.
 * (The paper has no flush; it is the snapshot operation a trainer needs.) */
int mpe_flush(mpe_handle* h);

/* Waits for the handle's stream, then frees everything. */
int mpe_destroy(mpe_handle* h);

/* ---- observation (all of these wait for the handle's stream) --------------------------------- */
/* Sticky device-detected condition since the last call of this function: *code is MPE_OK,
 * MPE_ERR_INDEX, MPE_ERR_OFFSETS or MPE_ERR_TIMEOUT; *detail counts the offending items.  Clears the
 * condition.  (MPE_ERR_TIMEOUT: the sort's tiles learn their output positions from the tiles before them;
 * every such wait gives up after about a second, the step that met it changes nothing from there on and
 * the handle stays usable.  It is not expected to occur.) */
int mpe_last_error(mpe_handle* h, int32_t* code, int64_t* detail);
/* Counters of table `table` accumulated by mpe_backward: out8 = {lookups, hits (per index),
 * unique rows, unique hits, admissions, evictions, bypasses, steps}. */
int mpe_stats(mpe_handle* h, int32_t table, uint64_t* out8);
/* Bytes of each component of the appendix's memory accounting (Appendix Eq. 2-3), summed over
 * tables: out6 = {low-precision table incl. scale/bias, FP32 cache, tags, LFU counters or LRU
 * timestamps, optimizer state, the FP32 table this replaces}. */
int mpe_memory_bytes(mpe_handle* h, uint64_t* out6);
/* Device memory the handle holds beyond the model state: out2 = {bytes of the per-step workspace (sized by
 * mpe_reserve or by the largest batch seen; twice that once mpe_prepare has been used), bytes of the two staging sets of mpe_step_host / _submit}. */
int mpe_workspace_bytes(mpe_handle* h, uint64_t* out2);

/* Self-checks of the library's own safety nets, for tests.  They change no table, cache or policy state and need the
 * workspace to exist (after mpe_reserve or a forward; else MPE_ERR_SEQUENCE).
 *   MPE_SELFTEST_LOOK_BACK_TIMEOUT: on the handle's stream, one warp performs the sort's look-back for a tile whose
 *     predecessor belongs to nobody, with the wait cut to a few thousand polls (about a millisecond).  The wait gives
 *     up as designed: the next mpe_last_error reports MPE_ERR_TIMEOUT with detail 1, exactly as after a real one, and
 *     the handle goes on working.  Nothing hangs or faults.  Not between a forward and its backward.
 *   MPE_SELFTEST_RENEW_TAGS: the next mpe_forward starts the sort's pass numbers over (waits for the device, clears the
 *     per-tile words), which otherwise happens once in hundreds of millions of steps. */
#define MPE_SELFTEST_LOOK_BACK_TIMEOUT 1
#define MPE_SELFTEST_RENEW_TAGS 2
int mpe_selftest(mpe_handle* h, int32_t which);
/* Geometry of table `table`'s cache. */
int mpe_cache_geometry(mpe_handle* h, int32_t table, int32_t* n_sets, int32_t* ways);
/* Figures of the last step: out6 = {valid indices, distinct rows, dropped indices, rows whose gradient
 * is summed by the multi-block tree (more than 256 occurrences), indices that belong to such rows,
 * newcomers that had to wait for the write-back of a row updated in the same step (known after
 * mpe_backward)}. */
int mpe_step_info(mpe_handle* h, int64_t* out6);
/* Low-precision entries of n rows: h_codes[n][dim*bits/8] (INT4: column 2k in the low nibble of
 * byte k), h_scale[n], h_bias[n].  The entry of a cache-resident row is stale until it is evicted
 * or flushed. */
int mpe_export_rows(mpe_handle* h, int32_t table, const int64_t* h_rows, int64_t n, uint8_t* h_codes,
                    float* h_scale, float* h_bias);
/* Whole cache of one table: h_tags[n_sets*ways] (-1 = empty), h_rows[n_sets*ways][dim],
 * h_ts[n_sets*ways] (LRU timestamps; pass NULL to skip, zeros under LFU). */
int mpe_export_cache(mpe_handle* h, int32_t table, int32_t* h_tags, float* h_rows, uint32_t* h_ts);
/* Per-row auxiliary state of n rows: LFU counters and/or Adagrad accumulators (NULL to skip). */
int mpe_export_aux(mpe_handle* h, int32_t table, const int64_t* h_rows, int64_t n, uint32_t* h_cnt,
                   float* h_adagrad);

/* Steps of up to about four million indices are bound by kernel-launch latency, so by default each half of
 * the step is captured once into a CUDA graph (sized for the reserved workspace) and replayed; the per-call
 * arguments reach the kernels through device memory.  enable = 0 switches to plain launches (larger steps and
 * steps issued while profiling or while the caller captures the stream always use plain launches).  A backward
 * is replayed only if its forward was.  Not allowed between a forward and its backward (MPE_ERR_SEQUENCE).
 * A graph the CALLER captured around steps of this library may be replayed about 10^8 times in a row: the pass
 * numbers in the sort's per-tile words (30 bits) are started over by mpe_forward's host code, which counts the calls
 * it sees, not by the captured kernels.  For more replays, every 10^8 of them call
 * mpe_selftest(h, MPE_SELFTEST_RENEW_TAGS) and then one mpe_forward / mpe_backward outside the graph. */
int mpe_use_graphs(mpe_handle* h, int32_t enable);

/* ---- instrumentation ---------------------------------------------------------------------------- */
/* Number of kernels this handle has launched so far. */
int mpe_kernel_launches(mpe_handle* h, uint64_t* count);
/* With profiling on, every kernel launch is bracketed by CUDA events on the launching stream.  Waits for the
 * handle's stream; not allowed between a forward and its backward (MPE_ERR_SEQUENCE). */
int mpe_profile(mpe_handle* h, int32_t enable);
/* Waits for the stream, then reports per kernel name the launches and the summed event time since
 * profiling was switched on (or last read): up to `cap` entries, names are 32-byte C strings.
 * *n receives the number of distinct kernels. */
int mpe_profile_read(mpe_handle* h, int32_t cap, char* names /*[cap][32]*/, double* ms, uint64_t* launches,
                     int32_t* n);
const char* mpe_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif

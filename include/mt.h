/*
 * mt.h - C ABI of the mixed-tenant batched inference library (one B200, sm_100a).
 *
 * The paper (arXiv 1901.06887) frames DNN inference as a narrow interface: a
 * tenant uploads a model as a declarative list of standard layers (Sec. 3.1:
 * no user code, a fixed layer catalogue), then sends requests; a DNN is a
 * stateless deterministic function evaluated layer by layer (Sec. 1.1); a
 * worker hosts many tenants' models at once and multiplexes incoming requests
 * across them (Sec. 3).  This library is that worker's execution step:
 * mt_infer evaluates ONE mixed batch of requests, each tagged with the id of
 * its model, in a single pass over all co-resident models.
 *
 * Threading: all calls are serialised by one internal mutex.  A context has
 * one workspace, so two mt_infer calls must not be in flight on different
 * streams at the same time (order them with events, or use one stream;
 * mt_infer_host_async does that ordering itself and may be used on two streams).
 *
 * Every function returns an mt_status; MT_OK (0) is success.  No function
 * throws, traps or aborts.  There is no CPU fallback: on a device that is not
 * compute capability 10.x mt_init fails with MT_ERR_ARCH.
 */
#ifndef MT_H_
#define MT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MT_OK = 0,
    MT_ERR_INVALID_ARG = 1,   /* null pointer, negative size, bad enum value */
    MT_ERR_BAD_MODEL_ID = 2,  /* id never issued, already released, or (async) seen in a batch */
    MT_ERR_SHAPE = 3,         /* layer chain inconsistent, or model does not match the hosted family */
    MT_ERR_UNSUPPORTED = 4,   /* a dimension outside what the kernels handle (see mt_register_model) */
    MT_ERR_OOM = 5,           /* device or host allocation failed, or table full */
    MT_ERR_CUDA = 6,          /* a CUDA runtime/driver call failed */
    MT_ERR_ARCH = 7,          /* device is not sm_100 */
    MT_ERR_TIMEOUT = 8,       /* (async) a bounded device-side wait gave up */
    MT_ERR_NOT_INIT = 9,
    MT_ERR_NOT_RESIDENT = 10  /* (async) a request names a registered model whose weights are not on the device now */
} mt_status;

typedef enum { MT_DENSE = 0, MT_CONV3X3 = 1, MT_GLOBAL_AVG_POOL = 2, MT_CONV1X1 = 3 } mt_layer_kind;

#define MT_MAX_LAYERS 8

/* One layer of a declarative model description (Sec. 3.1).
 *   MT_DENSE            y = act(W x + b), W bf16 [out_ch][in_ch] row-major (Sec. 1.1, fully-connected layer)
 *   MT_CONV3X3          NHWC, stride 1, zero pad 1, cross-correlation; W bf16 [out_ch][3][3][in_ch];
 *                       tap (ky,kx) reads pixel (y+ky-1, x+kx-1)
 *   MT_GLOBAL_AVG_POOL  mean over the h*w positions of each channel; no weights
 *   MT_CONV1X1          pointwise conv, NHWC: the fully-connected layer applied at every pixel; W bf16 [out_ch][in_ch]
 * residual (MT_CONV3X3 only, the layer before it a conv too): the layer closes a two-layer residual block with an
 * identity shortcut, the building block of the network the paper uses as its running example (Sec. 1.1, resnet18):
 * a[l+1] = act(conv(a[l]) + b + a[l-1]), where a[l-1] is the INPUT of the layer before.  Tenants of one conv family
 * may differ in which layers carry it.
 * weight / bias may be host or device pointers; the library copies them during mt_register_model and
 * keeps no reference, so the caller may free them on return.  bias == NULL means zeros. */
typedef struct {
    int32_t kind;          /* mt_layer_kind */
    int32_t in_ch, out_ch; /* dense: in/out features; conv: C_in/C_out; pool: in_ch == out_ch */
    int32_t h, w;          /* conv/pool spatial size; 0 for dense */
    int32_t relu;          /* 1: apply max(.,0) after bias (and after the shortcut's sum) */
    int32_t residual;      /* 1: add the previous layer's input before the activation (see above); else 0 */
    const void* weight;    /* bf16 */
    const void* bias;      /* fp32 [out_ch] */
} mt_layer_desc;

/* Set-up and tear-down of the worker's context (no passage of the paper: it describes the service, not a library).
 * Create the context on CUDA device `device`.  max_models bounds the id space (<= 8192), max_batch is
 * a hint for the first workspace allocation (the workspace grows on demand, see mt_infer).  Calling
 * mt_register_model before mt_init initialises device 0 with defaults (1024 models).
 * Errors: MT_ERR_ARCH, MT_ERR_CUDA, MT_ERR_OOM, MT_ERR_INVALID_ARG (already initialised with other
 * arguments is accepted and ignored). */
mt_status mt_init(int32_t device, int32_t max_models, int32_t max_batch);

/* Release every model, workspace and the context.  Synchronises the device. */
mt_status mt_shutdown(void);

/* A tenant hands its model to the service (Sec. 1.2 / Sec. 3): validate the layer list, copy the weights to the device in
 * the executor's tiled layout and return a small dense id (lowest free slot first) in *model_id_out.
 * All models hosted by one context form one family: the same layer kinds index by index.  MLPs (dense layers only)
 * may differ in depth and in every width - input, hidden and output; conv families keep one depth, geometry, input and
 * output width.  The row stride of mt_infer's output buffer is the WIDEST registered model's output
 * (mt_output_elems); a model with fewer outputs writes the first out_ch columns of its requests' rows and leaves the rest
 * untouched.  The row stride of the input buffer is the WIDEST registered model's input (mt_input_elems); a request of a
 * model with fewer inputs carries them at the start of its row and the rest of the row is never read.
 * Kernel limits (else MT_ERR_UNSUPPORTED): 1..MT_MAX_LAYERS layers; dense in_ch a multiple of 64;
 * conv3x3 in_ch == out_ch == 64, w <= 126; conv1x1 in_ch a multiple of 64, between two conv layers (it follows a conv3x3
 * or conv1x1 and is followed by one); a pool must follow a conv3x3; a dense layer may not precede a conv; residual only
 * on a conv3x3 layer that follows a conv3x3 layer.
 * The call does not wait for the device: weights and biases in HOST memory are copied into the library's pinned
 * staging before it returns (the caller may free them at once), and the copy to the device and the re-layout run on
 * an internal stream, under whatever batches are in flight; the first mt_infer* / mt_prefetch that follows waits, on
 * its own stream, for exactly the models it is the first to see.  Weights given as DEVICE pointers are read by that
 * internal stream, for which the call then waits (not for the device).  A model wider than any before makes the next
 * mt_infer* reallocate its workspace, which does synchronise the device.  MT_ASYNC_REGISTER=0 (option
 * "async_register") selects the older path that synchronises the device once per layer. */
mt_status mt_register_model(const mt_layer_desc* layers, int32_t n_layers, int32_t* model_id_out);

/* Elements per row of the output buffer as of now: the widest output among the models registered since the context
 * last held none (0 if none is registered); releasing a model never shortens the rows. */
mt_status mt_output_elems(int32_t* out_elems_out);

/* Elements per row of the input buffer as of now: the widest input among the models registered since the context
 * last held none (0 if none is registered). */
mt_status mt_input_elems(int32_t* in_elems_out);

/* One inference per request for a whole mixed batch (Sec. 3: a worker multiplexes requests across models).
 *   inputs    device, bf16, [n][in_elems] row-major (NHWC per request for conv), arrival order (in_elems: see
 *             mt_input_elems)
 *   model_ids device, int32 [n]; request i is evaluated by model model_ids[i]
 *   outputs   device, fp32, [n][out_elems], arrival order (out_elems: see mt_output_elems)
 *   stream    cudaStream_t (NULL = default stream)
 * Only enqueues work on `stream`: bucketing (histogram, exclusive scan, stable scatter, row gather), one
 * persistent grouped launch per layer (the last one writes its rows straight back in arrival order).  A batch
 * of at most 512 requests against dense layers at most 256 wide runs as ONE launch that does all of it; a conv
 * batch of at most 512 requests is bucketed inside its first conv launch.  No host<->device synchronisation happens unless the
 * workspace must grow (n larger than any earlier call, or a wider model registered since): then the
 * call synchronises the device and reallocates first - make one call at the largest n before timing.
 * inputs must be 16-byte aligned.  n == 0 is a no-op.  Once the workspace exists and the models in use have been seen by
 * one earlier call, the call only launches kernels on `stream`, so it may be captured into a CUDA graph and replayed on
 * new contents of the same buffers (tests/test_gpu_parity.py does).
 * A request whose id is not a live model never faults: its output row is NaN, a sticky status is set
 * (see mt_get_async_status) and all other requests complete normally. */
mt_status mt_infer(const void* inputs, const int32_t* model_ids, int32_t n, void* outputs, void* stream);

/* Same as mt_infer with HOST buffers (pinned memory recommended): copies inputs and ids to device
 * staging buffers on `stream`, runs the pass, copies the outputs back and synchronises `stream`.
 * The whole [n][out_elems] buffer is written: where models differ in output width, the columns of a row beyond its
 * model's own come back as NaN (mt_infer, which writes the caller's device buffer directly, leaves them untouched). */
mt_status mt_infer_host(const void* inputs_host, const int32_t* model_ids_host, int32_t n,
                        void* outputs_host, void* stream);

/* The same, without the final synchronisation, for callers that keep several batches in flight: everything is
 * enqueued on `stream` (copy in, the pass, copy out) and the call returns at once; synchronise `stream` before
 * reading outputs_host.  Host buffers must be pinned (cudaHostAlloc / cudaHostRegister) for the copies to be
 * asynchronous, and must stay untouched until the stream has passed the call.  Two device staging slots are used
 * in turn: a caller that alternates between TWO streams overlaps one batch's copies with its neighbours' kernels
 * (the kernels themselves run one batch after the other, since they share one workspace; the library orders them
 * with events).  mt_infer and mt_infer_host must not be in flight on other streams at the same time. */
mt_status mt_infer_host_async(const void* inputs_host, const int32_t* model_ids_host, int32_t n,
                              void* outputs_host, void* stream);

/* A tenant withdraws its model (Sec. 3: tenants upload models to the service and may remove them again; the paper
 * names no call for it).  Marks the id dead and frees its weights.  Synchronises the device first, so it cannot race
 * an mt_infer in flight.  The id may be re-issued by a later mt_register_model. */
mt_status mt_release(int32_t model_id);

/* Weight residency (Sec. 3.3: weights are cached at every level of the memory hierarchy; a model's footprint is fixed,
 * so the time to bring it in is predictable, and GPU memory need only hold the models in demand).  By default every
 * registered model stays on the device.  mt_set_cache_bytes(B), called after mt_init while no model is registered,
 * switches to a cache of B device bytes (one arena, allocated once; 0 switches back): registration then also keeps the
 * model's block - weights in the executor's layout and biases - in pinned host memory (copied back from the device on
 * the internal stream once the re-layout has run), and the device holds the least
 * recently used subset that fits.  MT_ERR_OOM: the arena cannot be allocated; a model larger than B is refused at
 * registration with MT_ERR_OOM.
 *
 * Who decides what is resident:
 *   mt_infer_host / mt_infer_host_async  read the batch's ids on the host and bring in exactly its tenants: blocks
 *       missing on the device are copied from their host images on an internal stream (over least-recently-used
 *       blocks if need be; blocks of this batch are never victims), the batch waits for the copies only, and copies
 *       for the next batch run under the kernels of the current one.  MT_ERR_OOM (nothing enqueued) if the batch's
 *       tenants do not fit the cache together.
 *   mt_prefetch(ids, count, stream)       the same for a caller that keeps ids on the device: name the tenants of the
 *       coming batch(es) (host array, duplicates allowed); work later enqueued on `stream` sees them resident.
 *       MT_ERR_BAD_MODEL_ID for an id that is not live, MT_ERR_OOM if the set does not fit.
 *   mt_infer                              never loads: a request for a registered but evicted model gets a NaN row and
 *       the sticky status MT_ERR_NOT_RESIDENT (see mt_get_async_status); all other requests complete.
 * A block that comes back is the same bytes as before, so outputs are bit-identical across evictions.
 * mt_get_cache_stats fills the counters since the cache was set up (or since the last call with reset != 0). */
typedef struct {
    uint64_t capacity_bytes, resident_bytes;
    uint64_t tenant_hits, tenant_misses;       /* per (batch or prefetch, tenant): block already there / had to be copied */
    uint64_t request_hits, request_misses;     /* the same weighted by the tenant's requests in the batch (host-id entry points) */
    uint64_t evictions, bytes_loaded;          /* blocks displaced; bytes copied host -> device for misses (registration included) */
} mt_cache_stats;
mt_status mt_set_cache_bytes(size_t device_bytes);
mt_status mt_prefetch(const int32_t* model_ids_host, int32_t count, void* stream);
mt_status mt_get_cache_stats(mt_cache_stats* out, int32_t reset);

/* The cache's policy by itself - first-fit arena, least-recently-used eviction on a clock the caller makes up - for
 * tests without a GPU.  access: result 0 = hit, 1 = placed (ids evicted to make room in evicted_out, at most
 * evicted_cap of them, their number in *n_evicted_out), -1 = does not fit beside the blocks touched at `tick`. */
mt_status mt_cache_sim_create(size_t capacity_bytes, void** sim_out);
mt_status mt_cache_sim_access(void* sim, int32_t id, size_t bytes, uint64_t tick, int32_t* result_out, int64_t* offset_out,
                              int32_t* evicted_out, int32_t evicted_cap, int32_t* n_evicted_out);
mt_status mt_cache_sim_release(void* sim, int32_t id);
mt_status mt_cache_sim_stats(void* sim, mt_cache_stats* out);
mt_status mt_cache_sim_destroy(void* sim);

/* Synchronise `stream`, then report and clear the sticky device-side status of the calls so far:
 * *status_out is MT_OK, MT_ERR_BAD_MODEL_ID or MT_ERR_NOT_RESIDENT (with the smallest offending arrival index of the
 * first such batch in *bad_request_index_out, else -1) or MT_ERR_TIMEOUT.  Either out pointer may be NULL. */
mt_status mt_get_async_status(void* stream, int32_t* status_out, int32_t* bad_request_index_out);

const char* mt_status_string(mt_status s);

/* Test hook: synchronise the device and copy the bucketing results of the last mt_infer to HOST arrays:
 * counts [T], offsets [T+2] (offsets[T+1] == n; [offsets[T], offsets[T+1]) holds rejected ids), perm [n],
 * inv [n], with n the batch size of that call and T = highest id ever issued + 1, returned in
 * *n_tenants_out (call once with null arrays to size them).  Any pointer may be NULL. */
mt_status mt_debug_last_bucketing(int32_t* counts_host, int32_t* offsets_host, int32_t* perm_host,
                                  int32_t* inv_host, int32_t* n_tenants_out);

/* Test hook for the bounded device-side waits (the executors never spin forever on a barrier: after a time limit
 * they give up, report MT_ERR_TIMEOUT and tear down normally, so a lost signal cannot hang the GPU).  Enqueues a
 * one-thread kernel that waits, for at most limit_ms (1..1000) milliseconds, on a barrier that nothing completes.
 * Afterwards mt_get_async_status reports MT_ERR_TIMEOUT and the context stays usable. */
mt_status mt_debug_wait_timeout(int32_t limit_ms, void* stream);

/* Test / bench hook: *count_out = number of kernels this library has enqueued on behalf of mt_infer and
 * mt_infer_host since it was loaded (registration and the no-allocation call are not counted). */
mt_status mt_debug_launch_count(int64_t* count_out);

/* Cost-aware scheduling (Sec. 3.2: a DNN's work per layer is fixed by its shape, so the cost of every work item is
 * known before a request arrives).  Each dense layer's work items are laid out heaviest first - tenants ranked on the
 * host, at registration, by the modelled cost of one of their items - and dealt back and forth over the CTAs.
 * mt_debug_item_cost: the model itself (pure host code, usable without a GPU): SM cycles of an item with k_blocks
 * K blocks of 64, n_cols output columns and `rows` requests (<= 64: transposed form); 0 for an empty item.
 * mt_debug_schedule_balance: for dense layer `layer` of the LAST mt_infer (layer-by-layer path), the heaviest CTA's
 * modelled cost over the mean (*max_over_mean_out; 1.0 = perfectly even), the number of work items and of CTAs (or
 * CTA pairs) they were dealt to.  Synchronises the device. */
mt_status mt_debug_item_cost(int32_t k_blocks, int32_t n_cols, int32_t rows, double* cycles_out);
mt_status mt_debug_schedule_balance(int32_t layer, double* max_over_mean_out, int32_t* n_items_out, int32_t* n_ctas_out);

/* Bench hook: enqueue `count` (0..100000) kernels that do nothing, chained on `stream` by programmatic dependent
 * launch exactly like the kernels of the path.  Timing a long chain gives the least a launch of the path can cost
 * (the launch floor that bounds a batch as small as 64 requests); not counted by mt_debug_launch_count. */
mt_status mt_debug_empty_launches(int32_t count, void* stream);

/* Test / A-B timing hook: which executor a batch takes.  Each switch starts from the environment variable read ONCE
 * by mt_init ("0" = off) and can be changed afterwards with this call; nothing reads the environment per batch.
 *   "fused"      (MT_FUSED)      one launch for a small batch of narrow MLPs; off: the layer-by-layer path
 *   "pair"       (MT_PAIR)       CTA-pair dense executor for batches with >= 1024 requests per tenant
 *   "conv_pair"  (MT_CONV_PAIR)  CTA-pair conv executor for padded rows of 64 pixels; off: the one-CTA executor
 *   "conv_stack" (MT_CONV_STACK) consecutive conv layers of the CTA-pair executor as one launch with grid-wide barriers;
 *                off: one launch per conv layer
 *   "conv_balance" (MT_CONV_BALANCE) the CTA-pair conv executor cuts its clusters' ranges by cost, a tenant border inside a
 *                range counting as two units of work; off: ranges of equal length
 *   "async_register" (MT_ASYNC_REGISTER) registration without device synchronisation; off: synchronous registration
 *   "pool_head"  (MT_POOL_HEAD)  pool + narrow head as one launch; off: pool_finalize + a grouped dense launch
 *   "perm_gather" (MT_PERM_GATHER) first dense layer reads the caller's rows through the permutation with TMA gathers
 *                instead of a row-move pass: 0 never, 1 (default) for batches of at most 256 requests, 2 always
 * Unknown name: MT_ERR_INVALID_ARG.  Results agree with the oracle on every setting. */
mt_status mt_debug_set_option(const char* name, int32_t value);

/* Per-kernel device timing.  enable = 1: every kernel launch of mt_infer is bracketed by CUDA events on the
 * caller's stream; enable = 2: only the layer executors (dense / conv / the one-launch path) are, and consecutive
 * launches of the same executor (also across calls, when a call is a single launch) share one pair of events, so
 * that the launches still overlap as they do untimed; enable = 3: as 2, on every fourth call only (an event between
 * two kernels still costs the overlap at that boundary, a few microseconds per pair);
 * 0: off.  mt_get_kernel_times synchronises those events, then fills up to `cap`
 * entries: names[i] (static strings), total_ms[i], launches[i]; *n_out = number of kernels seen.
 * Reading resets the accumulators. */
mt_status mt_set_kernel_timing(int32_t enable);
mt_status mt_get_kernel_times(const char** names, double* total_ms, int32_t* launches, int32_t cap,
                              int32_t* n_out);

/* Bucketing without any allocation.  (The paper has no counterpart to this call; it exists for callers
 * of this library that are not allowed to allocate device memory.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits - inside another allocator's
 * callback or a framework memory-pool hook, in a serving loop that froze its memory map after start-up, or
 * in a process whose device memory belongs wholly to a different allocator.  mt_infer cannot serve them,
 * because its workspace is allocated (and grown) with cudaMalloc.  This call does the same stable counting
 * sort of a batch by model id, using a fixed scratch array that is part of the library image: each GPU that
 * loads the library holds 1,057,804 bytes (1.01 MiB) for it until the process exits.  It never calls cudaMalloc,
 * cudaFree or any allocating routine, and needs no mt_init.  One caveat: the FIRST call on each device is where the
 * driver loads this part of the library (kernels and the scratch array itself, under lazy module loading) and where
 * the array's address is looked up, so that one call may allocate inside the driver.  Make it at start-up, outside
 * any allocator hook or frozen-memory phase - a call with n = 0 is enough; later calls allocate nothing.
 *
 *   model_ids   device, int32 [n]
 *   n           0 .. MT_NOALLOC_MAX_BATCH        (larger: MT_ERR_UNSUPPORTED, nothing enqueued)
 *   n_models    1 .. MT_NOALLOC_MAX_MODELS       (larger: MT_ERR_UNSUPPORTED, nothing enqueued)
 *   counts_out  device, int32 [n_models]         requests per id
 *   offsets_out device, int32 [n_models + 1]     exclusive prefix of counts; [n_models] = number of valid requests
 *   perm_out    device, int32 [n]                arrival index at each bucketed position (arrival order kept
 *                                                inside a segment); ids outside [0, n_models) sort behind all
 *                                                valid segments, in arrival order
 *   inv_out     device, int32 [n]                bucketed position of each arrival index
 *   stream      cudaStream_t; the work is enqueued there and runs on the CURRENT device
 *
 * The first call on each device looks up the scratch array's device address (with that device current);
 * make that first call before starting any stream capture.  All calls on a device share the one scratch
 * array, which still holds the previous call's contents when the next one starts; every entry a call reads
 * is written by that call first, so nothing needs clearing, but two calls whose kernels overlap on the GPU
 * (different streams without ordering) race and give wrong results - serialise them. */
#define MT_NOALLOC_MAX_BATCH 65536
#define MT_NOALLOC_MAX_MODELS 1024
mt_status mt_bucket_noalloc(const int32_t* model_ids, int32_t n, int32_t n_models, int32_t* counts_out,
                            int32_t* offsets_out, int32_t* perm_out, int32_t* inv_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MT_H_ */

// C-ABI layer: model registry, device workspace, tensor maps and the per-batch launch sequence.
// Everything that computes runs in the CUDA kernels of the other files; this file only validates,
// allocates, copies weights at registration and enqueues launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/mt.h"
#include "mt_device.cuh"
#include "mt_host.h"
#include "weight_cache.h"

namespace mt {
unsigned long long g_kernel_launches = 0;
}

namespace {

using namespace mt;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// kind is the EXECUTOR's kind: a pointwise conv (MT_CONV1X1 at the interface) is a dense layer over the pixels of the
// request's image, i.e. MT_DENSE with hw = H * W matrix rows per request (hw = 1 for a fully-connected layer).
struct HostLayer {
    int kind, in_ch, out_ch, h, w, relu, residual, hw;
};

struct HostModel {
    bool alive = false;
    std::vector<HostLayer> layers;
    void* dev_block = nullptr;             // without the weight cache: the model's own allocation
    // with the weight cache: the block lives in the arena while resident; its image is kept in pinned host memory
    size_t block_bytes = 0;
    void* host_image = nullptr;
    std::vector<size_t> w_off, b_off;      // per layer: offsets of weights and bias inside the block
    uint64_t last_batch = 0;               // number of the last batch that may have read the block
    cudaEvent_t ready = nullptr;           // asynchronous registration: the block's copies and re-layout have finished
};

// A change of the device tables that waits for the next call that names a stream (registration has none).
struct PendingOp {
    int id;
    int kind;                              // 1: the model's block is (being made) ready - publish its entry; 2: evicted
};

// What a tenant's entry in the device tables becomes when its block is (re)loaded or evicted: passed BY VALUE to a
// one-CTA kernel on the caller's stream, so the change is ordered with the batches before and after it and no host
// buffer has to outlive the call.
struct TableUpdate {
    ModelDev md;
    CUtensorMap wmaps[MT_MAX_LAYERS];
    int32_t alive;                         // 1 resident, 2 registered but not resident
    int32_t id, n_wmaps;
};

__global__ void table_update_kernel(const __grid_constant__ TableUpdate u, ModelDev* models, int32_t* brief, int brief_ld,
                                    CUtensorMap* wmaps) {
    const int t = threadIdx.x;
    if (u.alive == 1) {
        const int n_words = sizeof(ModelDev) / 4;
        const int32_t* src = reinterpret_cast<const int32_t*>(&u.md);
        int32_t* dst = reinterpret_cast<int32_t*>(models + u.id);
        for (int i = t; i < n_words; i += blockDim.x) dst[i] = src[i];
        const int map_words = sizeof(CUtensorMap) / 4;
        for (int l = 0; l < u.n_wmaps; ++l) {
            const int32_t* ms = reinterpret_cast<const int32_t*>(&u.wmaps[l]);
            int32_t* md = reinterpret_cast<int32_t*>(wmaps + (size_t)u.id * MT_MAX_LAYERS + l);
            for (int i = t; i < map_words; i += blockDim.x) md[i] = ms[i];
        }
    } else if (t == 0) {
        models[u.id].alive = u.alive;
    }
    if (t == 0) brief[u.id] = u.alive;
    if (u.alive == 1 && t >= 1 && t <= MT_MAX_LAYERS)      // rows 1..: out features per layer (0: the model has no such layer)
        brief[(size_t)t * brief_ld + u.id] = (t - 1 < u.md.n_layers) ? u.md.layer[t - 1].N : 0;
}

enum KernelId { K_BUCKET = 0, K_GATHER, K_GEMM, K_CONV, K_POOL, K_FUSED, K_COUNT };
const char* const kKernelNames[K_COUNT] = {"bucketing (histogram, scans, scatter, row move, work items)", "gather_rows",
                                           "grouped_gemm", "grouped_conv3x3", "pool (finalize, or pool + head)", "fused_mlp"};

struct TimedLaunch {
    int kernel;
    cudaEvent_t start, stop;
    int count;                           // launches between the two events
};

struct Ctx {
    bool init = false;
    int device = 0, sm_count = 0, max_models = 0;
    int T = 0;                           // id slots in use (highest issued id + 1)
    std::vector<HostModel> models;
    ModelDev* d_models = nullptr;
    int32_t* d_brief = nullptr;          // [1 + MT_MAX_LAYERS][max_models]: alive, out features per layer (bucketing passes)
    unsigned* d_grid_bar = nullptr;      // [8] barrier counters of a call's multi-layer conv launches (zeroed by the bucketing kernel)
    int32_t* d_order = nullptr;          // [MT_MAX_LAYERS][max_models]: per layer, tenants by descending a-priori item cost
    bool last_pair[MT_MAX_LAYERS] = {false};   // executor form of each dense layer in the last mt_infer (balance report)
    CUtensorMap* d_wmaps = nullptr;      // [max_models][MT_MAX_LAYERS]: dense weights as 128 x 64 boxes of the tiled image
    EncodeTiledFn encode = nullptr;

    // the hosted family (fixed by the first registered model)
    bool has_family = false;
    std::vector<HostLayer> family;       // kinds and geometry; dense hidden widths are per model
    int in_elems = 0, out_elems = 0;
    int width[MT_MAX_LAYERS + 1] = {0};  // per layer boundary: widest input row (elements) over all models
    int live = 0;
    ConvPlan conv;                       // strip geometry of the conv layers (one geometry per family)
    int tile_n[MT_MAX_LAYERS] = {0};     // per dense layer: output columns per work item (128 or 256)

    // workspace
    int cap_n = 0;
    bool ws_dirty = true;
    int32_t *d_block_hist = nullptr, *d_counts = nullptr, *d_offsets = nullptr, *d_tile_prefix = nullptr,
            *d_perm = nullptr, *d_inv = nullptr, *d_status = nullptr, *d_ticket = nullptr;
    void* act[MT_MAX_LAYERS + 1] = {nullptr};
    int act_ld[MT_MAX_LAYERS + 1] = {0};
    CUtensorMap act_map[MT_MAX_LAYERS + 1];
    CUtensorMap act_map32[MT_MAX_LAYERS + 1];   // dense inputs again, as 32-row boxes
    CUtensorMap act_store_map[MT_MAX_LAYERS + 1];   // conv activations as the store boxes of the CTA-pair executor
    CUtensorMap act_rows2_map[MT_MAX_LAYERS + 1];   // ... and as its load boxes of two rows and of one row
    CUtensorMap act_rows1_map[MT_MAX_LAYERS + 1];
    float* d_pool_partial = nullptr;     // per-strip channel sums of a conv layer that feeds a pool
    WorkItem* d_items[MT_MAX_LAYERS] = {nullptr};   // per dense layer
    size_t items_cap[MT_MAX_LAYERS] = {0};
    int last_n = 0;

    // staging for mt_infer_host
    void* st_in = nullptr;
    int32_t* st_ids = nullptr;
    float* st_out = nullptr;
    int n_residual[MT_MAX_LAYERS] = {0};     // live models whose layer l carries an identity shortcut
    bool out_mixed = false;                  // models of different output widths have been registered in this family
    size_t st_cap_in = 0, st_cap_ids = 0, st_cap_out = 0;   // bytes: a new family changes the row sizes, not only n

    // staging for mt_infer_host_async: two slots used in turn, so that the copies of one call overlap the compute
    // of its neighbours when the caller alternates between two streams
    void* as_in[2] = {nullptr, nullptr};
    int32_t* as_ids[2] = {nullptr, nullptr};
    float* as_out[2] = {nullptr, nullptr};
    size_t as_cap_in = 0, as_cap_ids = 0, as_cap_out = 0;   // bytes, per slot
    int as_next = 0;
    cudaEvent_t as_slot_done[2] = {nullptr, nullptr};   // the slot's device-to-host copy has finished
    bool as_slot_used[2] = {false, false};
    cudaEvent_t as_compute_done = nullptr;               // the previous call's kernels have finished (shared workspace)
    bool as_have_compute = false;

    // switches for tests and A/B timing: read from the environment once, at mt_init (MT_FUSED, MT_PAIR, MT_CONV_PAIR,
    // MT_POOL_HEAD; "0" turns the path off), changed afterwards only through mt_debug_set_option
    bool opt_fused = true, opt_pair = true, opt_conv_pair = true, opt_pool_head = true, opt_conv_stack = true, opt_conv_balance = true,
         opt_conv_self_bucket = true;
    int opt_gather = 1;                  // 0 never, 1 small batches, 2 always

    // tensor maps over the caller's images (first conv layer), kept while pointer and batch size stay the same
    const void* in_map_ptr = nullptr;
    int in_map_n = 0;
    CUtensorMap in_map, in_rows2_map, in_rows1_map;

    // weight cache (off while cache_bytes == 0: every registered model stays resident in its own allocation)
    size_t cache_bytes = 0;
    uint8_t* arena = nullptr;
    WeightCache cache;
    cudaStream_t load_stream = nullptr;
    uint64_t batch_no = 0;                              // batches enqueued so far (with the cache on)
    uint64_t synced_batch = 0;                          // batches up to this one are known to have finished
    uint64_t cache_tick = 0;                            // logical clock of the eviction policy
    static constexpr int kBatchEvents = 8;
    cudaEvent_t batch_done[kBatchEvents] = {nullptr};   // batch b's kernels have finished: batch_done[b % kBatchEvents]
    cudaEvent_t loads_done = nullptr;
    uint64_t request_hits = 0, request_misses = 0;

    // asynchronous registration: staging for the caller's weights (pinned host + device mirror), table changes that
    // wait for a stream, and the host mirror of the per-layer tenant order
    void* reg_host = nullptr;
    void* reg_dev = nullptr;
    size_t reg_host_cap = 0, reg_dev_cap = 0;
    cudaEvent_t reg_h2d_done = nullptr;                 // the staging copy of the last registration has left pinned memory
    bool reg_h2d_pending = false;
    std::vector<PendingOp> pending_ops;
    int32_t* h_order = nullptr;                         // pinned, [MT_MAX_LAYERS][max_models]
    bool order_dirty = false, order_copy_pending = false;
    cudaEvent_t order_copied = nullptr;
    bool opt_async_register = true;

    // timing
    int timing = 0;                      // 0 off, 1 every kernel, 2 only the layer executors, 3 the same on every 4th call
    int timing_now = 0;                  // the mode in force for the current call (0, 1 or 2)
    unsigned timing_calls = 0;
    std::vector<TimedLaunch> timed;
    std::vector<cudaEvent_t> event_pool;
};

Ctx g;
std::mutex g_mu;

#define CU_OK(call)                                                   \
    do {                                                              \
        cudaError_t e__ = (call);                                     \
        if (e__ != cudaSuccess) {                                     \
            if (getenv("MT_LOG"))                                     \
                fprintf(stderr, "[mt] %s:%d %s -> %s\n", __FILE__, __LINE__, #call, cudaGetErrorString(e__)); \
            return (e__ == cudaErrorMemoryAllocation) ? MT_ERR_OOM : MT_ERR_CUDA; \
        }                                                             \
    } while (0)

mt_status reset_status_word() {
    const int32_t init[ST_WORDS] = {MT_OK, INT_MAX, 0, 0};
    CU_OK(cudaMemcpy(g.d_status, init, sizeof init, cudaMemcpyHostToDevice));
    return MT_OK;
}

mt_status do_init(int device, int max_models, int /*max_batch*/) {
    if (g.init) return MT_OK;
    if (max_models <= 0 || max_models > 8192) return MT_ERR_INVALID_ARG;
    int n_dev = 0;
    CU_OK(cudaGetDeviceCount(&n_dev));
    if (device < 0 || device >= n_dev) return MT_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    CU_OK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return MT_ERR_ARCH;
    CU_OK(cudaSetDevice(device));
    g.device = device;
    g.sm_count = prop.multiProcessorCount;
    g.max_models = max_models;
    g.models.assign(max_models, HostModel());
    CU_OK(cudaMalloc(&g.d_models, sizeof(ModelDev) * (size_t)max_models));
    CU_OK(cudaMemset(g.d_models, 0, sizeof(ModelDev) * (size_t)max_models));
    CU_OK(cudaMalloc(&g.d_brief, sizeof(int32_t) * (size_t)(1 + MT_MAX_LAYERS) * max_models));
    CU_OK(cudaMemset(g.d_brief, 0, sizeof(int32_t) * (size_t)(1 + MT_MAX_LAYERS) * max_models));
    CU_OK(cudaMalloc(&g.d_grid_bar, sizeof(unsigned) * 8));
    CU_OK(cudaMemset(g.d_grid_bar, 0, sizeof(unsigned) * 8));
    CU_OK(cudaMalloc(&g.d_order, sizeof(int32_t) * (size_t)MT_MAX_LAYERS * max_models));
    CU_OK(cudaMallocHost(&g.h_order, sizeof(int32_t) * (size_t)MT_MAX_LAYERS * max_models));
    for (size_t i = 0; i < (size_t)MT_MAX_LAYERS * max_models; ++i) g.h_order[i] = (int32_t)(i % (size_t)max_models);
    CU_OK(cudaMemcpy(g.d_order, g.h_order, sizeof(int32_t) * (size_t)MT_MAX_LAYERS * max_models, cudaMemcpyHostToDevice));
    if (!g.load_stream) CU_OK(cudaStreamCreateWithFlags(&g.load_stream, cudaStreamNonBlocking));
    if (!g.reg_h2d_done) CU_OK(cudaEventCreateWithFlags(&g.reg_h2d_done, cudaEventDisableTiming));
    if (!g.order_copied) CU_OK(cudaEventCreateWithFlags(&g.order_copied, cudaEventDisableTiming));
    g.order_dirty = false; g.order_copy_pending = false; g.reg_h2d_pending = false;
    g.pending_ops.clear();
    CU_OK(cudaMalloc(&g.d_wmaps, sizeof(CUtensorMap) * (size_t)max_models * MT_MAX_LAYERS));
    CU_OK(cudaMalloc(&g.d_status, sizeof(int32_t) * ST_WORDS));
    CU_OK(cudaMalloc(&g.d_ticket, sizeof(int32_t)));
    CU_OK(cudaMemset(g.d_ticket, 0, sizeof(int32_t)));
    CU_OK(cudaMalloc(&g.d_counts, sizeof(int32_t) * (size_t)(max_models + 1)));
    CU_OK(cudaMalloc(&g.d_offsets, sizeof(int32_t) * (size_t)(max_models + 2)));
    CU_OK(cudaMalloc(&g.d_tile_prefix, sizeof(int32_t) * (size_t)MT_MAX_LAYERS * (max_models + 1)));
    CU_OK(cudaMemset(g.d_offsets, 0, sizeof(int32_t) * (size_t)(max_models + 2)));
    mt_status st = reset_status_word();
    if (st != MT_OK) return st;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CU_OK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return MT_ERR_CUDA;
    g.encode = reinterpret_cast<EncodeTiledFn>(fn);
    CU_OK(configure_bucketing());
    CU_OK(configure_grouped_gemm());
    CU_OK(configure_grouped_conv());
    CU_OK(configure_grouped_gemm_pair());
    CU_OK(configure_fused_mlp());
    CU_OK(configure_grouped_conv_pair());
    g.T = 0;
    g.live = 0;
    for (int l = 0; l < MT_MAX_LAYERS; ++l) g.n_residual[l] = 0;
    g.has_family = false;
    g.cap_n = 0;
    g.ws_dirty = true;
    g.in_map_ptr = nullptr;
    auto env_on = [](const char* name) { const char* v = getenv(name); return !(v && v[0] == '0'); };
    g.opt_fused = env_on("MT_FUSED");
    g.opt_pair = env_on("MT_PAIR");
    g.opt_conv_pair = env_on("MT_CONV_PAIR");
    g.opt_pool_head = env_on("MT_POOL_HEAD");
    g.opt_conv_stack = env_on("MT_CONV_STACK");
    g.opt_async_register = env_on("MT_ASYNC_REGISTER");
    g.opt_conv_balance = env_on("MT_CONV_BALANCE");
    g.opt_conv_self_bucket = env_on("MT_CONV_SELF_BUCKET");
    { const char* v = getenv("MT_PERM_GATHER"); g.opt_gather = (v && v[0] >= '0' && v[0] <= '2') ? v[0] - '0' : 1; }
    g.init = true;
    return MT_OK;
}

void free_workspace() {
    cudaFree(g.d_block_hist); g.d_block_hist = nullptr;
    cudaFree(g.d_perm); g.d_perm = nullptr;
    cudaFree(g.d_inv); g.d_inv = nullptr;
    cudaFree(g.d_pool_partial); g.d_pool_partial = nullptr;
    for (int b = 0; b <= MT_MAX_LAYERS; ++b) { cudaFree(g.act[b]); g.act[b] = nullptr; }
    for (int l = 0; l < MT_MAX_LAYERS; ++l) { cudaFree(g.d_items[l]); g.d_items[l] = nullptr; g.items_cap[l] = 0; }
    g.cap_n = 0;
}

// The host-buffer entry points' device staging.  Sized in bytes for the family's rows at the time; released when
// the context adopts another family (the caller has synchronised the device).
void free_staging() {
    cudaFree(g.st_in); cudaFree(g.st_ids); cudaFree(g.st_out);
    g.st_in = nullptr; g.st_ids = nullptr; g.st_out = nullptr;
    g.st_cap_in = g.st_cap_ids = g.st_cap_out = 0;
    for (int k = 0; k < 2; ++k) {
        cudaFree(g.as_in[k]); cudaFree(g.as_ids[k]); cudaFree(g.as_out[k]);
        g.as_in[k] = nullptr; g.as_ids[k] = nullptr; g.as_out[k] = nullptr;
        g.as_slot_used[k] = false;
    }
    g.as_cap_in = g.as_cap_ids = g.as_cap_out = 0;
    g.as_have_compute = false;
}

mt_status encode_2d(CUtensorMap* map, void* ptr, int ld, int rows, int box_rows = BM) {
    cuuint64_t dims[2] = {(cuuint64_t)ld, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MT_OK : MT_ERR_CUDA;
}

// A dense layer's tiled weight image seen as rows of 64 bf16 (128 bytes): tile (nt, kb) is rows
// [(nt * kblocks + kb) * 128, + 128).  The image is already swizzled, so the copy must not swizzle again.
mt_status encode_weight_tiles(CUtensorMap* map, const void* ptr, size_t n_tiles_total) {
    cuuint64_t dims[2] = {(cuuint64_t)BK, (cuuint64_t)n_tiles_total * BN};
    cuuint64_t strides[1] = {(cuuint64_t)BK * 2};
    cuuint32_t box[2] = {BK, BN};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MT_OK : MT_ERR_CUDA;
}

mt_status encode_nhwc(CUtensorMap* map, const void* ptr, int C, int W, int H, int n_img, int box_w, int box_h,
                      int box_c = 0) {
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)n_img};
    cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[4] = {(cuuint32_t)(box_c ? box_c : C), (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    // a box row of 64 channels is 128 bytes, of 32 channels 64 bytes: the swizzle span follows it
    CUresult r = g.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, box[0] == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? MT_OK : MT_ERR_CUDA;
}

// (Re)allocate everything whose size depends on the batch size or on the family's widest rows.
mt_status ensure_workspace(int n) {
    if (!g.ws_dirty && n <= g.cap_n) return MT_OK;
    CU_OK(cudaDeviceSynchronize());
    int cap = g.cap_n > n ? g.cap_n : n;
    free_workspace();
    const int L = (int)g.family.size();
    const size_t n_blocks = (size_t)(cap + kHistChunk - 1) / kHistChunk;
    CU_OK(cudaMalloc(&g.d_block_hist, sizeof(int32_t) * n_blocks * (size_t)(g.max_models + 1)));
    CU_OK(cudaMalloc(&g.d_perm, sizeof(int32_t) * (size_t)cap));
    CU_OK(cudaMalloc(&g.d_inv, sizeof(int32_t) * (size_t)cap));
    for (int b = 0; b < L; ++b) {
        const HostLayer& f = g.family[b];
        if (f.kind == MT_DENSE) {
            // rows: one per request, or one per pixel of every request's image (pointwise conv)
            const size_t rows = (size_t)cap * f.hw;
            if (rows > (size_t)INT_MAX) return MT_ERR_UNSUPPORTED;
            g.act_ld[b] = g.width[b];
            const size_t bytes = rows * g.act_ld[b] * 2;
            CU_OK(cudaMalloc(&g.act[b], bytes));
            CU_OK(cudaMemset(g.act[b], 0, bytes));
            mt_status st = encode_2d(&g.act_map[b], g.act[b], g.act_ld[b], (int)rows);
            if (st != MT_OK) return st;
            st = encode_2d(&g.act_map32[b], g.act[b], g.act_ld[b], (int)rows, 32);
            if (st != MT_OK) return st;
            if (b > 0 && g.family[b - 1].kind == MT_CONV3X3) {      // a conv3x3 stores its 64-channel pixels here
                st = encode_nhwc(&g.act_store_map[b], g.act[b], f.in_ch, f.w, f.h, cap, 32, 1, 32);
                if (st != MT_OK) return st;
            }
        } else {
            g.act_ld[b] = f.in_ch * f.h * f.w;
            if (b == 0) continue;   // the first conv layer reads the caller's buffer through perm
            const size_t bytes = (size_t)cap * g.act_ld[b] * 2;
            CU_OK(cudaMalloc(&g.act[b], bytes));
            CU_OK(cudaMemset(g.act[b], 0, bytes));
            if (f.kind == MT_CONV3X3) {
                mt_status st = encode_nhwc(&g.act_map[b], g.act[b], f.in_ch, f.w, f.h, cap, g.conv.Wp, g.conv.R + 2);
                if (st != MT_OK) return st;
                st = encode_nhwc(&g.act_store_map[b], g.act[b], f.in_ch, f.w, f.h, cap, 32, 1, 32);
                if (st != MT_OK) return st;
                if (g.conv.Wp == 64) {
                    st = encode_nhwc(&g.act_rows2_map[b], g.act[b], f.in_ch, f.w, f.h, cap, 64, 2);
                    if (st != MT_OK) return st;
                    st = encode_nhwc(&g.act_rows1_map[b], g.act[b], f.in_ch, f.w, f.h, cap, 64, 1);
                    if (st != MT_OK) return st;
                }
            }
        }
    }
    for (int l = 0; l + 1 < L; ++l)
        if (g.family[l].kind == MT_CONV3X3 && g.family[l + 1].kind == MT_GLOBAL_AVG_POOL && !g.d_pool_partial)
            CU_OK(cudaMalloc(&g.d_pool_partial, sizeof(float) * (size_t)cap * g.conv.strips_per_image * 64));
    // work items of the dense layers: at most (row tiles + one ragged tile per tenant) x column tiles of the widest model
    for (int l = 0; l < L; ++l) {
        if (g.family[l].kind != MT_DENSE) continue;
        int out_w = std::max((l + 1 < L) ? g.width[l + 1] : 0, g.out_elems);   // hidden, or some tenant's last layer
        if (l + 1 < L && g.family[l + 1].kind != MT_DENSE) out_w = g.family[l + 1].in_ch;   // pointwise conv in front of a conv3x3
        const size_t col_tiles = (size_t)(out_w + BN - 1) / BN;    // bound for either tile width
        g.items_cap[l] = ((size_t)cap * g.family[l].hw / BM + (size_t)g.max_models + 1) * col_tiles;
        CU_OK(cudaMalloc(&g.d_items[l], sizeof(WorkItem) * g.items_cap[l]));
    }
    g.cap_n = cap;
    g.ws_dirty = false;
    return MT_OK;
}

bool is_device_pointer(const void* p) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// 128-row weight tiles allocated for a layer: an even count once N >= 256, so that 256-column work items can
// always fetch two tiles (the padding tile is zero).
size_t padded_weight_tiles(const HostLayer& h) {
    size_t t = (h.out_ch + BN - 1) / BN;
    if (h.kind == MT_DENSE && h.out_ch >= 256 && (t & 1)) t += 1;
    return t;
}

// 256-column work items for a dense layer iff every live model is at least 256 wide there.
void recompute_tile_n() {
    for (int l = 0; l < MT_MAX_LAYERS; ++l) g.tile_n[l] = BN;
    if (!g.has_family) return;
    for (size_t l = 0; l < g.family.size(); ++l) {
        if (g.family[l].kind != MT_DENSE) continue;
        int min_n = INT_MAX;
        for (const HostModel& m : g.models)
            if (m.alive && l < m.layers.size() && m.layers[l].out_ch < min_n) min_n = m.layers[l].out_ch;
        g.tile_n[l] = (min_n != INT_MAX && min_n >= 256) ? 256 : BN;
    }
}

// ---------------------------------------------------------------------------------------------- weight cache
// Device-table entry of model `id` for a block that starts at `base`.
mt_status fill_table_update(int id, uint8_t* base, TableUpdate* u) {
    const HostModel& hm = g.models[id];
    memset(u, 0, sizeof *u);
    u->id = id;
    u->alive = 1;
    u->md.alive = 1;
    u->md.n_layers = (int)hm.layers.size();
    for (size_t l = 0; l < hm.layers.size(); ++l) {
        const HostLayer& h = hm.layers[l];
        LayerDev& d = u->md.layer[l];
        d.kind = h.kind; d.K = h.in_ch; d.N = h.out_ch; d.relu = h.relu; d.residual = h.residual;
        d.n_tiles = (int)padded_weight_tiles(h);
        d.k_blocks = h.kind == MT_DENSE ? h.in_ch / BK : 9;
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        d.w = reinterpret_cast<const uint16_t*>(base + hm.w_off[l]);
        d.bias = reinterpret_cast<const float*>(base + hm.b_off[l]);
        if (h.kind == MT_DENSE) {
            mt_status st = encode_weight_tiles(&u->wmaps[l], base + hm.w_off[l], padded_weight_tiles(h) * (size_t)(h.in_ch / BK));
            if (st != MT_OK) return st;
            u->n_wmaps = (int)l + 1;
        }
    }
    return MT_OK;
}

void launch_table_update(const TableUpdate& u, cudaStream_t s) {
    table_update_kernel<<<1, 128, 0, s>>>(u, g.d_models, g.d_brief, g.max_models, g.d_wmaps);
}

// Registration and release change the device tables without naming a stream; the changes are applied here, in stream
// order, by the next call that does: a model whose block is ready (or becomes ready on the load stream: `s` waits for
// its event) gets its table entry, an evicted one is marked, and the per-layer tenant order is uploaded from its
// pinned mirror.
mt_status flush_tables(cudaStream_t s) {
    if (!g.pending_ops.empty()) {
        for (const PendingOp& op : g.pending_ops) {
            HostModel& hm = g.models[op.id];
            TableUpdate u;
            if (op.kind == 1) {
                if (!hm.alive) continue;                                         // released in the meantime
                if (g.cache_bytes && !g.cache.resident(op.id)) continue;         // evicted again before it was ever used
                if (hm.ready) CU_OK(cudaStreamWaitEvent(s, hm.ready, 0));
                uint8_t* base = g.cache_bytes ? g.arena + g.cache.find(op.id)->off : static_cast<uint8_t*>(hm.dev_block);
                mt_status st = fill_table_update(op.id, base, &u);
                if (st != MT_OK) return st;
            } else {
                if (!hm.alive || !g.cache_bytes || g.cache.resident(op.id)) continue;   // gone, or back already
                memset(&u, 0, sizeof u);
                u.id = op.id; u.alive = 2;
            }
            launch_table_update(u, s);
        }
        g.pending_ops.clear();
        CU_OK(cudaGetLastError());
    }
    if (g.order_dirty) {
        CU_OK(cudaMemcpyAsync(g.d_order, g.h_order, sizeof(int32_t) * (size_t)MT_MAX_LAYERS * g.max_models,
                              cudaMemcpyHostToDevice, s));
        CU_OK(cudaEventRecord(g.order_copied, s));
        g.order_copy_pending = true;
        g.order_dirty = false;
    }
    return MT_OK;
}

// Make the given tenants resident for the batch that is about to be enqueued on `s` (ids unique and live; reqs[i] =
// requests of ids[i] in the batch, for the request-level hit count).  Blocks that are missing are copied from their
// pinned host images on the load stream, into free arena space or over least-recently-used blocks; `s` waits for the
// copies, then the device tables are switched by small kernels on `s`.  A victim's bytes may still be read by
// batches in flight, so the copies wait for the youngest batch that could have used one.  MT_ERR_OOM: the set does
// not fit the cache (nothing of this batch has been enqueued; tenants evicted on the way stay evicted).
mt_status ensure_resident(const std::vector<int>& ids, const std::vector<int>& reqs, cudaStream_t s) {
    if (!g.cache_bytes || ids.empty()) return MT_OK;
    {
        mt_status fs = flush_tables(s);
        if (fs != MT_OK) return fs;
    }
    const uint64_t tick = ++g.cache_tick;
    struct Load { int id; size_t off; };
    std::vector<Load> loads;
    std::vector<int> evicted;
    mt_status result = MT_OK;
    for (size_t i = 0; i < ids.size(); ++i) {
        HostModel& hm = g.models[ids[i]];
        size_t off = 0;
        const WeightCache::Result r = g.cache.acquire(ids[i], hm.block_bytes, tick, &off, &evicted);
        if (r == WeightCache::kNoRoom) { result = MT_ERR_OOM; break; }
        if (r == WeightCache::kLoaded) { loads.push_back({ids[i], off}); g.request_misses += reqs[i]; }
        else g.request_hits += reqs[i];
        hm.last_batch = g.batch_no + 1;          // the batch being prepared
    }
    uint64_t youngest = 0;
    for (int e : evicted) {
        TableUpdate u;
        memset(&u, 0, sizeof u);
        u.id = e; u.alive = 2;
        launch_table_update(u, s);
        if (g.models[e].last_batch > youngest) youngest = g.models[e].last_batch;
    }
    if (!loads.empty()) {
        if (youngest > g.synced_batch && youngest <= g.batch_no)
            CU_OK(cudaStreamWaitEvent(g.load_stream, g.batch_done[youngest % Ctx::kBatchEvents], 0));
        for (const Load& l : loads) {
            const HostModel& hm = g.models[l.id];
            CU_OK(cudaMemcpyAsync(g.arena + l.off, hm.host_image, hm.block_bytes, cudaMemcpyHostToDevice, g.load_stream));
        }
        CU_OK(cudaEventRecord(g.loads_done, g.load_stream));
        CU_OK(cudaStreamWaitEvent(s, g.loads_done, 0));
        for (const Load& l : loads) {
            TableUpdate u;
            mt_status st = fill_table_update(l.id, g.arena + l.off, &u);
            if (st != MT_OK) return st;
            launch_table_update(u, s);
        }
    }
    CU_OK(cudaGetLastError());
    return result;
}

// Tenant set of a batch whose ids the host can read: unique live ids and their request counts.
void tenant_set_of(const int32_t* ids_host, int n, std::vector<int>* ids, std::vector<int>* reqs) {
    std::vector<int> count(g.T, 0);
    for (int i = 0; i < n; ++i) {
        const int t = ids_host[i];
        if (t >= 0 && t < g.T && g.models[t].alive) count[t] += 1;
    }
    for (int t = 0; t < g.T; ++t)
        if (count[t]) { ids->push_back(t); reqs->push_back(count[t]); }
}

// Book-keeping around one batch when the cache is on: the batch number is the clock of "who may still be reading
// which block"; a batch whose ids live on the device may read any resident block.
void cache_begin_batch(bool ids_unknown) {
    if (!g.cache_bytes) return;
    if (ids_unknown) {
        g.cache.touch_all(++g.cache_tick);
        for (int t = 0; t < g.T; ++t)
            if (g.models[t].alive && g.cache.resident(t)) g.models[t].last_batch = g.batch_no + 1;
    }
}
mt_status cache_end_batch(cudaStream_t s) {
    if (!g.cache_bytes) return MT_OK;
    g.batch_no += 1;
    CU_OK(cudaEventRecord(g.batch_done[g.batch_no % Ctx::kBatchEvents], s));
    return MT_OK;
}

// A-priori cost of one dense work item in SM cycles (Sec. 3.2: the work of a layer is fixed by its shape and known
// before any request arrives).  Per K block of 64 the item either waits for its bytes - the rows of the weight tile
// that hold output features plus the activation rows it fetches, at one SM's share of the HBM stream - or for the
// tensor pipe; the larger of the two counts.  A fixed part per item covers the hand-over of the accumulator and the
// epilogue's tail.  rows <= 64 is the transposed form (32-row activation boxes, weights on M).
double item_cost_cycles(int k_blocks, int n_cols, int rows) {
    if (k_blocks <= 0 || n_cols <= 0 || rows <= 0) return 0.0;
    const double kBytesPerClk = 23.0;                 // 6.5 TB/s over 148 SMs at 1.9 GHz
    const double kFixed = 700.0;
    const int w_rows = (n_cols + 7) & ~7;
    const bool swap = rows <= 64;
    const double a_bytes = swap ? ((rows + 31) / 32) * 4096.0 : 16384.0;
    const double bytes = w_rows * 128.0 + a_bytes;
    const int w_tiles = (n_cols + 127) / 128;
    // four K = 16 instructions per weight tile: N = 32/64 columns of requests when transposed, else N = 128 or 256
    const double mma = swap ? w_tiles * 4 * (rows <= 32 ? 36.0 : 43.0) : (n_cols <= 128 ? 4 * 62.0 : 4 * 120.0);
    const double per_kb = bytes / kBytesPerClk > mma ? bytes / kBytesPerClk : mma;
    return kFixed + k_blocks * per_kb;
}

// Per dense layer: id slots 0 .. T-1 by descending cost of one full work item (dead slots last), ties in id order; the
// other layers keep id order.  The bucketing passes lay the work items out in this order and the executors deal them
// back and forth over their CTAs (longest-processing-time-first list scheduling with costs known a priori).
mt_status recompute_order() {
    if (!g.has_family || g.T == 0) return MT_OK;
    if (g.order_copy_pending) {             // the pinned mirror may still be the source of a copy in flight
        CU_OK(cudaEventSynchronize(g.order_copied));
        g.order_copy_pending = false;
    }
    std::vector<int32_t> row(g.T);
    std::vector<double> cost(g.T);
    for (size_t l = 0; l < g.family.size(); ++l) {
        for (int t = 0; t < g.T; ++t) {
            row[t] = t;
            cost[t] = -1.0;
            const HostModel& m = g.models[t];
            if (g.family[l].kind == MT_DENSE && m.alive && l < m.layers.size()) {
                const HostLayer& h = m.layers[l];
                cost[t] = item_cost_cycles(h.in_ch / BK, h.out_ch < g.tile_n[l] ? h.out_ch : g.tile_n[l], BM);
            }
        }
        if (g.family[l].kind == MT_DENSE)
            std::stable_sort(row.begin(), row.end(), [&](int32_t a, int32_t b) { return cost[a] > cost[b]; });
        memcpy(g.h_order + l * (size_t)g.max_models, row.data(), sizeof(int32_t) * g.T);
    }
    g.order_dirty = true;      // uploaded, in stream order, by the next call that names a stream (flush_tables)
    return MT_OK;
}

mt_status validate_layers(const mt_layer_desc* layers, int n_layers) {
    if (!layers || n_layers < 1 || n_layers > MT_MAX_LAYERS) return n_layers > MT_MAX_LAYERS ? MT_ERR_UNSUPPORTED : MT_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
        const mt_layer_desc& d = layers[l];
        if (d.kind < MT_DENSE || d.kind > MT_CONV1X1) return MT_ERR_INVALID_ARG;
        if (d.in_ch <= 0 || d.out_ch <= 0) return MT_ERR_INVALID_ARG;
        if (d.kind != MT_GLOBAL_AVG_POOL && !d.weight) return MT_ERR_INVALID_ARG;
        // an identity shortcut joins a conv layer's output with the input of the conv layer before it
        if (d.residual && (d.kind != MT_CONV3X3 || l == 0 || layers[l - 1].kind != MT_CONV3X3)) return MT_ERR_UNSUPPORTED;
        if (d.kind == MT_DENSE) {
            if (l > 0) {
                const mt_layer_desc& p = layers[l - 1];
                if (p.kind == MT_CONV3X3 || p.kind == MT_CONV1X1) return MT_ERR_UNSUPPORTED;   // needs a pool in between
                if (p.out_ch != d.in_ch) return MT_ERR_SHAPE;
            }
            if (d.in_ch % BK != 0) return MT_ERR_UNSUPPORTED;
        } else if (d.kind == MT_CONV1X1) {
            // the dense executor over the pixels of the image: it reads an activation tensor in bucketed order, so it
            // follows a conv layer, and what follows it reads 64-channel (conv3x3) or 64-multiple (conv1x1) pixels
            if (d.h <= 0 || d.w <= 0) return MT_ERR_INVALID_ARG;
            if (l == 0 || l + 1 >= n_layers) return MT_ERR_UNSUPPORTED;
            const mt_layer_desc& p = layers[l - 1];
            if (p.kind != MT_CONV3X3 && p.kind != MT_CONV1X1) return MT_ERR_UNSUPPORTED;
            if (p.out_ch != d.in_ch || p.h != d.h || p.w != d.w) return MT_ERR_SHAPE;
            if (d.in_ch % BK != 0) return MT_ERR_UNSUPPORTED;
            const int next = layers[l + 1].kind;
            if (next != MT_CONV3X3 && next != MT_CONV1X1) return MT_ERR_UNSUPPORTED;   // the pool is fused into a conv3x3 only
        } else {
            if (d.h <= 0 || d.w <= 0) return MT_ERR_INVALID_ARG;
            if (l > 0) {
                const mt_layer_desc& p = layers[l - 1];
                // conv/pool only after a conv; the pool only after a conv3x3, whose epilogue does the summing
                if (p.kind != MT_CONV3X3 && !(p.kind == MT_CONV1X1 && d.kind == MT_CONV3X3)) return MT_ERR_UNSUPPORTED;
                if (p.out_ch != d.in_ch || p.h != d.h || p.w != d.w) return MT_ERR_SHAPE;
            } else if (d.kind == MT_GLOBAL_AVG_POOL) {
                return MT_ERR_UNSUPPORTED;
            }
            if (d.kind == MT_CONV3X3 && (d.in_ch != 64 || d.out_ch != 64 || d.w > 126)) return MT_ERR_UNSUPPORTED;
            if (d.kind == MT_GLOBAL_AVG_POOL && d.in_ch != d.out_ch) return MT_ERR_SHAPE;
        }
    }
    if (layers[n_layers - 1].kind != MT_DENSE) return MT_ERR_UNSUPPORTED;   // the last layer writes the fp32 output
    return MT_OK;
}

int layer_in_elems(const HostLayer& l) { return l.kind == MT_DENSE ? l.in_ch : l.in_ch * l.h * l.w; }

bool all_dense(const std::vector<HostLayer>& m) {     // an MLP: fully-connected layers only
    for (const HostLayer& l : m)
        if (l.kind != MT_DENSE || l.hw != 1) return false;
    return true;
}

// What the models of one context share: the layer kinds index by index.  MLPs (dense layers only) may differ in
// depth and in every width, the input's included; a tenant's layer j runs in the family's j-th launch and its last
// layer, whichever launch that is, writes the output - its own out_ch columns of a row whose stride is the widest
// model's output.  Likewise the rows of the input buffer are as long as the widest model's input and a request's row
// holds its own model's features first.  Conv families keep one depth, geometry, input and output width.
mt_status check_family(const std::vector<HostLayer>& m) {
    if (!g.has_family || g.live == 0) return MT_OK;
    if (all_dense(m) && all_dense(g.family)) return MT_OK;      // MLPs: any depth, any input, hidden and output widths
    if (layer_in_elems(m[0]) != g.in_elems) return MT_ERR_SHAPE;
    if (m.back().out_ch != g.out_elems) return MT_ERR_SHAPE;
    if (m.size() != g.family.size()) return MT_ERR_SHAPE;
    for (size_t l = 0; l < m.size(); ++l) {
        const HostLayer &a = m[l], &f = g.family[l];
        if (a.kind != f.kind || a.hw != f.hw) return MT_ERR_SHAPE;
        if (a.kind != MT_DENSE && (a.in_ch != f.in_ch || a.out_ch != f.out_ch || a.h != f.h || a.w != f.w)) return MT_ERR_SHAPE;
    }
    return MT_OK;
}

cudaEvent_t pooled_event() {
    cudaEvent_t e;
    if (!g.event_pool.empty()) { e = g.event_pool.back(); g.event_pool.pop_back(); }
    else cudaEventCreate(&e);
    return e;
}

// Timing mode 1: one pair of events around every launch.  Mode 2: only the layer executors are timed, and
// consecutive launches of the same executor share ONE pair of events (start before the first, stop after the last):
// an event between two launches would serialise them and undo the programmatic dependent launch that lets the next
// layer's prologue run under the previous layer's tail, i.e. it would time something the untimed path never does.
struct Timer {
    static int open_kernel;              // mode 2: executor whose group of launches is open (-1 none)
    static cudaEvent_t open_start;
    static int open_count;
    static cudaStream_t open_stream;
    int kernel;
    cudaStream_t s;
    bool each;
    cudaEvent_t start = nullptr;
    static void close_group() { close_group(open_stream); }
    static void close_group(cudaStream_t st) {
        if (open_kernel < 0) return;
        cudaEvent_t stop = pooled_event();
        cudaEventRecord(stop, st);
        g.timed.push_back({open_kernel, open_start, stop, open_count});
        open_kernel = -1;
    }
    Timer(int k, cudaStream_t st) : kernel(k), s(st), each(g.timing_now == 1) {
        if (each) {
            start = pooled_event();
            cudaEventRecord(start, s);
        } else if (g.timing_now == 2) {
            const bool executor = (k == K_GEMM || k == K_CONV || k == K_FUSED);
            if (open_kernel >= 0 && (open_kernel != k || open_stream != s)) close_group();
            if (executor && open_kernel < 0) {
                open_start = pooled_event();
                cudaEventRecord(open_start, s);
                open_kernel = k;
                open_count = 0;
                open_stream = s;
            }
            if (executor) ++open_count;
        }
    }
    ~Timer() {
        if (!each) return;
        cudaEvent_t stop = pooled_event();
        cudaEventRecord(stop, s);
        g.timed.push_back({kernel, start, stop, 1});
    }
};
int Timer::open_kernel = -1;
cudaEvent_t Timer::open_start = nullptr;
int Timer::open_count = 0;
cudaStream_t Timer::open_stream = nullptr;

mt_status infer_device(const void* inputs, const int32_t* ids, int n, void* outputs, cudaStream_t s) {
    if (!g.init) return MT_ERR_NOT_INIT;
    if (n < 0) return MT_ERR_INVALID_ARG;
    if (n == 0) return MT_OK;
    if (!inputs || !ids || !outputs) return MT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(inputs) & 15) return MT_ERR_INVALID_ARG;
    if (!g.has_family || g.live == 0) return MT_ERR_BAD_MODEL_ID;
    CU_OK(cudaSetDevice(g.device));
    mt_status st = ensure_workspace(n);
    if (st != MT_OK) return st;
    st = flush_tables(s);
    if (st != MT_OK) return st;
    const int L = (int)g.family.size();
    const HostLayer& f0 = g.family[0];
    // mode 3 times the executors of every fourth call only (a call that is a single launch keeps its group open
    // across calls instead, which costs nothing per call)
    g.timing_now = (g.timing == 3) ? (((g.timing_calls++ & 3u) == 0) ? 2 : 0) : g.timing;
    // Small batch of narrow MLPs: the whole pass in one launch (MT_FUSED=0 forces the layer-by-layer path).
    {
        bool all_dense = true;
        int max_w = g.out_elems;
        for (int l = 0; l < L; ++l) {
            all_dense = all_dense && g.family[l].kind == MT_DENSE;
            if (g.width[l] > max_w) max_w = g.width[l];
        }
        if (all_dense && g.opt_fused && fused_mlp_fits(n, g.T, max_w)) {
            if (g.timing == 3) g.timing_now = 2;
            Timer t(K_FUSED, s);
            FusedArgs a;
            a.inputs = static_cast<const uint16_t*>(inputs); a.ids = ids; a.n = n; a.T = g.T; a.models = g.d_models;
            a.n_layers = L; a.K0 = g.in_elems; a.out_elems = g.out_elems; a.out = static_cast<float*>(outputs);
            a.counts = g.d_counts; a.offsets = g.d_offsets; a.perm = g.d_perm; a.inv = g.d_inv; a.status = g.d_status;
            // at most one unit per request, and one per live tenant plus one per full tile
            int grid = g.live + n / BM;
            if (grid > n) grid = n;
            if (grid > g.sm_count) grid = g.sm_count;
            CU_OK(launch_fused_mlp(a, grid, s));
            // the group of launches stays open: a step of this path is ONE launch, and the next call's joins it (an
            // event pair per launch costs more than the launch); it closes when the times are read or timing changes
            g.last_n = n;
            return MT_OK;
        }
    }
    // The CTA-pair executor (256 x 256 work items, two SMs per item) fits batches whose tenants have thousands of
    // requests each; the host only knows the average, which is enough to tell that regime from the long-tail ones.
    // There it moves half the weight bytes per SM from L2 and runs about 4 % faster under the power cap (at a lower
    // clock).  MT_PAIR=0 keeps the one-CTA executor.
    bool pair_mode[MT_MAX_LAYERS] = {false};
    const bool pair_ok = g.opt_pair && (g.sm_count >= 2) && (n / (g.live > 0 ? g.live : 1) >= 1024);
    for (int l = 0; l < L; ++l) pair_mode[l] = pair_ok && g.family[l].kind == MT_DENSE && g.tile_n[l] == 256;
    for (int l = 0; l < MT_MAX_LAYERS; ++l) g.last_pair[l] = l < L && pair_mode[l];
    int tiles_per_image = 0;
    for (const HostLayer& f : g.family)
        if (f.kind == MT_CONV3X3) tiles_per_image = g.conv.strips_per_image;
    // A global average pool followed by a narrow last dense layer (a classifier head) runs as one small launch.
    const bool pool_head = L >= 3 && g.family[L - 2].kind == MT_GLOBAL_AVG_POOL && g.family[L - 1].kind == MT_DENSE &&
                           g.family[L - 2].in_ch == 64 && g.family[L - 1].in_ch == 64 && g.out_elems <= 64 &&
                           g.opt_pool_head;
    // Conv layers run on CTA pairs (two images of a tenant per cluster) when the strip geometry allows the tap
    // pairing; MT_CONV_PAIR=0 forces the one-CTA executor.
    // (its shortcut path alternates two register buffers over a strip's tiles: an even number of them)
    const bool conv_pair = tiles_per_image > 0 && g.conv.Wp == 64 && g.sm_count >= 2 && g.opt_conv_pair &&
                           g.conv.tiles_per_strip % 2 == 0;

    // Dense families: the payload rows move into bucketed order inside the scatter pass when the batch is spread over
    // enough CTAs and small enough for them; otherwise as a gather pass of its own over the whole GPU.
    // Small batches (one bucketing CTA, which cannot move rows): the first dense layer reads the caller's rows through
    // perm, four rows per TMA gather, and no row pass runs at all.  Measured: a gather costs the producer about 130
    // cycles against one box load per 128 rows, and a tile is fetched once per column tile, so beyond a few hundred
    // requests moving each row once is cheaper (config 3: +57 us, config 5: +10 ms with gathers; at 512 requests the
    // two are level).  "perm_gather" = 2
    // forces the gather for any batch size (tests).
    // Small conv batches on the CTA-pair executor, when pool + head end the pass (so that no dense work items are
    // needed): no bucketing launch; the first conv launch sorts the ids itself, in every CTA (MT_CONV_SELF_BUCKET=0:
    // the bucketing launch as for larger batches).
    bool convs_then_pool = conv_pair && pool_head;
    for (int l = 0; l + 2 < L; ++l) convs_then_pool = convs_then_pool && g.family[l].kind == MT_CONV3X3;
    const bool self_bucket = convs_then_pool && g.opt_conv_self_bucket && n <= kConvSelfBucketMaxN && g.T <= kConvSelfBucketMaxT;
    const bool perm_gather = f0.kind == MT_DENSE && (g.opt_gather == 2 || (g.opt_gather == 1 && n <= 256));
    const bool rows_in_scatter = f0.kind == MT_DENSE && !perm_gather && n > 512 && (size_t)n * g.in_elems * 2 <= ((size_t)64 << 20);
    if (!self_bucket) {
        Timer t(K_BUCKET, s);
        BucketArgs a;
        a.ids = ids; a.n = n; a.T = g.T; a.models = g.d_models; a.n_layers = L; a.rows_per_unit = tiles_per_image;
        a.brief = g.d_brief; a.brief_ld = g.max_models; a.order = g.d_order;
        a.grid_bar = conv_pair ? g.d_grid_bar : nullptr;
        for (int l = 0; l < 8; ++l) a.kind[l] = (l < L) ? g.family[l].kind : -1;
        a.ticket = g.d_ticket;
        a.rows_src = rows_in_scatter ? inputs : nullptr; a.rows_dst = g.act[0];
        a.row_bytes = g.in_elems * 2; a.dst_ld_bytes = g.act_ld[0] * 2;
        for (int l = 0; l < 8; ++l) {
            a.tile_n[l] = g.tile_n[l]; a.tile_m[l] = pair_mode[l] ? 2 * BM : BM;
            if (l < L && g.family[l].kind == MT_CONV3X3) a.tile_m[l] = conv_pair ? 2 : 1;
            a.items[l] = (l < MT_MAX_LAYERS) ? g.d_items[l] : nullptr;
            if (pool_head && l == L - 1) a.items[l] = nullptr;     // the pool + head launch needs no work items
        }
        a.item_grid = g.sm_count;
        for (int l = 0; l < 8; ++l) a.row_scale[l] = (l < L && g.family[l].kind == MT_DENSE) ? g.family[l].hw : 1;
        a.block_hist = g.d_block_hist; a.counts = g.d_counts; a.offsets = g.d_offsets; a.tile_prefix = g.d_tile_prefix;
        a.perm = g.d_perm; a.inv = g.d_inv; a.status = g.d_status;
        launch_bucketing(a, s);
    }
    CUtensorMap &in_map = g.in_map, &in_rows2_map = g.in_rows2_map, &in_rows1_map = g.in_rows1_map;
    if (f0.kind == MT_DENSE) {
        if (perm_gather) {
            if (g.in_map_ptr != inputs || g.in_map_n != n) {
                g.in_map_ptr = nullptr;
                st = encode_2d(&in_map, const_cast<void*>(inputs), g.in_elems, n, 1);   // one-row boxes: the gather form
                if (st != MT_OK) return st;
                g.in_map_ptr = inputs;
                g.in_map_n = n;
            }
        } else if (!rows_in_scatter) {
            Timer t(K_GATHER, s);
            launch_gather_rows(inputs, g.d_perm, n, g.in_elems * 2, g.act[0], g.act_ld[0] * 2, g.sm_count, s);
        }
    } else if (g.in_map_ptr != inputs || g.in_map_n != n) {
        g.in_map_ptr = nullptr;
        st = encode_nhwc(&in_map, inputs, f0.in_ch, f0.w, f0.h, n, g.conv.Wp, g.conv.R + 2);
        if (st != MT_OK) return st;
        if (g.conv.Wp == 64) {
            st = encode_nhwc(&in_rows2_map, inputs, f0.in_ch, f0.w, f0.h, n, 64, 2);
            if (st != MT_OK) return st;
            st = encode_nhwc(&in_rows1_map, inputs, f0.in_ch, f0.w, f0.h, n, 64, 1);
            if (st != MT_OK) return st;
        }
        g.in_map_ptr = inputs;
        g.in_map_n = n;
    }
    int n_conv_launch = 0;
    for (int l = 0; l < L; ++l) {
        const HostLayer& f = g.family[l];
        const bool last = (l == L - 1);
        if (f.kind == MT_DENSE) {
            Timer t(K_GEMM, s);
            GemmArgs a;
            a.T = g.T;
            a.tile_prefix = g.d_tile_prefix + (size_t)l * (g.T + 1);
            a.items = g.d_items[l];
            a.wmaps = g.d_wmaps; a.layer = l;
            // a tenant's last layer (any launch, for a family of mixed depths) writes straight into the caller's buffer in
            // arrival order; the family's deepest launch also fills the rows of rejected requests
            a.out = last ? nullptr : g.act[l + 1];
            // (a pointwise conv in front of a conv3x3 writes that layer's 64-channel pixels)
            a.ld_out = last ? 0 : (g.family[l + 1].kind == MT_DENSE ? g.act_ld[l + 1] : g.family[l + 1].in_ch);
            a.final_out = static_cast<float*>(outputs);
            a.ld_final = g.out_elems;
            a.nan_fill = last ? 1 : 0;
            a.perm = g.d_perm;
            a.offsets = g.d_offsets;
            a.status = g.d_status;
            const bool gather = (l == 0) && perm_gather;
            a.gather_perm = gather ? g.d_perm : nullptr;
            if (pair_mode[l]) CU_OK(launch_grouped_gemm_pair(gather ? in_map : g.act_map[l], a, g.sm_count, s));
            else launch_grouped_gemm(gather ? in_map : g.act_map[l], g.act_map32[l], a, g.tile_n[l], g.sm_count, s);
        } else if (f.kind == MT_CONV3X3) {
            Timer t(K_CONV, s);
            ConvArgs a;
            a.models = g.d_models; a.layer = l; a.T = g.T; a.offsets = g.d_offsets;
            a.tile_prefix = g.d_tile_prefix + (size_t)l * (g.T + 1);
            a.perm = (l == 0) ? g.d_perm : nullptr;
            a.H = f.h; a.W = f.w;
            a.Wp = g.conv.Wp; a.R = g.conv.R; a.tiles_per_strip = g.conv.tiles_per_strip;
            a.stage_bytes = g.conv.stage_bytes; a.n_stages = g.conv.n_stages;
            a.strips_per_image = g.conv.strips_per_image; a.box_bytes = g.conv.box_bytes;
            a.status = g.d_status;
            const auto is_conv = [&](int k) { return k >= 0 && k < L && g.family[k].kind == MT_CONV3X3; };
            // what a residual layer k adds: the input of layer k - 1 (the caller's buffer, in arrival order, for k = 1)
            const auto skip_of = [&](int k) -> const uint16_t* {
                if (k < 1 || !is_conv(k - 1) || g.n_residual[k] == 0) return nullptr;   // no live model has one there
                return k == 1 ? static_cast<const uint16_t*>(inputs) : static_cast<const uint16_t*>(g.act[k - 1]);
            };
            const auto feeds_pool_at = [&](int k) { return k + 1 < L && g.family[k + 1].kind == MT_GLOBAL_AVG_POOL; };
            if (conv_pair) {
                // consecutive conv layers (at most kConvStackMax) as ONE launch with grid-wide barriers in between
                int n_stack = 1;
                while (n_stack < kConvStackMax && g.opt_conv_stack && is_conv(l + n_stack)) ++n_stack;
                const int l_last = l + n_stack - 1;
                ConvStackMaps maps;
                for (int k = 0; k < n_stack; ++k) {
                    const int lk = l + k;
                    maps.x2[k] = lk == 0 ? in_rows2_map : g.act_rows2_map[lk];
                    maps.x1[k] = lk == 0 ? in_rows1_map : g.act_rows1_map[lk];
                    // a layer that feeds the pool stores nothing: any valid map will do for it
                    maps.y[k] = feeds_pool_at(lk) ? (lk == 0 ? in_map : g.act_map[lk]) : g.act_store_map[lk + 1];
                }
                for (int k = 0; k < n_stack; ++k) {
                    a.skip[k] = skip_of(l + k);
                    a.skip_perm[k] = (l + k == 1) ? g.d_perm : nullptr;
                }
                if (self_bucket && l == 0) {
                    a.ids = ids; a.n = n;
                    a.counts_out = g.d_counts; a.offsets_out = g.d_offsets; a.perm_out = g.d_perm; a.inv_out = g.d_inv;
                    a.prefix_out = g.d_tile_prefix; a.prefix_rows = L - 2;      // one row per conv layer
                }
                a.n_stack = n_stack;
                a.border_units = g.opt_conv_balance ? 2 : 0;
                a.grid_bar = g.d_grid_bar + (n_conv_launch++ & 7);
                a.out = nullptr;
                a.pool_partial = feeds_pool_at(l_last) ? g.d_pool_partial : nullptr;
                a.late_trigger = is_conv(l_last + 1) ? 1 : 0;
                a.early_lookup = is_conv(l - 1) ? 1 : 0;
                CU_OK(launch_grouped_conv_pair(maps, a, g.sm_count, s));
                l = l_last;
            } else {
                a.out = (uint16_t*)g.act[l + 1];
                a.skip[0] = skip_of(l);
                a.skip_perm[0] = (l == 1) ? g.d_perm : nullptr;
                a.pool_partial = feeds_pool_at(l) ? g.d_pool_partial : nullptr;
                launch_grouped_conv(l == 0 ? in_map : g.act_map[l], a, g.conv.smem_bytes, g.sm_count, s);
            }
        } else if (pool_head && l == L - 2) {
            // pool + narrow last dense layer in one launch (the loop ends here: the head is done)
            Timer t(K_POOL, s);
            launch_pool_head(g.d_pool_partial, n, g.conv.strips_per_image, f.h * f.w, g.d_models, L - 1, g.d_offsets, g.T,
                             g.d_perm, (float*)outputs, g.out_elems, g.d_grid_bar, s);
            break;
        } else {
            Timer t(K_POOL, s);
            // a pool always follows a conv (checked at registration), whose epilogue already reduced every strip
            // to channel sums
            launch_pool_finalize(g.d_pool_partial, n, g.conv.strips_per_image, f.in_ch, f.h * f.w,
                                 (uint16_t*)g.act[l + 1], g.act_ld[l + 1], g.d_grid_bar, s);
        }
    }
    Timer::close_group(s);
    g.last_n = n;
    CU_OK(cudaGetLastError());
    return MT_OK;
}

// Host-side bookkeeping of a freshly registered model (both registration paths).
mt_status adopt_model(int id, const std::vector<HostLayer>& hl, uint8_t* block, size_t total, void* host_image,
                      const std::vector<size_t>& w_off, const std::vector<size_t>& b_off, cudaEvent_t ready) {
    const int n_layers = (int)hl.size();
    if (!g.has_family || g.live == 0) {
        g.family = hl;
        g.has_family = true;
        g.in_elems = layer_in_elems(hl[0]);
        g.out_elems = hl.back().out_ch;
        g.out_mixed = false;
        for (const HostLayer& f : hl)
            if (f.kind == MT_CONV3X3) plan_conv(f.h, f.w, &g.conv);   // cannot fail: validate_layers bounds w
        for (int b = 0; b <= MT_MAX_LAYERS; ++b) g.width[b] = 0;
        g.ws_dirty = true;
        g.in_map_ptr = nullptr;
        free_staging();   // sized for the previous family's rows (no model is live: nothing is in flight)
    }
    if ((size_t)n_layers > g.family.size()) {      // a deeper MLP joins: the family gains launches
        for (size_t l = g.family.size(); l < (size_t)n_layers; ++l) g.family.push_back(hl[l]);
        g.ws_dirty = true;
    }
    for (int l = 0; l < n_layers; ++l) {
        const int wd = layer_in_elems(hl[l]);
        if (wd > g.width[l]) { g.width[l] = wd; g.ws_dirty = true; }
    }
    if (hl.back().out_ch != g.out_elems) g.out_mixed = true;
    if (hl.back().out_ch > g.out_elems) {          // a wider output: the rows of the output buffer get longer
        g.out_elems = hl.back().out_ch;
        g.ws_dirty = true;
    }
    if (layer_in_elems(hl[0]) > g.in_elems) {      // a wider input (MLP families only): so do the input buffer's
        g.in_elems = layer_in_elems(hl[0]);
        g.ws_dirty = true;
        g.in_map_ptr = nullptr;
    }
    HostModel& hm = g.models[id];
    hm.alive = true;
    hm.layers = hl;
    for (int l = 0; l < n_layers; ++l) g.n_residual[l] += hl[l].residual ? 1 : 0;
    hm.dev_block = g.cache_bytes ? nullptr : block;
    hm.block_bytes = total;
    hm.host_image = host_image;
    hm.w_off = w_off;
    hm.b_off = b_off;
    hm.last_batch = 0;
    if (hm.ready && hm.ready != ready) cudaEventDestroy(hm.ready);
    hm.ready = ready;
    g.live += 1;
    if (id + 1 > g.T) g.T = id + 1;
    recompute_tile_n();
    return recompute_order();
}

// Registration without stalling the device.  The caller's weights and biases are copied into pinned staging on the
// host (so the caller may free them on return, as before), everything else - the copy to the device, the re-layout
// into the executor's tiled images, with the cache on also the copy of the finished block back to its pinned host
// image - is enqueued on the library's load stream and overlaps whatever batches are running.  The model's entry in
// the device tables is written by the next call that names a stream, which first waits for the model's event.
// Weights given as DEVICE pointers are read by the load stream directly; the call then waits for that stream alone.
mt_status register_async(const mt_layer_desc* layers, const std::vector<HostLayer>& hl, int id, size_t total,
                         const std::vector<size_t>& w_off, const std::vector<size_t>& b_off, int32_t* model_id_out) {
    const int n_layers = (int)hl.size();
    // staging layout: per layer the raw weights, then the bias, 256-byte aligned pieces
    std::vector<size_t> sw(n_layers, 0), sb(n_layers, 0);
    size_t need = 0;
    bool device_source = false;
    for (int l = 0; l < n_layers; ++l) {
        const HostLayer& h = hl[l];
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        const size_t raw = (size_t)h.out_ch * h.in_ch * 2 * (h.kind == MT_CONV3X3 ? 9 : 1);
        sw[l] = need; need += align_up(raw, 256);
        sb[l] = need; need += align_up(sizeof(float) * h.out_ch, 256);
        if (is_device_pointer(layers[l].weight) || (layers[l].bias && is_device_pointer(layers[l].bias))) device_source = true;
    }
    if (need > g.reg_host_cap || need > g.reg_dev_cap) {
        // grow the staging (rare: sized for the largest model seen, with headroom); the load stream must be done with it
        CU_OK(cudaStreamSynchronize(g.load_stream));
        g.reg_h2d_pending = false;
        const size_t cap = align_up(need + need / 2, (size_t)1 << 20);
        if (g.reg_host) cudaFreeHost(g.reg_host);
        cudaFree(g.reg_dev);
        g.reg_host = nullptr; g.reg_dev = nullptr; g.reg_host_cap = g.reg_dev_cap = 0;
        CU_OK(cudaMallocHost(&g.reg_host, cap));
        CU_OK(cudaMalloc(&g.reg_dev, cap));
        g.reg_host_cap = g.reg_dev_cap = cap;
    }
    uint8_t* block = nullptr;
    std::vector<int> evicted;
    if (g.cache_bytes) {
        size_t off = 0;
        const WeightCache::Result got = g.cache.acquire(id, total, ++g.cache_tick, &off, &evicted);
        block = g.arena + off;
        // the victims' bytes may still be read by batches in flight; their table entries flip at the next flush
        // (also when no room could be made in the end: what was evicted on the way stays evicted)
        uint64_t youngest = 0;
        for (int v : evicted) {
            g.pending_ops.push_back({v, 2});
            if (g.models[v].last_batch > youngest) youngest = g.models[v].last_batch;
        }
        if (got == WeightCache::kNoRoom) return MT_ERR_OOM;
        if (youngest > g.synced_batch && youngest <= g.batch_no)
            CU_OK(cudaStreamWaitEvent(g.load_stream, g.batch_done[youngest % Ctx::kBatchEvents], 0));
    } else {
        CU_OK(cudaMalloc(&block, total));
    }
    auto fail = [&](cudaError_t e) {
        if (g.cache_bytes) g.cache.release(id); else cudaFree(block);
        cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? MT_ERR_OOM : MT_ERR_CUDA;
    };
    // the previous registration's staging copy must have left pinned memory before it is overwritten
    if (g.reg_h2d_pending) {
        cudaError_t e = cudaEventSynchronize(g.reg_h2d_done);
        if (e != cudaSuccess) return fail(e);
        g.reg_h2d_pending = false;
    }
    uint8_t* hs = static_cast<uint8_t*>(g.reg_host);
    uint8_t* ds = static_cast<uint8_t*>(g.reg_dev);
    cudaStream_t ls = g.load_stream;
    cudaError_t e = cudaMemsetAsync(block, 0, total, ls);
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
        const HostLayer& h = hl[l];
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        const size_t raw = (size_t)h.out_ch * h.in_ch * 2 * (h.kind == MT_CONV3X3 ? 9 : 1);
        if (is_device_pointer(layers[l].weight)) e = cudaMemcpyAsync(ds + sw[l], layers[l].weight, raw, cudaMemcpyDeviceToDevice, ls);
        else memcpy(hs + sw[l], layers[l].weight, raw);
        if (e != cudaSuccess) break;
        if (layers[l].bias) {
            if (is_device_pointer(layers[l].bias)) e = cudaMemcpyAsync(ds + sb[l], layers[l].bias, sizeof(float) * h.out_ch, cudaMemcpyDeviceToDevice, ls);
            else memcpy(hs + sb[l], layers[l].bias, sizeof(float) * h.out_ch);
        }
    }
    // host-resident pieces: one copy of the staging per piece (device-resident pieces were copied above)
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
        const HostLayer& h = hl[l];
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        const size_t raw = (size_t)h.out_ch * h.in_ch * 2 * (h.kind == MT_CONV3X3 ? 9 : 1);
        if (!is_device_pointer(layers[l].weight)) e = cudaMemcpyAsync(ds + sw[l], hs + sw[l], raw, cudaMemcpyHostToDevice, ls);
        if (e == cudaSuccess && layers[l].bias && !is_device_pointer(layers[l].bias))
            e = cudaMemcpyAsync(ds + sb[l], hs + sb[l], sizeof(float) * h.out_ch, cudaMemcpyHostToDevice, ls);
    }
    if (e == cudaSuccess) e = cudaEventRecord(g.reg_h2d_done, ls);
    if (e != cudaSuccess) return fail(e);
    g.reg_h2d_pending = true;
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
        const HostLayer& h = hl[l];
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        const uint16_t* src = reinterpret_cast<const uint16_t*>(ds + sw[l]);
        if (h.kind == MT_DENSE) launch_pretile_dense(src, h.out_ch, h.in_ch, (uint16_t*)(block + w_off[l]), ls);
        else {
            launch_pretile_conv(src, h.out_ch, h.in_ch, (uint16_t*)(block + w_off[l]), ls);
            launch_pretile_conv_pair(src, (uint16_t*)(block + w_off[l]) + kConvPairImageOffset, ls);
        }
        e = cudaGetLastError();
        if (e == cudaSuccess && layers[l].bias)
            e = cudaMemcpyAsync(block + b_off[l], ds + sb[l], sizeof(float) * h.out_ch, cudaMemcpyDeviceToDevice, ls);
    }
    void* host_image = nullptr;
    if (e == cudaSuccess && g.cache_bytes) {        // the host tier: the block's image in pinned memory
        e = cudaMallocHost(&host_image, total);
        if (e == cudaSuccess) e = cudaMemcpyAsync(host_image, block, total, cudaMemcpyDeviceToHost, ls);
    }
    cudaEvent_t ready = nullptr;
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ready, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventRecord(ready, ls);
    if (e == cudaSuccess && device_source) e = cudaStreamSynchronize(ls);   // the caller's device buffers may go away on return
    if (e != cudaSuccess) {
        if (host_image) cudaFreeHost(host_image);
        if (ready) cudaEventDestroy(ready);
        return fail(e);
    }
    g.pending_ops.push_back({id, 1});
    mt_status st = adopt_model(id, hl, block, total, host_image, w_off, b_off, ready);
    if (st != MT_OK) return st;
    *model_id_out = id;
    return MT_OK;
}

}  // namespace

extern "C" {

mt_status mt_init(int32_t device, int32_t max_models, int32_t max_batch) {
    std::lock_guard<std::mutex> lk(g_mu);
    return do_init(device, max_models, max_batch);
}

mt_status mt_shutdown(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_OK;
    cudaSetDevice(g.device);
    cudaDeviceSynchronize();
    for (HostModel& m : g.models) {
        if (m.dev_block) { cudaFree(m.dev_block); m.dev_block = nullptr; }
        if (m.host_image) { cudaFreeHost(m.host_image); m.host_image = nullptr; }
        if (m.ready) { cudaEventDestroy(m.ready); m.ready = nullptr; }
    }
    if (g.h_order) { cudaFreeHost(g.h_order); g.h_order = nullptr; }
    if (g.reg_host) { cudaFreeHost(g.reg_host); g.reg_host = nullptr; }
    cudaFree(g.reg_dev); g.reg_dev = nullptr;
    g.reg_host_cap = g.reg_dev_cap = 0;
    if (g.reg_h2d_done) { cudaEventDestroy(g.reg_h2d_done); g.reg_h2d_done = nullptr; }
    if (g.order_copied) { cudaEventDestroy(g.order_copied); g.order_copied = nullptr; }
    g.pending_ops.clear();
    g.order_dirty = g.order_copy_pending = g.reg_h2d_pending = false;
    g.models.clear();
    cudaFree(g.arena); g.arena = nullptr;
    g.cache.reset(0);
    g.cache_bytes = 0;
    if (g.load_stream) { cudaStreamDestroy(g.load_stream); g.load_stream = nullptr; }
    for (cudaEvent_t& ev : g.batch_done)
        if (ev) { cudaEventDestroy(ev); ev = nullptr; }
    if (g.loads_done) { cudaEventDestroy(g.loads_done); g.loads_done = nullptr; }
    g.batch_no = g.synced_batch = g.cache_tick = 0;
    g.request_hits = g.request_misses = 0;
    free_workspace();
    cudaFree(g.d_models); g.d_models = nullptr;
    cudaFree(g.d_brief); g.d_brief = nullptr;
    cudaFree(g.d_order); g.d_order = nullptr;
    cudaFree(g.d_grid_bar); g.d_grid_bar = nullptr;
    cudaFree(g.d_wmaps); g.d_wmaps = nullptr;
    cudaFree(g.d_status); g.d_status = nullptr;
    cudaFree(g.d_ticket); g.d_ticket = nullptr;
    cudaFree(g.d_counts); g.d_counts = nullptr;
    cudaFree(g.d_offsets); g.d_offsets = nullptr;
    cudaFree(g.d_tile_prefix); g.d_tile_prefix = nullptr;
    cudaFree(g.st_in); g.st_in = nullptr;
    cudaFree(g.st_ids); g.st_ids = nullptr;
    free_staging();
    for (int k = 0; k < 2; ++k)
        if (g.as_slot_done[k]) { cudaEventDestroy(g.as_slot_done[k]); g.as_slot_done[k] = nullptr; }
    if (g.as_compute_done) { cudaEventDestroy(g.as_compute_done); g.as_compute_done = nullptr; }
    g.as_next = 0;
    Timer::close_group();
    for (TimedLaunch& t : g.timed) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
    g.timed.clear();
    for (cudaEvent_t e : g.event_pool) cudaEventDestroy(e);
    g.event_pool.clear();
    g.timing = 0;
    g.init = false;
    g.has_family = false;
    g.family.clear();
    g.live = 0;
    for (int l = 0; l < MT_MAX_LAYERS; ++l) g.n_residual[l] = 0;
    g.T = 0;
    return MT_OK;
}

mt_status mt_register_model(const mt_layer_desc* layers, int32_t n_layers, int32_t* model_id_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!model_id_out) return MT_ERR_INVALID_ARG;
    mt_status st = validate_layers(layers, n_layers);
    if (st != MT_OK) return st;
    if (!g.init) {
        st = do_init(0, 1024, 0);
        if (st != MT_OK) return st;
    }
    CU_OK(cudaSetDevice(g.device));
    std::vector<HostLayer> hl(n_layers);
    for (int l = 0; l < n_layers; ++l) {
        hl[l] = {layers[l].kind, layers[l].in_ch, layers[l].out_ch, layers[l].h, layers[l].w, layers[l].relu ? 1 : 0,
                 layers[l].residual ? 1 : 0, 1};
        if (layers[l].kind == MT_CONV1X1) { hl[l].kind = MT_DENSE; hl[l].hw = layers[l].h * layers[l].w; }
    }
    st = check_family(hl);
    if (st != MT_OK) return st;
    int id = -1;
    for (int i = 0; i < g.max_models; ++i)
        if (!g.models[i].alive) { id = i; break; }
    if (id < 0) return MT_ERR_OOM;

    // one device block per model: [tiled weights | padded bias] per layer, 1024-byte aligned pieces
    size_t total = 0, raw_max = 0;
    std::vector<size_t> w_off(n_layers, 0), b_off(n_layers, 0);
    for (int l = 0; l < n_layers; ++l) {
        const HostLayer& h = hl[l];
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        const size_t n_tiles = padded_weight_tiles(h);
        size_t wbytes, raw;
        if (h.kind == MT_DENSE) { wbytes = n_tiles * (size_t)(h.in_ch / BK) * TILE_BYTES; raw = (size_t)h.out_ch * h.in_ch * 2; }
        else { raw = (size_t)9 * h.out_ch * h.in_ch * 2; wbytes = raw + 2 * (size_t)kConvPairWeightBytes; }   // one-CTA image + the pair's two
        w_off[l] = total; total += align_up(wbytes, 1024);
        b_off[l] = total; total += align_up(n_tiles * BN * sizeof(float), 1024);
        if (raw > raw_max) raw_max = raw;
    }
    if (g.opt_async_register) return register_async(layers, hl, id, total, w_off, b_off, model_id_out);

    uint8_t* block = nullptr;
    if (g.cache_bytes) {
        // a place in the arena, over least-recently-used tenants if need be (registration is synchronous: nothing is
        // in flight once the device has been synchronised, so the victims' table entries are switched directly)
        std::vector<int> evicted;
        size_t off = 0;
        const WeightCache::Result got = g.cache.acquire(id, total, ++g.cache_tick, &off, &evicted);
        CU_OK(cudaDeviceSynchronize());
        g.synced_batch = g.batch_no;
        for (int v : evicted) {     // also when no room could be made in the end: what was evicted on the way stays evicted
            const int32_t two = 2;
            CU_OK(cudaMemcpy(g.d_brief + v, &two, sizeof two, cudaMemcpyHostToDevice));
            CU_OK(cudaMemcpy(&g.d_models[v].alive, &two, sizeof two, cudaMemcpyHostToDevice));
        }
        if (got == WeightCache::kNoRoom) return MT_ERR_OOM;
        block = g.arena + off;
    } else {
        CU_OK(cudaMalloc(&block, total));
    }
    cudaError_t e = cudaMemset(block, 0, total);
    void* raw_dev = nullptr;
    ModelDev md;
    memset(&md, 0, sizeof md);
    md.alive = 1;
    md.n_layers = n_layers;
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
        const HostLayer& h = hl[l];
        LayerDev& d = md.layer[l];
        d.kind = h.kind; d.K = h.in_ch; d.N = h.out_ch; d.relu = h.relu; d.residual = h.residual;
        d.n_tiles = (int)padded_weight_tiles(h);
        d.k_blocks = h.kind == MT_DENSE ? h.in_ch / BK : 9;
        if (h.kind == MT_GLOBAL_AVG_POOL) continue;
        d.w = reinterpret_cast<const uint16_t*>(block + w_off[l]);
        d.bias = reinterpret_cast<const float*>(block + b_off[l]);
        const size_t raw = (size_t)h.out_ch * h.in_ch * 2 * (h.kind == MT_CONV3X3 ? 9 : 1);
        const uint16_t* src = static_cast<const uint16_t*>(layers[l].weight);
        if (!is_device_pointer(src) || (reinterpret_cast<uintptr_t>(src) & 15)) {
            if (!raw_dev) e = cudaMalloc(&raw_dev, raw_max);
            if (e == cudaSuccess) e = cudaMemcpy(raw_dev, src, raw, cudaMemcpyDefault);
            src = static_cast<const uint16_t*>(raw_dev);
        }
        if (e != cudaSuccess) break;
        if (h.kind == MT_DENSE) launch_pretile_dense(src, h.out_ch, h.in_ch, (uint16_t*)(block + w_off[l]), 0);
        else {
            launch_pretile_conv(src, h.out_ch, h.in_ch, (uint16_t*)(block + w_off[l]), 0);
            launch_pretile_conv_pair(src, (uint16_t*)(block + w_off[l]) + kConvPairImageOffset, 0);
        }
        e = cudaGetLastError();
        if (e == cudaSuccess && layers[l].bias)
            e = cudaMemcpy(block + b_off[l], layers[l].bias, sizeof(float) * h.out_ch, cudaMemcpyDefault);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();   // raw_dev is reused by the next layer
    }
    for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
        if (hl[l].kind != MT_DENSE) continue;
        CUtensorMap wm;
        if (encode_weight_tiles(&wm, block + w_off[l], padded_weight_tiles(hl[l]) * (size_t)(hl[l].in_ch / BK)) != MT_OK) {
            e = cudaErrorInvalidValue;
            break;
        }
        e = cudaMemcpy(g.d_wmaps + (size_t)id * MT_MAX_LAYERS + l, &wm, sizeof wm, cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess) e = cudaMemcpy(g.d_models + id, &md, sizeof md, cudaMemcpyHostToDevice);
    for (int r = 0; r <= MT_MAX_LAYERS && e == cudaSuccess; ++r) {   // the compact copy: alive, then out features per layer
        const int32_t v = (r == 0) ? 1 : (r <= n_layers ? hl[r - 1].out_ch : 0);   // 0: the model has no such layer
        e = cudaMemcpy(g.d_brief + (size_t)r * g.max_models + id, &v, sizeof v, cudaMemcpyHostToDevice);
    }
    if (raw_dev) cudaFree(raw_dev);
    void* host_image = nullptr;
    if (e == cudaSuccess && g.cache_bytes) {        // the host tier: the block's image in pinned memory
        e = cudaMallocHost(&host_image, total);
        if (e == cudaSuccess) e = cudaMemcpy(host_image, block, total, cudaMemcpyDeviceToHost);
    }
    if (e != cudaSuccess) {
        if (g.cache_bytes) g.cache.release(id); else cudaFree(block);
        if (host_image) cudaFreeHost(host_image);
        cudaGetLastError();
        return e == cudaErrorMemoryAllocation ? MT_ERR_OOM : MT_ERR_CUDA;
    }

    st = adopt_model(id, hl, block, total, host_image, w_off, b_off, nullptr);
    if (st != MT_OK) return st;
    *model_id_out = id;
    return MT_OK;
}

mt_status mt_release(int32_t model_id) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (model_id < 0 || model_id >= g.max_models || !g.models[model_id].alive) return MT_ERR_BAD_MODEL_ID;
    CU_OK(cudaSetDevice(g.device));
    CU_OK(cudaDeviceSynchronize());
    ModelDev md;
    memset(&md, 0, sizeof md);
    CU_OK(cudaMemcpy(g.d_models + model_id, &md, sizeof md, cudaMemcpyHostToDevice));
    const int32_t dead = 0;
    CU_OK(cudaMemcpy(g.d_brief + model_id, &dead, sizeof dead, cudaMemcpyHostToDevice));
    HostModel& hm = g.models[model_id];
    g.synced_batch = g.batch_no;
    if (g.cache_bytes) g.cache.release(model_id);
    if (hm.host_image) { cudaFreeHost(hm.host_image); hm.host_image = nullptr; }
    cudaFree(hm.dev_block);
    hm.dev_block = nullptr;
    hm.alive = false;
    for (size_t l = 0; l < hm.layers.size(); ++l) g.n_residual[l] -= hm.layers[l].residual ? 1 : 0;
    hm.layers.clear();
    g.live -= 1;
    recompute_tile_n();
    return recompute_order();
}

mt_status mt_infer(const void* inputs, const int32_t* model_ids, int32_t n, void* outputs, void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    cache_begin_batch(true);      // ids on the device: the batch may read any resident tenant
    mt_status st = infer_device(inputs, model_ids, n, outputs, static_cast<cudaStream_t>(stream));
    if (st != MT_OK || n == 0) return st;
    return cache_end_batch(static_cast<cudaStream_t>(stream));
}

mt_status mt_infer_host(const void* inputs_host, const int32_t* model_ids_host, int32_t n, void* outputs_host,
                        void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (n < 0) return MT_ERR_INVALID_ARG;
    if (n == 0) return MT_OK;
    if (!inputs_host || !model_ids_host || !outputs_host) return MT_ERR_INVALID_ARG;
    if (!g.has_family || g.live == 0) return MT_ERR_BAD_MODEL_ID;
    CU_OK(cudaSetDevice(g.device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t in_bytes = (size_t)n * g.in_elems * 2, id_bytes = (size_t)n * sizeof(int32_t),
                 out_bytes = (size_t)n * g.out_elems * sizeof(float);
    if (in_bytes > g.st_cap_in || id_bytes > g.st_cap_ids || out_bytes > g.st_cap_out) {
        CU_OK(cudaDeviceSynchronize());
        cudaFree(g.st_in); cudaFree(g.st_ids); cudaFree(g.st_out);
        g.st_in = nullptr; g.st_ids = nullptr; g.st_out = nullptr;
        g.st_cap_in = g.st_cap_ids = g.st_cap_out = 0;
        CU_OK(cudaMalloc(&g.st_in, in_bytes));
        CU_OK(cudaMalloc(&g.st_ids, id_bytes));
        CU_OK(cudaMalloc(&g.st_out, out_bytes));
        g.st_cap_in = in_bytes; g.st_cap_ids = id_bytes; g.st_cap_out = out_bytes;
    }
    if (g.cache_bytes) {          // the host sees the ids: bring exactly this batch's tenants in
        std::vector<int> set, reqs;
        tenant_set_of(model_ids_host, n, &set, &reqs);
        mt_status rs = ensure_resident(set, reqs, s);
        if (rs != MT_OK) return rs;
    }
    CU_OK(cudaMemcpyAsync(g.st_in, inputs_host, in_bytes, cudaMemcpyHostToDevice, s));
    CU_OK(cudaMemcpyAsync(g.st_ids, model_ids_host, id_bytes, cudaMemcpyHostToDevice, s));
    // columns beyond a model's own are never written: what the caller gets there must not be an earlier batch's values
    if (g.out_mixed) CU_OK(cudaMemsetAsync(g.st_out, 0xFF, out_bytes, s));      // all ones: a NaN
    mt_status st = infer_device(g.st_in, g.st_ids, n, g.st_out, s);
    if (st != MT_OK) return st;
    st = cache_end_batch(s);
    if (st != MT_OK) return st;
    CU_OK(cudaMemcpyAsync(outputs_host, g.st_out, out_bytes, cudaMemcpyDeviceToHost, s));
    CU_OK(cudaStreamSynchronize(s));
    return MT_OK;
}

mt_status mt_infer_host_async(const void* inputs_host, const int32_t* model_ids_host, int32_t n, void* outputs_host,
                              void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (n < 0) return MT_ERR_INVALID_ARG;
    if (n == 0) return MT_OK;
    if (!inputs_host || !model_ids_host || !outputs_host) return MT_ERR_INVALID_ARG;
    if (!g.has_family || g.live == 0) return MT_ERR_BAD_MODEL_ID;
    CU_OK(cudaSetDevice(g.device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t in_bytes = (size_t)n * g.in_elems * 2, id_bytes = (size_t)n * sizeof(int32_t),
                 out_bytes = (size_t)n * g.out_elems * sizeof(float);
    if (in_bytes > g.as_cap_in || id_bytes > g.as_cap_ids || out_bytes > g.as_cap_out) {
        CU_OK(cudaDeviceSynchronize());
        for (int k = 0; k < 2; ++k) {
            cudaFree(g.as_in[k]); cudaFree(g.as_ids[k]); cudaFree(g.as_out[k]);
            g.as_in[k] = nullptr; g.as_ids[k] = nullptr; g.as_out[k] = nullptr;
            g.as_slot_used[k] = false;
        }
        g.as_cap_in = g.as_cap_ids = g.as_cap_out = 0;
        for (int k = 0; k < 2; ++k) {
            CU_OK(cudaMalloc(&g.as_in[k], in_bytes));
            CU_OK(cudaMalloc(&g.as_ids[k], id_bytes));
            CU_OK(cudaMalloc(&g.as_out[k], out_bytes));
            if (!g.as_slot_done[k]) CU_OK(cudaEventCreateWithFlags(&g.as_slot_done[k], cudaEventDisableTiming));
        }
        if (!g.as_compute_done) CU_OK(cudaEventCreateWithFlags(&g.as_compute_done, cudaEventDisableTiming));
        g.as_have_compute = false;
        g.as_cap_in = in_bytes; g.as_cap_ids = id_bytes; g.as_cap_out = out_bytes;
    }
    // grow the workspace (a device-wide synchronisation) before anything of this call is in flight
    mt_status st = ensure_workspace(n);
    if (st != MT_OK) return st;
    const int k = g.as_next;
    g.as_next ^= 1;
    // the slot's previous user must have copied its outputs out
    if (g.as_slot_used[k]) CU_OK(cudaStreamWaitEvent(s, g.as_slot_done[k], 0));
    CU_OK(cudaMemcpyAsync(g.as_in[k], inputs_host, in_bytes, cudaMemcpyHostToDevice, s));
    CU_OK(cudaMemcpyAsync(g.as_ids[k], model_ids_host, id_bytes, cudaMemcpyHostToDevice, s));
    // the kernels of consecutive calls share one workspace: they run one call after the other, whatever the streams
    if (g.as_have_compute) CU_OK(cudaStreamWaitEvent(s, g.as_compute_done, 0));
    if (g.cache_bytes) {          // after the wait: the table switches are ordered behind the previous batch's kernels
        std::vector<int> set, reqs;
        tenant_set_of(model_ids_host, n, &set, &reqs);
        mt_status rs = ensure_resident(set, reqs, s);
        if (rs != MT_OK) return rs;
    }
    if (g.out_mixed) CU_OK(cudaMemsetAsync(g.as_out[k], 0xFF, out_bytes, s));   // see mt_infer_host
    st = infer_device(g.as_in[k], g.as_ids[k], n, g.as_out[k], s);
    if (st != MT_OK) return st;
    st = cache_end_batch(s);
    if (st != MT_OK) return st;
    CU_OK(cudaEventRecord(g.as_compute_done, s));
    g.as_have_compute = true;
    CU_OK(cudaMemcpyAsync(outputs_host, g.as_out[k], out_bytes, cudaMemcpyDeviceToHost, s));
    CU_OK(cudaEventRecord(g.as_slot_done[k], s));
    g.as_slot_used[k] = true;
    return MT_OK;
}

mt_status mt_output_elems(int32_t* out_elems_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (!out_elems_out) return MT_ERR_INVALID_ARG;
    *out_elems_out = (g.has_family && g.live > 0) ? g.out_elems : 0;
    return MT_OK;
}

mt_status mt_input_elems(int32_t* in_elems_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (!in_elems_out) return MT_ERR_INVALID_ARG;
    *in_elems_out = (g.has_family && g.live > 0) ? g.in_elems : 0;
    return MT_OK;
}

mt_status mt_set_cache_bytes(size_t device_bytes) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (g.live != 0) return MT_ERR_INVALID_ARG;          // only while no model is registered
    CU_OK(cudaSetDevice(g.device));
    CU_OK(cudaDeviceSynchronize());
    cudaFree(g.arena); g.arena = nullptr;
    g.cache.reset(0);
    g.cache_bytes = 0;
    if (device_bytes == 0) return MT_OK;
    const size_t cap = device_bytes / 1024 * 1024;
    if (cap == 0) return MT_ERR_INVALID_ARG;
    cudaError_t e = cudaMalloc(&g.arena, cap);
    if (e != cudaSuccess) { cudaGetLastError(); g.arena = nullptr; return e == cudaErrorMemoryAllocation ? MT_ERR_OOM : MT_ERR_CUDA; }
    if (!g.load_stream) CU_OK(cudaStreamCreateWithFlags(&g.load_stream, cudaStreamNonBlocking));
    for (cudaEvent_t& ev : g.batch_done)
        if (!ev) CU_OK(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    if (!g.loads_done) CU_OK(cudaEventCreateWithFlags(&g.loads_done, cudaEventDisableTiming));
    g.cache.reset(cap);
    g.cache_bytes = cap;
    g.batch_no = g.synced_batch = g.cache_tick = 0;
    g.request_hits = g.request_misses = 0;
    return MT_OK;
}

mt_status mt_prefetch(const int32_t* model_ids_host, int32_t count, void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (count < 0 || (count > 0 && !model_ids_host)) return MT_ERR_INVALID_ARG;
    if (!g.cache_bytes || count == 0) return MT_OK;       // without the cache every model is resident
    for (int i = 0; i < count; ++i) {
        const int t = model_ids_host[i];
        if (t < 0 || t >= g.max_models || !g.models[t].alive) return MT_ERR_BAD_MODEL_ID;
    }
    CU_OK(cudaSetDevice(g.device));
    std::vector<int> set, reqs;
    tenant_set_of(model_ids_host, count, &set, &reqs);
    for (int& r : reqs) r = 0;                            // a prefetch serves no request yet
    return ensure_resident(set, reqs, static_cast<cudaStream_t>(stream));
}

mt_status mt_get_cache_stats(mt_cache_stats* out, int32_t reset) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (!out) return MT_ERR_INVALID_ARG;
    const WeightCache::Stats& cs = g.cache.stats();
    out->capacity_bytes = g.cache_bytes;
    out->resident_bytes = g.cache.resident_bytes();
    out->tenant_hits = cs.hits; out->tenant_misses = cs.misses;
    out->evictions = cs.evictions; out->bytes_loaded = cs.bytes_loaded;
    out->request_hits = g.request_hits; out->request_misses = g.request_misses;
    if (reset) { g.cache.clear_stats(); g.request_hits = g.request_misses = 0; }
    return MT_OK;
}

// The eviction policy by itself, on a made-up clock (host code only: usable without a GPU).
struct CacheSim { mt::WeightCache c; };
mt_status mt_cache_sim_create(size_t capacity_bytes, void** sim_out) {
    if (!sim_out) return MT_ERR_INVALID_ARG;
    CacheSim* s = new CacheSim();
    s->c.reset(capacity_bytes);
    *sim_out = s;
    return MT_OK;
}
mt_status mt_cache_sim_access(void* sim, int32_t id, size_t bytes, uint64_t tick, int32_t* result_out, int64_t* offset_out,
                              int32_t* evicted_out, int32_t evicted_cap, int32_t* n_evicted_out) {
    if (!sim || !result_out) return MT_ERR_INVALID_ARG;
    std::vector<int> ev;
    size_t off = 0;
    const mt::WeightCache::Result r = static_cast<CacheSim*>(sim)->c.acquire(id, bytes, tick, &off, &ev);
    *result_out = (int32_t)r;
    if (offset_out) *offset_out = r == mt::WeightCache::kNoRoom ? -1 : (int64_t)off;
    if (n_evicted_out) *n_evicted_out = (int32_t)ev.size();
    for (size_t i = 0; i < ev.size() && evicted_out && (int)i < evicted_cap; ++i) evicted_out[i] = ev[i];
    return MT_OK;
}
mt_status mt_cache_sim_release(void* sim, int32_t id) {
    if (!sim) return MT_ERR_INVALID_ARG;
    static_cast<CacheSim*>(sim)->c.release(id);
    return MT_OK;
}
mt_status mt_cache_sim_stats(void* sim, mt_cache_stats* out) {
    if (!sim || !out) return MT_ERR_INVALID_ARG;
    const mt::WeightCache& c = static_cast<CacheSim*>(sim)->c;
    memset(out, 0, sizeof *out);
    out->capacity_bytes = c.capacity(); out->resident_bytes = c.resident_bytes();
    out->tenant_hits = c.stats().hits; out->tenant_misses = c.stats().misses;
    out->evictions = c.stats().evictions; out->bytes_loaded = c.stats().bytes_loaded;
    return MT_OK;
}
mt_status mt_cache_sim_destroy(void* sim) {
    delete static_cast<CacheSim*>(sim);
    return MT_OK;
}

mt_status mt_get_async_status(void* stream, int32_t* status_out, int32_t* bad_request_index_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    CU_OK(cudaSetDevice(g.device));
    CU_OK(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    int32_t w[ST_WORDS];
    CU_OK(cudaMemcpy(w, g.d_status, sizeof w, cudaMemcpyDeviceToHost));
    if (status_out) *status_out = w[ST_CODE];
    if (bad_request_index_out) *bad_request_index_out = (w[ST_BAD_INDEX] == INT_MAX) ? -1 : w[ST_BAD_INDEX];
    if (w[ST_CODE] == MT_ERR_TIMEOUT && getenv("MT_LOG")) fprintf(stderr, "[mt] device wait gave up at site %d\n", w[ST_WHERE]);
    return reset_status_word();
}

const char* mt_status_string(mt_status s) {
    switch (s) {
        case MT_OK: return "ok";
        case MT_ERR_INVALID_ARG: return "invalid argument";
        case MT_ERR_BAD_MODEL_ID: return "bad model id";
        case MT_ERR_SHAPE: return "shape mismatch";
        case MT_ERR_UNSUPPORTED: return "unsupported layer or dimension";
        case MT_ERR_OOM: return "out of memory";
        case MT_ERR_CUDA: return "CUDA error";
        case MT_ERR_ARCH: return "device is not sm_100";
        case MT_ERR_TIMEOUT: return "device-side wait timed out";
        case MT_ERR_NOT_INIT: return "not initialised";
        case MT_ERR_NOT_RESIDENT: return "model registered but not resident on the device";
    }
    return "unknown status";
}

mt_status mt_debug_last_bucketing(int32_t* counts_host, int32_t* offsets_host, int32_t* perm_host,
                                  int32_t* inv_host, int32_t* n_tenants_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    CU_OK(cudaSetDevice(g.device));
    CU_OK(cudaDeviceSynchronize());
    const size_t i4 = sizeof(int32_t);
    if (n_tenants_out) *n_tenants_out = g.T;
    if (counts_host && g.T) CU_OK(cudaMemcpy(counts_host, g.d_counts, i4 * g.T, cudaMemcpyDeviceToHost));
    if (offsets_host) CU_OK(cudaMemcpy(offsets_host, g.d_offsets, i4 * (g.T + 2), cudaMemcpyDeviceToHost));
    if (perm_host && g.last_n) CU_OK(cudaMemcpy(perm_host, g.d_perm, i4 * g.last_n, cudaMemcpyDeviceToHost));
    if (inv_host && g.last_n) CU_OK(cudaMemcpy(inv_host, g.d_inv, i4 * g.last_n, cudaMemcpyDeviceToHost));
    return MT_OK;
}

mt_status mt_debug_wait_timeout(int32_t limit_ms, void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (limit_ms < 1 || limit_ms > 1000) return MT_ERR_INVALID_ARG;
    CU_OK(cudaSetDevice(g.device));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    launch_wait_timeout_probe(g.d_status, (unsigned long long)limit_ms * 1000000ull, g.d_status + 3, s);
    CU_OK(cudaGetLastError());
    return MT_OK;
}

mt_status mt_debug_item_cost(int32_t k_blocks, int32_t n_cols, int32_t rows, double* cycles_out) {
    if (!cycles_out || k_blocks < 0 || n_cols < 0 || rows < 0) return MT_ERR_INVALID_ARG;
    *cycles_out = item_cost_cycles(k_blocks, n_cols, rows);
    return MT_OK;
}

mt_status mt_debug_schedule_balance(int32_t layer, double* max_over_mean_out, int32_t* n_items_out, int32_t* n_ctas_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (!max_over_mean_out || layer < 0 || layer >= (int)g.family.size() || g.family[layer].kind != MT_DENSE || !g.d_items[layer])
        return MT_ERR_INVALID_ARG;
    CU_OK(cudaSetDevice(g.device));
    CU_OK(cudaDeviceSynchronize());
    int32_t n_items = 0;
    CU_OK(cudaMemcpy(&n_items, g.d_tile_prefix + (size_t)layer * (g.T + 1) + g.T, sizeof n_items, cudaMemcpyDeviceToHost));
    if (n_items < 0 || (size_t)n_items > g.items_cap[layer]) return MT_ERR_CUDA;
    std::vector<WorkItem> items(n_items);
    if (n_items) CU_OK(cudaMemcpy(items.data(), g.d_items[layer], sizeof(WorkItem) * (size_t)n_items, cudaMemcpyDeviceToHost));
    const bool pair = g.last_pair[layer];
    const int grid = pair ? (g.sm_count & ~1) / 2 : g.sm_count;
    const int tn = pair ? 256 : g.tile_n[layer];
    std::vector<double> per(grid, 0.0);
    double sum = 0.0;
    for (int i = 0; i < n_items; ++i) {
        const WorkItem& w = items[i];
        const int cols = w.N - w.n_tile * tn < tn ? w.N - w.n_tile * tn : tn;
        const double c = item_cost_cycles(w.k_blocks, cols, w.rows_valid < BM ? w.rows_valid : BM);
        const int k = i / grid, r = i % grid;
        per[(k & 1) ? grid - 1 - r : r] += c;     // the executors' dealing (dealt_item)
        sum += c;
    }
    double mx = 0.0;
    for (double v : per) mx = v > mx ? v : mx;
    *max_over_mean_out = sum > 0 ? mx / (sum / grid) : 1.0;
    if (n_items_out) *n_items_out = n_items;
    if (n_ctas_out) *n_ctas_out = grid;
    return MT_OK;
}

mt_status mt_debug_empty_launches(int32_t count, void* stream) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (count < 0 || count > 100000) return MT_ERR_INVALID_ARG;
    CU_OK(cudaSetDevice(g.device));
    launch_empty_chain(count, static_cast<cudaStream_t>(stream));
    CU_OK(cudaGetLastError());
    return MT_OK;
}

mt_status mt_debug_launch_count(int64_t* count_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!count_out) return MT_ERR_INVALID_ARG;
    *count_out = (int64_t)mt::g_kernel_launches;
    return MT_OK;
}

mt_status mt_debug_set_option(const char* name, int32_t value) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g.init) return MT_ERR_NOT_INIT;
    if (!name) return MT_ERR_INVALID_ARG;
    const bool on = value != 0;
    if (!strcmp(name, "fused")) g.opt_fused = on;
    else if (!strcmp(name, "pair")) g.opt_pair = on;
    else if (!strcmp(name, "conv_pair")) g.opt_conv_pair = on;
    else if (!strcmp(name, "pool_head")) g.opt_pool_head = on;
    else if (!strcmp(name, "conv_stack")) g.opt_conv_stack = on;
    else if (!strcmp(name, "async_register")) g.opt_async_register = on;
    else if (!strcmp(name, "conv_balance")) g.opt_conv_balance = on;
    else if (!strcmp(name, "conv_self_bucket")) g.opt_conv_self_bucket = on;
    else if (!strcmp(name, "perm_gather")) g.opt_gather = value < 0 ? 0 : (value > 2 ? 2 : value);
    else return MT_ERR_INVALID_ARG;
    return MT_OK;
}

mt_status mt_set_kernel_timing(int32_t enable) {
    std::lock_guard<std::mutex> lk(g_mu);
    Timer::close_group();
    g.timing = enable < 0 ? 0 : (enable > 3 ? 1 : enable);
    g.timing_now = 0;
    g.timing_calls = 0;
    return MT_OK;
}

mt_status mt_get_kernel_times(const char** names, double* total_ms, int32_t* launches, int32_t cap, int32_t* n_out) {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!names || !total_ms || !launches || !n_out || cap < 0) return MT_ERR_INVALID_ARG;
    Timer::close_group();
    double ms[K_COUNT] = {0};
    int cnt[K_COUNT] = {0};
    for (TimedLaunch& t : g.timed) {
        CU_OK(cudaEventSynchronize(t.stop));
        float f = 0.f;
        CU_OK(cudaEventElapsedTime(&f, t.start, t.stop));
        ms[t.kernel] += f;
        cnt[t.kernel] += t.count;
        g.event_pool.push_back(t.start);
        g.event_pool.push_back(t.stop);
    }
    g.timed.clear();
    int k = 0;
    for (int i = 0; i < K_COUNT && k < cap; ++i) {
        if (cnt[i] == 0) continue;
        names[k] = kKernelNames[i];
        total_ms[k] = ms[i];
        launches[k] = cnt[i];
        ++k;
    }
    *n_out = k;
    return MT_OK;
}

}  // extern "C"

// Host-side declarations of the kernel launchers (one per .cu file) used by the C-ABI layer.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mt {

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the stream is
// still draining; it must call pdl_wait() before it touches anything the predecessor wrote or still reads.
extern unsigned long long g_kernel_launches;   // kernels enqueued through launch_pdl since the library was loaded
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    ++g_kernel_launches;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

struct ModelDev;
struct WorkItem;

// Dealing of a layer's work items to the CTAs (or CTA pairs) of a persistent launch: rounds of `grid` consecutive
// items, forwards in even rounds and backwards in odd ones.  The list is laid out heaviest items first, so a plain
// round-robin would hand CTA 0 the largest item of every round; the back-and-forth order evens the sums out.
__host__ __device__ inline int dealt_item(int k, int b, int grid) { return k * grid + ((k & 1) ? grid - 1 - b : b); }

constexpr int kBucketChunk = 64;    // requests per CTA in the scatter pass (kHistChunk is a multiple of it)
constexpr int kScatterThreads = 256;
constexpr int kHistChunk = 1024;    // requests per CTA (and per row of block_hist) in the histogram pass

struct BucketArgs {
    const int32_t* ids;
    int n;
    int T;                    // id slots in use (highest issued id + 1)
    const ModelDev* models;
    const int32_t* brief;     // compact tenant fields, rows of brief_ld ints: row 0 alive, row 1 + l out features of layer l
    int brief_ld;
    const int32_t* order;     // rows of brief_ld ints, one per layer: tenants in the order their work items are laid out
                              // (heaviest a-priori cost per item first for dense layers; id order for the others)
    int kind[8];              // layer kinds of the hosted family
    int n_layers;
    int rows_per_unit;        // conv: tiles per image
    int tile_n[8];            // dense: output columns per work item of each layer (128 or 256)
    int tile_m[8];            // dense: rows per work item of each layer (128, or 256 for the CTA-pair executor);
                              // conv: images per work unit (1, or 2 for the CTA-pair executor)
    int row_scale[8] = {0, 0, 0, 0, 0, 0, 0, 0};   // dense: matrix rows per request (0 or 1: one; H * W for a pointwise conv)
    int32_t* block_hist;      // [ceil(n / kHistChunk)][T + 1]
    int32_t* counts;          // [T + 1]
    int32_t* offsets;         // [T + 2]
    int32_t* tile_prefix;     // [n_layers][T + 1]
    int32_t* perm;            // [n]
    int32_t* inv;             // [n]
    int32_t* ticket;          // one zero-initialised word: arrival counter of pass 1 (left at zero by every call)
    const void* rows_src;     // non-null: payload rows [n][row_bytes] in arrival order, moved by pass 2 ...
    void* rows_dst;           // ... to bucketed order, rows dst_ld_bytes apart (both multiples of 16 bytes)
    int row_bytes;
    int dst_ld_bytes;
    int item_grid;            // least number of CTAs of pass 2 (the work-item expansion wants the whole GPU)
    WorkItem* items[8];       // per dense layer: expanded work items (null for other layers)
    unsigned* grid_bar;       // non-null: a word this call's conv launches use as their barrier counter; zeroed here
    int32_t* status;
};

cudaError_t configure_bucketing();
void launch_bucketing(const BucketArgs& a, cudaStream_t s);
// One thread waits (bounded by limit_ns) on a barrier nobody completes; *gave_up = 1 and the status word is set.
void launch_wait_timeout_probe(int32_t* status, unsigned long long limit_ns, int32_t* gave_up, cudaStream_t s);
// `count` empty kernels chained by programmatic dependent launch (the launch floor of the path).
void launch_empty_chain(int count, cudaStream_t s);
void launch_gather_rows(const void* src, const int32_t* perm, int n, int row_bytes, void* dst, int dst_ld_bytes,
                        int sm_count, cudaStream_t s);

// Re-lay a dense weight matrix W[N][K] (bf16, row-major) as ceil(N/128) x (K/64) tiles of 128 rows x 64
// columns, each tile 16 KiB in the 128-byte-swizzled shared-memory image the tensor-core kernels consume;
// rows >= N are zero.  Tile (nt, kb) starts at element offset (nt * (K/64) + kb) * 8192.
void launch_pretile_dense(const uint16_t* w, int N, int K, uint16_t* out, cudaStream_t s);
// Conv weights W[64][3][3][64] -> 9 tap tiles of 64 rows (out channel) x 64 columns (in channel), 8 KiB each,
// in the tile order the conv executor pairs them in.
void launch_pretile_conv(const uint16_t* w, int C_out, int C_in, uint16_t* out, cudaStream_t s);

struct GemmArgs {
    int T;
    const int32_t* tile_prefix;   // [T + 1] of this layer; tile_prefix[T] = number of work items
    const WorkItem* items;        // the layer's work items
    const CUtensorMap* wmaps;     // [model][MT_MAX_LAYERS] tensor maps of the tiled dense weights (CTA-pair executor)
    int layer;
    void* out;                    // bf16 hidden activations of the next layer, rows in bucketed order (may be null
                                  // when every item of the launch is a tenant's last layer)
    int ld_out;                   // elements between rows of `out`
    // Items flagged kItemFinal (the tenant's last layer; models of a family may differ in depth, so any launch can
    // hold some) write fp32 rows straight to row perm[j] of final_out, the caller's buffer in arrival order - there
    // is no separate un-permute pass.  The launch with nan_fill set (the family's deepest layer) also fills the rows of
    // rejected requests, bucketed rows [offsets[T], offsets[T + 1]), with NaN.
    float* final_out;
    int ld_final;
    int nan_fill;
    const int32_t* perm;
    const int32_t* offsets;       // [T + 2]
    // First layer only: non-null gather_perm makes the executor read its input rows from the caller's buffer (arrival
    // order) through the permutation - bucketed row j is row gather_perm[j] of the tensor behind the gather map (boxes
    // of one row x 64 columns), fetched four rows per TMA gather - so the payload is never moved into bucketed order.
    const int32_t* gather_perm;
    int32_t* status;
};
cudaError_t configure_grouped_gemm();
// tile_n: 128 or 256 output columns per work item; must match BucketArgs::tile_n of that layer.
// tmap_a: 128-row boxes of the layer's input; tmap_a32: 32-row boxes of the same buffer (transposed small items).
// With GemmArgs::gather_perm set, tmap_a is the gather map over the caller's rows (tmap_a32 is then unused).
void launch_grouped_gemm(const CUtensorMap& tmap_a, const CUtensorMap& tmap_a32, const GemmArgs& a, int tile_n,
                         int sm_count, cudaStream_t s);

// Whole-pass executor for small batches of narrow MLPs (fused_mlp.cu): bucketing, all dense layers and the return to
// arrival order in one launch.
struct FusedArgs {
    const uint16_t* inputs;   // bf16 [n][K0], arrival order
    const int32_t* ids;       // [n]
    int n;
    int T;
    const ModelDev* models;
    int n_layers;
    int K0;                   // features per row of `inputs`: the widest model's input (multiple of 64, at most 256)
    int out_elems;            // output features (at most 256)
    float* out;               // fp32 [n][out_elems], arrival order (the caller's buffer)
    int32_t* counts;          // [T + 1]   bucketing results, written by CTA 0
    int32_t* offsets;         // [T + 2]
    int32_t* perm;            // [n]
    int32_t* inv;             // [n]
    int32_t* status;
};
// n <= 512, every layer at most max_width <= 256 wide, and the per-chunk histograms fit the operand buffer
bool fused_mlp_fits(int n, int T, int max_width);
cudaError_t configure_fused_mlp();
cudaError_t launch_fused_mlp(const FusedArgs& a, int grid, cudaStream_t s);

// CTA-pair form (grouped_gemm_pair.cu): work items of 256 rows x 256 columns (BucketArgs::tile_m = tile_n = 256).
cudaError_t configure_grouped_gemm_pair();
cudaError_t launch_grouped_gemm_pair(const CUtensorMap& tmap_a, const GemmArgs& a, int sm_count, cudaStream_t s);

// Strip geometry of the conv executor (see grouped_conv.cu).
struct ConvPlan {
    int Wp;                // padded row length in shared memory: W + 2 rounded up to 32, 64 or 128 pixels
    int R;                 // output rows per strip
    int tiles_per_strip;   // 128-pixel accumulator tiles per strip
    int stage_bytes;       // shared memory per strip stage (multiple of 1024)
    int n_stages;
    int strips_per_image;
    int box_bytes;         // bytes one TMA box delivers: (R + 2) * Wp * 128
    int smem_bytes;        // dynamic shared memory of the launch
};
bool plan_conv(int H, int W, ConvPlan* plan);

struct ConvArgs {
    const ModelDev* models;
    int layer;
    int T;
    const int32_t* offsets;
    const int32_t* tile_prefix;   // work units = strips
    const int32_t* perm;          // non-null: image index = perm[j] (first layer reads the caller's buffer)
    uint16_t* out;                // bf16 NHWC, bucketed order (unused when pool_partial is set)
    float* pool_partial;          // non-null: the layer feeds a global average pool; [n][strips_per_image][64] sums
    int H, W;
    int Wp, R, tiles_per_strip, stage_bytes, n_stages, strips_per_image, box_bytes;
    // CTA-pair executor, consecutive conv layers of one call (programmatic dependent launch).  late_trigger: let the next
    // launch start only after this one's dependency wait has returned, so that everything older than this launch's
    // predecessor is complete when the next one starts.  early_lookup (only behind a launch with late_trigger, which is
    // not the bucketing itself): read the bucketing results and request the first weights BEFORE the dependency wait.
    int late_trigger = 0, early_lookup = 0;
    int border_units = 0;         // CTA-pair executor: work units a tenant border inside a cluster's range is charged when
                                  // the ranges are cut (0: ranges of equal length)
    int n_stack = 1;              // CTA-pair executor: conv layers run by this launch
    unsigned* grid_bar = nullptr; // ... and the counter of their grid-wide barrier (zero when the launch starts)
    // Identity shortcuts: per layer of the launch (index 0 for the one-CTA executor) the bf16 NHWC tensor that a tenant
    // whose layer is marked residual adds before the activation - the input of the layer before - or nullptr when no
    // such tensor exists (the family's first layer).  skip_perm non-null: that tensor is the caller's buffer, image
    // index = skip_perm[j]; else it is in bucketed order.
    const uint16_t* skip[4] = {nullptr, nullptr, nullptr, nullptr};
    const int32_t* skip_perm[4] = {nullptr, nullptr, nullptr, nullptr};
    // CTA-pair executor, small batches (kConvSelfBucketMaxN requests, kConvSelfBucketMaxT tenants at most): ids non-null
    // = no bucketing launch ran for this call; every CTA repeats the stable counting sort of the n ids in shared memory
    // (as the one-launch MLP path does) and takes offsets, unit prefixes and perm from there; CTA 0 also writes them,
    // counts and inv to the arrays below for the launches that follow (prefix_rows rows of T + 1 unit prefixes).
    const int32_t* ids = nullptr;
    int n = 0;
    int32_t* counts_out = nullptr;
    int32_t* offsets_out = nullptr;
    int32_t* perm_out = nullptr;
    int32_t* inv_out = nullptr;
    int32_t* prefix_out = nullptr;
    int prefix_rows = 0;
    int32_t* status;
};
constexpr int kConvSelfBucketMaxN = 512;
constexpr int kConvSelfBucketMaxT = 512;

cudaError_t configure_grouped_conv();
void launch_grouped_conv(const CUtensorMap& tmap_x, const ConvArgs& a, int smem_bytes, int sm_count, cudaStream_t s);

// CTA-pair form of the conv executor (grouped_conv_pair.cu; padded row length 64 only).  Its weight images (two of
// kConvPairWeightBytes, rank 0 first) follow the one-CTA image in the layer's weight block, kConvPairImageOffset
// elements in.  ConvArgs::tile_prefix must count (pair of images, strip) units: BucketArgs::tile_m = 2 for the layer.
constexpr int kConvPairWeightBytes = 60 * 1024;
constexpr int kConvPairImageOffset = 9 * 64 * 64;          // bf16 elements of the one-CTA image
void launch_pretile_conv_pair(const uint16_t* w, uint16_t* out, cudaStream_t s);
int conv_pair_smem_bytes();
cudaError_t configure_grouped_conv_pair();
// Up to kConvStackMax consecutive conv layers of one geometry run as ONE launch (ConvArgs::n_stack, from ConvArgs::layer
// on; grid-wide barrier between layers on ConvArgs::grid_bar, a word the bucketing kernel of the call has zeroed).
// Per layer of the stack: x2, x1 = its input (NHWC bf16) as boxes of 64 channels x 64 pixels x 2 rows and x 1 row (the
// executor fetches the image in blocks of two rows, whatever ConvArgs says about strip stages); y = its output as boxes
// of 32 channels x 32 pixels x 1 row, 64-byte swizzle (unused by a layer that feeds the pool).  ConvArgs::perm applies to
// the stack's first layer, ConvArgs::pool_partial to its last.
constexpr int kConvStackMax = 4;
static_assert(kConvStackMax <= 4, "ConvArgs::skip holds one entry per stacked layer");
struct ConvStackMaps {
    CUtensorMap x2[kConvStackMax], x1[kConvStackMax], y[kConvStackMax];
};
cudaError_t launch_grouped_conv_pair(const ConvStackMaps& maps, const ConvArgs& a, int sm_count, cudaStream_t s);

// Second half of the fused pooling: sums the per-strip channel sums of each image and divides by H*W.
// grid_bar (may be null): the eight barrier counters of the call's stacked conv launches, set back to zero here - a
// pool always follows the last conv layer, so the counters are zero whenever a call starts.
void launch_pool_finalize(const float* partial, int n, int strips, int C, int HW, uint16_t* out, int ld_out,
                          unsigned* grid_bar, cudaStream_t s);

// The same fused with the model's last layer when that is a dense layer from the pooled 64 channels to at most 64
// outputs: pooled values (rounded to bf16) x head weights, bias, optional ReLU, fp32 rows written to arrival order.
void launch_pool_head(const float* partial, int n, int strips, int HW, const ModelDev* models, int layer,
                      const int32_t* offsets, int T, const int32_t* perm, float* out, int out_elems, unsigned* grid_bar,
                      cudaStream_t s);

}  // namespace mt

// Request bucketing and its inverse: group the requests of one mixed batch by model id into
// contiguous segments (a stable counting sort), keep the permutation back to arrival order,
// move payload rows into bucketed order, and restore arrival order at the end.
//
// The paper (Sec. 3) has a worker receive requests for many tenants' models; grouping them by model is a
// pure re-ordering, made unique by stability: inside a segment, requests keep their arrival order.
//
//   pass 1  bucket_block_hist   per-block histogram of ids (warp-level match + one shared atomic per group)
//   pass 2  bucket_scan         per-tenant exclusive scan over blocks, exclusive scan over tenants
//                               (offsets), per-layer tile prefix sums for the grouped executors
//   pass 3  bucket_scatter      stable position of every request -> perm / inv
//           gather_rows         X_b[j, :] = X[perm[j], :]          (128-bit copies)
//           unpermute_rows      out[perm[j], :] = out_b[j, :]      (128-bit copies where rows allow)
#include <limits>

#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kScanThreads = 1024;

struct LayerTileN { int v[8]; int m[8]; };   // per layer: columns (v) and rows (m) of one dense work item

// ids outside [0, T) or of dead models go to the extra bucket T, so they sort behind every live segment.
__device__ __forceinline__ int classify(int id, int T, const ModelDev* models) {
    if (id < 0 || id >= T) return T;
    return models[id].alive ? id : T;
}

__global__ void __launch_bounds__(kBucketChunk)
bucket_block_hist(const int32_t* __restrict__ ids, int n, int T, const ModelDev* __restrict__ models,
                  int32_t* __restrict__ block_hist, int32_t* __restrict__ status) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ int32_t s_hist[];   // T + 1
    const int T1 = T + 1;
    for (int t = threadIdx.x; t < T1; t += blockDim.x) s_hist[t] = 0;
    __syncthreads();
    const int i = blockIdx.x * kBucketChunk + threadIdx.x;
    if (i < n) {
        const int b = classify(ids[i], T, models);
        if (b == T) {
            atomicCAS(&status[ST_CODE], MT_OK, MT_ERR_BAD_MODEL_ID);
            atomicMin(&status[ST_BAD_INDEX], i);
        }
        const unsigned peers = __match_any_sync(__activemask(), b);
        if ((__ffs(peers) - 1) == (threadIdx.x & 31)) atomicAdd(&s_hist[b], __popc(peers));
    }
    __syncthreads();
    for (int t = threadIdx.x; t < T1; t += blockDim.x) block_hist[(size_t)blockIdx.x * T1 + t] = s_hist[t];
}

// Exclusive scan across the threads of a CTA (any multiple of 32 threads up to 1024): returns the sum of `v` over
// all lower-numbered threads; *total = sum over the CTA.  s_warp: 33 ints of shared memory.  Two barriers.
__device__ __forceinline__ int cta_excl_scan(int v, int32_t* s_warp, int* total) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += u;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = (lane < n_warps) ? s_warp[lane] : 0;
        int wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += u;
        }
        s_warp[lane] = wi - w;                 // exclusive prefix of the warp totals
        if (lane == 31) s_warp[32] = wi;       // grand total
    }
    __syncthreads();
    const int r = incl - v + s_warp[warp];
    *total = s_warp[32];
    __syncthreads();                           // s_warp may be reused right away
    return r;
}

// Work units (tiles / strips) tenant t contributes to layer l, given its request count c.
__device__ __forceinline__ int layer_units(const ModelDev* models, int t, int l, int c, int rows_per_unit, int tile_n,
                                           int tile_m) {
    if (c <= 0) return 0;
    const LayerDev& L = models[t].layer[l];
    if (L.kind == MT_DENSE) return ((c + tile_m - 1) / tile_m) * ((L.N + tile_n - 1) / tile_n);
    if (L.kind == MT_CONV3X3) return c * rows_per_unit;
    return 0;
}

// Per bucket t (one warp each): counts[t] = sum over blocks, block_hist[b][t] <- exclusive prefix over blocks.
__device__ __forceinline__ void column_scan(int t, int n_blocks, int T1, int32_t* __restrict__ block_hist,
                                            int32_t* __restrict__ counts) {
    const int lane = threadIdx.x & 31;
    int carry = 0;
    for (int b0 = 0; b0 < n_blocks; b0 += 32) {
        const int b = b0 + lane;
        const int v = (b < n_blocks) ? block_hist[(size_t)b * T1 + t] : 0;
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += u;
        }
        if (b < n_blocks) block_hist[(size_t)b * T1 + t] = carry + incl - v;
        carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) counts[t] = carry;
}

// Many tenants x many blocks: the per-tenant scans over blocks run as a grid of warps.
__global__ void __launch_bounds__(256)
bucket_column_scan(int n_blocks, int T, int32_t* __restrict__ block_hist, int32_t* __restrict__ counts) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t < T + 1) column_scan(t, n_blocks, T + 1, block_hist, counts);
}

// One CTA: (optionally the per-tenant scans over blocks,) offsets = exclusive scan of counts over the T + 1
// buckets (offsets[T + 1] = n), and per layer the prefix sums of the work units each tenant contributes.
__global__ void __launch_bounds__(kScanThreads)
bucket_scan(int n_blocks, int T, const ModelDev* __restrict__ models, int n_layers, int rows_per_unit, LayerTileN tn,
            int do_columns, int32_t* __restrict__ block_hist, int32_t* __restrict__ counts,
            int32_t* __restrict__ offsets, int32_t* __restrict__ tile_prefix) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int32_t s_warp[33];
    const int T1 = T + 1;
    if (do_columns) {
        for (int t = threadIdx.x >> 5; t < T1; t += kScanThreads / 32) column_scan(t, n_blocks, T1, block_hist, counts);
        __syncthreads();
    }
    // each thread owns `per` consecutive buckets
    const int per = (T1 + kScanThreads - 1) / kScanThreads;
    const int lo = min((int)threadIdx.x * per, T1), hi = min(lo + per, T1);
    int sum = 0;
    for (int t = lo; t < hi; ++t) sum += counts[t];
    int total;
    int run = cta_excl_scan(sum, s_warp, &total);
    for (int t = lo; t < hi; ++t) { offsets[t] = run; run += counts[t]; }
    if (threadIdx.x == 0) offsets[T1] = total;
    for (int l = 0; l < n_layers; ++l) {
        int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        const int hi_t = min(hi, T);           // the extra bucket of rejected ids contributes no work
        int usum = 0;
        for (int t = lo; t < hi_t; ++t) usum += layer_units(models, t, l, counts[t], rows_per_unit, tn.v[l], tn.m[l]);
        int urun = cta_excl_scan(usum, s_warp, &total);
        for (int t = lo; t < hi_t; ++t) { prefix[t] = urun; urun += layer_units(models, t, l, counts[t], rows_per_unit, tn.v[l], tn.m[l]); }
        if (threadIdx.x == 0) prefix[T] = total;
    }
}

struct ItemPtrs { WorkItem* v[8]; };

// Work item `item` of dense layer l: (tenant, row tile, column tile) and what the executor needs to know about it.
__device__ __forceinline__ WorkItem make_work_item(int item, int l, int T, const ModelDev* __restrict__ models,
                                                   const int32_t* __restrict__ offsets,
                                                   const int32_t* __restrict__ prefix, int tile_m) {
    int lo = 0, hi = T;   // largest t with prefix[t] <= item
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (prefix[mid] <= item) lo = mid; else hi = mid;
    }
    const LayerDev& L = models[lo].layer[l];
    const int seg0 = offsets[lo], n_t = offsets[lo + 1] - seg0;
    const int m_tiles = (n_t + tile_m - 1) / tile_m;
    const int local = item - prefix[lo];
    const int n_tile = local / m_tiles, m_tile = local - n_tile * m_tiles;
    WorkItem w;
    w.row0 = seg0 + m_tile * tile_m;
    w.rows_valid = min(tile_m, n_t - m_tile * tile_m);
    w.n_tile = n_tile;
    w.k_blocks = L.k_blocks;
    w.w = L.w;
    w.bias = L.bias;
    w.N = L.N;
    w.relu = L.relu;
    w.t = lo;
    w.pad = 0;
    return w;
}


// A batch that fits one CTA (n <= kSingleCtaMax): histogram, scans, stable scatter and the work-item expansion in
// ONE launch.  blockDim.x is 256 or 1024; the requests are taken in rounds of blockDim.x.
constexpr int kSingleCtaMax = 4096;

__global__ void __launch_bounds__(1024)
bucket_single_cta(const int32_t* __restrict__ ids, int n, int T, const ModelDev* __restrict__ models, int n_layers,
                  int rows_per_unit, LayerTileN tn, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                  int32_t* __restrict__ tile_prefix, int32_t* __restrict__ perm, int32_t* __restrict__ inv,
                  ItemPtrs items, int32_t* __restrict__ status) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ int32_t s_mem[];          // s_cnt[T + 1], s_next[T + 1]
    __shared__ int32_t s_warp[33];
    const int T1 = T + 1;
    int32_t* s_cnt = s_mem;
    int32_t* s_next = s_mem + T1;
    const int nthr = blockDim.x, n_warps = nthr >> 5;
    const int rounds = (n + nthr - 1) / nthr;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int t = threadIdx.x; t < T1; t += nthr) s_cnt[t] = 0;
    __syncthreads();
    int bucket[kSingleCtaMax / 256];            // this thread's requests, one per round (at most 16 rounds of 256)
#pragma unroll
    for (int r = 0; r < kSingleCtaMax / 256; ++r) {
        bucket[r] = -1;
        const int i = r * nthr + threadIdx.x;
        if (r < rounds && i < n) {
            const int b = classify(ids[i], T, models);
            bucket[r] = b;
            if (b == T) {
                atomicCAS(&status[ST_CODE], MT_OK, MT_ERR_BAD_MODEL_ID);
                atomicMin(&status[ST_BAD_INDEX], i);
            }
            const unsigned peers = __match_any_sync(__activemask(), b);
            if ((__ffs(peers) - 1) == lane) atomicAdd(&s_cnt[b], __popc(peers));
        }
    }
    __syncthreads();
    const int per = (T1 + nthr - 1) / nthr;
    const int lo = min((int)threadIdx.x * per, T1), hi = min(lo + per, T1);
    int sum = 0;
    for (int t = lo; t < hi; ++t) sum += s_cnt[t];
    int total;
    int run = cta_excl_scan(sum, s_warp, &total);
    for (int t = lo; t < hi; ++t) { offsets[t] = run; s_next[t] = run; counts[t] = s_cnt[t]; run += s_cnt[t]; }
    if (threadIdx.x == 0) offsets[T1] = total;
    for (int l = 0; l < n_layers; ++l) {
        int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        const int hi_t = min(hi, T);
        int usum = 0;
        for (int t = lo; t < hi_t; ++t) usum += layer_units(models, t, l, s_cnt[t], rows_per_unit, tn.v[l], tn.m[l]);
        int urun = cta_excl_scan(usum, s_warp, &total);
        for (int t = lo; t < hi_t; ++t) { prefix[t] = urun; urun += layer_units(models, t, l, s_cnt[t], rows_per_unit, tn.v[l], tn.m[l]); }
        if (threadIdx.x == 0) prefix[T] = total;
    }
    __syncthreads();
    // rounds in order, and inside a round the warps take turns: positions inside a bucket ascend with arrival index
#pragma unroll
    for (int r = 0; r < kSingleCtaMax / 256; ++r) {
        if (r >= rounds) break;
        const int i = r * nthr + threadIdx.x;
        const int b = bucket[r];
        for (int w = 0; w < n_warps; ++w) {
            if (warp == w && i < n) {
                const unsigned peers = __match_any_sync(__activemask(), b);
                const int rank = __popc(peers & ((1u << lane) - 1u));
                const int pos = s_next[b] + rank;
                __syncwarp(__activemask());
                if (rank == 0) s_next[b] += __popc(peers);
                perm[pos] = i;
                inv[i] = pos;
            }
            __syncthreads();
        }
    }
    // work items of the dense layers (offsets and prefixes were written by this CTA: make them visible first)
    __threadfence_block();
    __syncthreads();
    for (int l = 0; l < n_layers; ++l) {
        WorkItem* out = items.v[l];
        if (!out) continue;
        const int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        const int n_items = prefix[T];
        for (int item = threadIdx.x; item < n_items; item += nthr) out[item] = make_work_item(item, l, T, models, offsets, prefix, tn.m[l]);
    }
}

// Expand every dense layer's work list: item i of layer l -> (tenant, row tile, column tile) and everything the
// executor needs to know about it.  Row tiles of one weight slab are adjacent items, so concurrent CTAs share it in L2.
__global__ void build_work_items(int T, const ModelDev* __restrict__ models, int n_layers, LayerTileN tn,
                                 const int32_t* __restrict__ offsets, const int32_t* __restrict__ tile_prefix,
                                 ItemPtrs items) {
    pdl_launch_dependents();
    pdl_wait();
    for (int l = 0; l < n_layers; ++l) {
        WorkItem* out = items.v[l];
        if (!out) continue;
        const int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        const int total = prefix[T];
        for (int item = blockIdx.x * blockDim.x + threadIdx.x; item < total; item += gridDim.x * blockDim.x) {
            out[item] = make_work_item(item, l, T, models, offsets, prefix, tn.m[l]);
        }
    }
}

__global__ void __launch_bounds__(kBucketChunk)
bucket_scatter(const int32_t* __restrict__ ids, int n, int T, const ModelDev* __restrict__ models,
               const int32_t* __restrict__ block_hist, const int32_t* __restrict__ offsets,
               int32_t* __restrict__ perm, int32_t* __restrict__ inv) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ int32_t s_next[];   // next free position of every bucket for this block
    const int T1 = T + 1;
    for (int t = threadIdx.x; t < T1; t += blockDim.x)
        s_next[t] = offsets[t] + block_hist[(size_t)blockIdx.x * T1 + t];
    __syncthreads();
    const int i = blockIdx.x * kBucketChunk + threadIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = (i < n) ? classify(ids[i], T, models) : -1;
    // warps take turns in arrival order, so positions inside a bucket ascend with the arrival index
    for (int w = 0; w < kBucketChunk / 32; ++w) {
        if (warp == w && i < n) {
            const unsigned peers = __match_any_sync(__activemask(), b);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            const int pos = s_next[b] + rank;
            __syncwarp(__activemask());
            if (rank == 0) s_next[b] += __popc(peers);
            perm[pos] = i;
            inv[i] = pos;
        }
        __syncthreads();
    }
}

// X_b[j, :] = X[perm[j], :]; rows of `row_vec` 16-byte vectors; dst rows `dst_ld_vec` vectors apart.
__global__ void gather_rows(const uint4* __restrict__ src, const int32_t* __restrict__ perm, int n, int row_vec,
                            uint4* __restrict__ dst, int dst_ld_vec) {
    pdl_launch_dependents();
    pdl_wait();
    const long long total = (long long)n * row_vec;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int j = (int)(idx / row_vec), v = (int)(idx % row_vec);
        dst[(size_t)j * dst_ld_vec + v] = __ldg(&src[(size_t)perm[j] * row_vec + v]);
    }
}

// out[perm[j], :] = out_b[j, :] for j < n_valid; rows of rejected requests (j >= n_valid) become NaN.
template <typename V>
__global__ void unpermute_rows(const V* __restrict__ src, const int32_t* __restrict__ perm,
                               const int32_t* __restrict__ offsets, int T, int n, int row_vec,
                               V* __restrict__ dst, V nan_v) {
    pdl_launch_dependents();
    pdl_wait();
    const int n_valid = offsets[T];
    const long long total = (long long)n * row_vec;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int j = (int)(idx / row_vec), v = (int)(idx % row_vec);
        dst[(size_t)perm[j] * row_vec + v] = (j < n_valid) ? src[idx] : nan_v;
    }
}

// Self-test of the bounded wait every executor relies on: one thread waits on an mbarrier that nobody ever
// completes; after limit_ns it must give up, raise the abort flag and report MT_ERR_TIMEOUT - and return.
__global__ void wait_timeout_probe(int32_t* status, unsigned long long limit_ns, int32_t* gave_up) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_mbar_init();
        const bool done = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, 99, limit_ns);
        *gave_up = done ? 0 : 1;
    }
}

void launch_wait_timeout_probe(int32_t* status, unsigned long long limit_ns, int32_t* gave_up, cudaStream_t s) {
    wait_timeout_probe<<<1, 32, 0, s>>>(status, limit_ns, gave_up);
}

// ------------------------------------------------------------------------------------------ launchers
static int grid_for(long long total, int threads, int sm_count) {
    long long blocks = (total + threads - 1) / threads;
    const long long cap = (long long)sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

void launch_bucketing(const BucketArgs& a, cudaStream_t s) {
    const int n_blocks = (a.n + kBucketChunk - 1) / kBucketChunk;
    const size_t smem = sizeof(int32_t) * (size_t)(a.T + 1);
    LayerTileN tn;
    for (int l = 0; l < 8; ++l) { tn.v[l] = a.tile_n[l] > 0 ? a.tile_n[l] : BN; tn.m[l] = a.tile_m[l] > 0 ? a.tile_m[l] : BM; }
    ItemPtrs ip;
    bool any = false;
    for (int l = 0; l < 8; ++l) { ip.v[l] = a.items[l]; any = any || a.items[l]; }
    // measured: one CTA wins up to a few hundred requests; beyond that its serial scatter and the item expansion
    // by a single CTA cost more than the extra launches of the multi-CTA path
    if (a.n <= 512 && a.T + 1 <= 4096) {
        const int threads = (a.n <= 256) ? 256 : 1024;
        launch_pdl(bucket_single_cta, dim3(1), dim3(threads), 2 * smem, s, a.ids, a.n, a.T, a.models, a.n_layers, a.rows_per_unit, tn, a.counts,
                                                      a.offsets, a.tile_prefix, a.perm, a.inv, ip, a.status);
        return;
    }
    launch_pdl(bucket_block_hist, dim3(n_blocks), dim3(kBucketChunk), smem, s, a.ids, a.n, a.T, a.models, a.block_hist, a.status);
    // few buckets x few blocks: the per-tenant scans over blocks ride along in the single-CTA scan kernel
    const int col_iters = ((a.T + 1 + 31) / 32) * ((n_blocks + 31) / 32);
    const int fused = col_iters <= 4;
    if (!fused) launch_pdl(bucket_column_scan, dim3((a.T + 1 + 7) / 8), dim3(256), 0, s, n_blocks, a.T, a.block_hist, a.counts);
    launch_pdl(bucket_scan, dim3(1), dim3(kScanThreads), 0, s, n_blocks, a.T, a.models, a.n_layers, a.rows_per_unit, tn, fused, a.block_hist,
                                           a.counts, a.offsets, a.tile_prefix);
    launch_pdl(bucket_scatter, dim3(n_blocks), dim3(kBucketChunk), smem, s, a.ids, a.n, a.T, a.models, a.block_hist, a.offsets, a.perm,
                                                        a.inv);
    if (any) launch_pdl(build_work_items, dim3(a.item_grid), dim3(256), 0, s, a.T, a.models, a.n_layers, tn, a.offsets, a.tile_prefix, ip);
}

void launch_gather_rows(const void* src, const int32_t* perm, int n, int row_bytes, void* dst, int dst_ld_bytes,
                        int sm_count, cudaStream_t s) {
    const int row_vec = row_bytes / 16;
    launch_pdl(gather_rows, dim3(grid_for((long long)n * row_vec, 256, sm_count)), dim3(256), 0, s,
        (const uint4*)src, perm, n, row_vec, (uint4*)dst, dst_ld_bytes / 16);
}

void launch_unpermute(const float* src, const int32_t* perm, const int32_t* offsets, int T, int n, int out_elems,
                      float* dst, int sm_count, cudaStream_t s) {
    const float qnan = std::numeric_limits<float>::quiet_NaN();
    const bool vec_ok = (out_elems % 4 == 0) && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0);
    if (vec_ok) {
        const int row_vec = out_elems / 4;
        launch_pdl(unpermute_rows<float4>, dim3(grid_for((long long)n * row_vec, 256, sm_count)), dim3(256), 0, s,
            (const float4*)src, perm, offsets, T, n, row_vec, (float4*)dst, make_float4(qnan, qnan, qnan, qnan));
    } else {
        launch_pdl(unpermute_rows<float>, dim3(grid_for((long long)n * out_elems, 256, sm_count)), dim3(256), 0, s,
            src, perm, offsets, T, n, out_elems, dst, qnan);
    }
}

}  // namespace mt

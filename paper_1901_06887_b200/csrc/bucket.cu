// Request bucketing and its inverse: group the requests of one mixed batch by model id into
// contiguous segments (a stable counting sort), keep the permutation back to arrival order,
// move payload rows into bucketed order, and restore arrival order at the end.
//
// The paper (Sec. 3) has a worker receive requests for many tenants' models; grouping them by model is a
// pure re-ordering, made unique by stability: inside a segment, requests keep their arrival order.
//
//   pass 1  bucket_hist_scan       per-block histogram of ids (warp-level match + one shared atomic per group); the
//                                  CTA that finishes last scans per tenant over the blocks and over the tenants
//                                  (offsets) and builds the per-layer unit prefix sums for the grouped executors
//   pass 2  bucket_scatter_expand  stable position of every request -> perm / inv, payload rows moved into
//                                  bucketed order (128-bit copies), work items of the dense layers
//           bucket_single_cta      both passes in one CTA for batches of at most 512 requests
//           gather_rows            X_b[j, :] = X[perm[j], :] as a pass of its own (payloads too large for pass 2)
//           (the return to arrival order, out[perm[j], :] = out_b[j, :], happens in the last layer's epilogue)
#include <climits>

#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {


// Per layer: columns (v) and rows (m) of one dense work item, the layer's kind (the same for every tenant of the
// hosted family) and, for dense layers, the matrix rows one request contributes (scale: 1, or H * W when the layer is a
// pointwise conv, i.e. the dense layer applied at every pixel of the request's image).
struct LayerTileN { int v[8]; int m[8]; int kind[8]; };   // kind[l]: layer kind in the low byte, row scale above it

// Compact copy of what the bucketing passes need from the tenant table, one row of `ld` ints per field: row 0 =
// alive flag, row 1 + l = out features of layer l.  (Reading these through the 328-byte ModelDev records costs one
// memory sector per tenant and field; a thousand tenants' worth from a single CTA took several microseconds.)
// `order` (rows of `ld` ints, one per layer) lists the tenants of a layer in the order their work items are laid out:
// heaviest per-item cost first, as ranked on the host from the layer shapes (known before any request arrives).
struct Brief { const int32_t* p; int ld; const int32_t* order; };
__device__ __forceinline__ int tenant_at(Brief br, int l, int rank) { return __ldg(br.order + (size_t)l * br.ld + rank); }

// ids outside [0, T) or of dead models go to the extra bucket T, so they sort behind every live segment.
// (Row 0 of the compact table: 0 = no model, 1 = live and resident, 2 = registered but evicted from the device.)
__device__ __forceinline__ int classify(int id, int T, Brief br) {
    if (id < 0 || id >= T) return T;
    return __ldg(br.p + id) == 1 ? id : T;
}
// Sticky status of a rejected request: its model is unknown, or known but not resident right now.
__device__ __forceinline__ void report_rejected(int id, int i, int T, Brief br, int32_t* status) {
    const bool evicted = id >= 0 && id < T && __ldg(br.p + id) == 2;
    atomicCAS(&status[ST_CODE], MT_OK, evicted ? MT_ERR_NOT_RESIDENT : MT_ERR_BAD_MODEL_ID);
    atomicMin(&status[ST_BAD_INDEX], i);
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

// The same for MT_MAX_LAYERS values per thread at once (three barriers for all of them instead of three each).
// s_vec: MT_MAX_LAYERS x 33 ints of shared memory.
__device__ __forceinline__ void cta_excl_scan_vec(const int (&v)[MT_MAX_LAYERS], int (&excl)[MT_MAX_LAYERS],
                                                  int (&total)[MT_MAX_LAYERS], int32_t* s_vec, int n_used) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
    int incl[MT_MAX_LAYERS];
#pragma unroll
    for (int l = 0; l < MT_MAX_LAYERS; ++l) {
        incl[l] = v[l];
        if (l >= n_used) continue;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, incl[l], d);
            if (lane >= d) incl[l] += u;
        }
        if (lane == 31) s_vec[l * 33 + warp] = incl[l];
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int l = 0; l < MT_MAX_LAYERS; ++l) {
            if (l >= n_used) continue;
            const int w = (lane < n_warps) ? s_vec[l * 33 + lane] : 0;
            int wi = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= d) wi += u;
            }
            s_vec[l * 33 + lane] = wi - w;
            if (lane == 31) s_vec[l * 33 + 32] = wi;
        }
    }
    __syncthreads();
#pragma unroll
    for (int l = 0; l < MT_MAX_LAYERS; ++l) {
        if (l >= n_used) { excl[l] = 0; total[l] = 0; continue; }
        excl[l] = incl[l] - v[l] + s_vec[l * 33 + warp];
        total[l] = s_vec[l * 33 + 32];
    }
    __syncthreads();
}

// What the unit count of a layer depends on, read from the tenant table without looking at the request count first:
// callers fetch the heads of all layers back to back, so the loads are in flight together (a load behind a branch on
// the count costs one memory round trip per layer on the single CTA's critical path).
struct LayerHead { int kind, N; };
__device__ __forceinline__ LayerHead load_head(Brief br, const LayerTileN& tn, int t, int l) {
    LayerHead h;
    h.kind = tn.kind[l] & 0xff;
    h.N = __ldg(br.p + (size_t)(1 + l) * br.ld + t);
    return h;
}
// Work units (tiles / strips) a tenant with c requests contributes to a layer.
__device__ __forceinline__ int units_of(LayerHead h, int c, int rows_per_unit, int tile_n, int tile_m, int scale) {
    if (c <= 0) return 0;
    if (h.kind == MT_DENSE) return ((c * scale + tile_m - 1) / tile_m) * ((h.N + tile_n - 1) / tile_n);
    if (h.kind == MT_CONV3X3) return ((c + tile_m - 1) / tile_m) * rows_per_unit;   // tile_m = images per unit
    return 0;
}
__device__ __forceinline__ int layer_units(Brief br, const LayerTileN& tn, int t, int l, int c, int rows_per_unit) {
    return units_of(load_head(br, tn, t, l), c, rows_per_unit, tn.v[l], tn.m[l], (tn.kind[l] >> 8));
}

// Offsets (exclusive scan of counts over the T + 1 buckets, offsets[T + 1] = n) and, per layer, the prefix sums of
// the work units each tenant contributes, taken in the layer's cost order (tile_prefix[l][r] belongs to the tenant of
// rank r).  Run by one CTA of any multiple of 32 threads; counts[] must be visible (cnt may be a shared-memory copy).
__device__ __forceinline__ void scan_buckets(int T, Brief br, int n_layers, int rows_per_unit,
                                             const LayerTileN& tn, const int32_t* cnt, int32_t* __restrict__ offsets,
                                             int32_t* __restrict__ tile_prefix, int32_t* s_warp, int32_t* s_vec,
                                             int own_count = -1) {
    // own_count >= 0: the caller has counts[threadIdx.x] in a register (one bucket per thread), no need to read it back
    const int T1 = T + 1;
    const int per = (T1 + (int)blockDim.x - 1) / (int)blockDim.x;     // each thread owns `per` consecutive buckets
    const int lo = min((int)threadIdx.x * per, T1), hi = min(lo + per, T1);
    const bool have_own = own_count >= 0 && per == 1;
    int sum = 0;
    if (have_own) sum = (lo < hi) ? own_count : 0;
    else for (int t = lo; t < hi; ++t) sum += cnt[t];
    int total;
    int run = cta_excl_scan(sum, s_warp, &total);
    if (have_own) { if (lo < hi) offsets[lo] = run; }
    else for (int t = lo; t < hi; ++t) { offsets[t] = run; run += cnt[t]; }
    if (threadIdx.x == 0) offsets[T1] = total;
    const int hi_t = min(hi, T);               // the extra bucket of rejected ids contributes no work
    if (per == 1) {
        // one rank per thread (the usual case): the tenants of that rank in every layer first, then their shapes, then
        // their counts, so that each kind of load is in flight for all layers together
        const int r_own = min(lo, T - 1);
        int t_l[MT_MAX_LAYERS];
#pragma unroll
        for (int l = 0; l < MT_MAX_LAYERS; ++l) t_l[l] = (l < n_layers) ? tenant_at(br, l, r_own) : 0;
        LayerHead head[MT_MAX_LAYERS];
#pragma unroll
        for (int l = 0; l < MT_MAX_LAYERS; ++l) head[l] = (l < n_layers) ? load_head(br, tn, t_l[l], l) : LayerHead{-1, 0};
        int units[MT_MAX_LAYERS];
#pragma unroll
        for (int l = 0; l < MT_MAX_LAYERS; ++l)
            units[l] = (l < n_layers && lo < hi_t) ? units_of(head[l], cnt[t_l[l]], rows_per_unit, tn.v[l], tn.m[l], (tn.kind[l] >> 8)) : 0;
        int urun[MT_MAX_LAYERS], utotal[MT_MAX_LAYERS];
        cta_excl_scan_vec(units, urun, utotal, s_vec, n_layers);
#pragma unroll
        for (int l = 0; l < MT_MAX_LAYERS; ++l) {
            if (l >= n_layers) break;
            if (lo < hi_t) tile_prefix[(size_t)l * (T + 1) + lo] = urun[l];
            if (threadIdx.x == 0) tile_prefix[(size_t)l * (T + 1) + T] = utotal[l];
        }
        return;
    }
    for (int l = 0; l < n_layers; ++l) {
        int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        int usum = 0;
        for (int r = lo; r < hi_t; ++r) { const int t = tenant_at(br, l, r); usum += layer_units(br, tn, t, l, cnt[t], rows_per_unit); }
        int urun = cta_excl_scan(usum, s_warp, &total);
        for (int r = lo; r < hi_t; ++r) {
            const int t = tenant_at(br, l, r);
            prefix[r] = urun;
            urun += layer_units(br, tn, t, l, cnt[t], rows_per_unit);
        }
        if (threadIdx.x == 0) prefix[T] = total;
    }
}

// Pass 1 of a batch that needs several CTAs: per-block histogram of ids (blocks of kHistChunk requests; warp-level
// match, one shared atomic per group of equal ids), and the CTA that finishes LAST (a ticket counter; nobody waits)
// turns the block histograms into per-tenant exclusive prefixes over the blocks, the counts, the offsets and the
// per-layer unit prefixes.
__global__ void __launch_bounds__(kHistChunk)
bucket_hist_scan(const int32_t* __restrict__ ids, int n, int T, Brief br, int n_layers,
                 int rows_per_unit, LayerTileN tn, int32_t* block_hist, int32_t* counts, int32_t* __restrict__ offsets,
                 int32_t* __restrict__ tile_prefix, int32_t* ticket, int32_t* __restrict__ status, unsigned* grid_bar) {
    pdl_launch_dependents();
    pdl_wait();
    if (grid_bar && blockIdx.x == 0 && threadIdx.x < 8) grid_bar[threadIdx.x] = 0u;   // barrier counters of this call's conv launches
    extern __shared__ int32_t s_hist[];   // T + 1
    __shared__ int32_t s_warp[33];
    __shared__ int32_t s_vec[MT_MAX_LAYERS * 33];
    __shared__ int s_last;
    const int T1 = T + 1;
    for (int t = threadIdx.x; t < T1; t += blockDim.x) s_hist[t] = 0;
    __syncthreads();
    const int i = blockIdx.x * kHistChunk + threadIdx.x;
    if (i < n) {
        const int b = classify(ids[i], T, br);
        if (b == T) report_rejected(ids[i], i, T, br, status);
        const unsigned peers = __match_any_sync(__activemask(), b);
        if ((__ffs(peers) - 1) == (threadIdx.x & 31)) atomicAdd(&s_hist[b], __popc(peers));
    }
    __syncthreads();
    for (int t = threadIdx.x; t < T1; t += blockDim.x) block_hist[(size_t)blockIdx.x * T1 + t] = s_hist[t];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int prev = atomicAdd(ticket, 1);
        s_last = (prev == (int)gridDim.x - 1);
        if (s_last) *ticket = 0;               // ready for the next batch
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // per bucket (one thread each; neighbouring threads read neighbouring words): exclusive prefix over the blocks
    const int n_blocks = gridDim.x;
    int own_count = -1;                        // counts[threadIdx.x] when every bucket has a thread of its own
    for (int t = threadIdx.x; t < T1; t += blockDim.x) {
        int run = 0;
        int b = 0;
        for (; b + 16 <= n_blocks; b += 16) {      // sixteen independent loads in flight
            int v[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) v[k] = __ldcg(&block_hist[(size_t)(b + k) * T1 + t]);
#pragma unroll
            for (int k = 0; k < 16; ++k) { block_hist[(size_t)(b + k) * T1 + t] = run; run += v[k]; }
        }
        for (; b < n_blocks; ++b) {
            const int v = __ldcg(&block_hist[(size_t)b * T1 + t]);
            block_hist[(size_t)b * T1 + t] = run;
            run += v;
        }
        counts[t] = run;
        s_hist[t] = run;                       // the scan below reads counts by tenant rank: keep them on the SM
        own_count = run;
    }
    if (T1 > (int)blockDim.x) own_count = -1;
    else if ((int)threadIdx.x >= T1) own_count = 0;
    __syncthreads();
    scan_buckets(T, br, n_layers, rows_per_unit, tn, s_hist, offsets, tile_prefix, s_warp, s_vec, own_count);
}

struct ItemPtrs { WorkItem* v[8]; };

// Work item `item` of dense layer l: (tenant, row tile, column tile) and what the executor needs to know about it.
__device__ __forceinline__ WorkItem make_work_item(int item, int l, int T, const ModelDev* __restrict__ models,
                                                   const int32_t* order_row, const int32_t* __restrict__ offsets,
                                                   const int32_t* __restrict__ prefix, int tile_m, int row_scale) {
    int lo = 0, hi = T;   // largest rank r with prefix[r] <= item
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (prefix[mid] <= item) lo = mid; else hi = mid;
    }
    const int t = order_row[lo];               // lo is a rank in the layer's cost order
    const LayerDev& L = models[t].layer[l];
    const int seg0 = offsets[t] * row_scale, n_t = (offsets[t + 1] - offsets[t]) * row_scale;   // matrix rows of the tenant
    const int m_tiles = (n_t + tile_m - 1) / tile_m;
    const int local = item - prefix[lo];
    // Order of a tenant's items: column tiles in groups of kColGroup, inside a group row tile by row tile.  Items in
    // flight together (one per CTA) then share a few weight slabs AND a few activation row tiles, instead of one
    // weight slab and every row tile of the tenant: for segments of thousands of requests that halves what a wave
    // of CTAs pulls through L2.  Row tiles of one weight slab stay at most kColGroup items apart.
    constexpr int kColGroup = 8;
    const int n_tiles = (prefix[lo + 1] - prefix[lo]) / m_tiles;
    const int per_group = m_tiles * kColGroup;
    const int grp = local / per_group, rem = local - grp * per_group;
    const int gn = min(kColGroup, n_tiles - grp * kColGroup);
    const int m_tile = rem / gn, n_tile = grp * kColGroup + (rem - m_tile * gn);
    WorkItem w;
    w.row0 = seg0 + m_tile * tile_m;
    w.rows_valid = min(tile_m, n_t - m_tile * tile_m);
    w.n_tile = n_tile;
    w.k_blocks = L.k_blocks;
    w.w = L.w;
    w.bias = L.bias;
    w.N = L.N;
    w.relu = L.relu;
    w.t = t;
    w.flags = (l == models[t].n_layers - 1) ? kItemFinal : 0;    // models of one family may differ in depth
    return w;
}


// A batch that fits one CTA (n <= kSingleCtaMax): histogram, scans, stable scatter and the work-item expansion in
// ONE launch.  blockDim.x is 256 or 1024; the requests are taken in rounds of blockDim.x.
constexpr int kSingleCtaMax = 4096;

__global__ void __launch_bounds__(1024)
bucket_single_cta(const int32_t* __restrict__ ids, int n, int T, const ModelDev* __restrict__ models, Brief br, int n_layers,
                  int rows_per_unit, LayerTileN tn, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                  int32_t* __restrict__ tile_prefix, int32_t* __restrict__ perm, int32_t* __restrict__ inv,
                  ItemPtrs items, int32_t* __restrict__ status, unsigned* grid_bar) {
    pdl_launch_dependents();
    pdl_wait();
    if (grid_bar && threadIdx.x < 8) grid_bar[threadIdx.x] = 0u;   // barrier counters of this call's conv launches
    extern __shared__ int32_t s_mem[];          // s_cnt[T + 1], s_next[T + 1]
    __shared__ int32_t s_warp[33];
    __shared__ int32_t s_vec[MT_MAX_LAYERS * 33];
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
            const int b = classify(ids[i], T, br);
            bucket[r] = b;
            if (b == T) report_rejected(ids[i], i, T, br, status);
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
    {
        const int hi_t = min(hi, T);
        if (per == 1) {
            // one rank per thread: tenants of that rank, their shapes and their counts for all layers together
            const int r_own = min(lo, T - 1);
            int t_l[MT_MAX_LAYERS];
#pragma unroll
            for (int l = 0; l < MT_MAX_LAYERS; ++l) t_l[l] = (l < n_layers) ? tenant_at(br, l, r_own) : 0;
            LayerHead head[MT_MAX_LAYERS];
#pragma unroll
            for (int l = 0; l < MT_MAX_LAYERS; ++l) head[l] = (l < n_layers) ? load_head(br, tn, t_l[l], l) : LayerHead{-1, 0};
            int units[MT_MAX_LAYERS];
#pragma unroll
            for (int l = 0; l < MT_MAX_LAYERS; ++l)
                units[l] = (l < n_layers && lo < hi_t) ? units_of(head[l], s_cnt[t_l[l]], rows_per_unit, tn.v[l], tn.m[l], (tn.kind[l] >> 8)) : 0;
            int urun[MT_MAX_LAYERS], utotal[MT_MAX_LAYERS];
            cta_excl_scan_vec(units, urun, utotal, s_vec, n_layers);
#pragma unroll
            for (int l = 0; l < MT_MAX_LAYERS; ++l) {
                if (l >= n_layers) break;
                if (lo < hi_t) tile_prefix[(size_t)l * (T + 1) + lo] = urun[l];
                if (threadIdx.x == 0) tile_prefix[(size_t)l * (T + 1) + T] = utotal[l];
            }
        } else {
            for (int l = 0; l < n_layers; ++l) {
                int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
                int usum = 0;
                for (int r = lo; r < hi_t; ++r) { const int t = tenant_at(br, l, r); usum += layer_units(br, tn, t, l, s_cnt[t], rows_per_unit); }
                int urun = cta_excl_scan(usum, s_warp, &total);
                for (int r = lo; r < hi_t; ++r) {
                    const int t = tenant_at(br, l, r);
                    prefix[r] = urun;
                    urun += layer_units(br, tn, t, l, s_cnt[t], rows_per_unit);
                }
                if (threadIdx.x == 0) prefix[T] = total;
            }
        }
    }
    __syncthreads();
    // rounds in order, and inside a round the warps take turns: positions inside a bucket ascend with arrival index
#pragma unroll
    for (int r = 0; r < kSingleCtaMax / 256; ++r) {
        if (r >= rounds) break;
        const int i = r * nthr + threadIdx.x;
        const int b = bucket[r];
        // the lanes that hold a request, agreed on by the whole warp BEFORE the divergent branch: the ranks below
        // are only right if every such lane takes part in the match, which __activemask() would not promise
        const unsigned live = __ballot_sync(0xffffffffu, i < n);
        for (int w = 0; w < n_warps; ++w) {
            if (warp == w && i < n) {
                const unsigned peers = __match_any_sync(live, b);
                const int rank = __popc(peers & ((1u << lane) - 1u));
                const int pos = s_next[b] + rank;
                __syncwarp(live);
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
        // the layer's unit prefixes into shared memory (s_cnt is free by now): the search per item stays on the SM
        const int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        for (int t = threadIdx.x; t < T1; t += nthr) s_cnt[t] = prefix[t];
        __syncthreads();
        const int n_items = s_cnt[T];
        for (int item = threadIdx.x; item < n_items; item += nthr) out[item] = make_work_item(item, l, T, models, br.order + (size_t)l * br.ld, offsets, s_cnt, tn.m[l], (tn.kind[l] >> 8));
        __syncthreads();
    }
}

// Pass 2: stable position of every request (perm / inv), the move of its payload row into bucketed order
// (X_b[pos, :] = X[i, :]: the block's source rows are contiguous, so the reads stream), and the expansion of every
// dense layer's work list: item i of layer l -> (tenant, row tile, column tile) and everything the executor needs to
// know about it.  Row tiles of one weight slab are adjacent items, so concurrent CTAs share the slab in L2.
// A CTA takes kBucketChunk requests (small, so that the row move spreads over many SMs); CTAs beyond the last block
// of requests only expand work items.
__global__ void __launch_bounds__(kScatterThreads)
bucket_scatter_expand(const int32_t* __restrict__ ids, int n, int T, const ModelDev* __restrict__ models, Brief br,
                      const int32_t* __restrict__ block_hist, const int32_t* __restrict__ offsets,
                      int32_t* __restrict__ perm, int32_t* __restrict__ inv, const uint4* __restrict__ rows_src,
                      uint4* __restrict__ rows_dst, int row_vec, int dst_ld_vec, int n_layers, LayerTileN tn,
                      const int32_t* __restrict__ tile_prefix, ItemPtrs items, int all_layers_at_once) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ int32_t s_next[];   // T + 1: next free position of every bucket for this block; then s_pos[chunk]
    const int T1 = T + 1;
    int32_t* s_pos = s_next + T1;
    const int n_blocks = (n + kBucketChunk - 1) / kBucketChunk;
    if ((int)blockIdx.x < n_blocks) {
        // pass 1 counted blocks of kHistChunk requests; this CTA first counts the requests of its pass-1 block that
        // come before its own kBucketChunk
        const int chunk0 = blockIdx.x * kBucketChunk;
        const int hist_block = chunk0 / kHistChunk;
        for (int t = threadIdx.x; t < T1; t += blockDim.x)
            s_next[t] = offsets[t] + block_hist[(size_t)hist_block * T1 + t];
        __syncthreads();
        // (chunk0 - first id of the pass-1 block) is a multiple of kBucketChunk = 64: whole warps only
        // (at most kHistChunk / kScatterThreads rounds; the ids of all rounds are fetched first, then the tenant
        // table entries, so that each kind of load costs one round trip instead of one per round)
        constexpr int kRounds = kHistChunk / kScatterThreads;
        int pre_id[kRounds], pre_b[kRounds];
#pragma unroll
        for (int q = 0; q < kRounds; ++q) {
            const int i = hist_block * kHistChunk + q * kScatterThreads + (int)threadIdx.x;
            pre_id[q] = (i < chunk0) ? ids[i] : INT_MIN;
        }
#pragma unroll
        for (int q = 0; q < kRounds; ++q) pre_b[q] = (pre_id[q] == INT_MIN) ? -1 : classify(pre_id[q], T, br);
#pragma unroll
        for (int q = 0; q < kRounds; ++q) {
            if (pre_b[q] >= 0) {      // whole warps: the part before this CTA's requests is a multiple of 64 long
                const unsigned peers = __match_any_sync(__activemask(), pre_b[q]);
                if ((__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&s_next[pre_b[q]], __popc(peers));
            }
        }
        __syncthreads();
        const int i = chunk0 + threadIdx.x;
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const bool mine = threadIdx.x < kBucketChunk && i < n;
        const int b = mine ? classify(ids[i], T, br) : -1;
        // warps take turns in arrival order, so positions inside a bucket ascend with the arrival index
        // (the participating lanes are agreed on before the divergent branch; see bucket_single_cta)
        const unsigned live = __ballot_sync(0xffffffffu, mine);
        for (int w = 0; w < kBucketChunk / 32; ++w) {
            if (warp == w && mine) {
                const unsigned peers = __match_any_sync(live, b);
                const int rank = __popc(peers & ((1u << lane) - 1u));
                const int pos = s_next[b] + rank;
                __syncwarp(live);
                if (rank == 0) s_next[b] += __popc(peers);
                perm[pos] = i;
                inv[i] = pos;
                s_pos[threadIdx.x] = pos;
            }
            __syncthreads();
        }
        if (rows_src) {
            const int rows_here = min(kBucketChunk, n - chunk0);
            const uint4* src = rows_src + (size_t)chunk0 * row_vec;
            const int total = rows_here * row_vec;
            int idx = threadIdx.x;
            for (; idx + 3 * (int)blockDim.x < total; idx += 4 * blockDim.x) {      // four independent copies in flight
                uint4 v[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) v[k] = __ldg(src + idx + k * blockDim.x);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int e = idx + k * blockDim.x;
                    const int r = e / row_vec;
                    rows_dst[(size_t)s_pos[r] * dst_ld_vec + (e - r * row_vec)] = v[k];
                }
            }
            for (; idx < total; idx += blockDim.x) {
                const int r = idx / row_vec;
                rows_dst[(size_t)s_pos[r] * dst_ld_vec + (idx - r * row_vec)] = __ldg(src + idx);
            }
        }
        __syncthreads();      // s_next is reused below
    }
    // work items: the layers' unit prefix sums (and their tenant orders) go to shared memory first, so the search per
    // item stays on the SM
    if (all_layers_at_once) {
        // every dense layer's rows at once and ONE loop over the items of all layers: the chain of dependent loads
        // (prefixes -> tenant -> its table entry and offsets) is paid once, not once per layer
        int32_t* s_all = s_next;                     // per item layer q: prefix row [T1], then order row [T1]
        int n_q = 0;
        for (int l = 0; l < n_layers; ++l) {
            if (!items.v[l]) continue;
            const int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
            const int32_t* ord = br.order + (size_t)l * br.ld;
            int32_t* row = s_all + (size_t)n_q * 2 * T1;
            for (int t = threadIdx.x; t < T1; t += blockDim.x) { row[t] = prefix[t]; row[T1 + t] = (t < T) ? __ldg(ord + t) : 0; }
            ++n_q;
        }
        __syncthreads();
        int done = 0, q = 0;                         // items of the layers before the current one
        for (int l = 0; l < n_layers; ++l) {
            WorkItem* out = items.v[l];
            if (!out) continue;
            const int32_t* row = s_all + (size_t)q * 2 * T1;
            const int total = row[T];
            // global item numbers [done, done + total) belong to this layer; a thread's items keep the grid stride
            const int first = blockIdx.x * blockDim.x + threadIdx.x, stride = gridDim.x * blockDim.x;
            int g = first + ((done > first) ? ((done - first + stride - 1) / stride) * stride : 0);
            for (; g < done + total; g += stride)
                out[g - done] = make_work_item(g - done, l, T, models, row + T1, offsets, row, tn.m[l], (tn.kind[l] >> 8));
            done += total;
            ++q;
        }
        return;
    }
    for (int l = 0; l < n_layers; ++l) {
        WorkItem* out = items.v[l];
        if (!out) continue;
        const int32_t* prefix = tile_prefix + (size_t)l * (T + 1);
        for (int t = threadIdx.x; t < T1; t += blockDim.x) s_next[t] = prefix[t];
        __syncthreads();
        const int total = s_next[T];
        for (int item = blockIdx.x * blockDim.x + threadIdx.x; item < total; item += gridDim.x * blockDim.x)
            out[item] = make_work_item(item, l, T, models, br.order + (size_t)l * br.ld, offsets, s_next, tn.m[l], (tn.kind[l] >> 8));
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

// A kernel that does nothing but take part in the programmatic dependent launch chain like every kernel of the path:
// `count` of them back to back measure what one link of such a chain costs at least (the launch floor).
__global__ void empty_chain_kernel() {
    pdl_launch_dependents();
    pdl_wait();
}

void launch_empty_chain(int count, cudaStream_t s) {
    for (int i = 0; i < count; ++i) launch_pdl(empty_chain_kernel, dim3(1), dim3(32), 0, s);
    g_kernel_launches -= (unsigned long long)count;    // not kernels of the inference path
}

// ------------------------------------------------------------------------------------------ launchers
static int grid_for(long long total, int threads, int sm_count) {
    long long blocks = (total + threads - 1) / threads;
    const long long cap = (long long)sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

constexpr size_t kScatterSmemMax = 96 * 1024;      // two CTAs of the scatter pass still fit an SM

cudaError_t configure_bucketing() {
    return cudaFuncSetAttribute(bucket_scatter_expand, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kScatterSmemMax);
}

void launch_bucketing(const BucketArgs& a, cudaStream_t s) {
    const int n_blocks = (a.n + kBucketChunk - 1) / kBucketChunk;
    const int n_hist_blocks = (a.n + kHistChunk - 1) / kHistChunk;
    const size_t smem = sizeof(int32_t) * (size_t)(a.T + 1);
    LayerTileN tn;
    for (int l = 0; l < 8; ++l) { tn.v[l] = a.tile_n[l] > 0 ? a.tile_n[l] : BN; tn.m[l] = a.tile_m[l] > 0 ? a.tile_m[l] : BM; tn.kind[l] = (a.kind[l] & 0xff) | ((a.row_scale[l] > 0 ? a.row_scale[l] : 1) << 8); }
    Brief br{a.brief, a.brief_ld, a.order};
    ItemPtrs ip;
    for (int l = 0; l < 8; ++l) ip.v[l] = a.items[l];
    // measured: one CTA wins up to a few hundred requests; beyond that its serial scatter and the item expansion
    // by a single CTA cost more than the extra launches of the multi-CTA path
    // (a pointwise conv multiplies the rows, and with them the work items one CTA would have to expand)
    int max_scale = 1;
    for (int l = 0; l < 8; ++l) if (a.row_scale[l] > max_scale) max_scale = a.row_scale[l];
    if (a.n <= 512 && a.T + 1 <= 4096 && (long long)a.n * max_scale <= 8192) {
        const int threads = (a.n <= 256) ? 256 : 1024;
        launch_pdl(bucket_single_cta, dim3(1), dim3(threads), 2 * smem, s, a.ids, a.n, a.T, a.models, br, a.n_layers, a.rows_per_unit, tn, a.counts,
                                                      a.offsets, a.tile_prefix, a.perm, a.inv, ip, a.status, a.grid_bar);
        return;
    }
    launch_pdl(bucket_hist_scan, dim3(n_hist_blocks), dim3(kHistChunk), smem, s, a.ids, a.n, a.T, br, a.n_layers, a.rows_per_unit, tn,
               a.block_hist, a.counts, a.offsets, a.tile_prefix, a.ticket, a.status, a.grid_bar);
    const int grid2 = n_blocks > a.item_grid ? n_blocks : a.item_grid;
    // shared memory: the scatter's positions, or (larger) prefix and order rows of every layer that has work items
    int item_layers = 0;
    for (int l = 0; l < a.n_layers && l < 8; ++l) item_layers += a.items[l] ? 1 : 0;
    const size_t smem_scatter = smem + sizeof(int32_t) * kBucketChunk;
    const size_t smem_items = sizeof(int32_t) * 2 * (size_t)(a.T + 1) * item_layers;
    const int at_once = (item_layers > 1 && smem_items <= kScatterSmemMax) ? 1 : 0;
    launch_pdl(bucket_scatter_expand, dim3(grid2), dim3(kScatterThreads), (at_once && smem_items > smem_scatter) ? smem_items : smem_scatter, s,
               a.ids, a.n, a.T, a.models, br,
               a.block_hist, a.offsets, a.perm, a.inv, (const uint4*)a.rows_src, (uint4*)a.rows_dst, a.row_bytes / 16,
               a.dst_ld_bytes / 16, a.n_layers, tn, a.tile_prefix, ip, at_once);
}

void launch_gather_rows(const void* src, const int32_t* perm, int n, int row_bytes, void* dst, int dst_ld_bytes,
                        int sm_count, cudaStream_t s) {
    const int row_vec = row_bytes / 16;
    launch_pdl(gather_rows, dim3(grid_for((long long)n * row_vec, 256, sm_count)), dim3(256), 0, s,
        (const uint4*)src, perm, n, row_vec, (uint4*)dst, dst_ld_bytes / 16);
}

}  // namespace mt

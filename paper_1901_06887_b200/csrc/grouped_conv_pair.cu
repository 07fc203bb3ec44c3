// Grouped 3x3 convolution executor, CTA-pair form (images whose padded row length is 64 pixels, i.e. the 56 x 56
// workload): the same implicit GEMM and tap pairing as grouped_conv.cu,
//     Y[r, y, x, o] = act(b_t[o] + sum_{ky,kx,c} X[r, y+ky-1, x+kx-1, c] * W_t[o, ky, kx, c]),
// but two CTAs of a cluster (two SMs) work in lockstep on the same strip of TWO images of one tenant, and ONE
// thread of the leader CTA issues tcgen05.mma.cta_group::2 (M = 256: 128 pixels of each image) for both.
//
// Why: with 64 output channels an instruction is short and bound by the operand reads from shared memory (an
// M = 128 x N = 64 x K = 16 step reads 4 KiB of pixels for 32 cycles of tensor work).  A pair instruction lets each CTA
// hold only its share of the B operand: for the N = 64 instructions its 32 output channels of the tap, for the paired
// N = 128 instructions one of the two stacked tap tiles (rank 0: W(2,kx), rank 1: W(0,kx)); 60 KiB per CTA instead of
// 72, which is what makes room for the ring of input blocks below, and half the B bytes per instruction.  The issuing
// thread's cost per instruction is the same as in the one-CTA form (half as many threads issue half as many each).
//
// Synchronisation inside the pair (every wait bounded, as everywhere):
//   bfull[k]   in the leader: announces the bytes of BOTH CTAs' loads of a block of two image rows; both report there;
//   bempty[k]  in each CTA: its own epilogue releases its own blocks;
//   tfull[a]   in both CTAs, signalled together by a multicast commit: each CTA drains its own 128 accumulator rows;
//   tempty[a]  in the leader: 16 arrivals (one per epilogue warp, 8 local and 8 remote);
//   wfull      in each CTA for its own weight image; the peer then arrives on wpeer in the leader;
//   wempty     in both CTAs, multicast commit once every MMA on the old weights is done.
// Input staging.  The image is fetched in blocks of two padded rows (128 pixels, 16 KiB, zero fill outside the image
// as the padding): block b of an image holds input rows 2b-1 and 2b, so the tile of output rows 2i, 2i+1 reads block
// i (tap row 0), block i shifted by one row (tap row 1: second row of block i, first row of block i+1) and block i+1
// (tap row 2).  Blocks go round a ring of eight slots in load order, so consecutive blocks are neighbours in shared
// memory and a shifted operand simply runs on into the next slot; behind the last slot sits a copy of the first row
// of the block in slot 0 for the operand that starts in the last slot.  Nothing is fetched twice (a strip with its
// own halo re-read half of its rows), a block is released as soon as the tile below it has been issued and
// completed, and loads run six tiles ahead of the tensor pipe instead of one or two strips.
// The two CTAs meet at a cluster barrier before they exit.  A tenant with an odd number of images leaves the peer
// of its last pair a copy of the leader's image, computed and not stored.
//
// The paper does not define convolution; it only names a catalogue of standard layers (Sec. 1.1, Sec. 3.1).
#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kCpThreads = 320;
constexpr int kCpEpiThreads = 256;
constexpr int kCpN = 64;                                  // output channels
constexpr int kCpHalfTap = 32 * BK * 2;                   // 4 KiB: 32 output channels x 64 input channels
constexpr int kCpFullTap = 64 * BK * 2;                   // 8 KiB
constexpr int kOffMid = 0;                                // ky = 1 taps, this CTA's 32 output channels, kx = 0..2
constexpr int kOffPair = 3 * kCpHalfTap;                  // stacked pairs: rank 0 holds W(2,kx), rank 1 W(0,kx)
constexpr int kOffBot = kOffPair + 3 * kCpFullTap;        // ky = 2 taps alone, this CTA's 32 output channels
constexpr int kOffTop = kOffBot + 3 * kCpHalfTap;         // ky = 0 taps alone
static_assert(kOffTop + 3 * kCpHalfTap == kConvPairWeightBytes, "weight image layout");
constexpr int kCpRing = 8;                                // slots of the block ring
constexpr int kCpBlockBytes = 2 * 64 * 128;               // two padded rows of 64 pixels x 64 channels
constexpr int kCpGhostBytes = 64 * 128 + 1024;            // first row of the block in slot 0, again, behind the last slot
constexpr int kCpSlots = 8;                               // TMEM ring: 8 accumulators of 64 columns
constexpr int kCpBarBytes = 2048;
constexpr int kCpRecords = 16;
constexpr int kCpOutStageBytes = 8 * 2048;                // per epilogue warp: 32 pixels x 64 bytes
// the launch's own bucketing results (small batches): offsets (T + 2), unit prefixes (T + 1), perm (n)
constexpr int kCpSortBytes = 4 * ((kConvSelfBucketMaxT + 2) + (kConvSelfBucketMaxT + 1) + kConvSelfBucketMaxN + 13);
constexpr int kCpSmemBytes = kConvPairWeightBytes + kCpRing * kCpBlockBytes + kCpGhostBytes + kCpOutStageBytes + kCpBarBytes +
                             kCpSortBytes + 1024;
static_assert(kCpSmemBytes <= 227 * 1024, "shared memory of the pair conv executor");
static_assert(16 * (kConvSelfBucketMaxT + 1) * 4 <= kCpRing * kCpBlockBytes, "chunk histograms borrow the block ring");

__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(leader_bar)
        : "memory");
}

struct PairStrip {
    int t, j, y0, strip_in_image, dummy;
};

// Consecutive conv layers of one geometry run in ONE launch (p.n_stack of them, from layer p.layer on): every cluster
// keeps its range of units through all layers, and between two layers all CTAs meet at a grid-wide barrier (a counter
// in global memory, every wait bounded) - a layer boundary inside a launch costs a few microseconds, one between two
// launches about three times that, since no CTA of the next launch can start while one of this launch holds its SM's
// shared memory.  The next layer's first weights are requested before the barrier.
// kSkip: the launch has layers with identity shortcuts (ConvArgs::skip); without it the epilogue carries none of that
// code - its registers and the predicated loads cost the plain path 5 % when they were compiled in unconditionally.
template <bool kSkip>
__global__ void __launch_bounds__(kCpThreads, 1)
grouped_conv3x3_pair_kernel(const __grid_constant__ ConvStackMaps maps, const ConvArgs p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t w_smem = base;
    const uint32_t ring0 = base + kConvPairWeightBytes;           // kCpRing blocks, then the ghost row
    const uint32_t ghost0 = ring0 + kCpRing * kCpBlockBytes;
    // output staging: one 2 KiB region per epilogue warp (32 pixels x 32 channels), the source of its TMA stores
    const uint32_t out_stage0 = ghost0 + kCpGhostBytes;
    uint8_t* out_stage_ptr = smem + kConvPairWeightBytes + kCpRing * kCpBlockBytes + kCpGhostBytes;
    const uint32_t bar0 = out_stage0 + kCpOutStageBytes;
    uint8_t* bar_ptr = out_stage_ptr + kCpOutStageBytes;
    auto bfull_bar = [&](int k) { return bar0 + 8u * k; };
    auto bempty_bar = [&](int k) { return bar0 + 8u * (kCpRing + k); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kCpRing + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kCpRing + kCpSlots + a); };
    const uint32_t wfull_bar = bar0 + 8u * (2 * kCpRing + 2 * kCpSlots);
    const uint32_t wempty_bar = wfull_bar + 8u;
    const uint32_t wpeer_bar = wfull_bar + 16u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * (2 * kCpRing + 2 * kCpSlots + 3));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    static_assert(8 * (2 * kCpRing + 2 * kCpSlots + 3) + 8 <= 320, "barriers, TMEM address and abort flag come before the bias");
    float* s_bias = reinterpret_cast<float*>(bar_ptr + 512);          // 64 floats
    // Per-strip record, producer -> epilogue of the same CTA: x = flags (1 new tenant, 2 the strip starts a segment, 8 copy
    // of the leader's image: do not store), y = image (bucketed index), z = first output row, w = tenant.
    int4* s_rec = reinterpret_cast<int4*>(bar_ptr + 768);             // kCpRecords x 16 bytes
    float* s_pool = reinterpret_cast<float*>(bar_ptr + 1024);         // 8 warps x 32 channel sums (fused pooling)
    int* s_first = reinterpret_cast<int*>(bar_ptr + 320);             // the first unit's tenant: id, units, requests
    const uint16_t** s_first_w = reinterpret_cast<const uint16_t**>(bar_ptr + 352);   // ... and its weight block
    int32_t* const s_off = reinterpret_cast<int32_t*>(bar_ptr + kCpBarBytes);        // own bucketing: offsets, T + 2
    int32_t* const s_prefix = s_off + kConvSelfBucketMaxT + 2;                        // ... unit prefixes, T + 1
    int32_t* const s_perm = s_prefix + kConvSelfBucketMaxT + 1;                       // ... perm, n

    if (!p.late_trigger) pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader (issues the MMAs), 1 = peer
    const bool is_leader = (rank == 0);
    if (threadIdx.x == 0) {
        for (int k = 0; k < kCpRing; ++k) { mbar_init(bfull_bar(k), 1); mbar_init(bempty_bar(k), 1); }
        for (int a = 0; a < kCpSlots; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * (kCpEpiThreads / 32)); }
        mbar_init(wfull_bar, 1);
        mbar_init(wempty_bar, 1);
        mbar_init(wpeer_bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
        for (int k = 0; k < p.n_stack; ++k) {
            prefetch_tensormap(&maps.x2[k]);
            prefetch_tensormap(&maps.x1[k]);
            prefetch_tensormap(&maps.y[k]);
        }
    }
    // Operands shifted by one or two pixels read a little past what the copies wrote, whatever the previous kernel left
    // there: rows of the product that belong to pad columns, which are neither stored nor pooled.
    if (warp == 1) {                                  // the same warp of both CTAs
        tmem_alloc_pair(smem_u32(tmem_slot), kCpSlots * kCpN);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Everything above overlapped the previous kernel's tail; its results are needed from here on.  Behind another conv
    // layer of the same call (early_lookup) the wait comes a little later: the bucketing results read next are older
    // than that layer's own dependency, which it let pass before it allowed this launch to start.
    if (!p.early_lookup) pdl_wait();
    // Where the bucketing results come from: the arrays a bucketing launch filled, or - small batches - this CTA's own
    // stable counting sort of the ids (every CTA of the launch repeats it; it costs a few microseconds where a launch of
    // its own costs about twenty, a twelfth of a step on 56 x 56 images).
    const int32_t* tile_prefix = p.tile_prefix;
    const int32_t* offsets = p.offsets;
    const int32_t* perm_first = p.perm;              // the launch's first layer reads the caller's images through it
    const bool self_bucket = p.ids != nullptr;
    if (self_bucket) {
        const int T = p.T, T1 = p.T + 1, n = p.n;
        const int n_chunks = (n + 31) >> 5;           // chunk c = requests [32c, 32c + 32)
        int32_t* s_chist = reinterpret_cast<int32_t*>(smem + kConvPairWeightBytes);   // [chunks][T1], in the idle block ring
        for (int k = threadIdx.x; k < n_chunks * T1; k += kCpThreads) s_chist[k] = 0;
        __syncthreads();
        constexpr int kWarps = kCpThreads / 32;
        constexpr int kMaxOwn = (kConvSelfBucketMaxN / 32 + kWarps - 1) / kWarps;     // chunks a warp may own
        int own_b[kMaxOwn], own_rank[kMaxOwn];
#pragma unroll
        for (int q = 0; q < kMaxOwn; ++q) {
            own_b[q] = -1; own_rank[q] = 0;
            const int c = warp + kWarps * q;
            const int i = c * 32 + lane;
            if (c < n_chunks && i < n) {
                const int id = p.ids[i];
                const int alive = (id < 0 || id >= T) ? 0 : p.models[id].alive;     // 1 resident, 2 registered but evicted
                const int b = alive == 1 ? id : T;
                if (b == T && blockIdx.x == 0) {
                    atomicCAS(&p.status[ST_CODE], MT_OK, alive == 2 ? MT_ERR_NOT_RESIDENT : MT_ERR_BAD_MODEL_ID);
                    atomicMin(&p.status[ST_BAD_INDEX], i);
                }
                // rank among the chunk's requests of the same bucket, from the warp's match mask (the lanes with a
                // request are lanes 0 .. n - 32c - 1)
                const unsigned live = (n - c * 32 >= 32) ? 0xffffffffu : ((1u << (n - c * 32)) - 1u);
                const unsigned peers = __match_any_sync(live, b);
                const int rank_in_chunk = __popc(peers & ((1u << lane) - 1u));
                if (rank_in_chunk == 0) s_chist[c * T1 + b] = __popc(peers);
                own_b[q] = b; own_rank[q] = rank_in_chunk;
            }
        }
        __syncthreads();
        for (int t = threadIdx.x; t < T1; t += kCpThreads) {      // per bucket: exclusive prefix over the chunks; the count
            int run = 0;
            for (int c = 0; c < n_chunks; ++c) {
                const int v = s_chist[c * T1 + t];
                s_chist[c * T1 + t] = run;
                run += v;
            }
            s_prefix[t] = run;                                    // (counts for now)
        }
        __syncthreads();
        if (warp == 0) {                                          // offsets and unit prefixes over the buckets
            const int per = (T1 + 31) >> 5;
            const int lo = min(lane * per, T1), hi = min(lo + per, T1);
            int sum = 0, usum = 0;
            for (int t = lo; t < hi; ++t) { sum += s_prefix[t]; if (t < T) usum += ((s_prefix[t] + 1) >> 1) * p.strips_per_image; }
            int incl = sum, uincl = usum;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, incl, d);
                const int uu = __shfl_up_sync(0xffffffffu, uincl, d);
                if (lane >= d) { incl += u; uincl += uu; }
            }
            int run = incl - sum, urun = uincl - usum;
            for (int t = lo; t < hi; ++t) {
                const int cnt = s_prefix[t];
                if (blockIdx.x == 0) p.counts_out[t] = cnt;
                s_off[t] = run; run += cnt;
                if (t < T) { s_prefix[t] = urun; urun += ((cnt + 1) >> 1) * p.strips_per_image; }
            }
            __syncwarp();
            if (lane == 31) { s_off[T1] = incl; s_prefix[T] = uincl; }
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxOwn; ++q) {
            const int c = warp + kWarps * q;
            const int i = c * 32 + lane;
            if (own_b[q] >= 0) {
                const int pos = s_off[own_b[q]] + s_chist[c * T1 + own_b[q]] + own_rank[q];
                s_perm[pos] = i;
                if (blockIdx.x == 0) { p.perm_out[pos] = i; p.inv_out[i] = pos; }
            }
        }
        if (blockIdx.x == 0) {        // for the launches that follow (more conv layers, the pool and the head)
            for (int t = threadIdx.x; t <= T1; t += kCpThreads) p.offsets_out[t] = s_off[t];
            for (int k = threadIdx.x; k < p.prefix_rows * T1; k += kCpThreads) p.prefix_out[k] = s_prefix[k % T1];
        }
        __syncthreads();              // the block ring is free again; s_off, s_prefix and s_perm are complete
        tile_prefix = s_prefix;
        offsets = s_off;
        perm_first = s_perm;
    }
    // contiguous range of pair-strips for this cluster: unit = (tenant, pair of images, strip of 2 tiles)
    const int total = tile_prefix[p.T];
    const int n_pairs = gridDim.x >> 1, pair_id = blockIdx.x >> 1;
    int s_begin = (int)(((long long)total * pair_id) / n_pairs);
    int s_end = (int)(((long long)total * (pair_id + 1)) / n_pairs);
    constexpr int Wp = 64;
    const int TS = p.tiles_per_strip;
    // Ranges of equal COST rather than equal length: a tenant border inside a range stops the tensor pipe while the
    // new weights come in, which is worth about p.border_units units of work (measured: the pairs that cross a border
    // issue for 3 us longer than the others, and everybody waits for them at the end of each layer).  Every tenant
    // border is charged that many units and the ranges split the total evenly; a range edge that falls into a border's
    // charge snaps to the border itself, so neither neighbour pays for it.  The cost prefix over the tenants is built in
    // shared memory (the output staging area is free before the first tile); more tenants than fit there keep the
    // equal-length split.
    constexpr int kMaxBalancedTenants = kCpOutStageBytes / 4 - 8;
    if (p.border_units > 0 && p.T <= kMaxBalancedTenants && total > 0) {
        int* s_cost = reinterpret_cast<int*>(out_stage_ptr);          // s_cost[t] = cost position of tenant t's first unit
        if (warp == 2) {
            // lane l scans its share of the tenants in order; the shares' border counts are then scanned across the warp
            const int per = (p.T + 31) >> 5;
            const int lo = min(lane * per, p.T), hi = min(lo + per, p.T);
            int mine = 0;
            for (int t = lo; t < hi; ++t) mine += (tile_prefix[t + 1] > tile_prefix[t]) ? 1 : 0;
            int incl = mine;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int u = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += u;
            }
            int before = incl - mine;                                 // tenants with units in front of this lane's share
            for (int t = lo; t < hi; ++t) {
                const int first = tile_prefix[t];
                s_cost[t] = first + p.border_units * before;
                before += (tile_prefix[t + 1] > first) ? 1 : 0;
            }
            if (lane == 31) s_cost[p.T] = total + p.border_units * max(before - 1, 0);   // total cost (the first tenant has no border)
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const long long total_cost = s_cost[p.T];
            // unit at which cost position c is reached: the last tenant whose border charge starts at or before c
            auto unit_at = [&](long long c) {
                if (c <= 0) return 0;
                if (c >= total_cost) return total;
                int lo = 0, hi = p.T;                                  // largest t with s_cost[t] - border_units <= c
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if ((long long)s_cost[mid] - p.border_units <= c) lo = mid; else hi = mid;
                }
                const int first = tile_prefix[lo], units = tile_prefix[lo + 1] - first;
                const long long into = c - s_cost[lo];
                return first + (int)min((long long)units, max(into, 0LL));
            };
            s_first[6] = unit_at(total_cost * pair_id / n_pairs);
            s_first[7] = unit_at(total_cost * (pair_id + 1) / n_pairs);
        }
        __syncthreads();
        s_begin = s_first[6];
        s_end = s_first[7];
        __syncthreads();                                              // the staging area goes back to the epilogue
    }

    // The first unit's tenant, its range of units and requests and its weight image: every thread looks at a few
    // tenants, all loads independent of one another, instead of a binary search of dependent loads by each role -
    // this sits between the previous layer's end and the first MMA.
    if (s_begin < s_end) {
        for (int i = threadIdx.x; i < p.T; i += blockDim.x) {
            const int lo = tile_prefix[i], hi = tile_prefix[i + 1];
            const int seg = offsets[i], seg_hi = offsets[i + 1];
            const uint16_t* w = p.models[i].layer[p.layer].w;
            if (lo <= s_begin && s_begin < hi) {
                s_first[0] = i; s_first[1] = lo; s_first[2] = hi; s_first[3] = seg; s_first[4] = seg_hi - seg;
                *s_first_w = w;
            }
        }
    }
    __syncthreads();
    if (p.early_lookup) {
        // the first weights (unchanged since registration) are on their way while the previous layer drains: at the
        // start of a launch they are what the first MMA waits for longest
        if (threadIdx.x == 0 && s_begin < s_end) {
            mbar_expect_tx(wfull_bar, kConvPairWeightBytes);
            bulk_load(w_smem, *s_first_w + kConvPairImageOffset + (size_t)rank * (kConvPairWeightBytes / 2), kConvPairWeightBytes, wfull_bar);
        }
        pdl_wait();
    }
    if (p.late_trigger) pdl_launch_dependents();

    // pair-strip -> (tenant, this CTA's image, first row); units of one tenant are consecutive: its range is cached
    int cur_t = -1, cur_lo = 0, cur_hi = 0, cur_seg = 0, cur_n = 0;
    if (s_begin < s_end) { cur_t = s_first[0]; cur_lo = s_first[1]; cur_hi = s_first[2]; cur_seg = s_first[3]; cur_n = s_first[4]; }
    auto locate = [&](int s) {
        if (s < cur_lo || s >= cur_hi) {
            int lo = 0, hi = p.T;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (tile_prefix[mid] <= s) lo = mid; else hi = mid;
            }
            cur_t = lo; cur_lo = tile_prefix[lo]; cur_hi = tile_prefix[lo + 1];
            cur_seg = offsets[lo]; cur_n = offsets[lo + 1] - cur_seg;
        }
        PairStrip c;
        const int local = s - cur_lo;
        const int pr = local / p.strips_per_image;
        const int mine = 2 * pr + (int)rank;
        c.t = cur_t;
        c.dummy = mine >= cur_n;
        c.j = cur_seg + (c.dummy ? 2 * pr : mine);
        c.strip_in_image = local - pr * p.strips_per_image;
        c.y0 = c.strip_in_image * p.R;
        return c;
    };

    // End of layer k of the stack, called by every thread of the CTA at a converged point: this CTA's outputs are
    // complete and visible (the storing lanes have waited for their tensor stores), then one thread arrives at the
    // grid-wide counter and waits, for a bounded time, until all CTAs of the launch have (p.grid_bar was zeroed by the
    // bucketing kernel of this call).  Afterwards the layer's outputs may be read by anyone, also through TMA.
    auto layer_sync = [&](int k) {
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();            // cumulative: covers what the CTA's other threads wrote before the barrier above
            atomicAdd(p.grid_bar, 1u);
            const unsigned want = (unsigned)(k + 1) * gridDim.x;
            const uint64_t t0 = global_timer_ns();
            unsigned seen;
            uint32_t it = 0;
            while (true) {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.grid_bar) : "memory");
                if (seen >= want) break;
                if ((++it & 0xFF) == 0) {
                    if (*abort_flag) break;
                    if (global_timer_ns() - t0 > kWaitLimitNs) {
                        *abort_flag = 1;
                        if (atomicCAS(&p.status[ST_CODE], MT_OK, MT_ERR_TIMEOUT) == MT_OK) p.status[ST_WHERE] = 60;
                        break;
                    }
                }
            }
            __threadfence();
            asm volatile("fence.proxy.async;" ::: "memory");
        }
        __syncthreads();
    };
    const int n_stack = p.n_stack;

    if (warp == 0) {
        // ------------------------------------------------------------------- TMA producer (lane 0 of both CTAs)
        int w_loads = 0, w_tenant = -1;
        int nb = 0;                     // blocks armed so far; block b goes to slot b % kCpRing
        bool ok = true;
        bool first_weights_out = p.early_lookup != 0;      // the stack's first weights were requested before the wait
        for (int k = 0; k < n_stack; ++k) {
          if (lane == 0 && ok && !*abort_flag) {
            const int layer = p.layer + k;
            const CUtensorMap* const tmap_x = &maps.x2[k];
            const CUtensorMap* const tmap_x1 = &maps.x1[k];
            const int32_t* const perm = (k == 0) ? perm_first : nullptr;
            if (k > 0) w_tenant = -1;   // same tenants, other weights
            {
            // (indentation kept from the single-layer form)
            
            const uint32_t wpeer_leader = map_to_cta(wpeer_bar, 0);
            const uint32_t bfull_leader0 = map_to_cta(bfull_bar(0), 0);
            auto start_weights = [&](int t, const uint16_t* w) {
                // The issuer releases the old weights when it reaches the tenant's first strip in its own order.
                if (w_loads > 0 && !mbar_wait_spin(wempty_bar, (uint32_t)((w_loads - 1) & 1), abort_flag, p.status, 51, 64)) return false;
                mbar_expect_tx(wfull_bar, kConvPairWeightBytes);
                bulk_load(w_smem, w + kConvPairImageOffset + (size_t)rank * (kConvPairWeightBytes / 2), kConvPairWeightBytes, wfull_bar);
                w_tenant = t;
                return true;
            };
            auto announce_weights = [&]() {
                if (!is_leader) {      // tell the leader's issuer once this CTA's share has landed
                    if (!mbar_wait(wfull_bar, (uint32_t)(w_loads & 1), abort_flag, p.status, 53)) return false;
                    mbar_arrive_remote(wpeer_leader);
                }
                ++w_loads;
                return true;
            };
            for (int s = s_begin; ok && s < s_end; ++s) {
                const PairStrip c = locate(s);
                const bool new_tenant = (c.t != w_tenant);
                const int img = perm ? perm[c.j] : c.j;
                const bool seg_start = (s == s_begin) || c.strip_in_image == 0;
                // the very first weights go out before the first blocks: the first MMA needs both, and this is the
                // larger copy (later ones must wait for the issuer to let go of the old weights, so the blocks go first)
                const bool weights_first = new_tenant && s == s_begin;
                if (weights_first) {
                    if (first_weights_out) w_tenant = c.t;     // requested before the dependency wait / the layer barrier
                    else if (!start_weights(c.t, k == 0 ? *s_first_w : p.models[c.t].layer[layer].w)) { ok = false; break; }
                }
                // published to this CTA's epilogue with the strip's first block (the issuer starts the strip's first
                // tile only after that block has landed)
                s_rec[(s - s_begin) & (kCpRecords - 1)] =
                    make_int4((new_tenant ? 1 : 0) | (seg_start ? 2 : 0) | (c.dummy ? 8 : 0), c.j, c.y0, c.t);
                // blocks of the strip: kb = 0 is the block of its first tile (loaded by the strip above unless the strip
                // starts a segment), kb = k the block of tile k, kb = TS the block under its last tile
                for (int kb = seg_start ? 0 : 1; kb <= TS; ++kb) {
                    const int slot = nb & (kCpRing - 1);
                    if (!mbar_wait(bempty_bar(slot), (uint32_t)(((nb / kCpRing) & 1) ^ 1), abort_flag, p.status, 52)) { ok = false; break; }
                    const int y_in = c.y0 + 2 * kb - 1;              // first input row of the block
                    const uint32_t bytes = kCpBlockBytes + (slot == 0 ? 64u * 128u : 0u);
                    if (is_leader) mbar_expect_tx(bfull_bar(slot), 2u * bytes);   // both CTAs' bytes
                    tma_load_4d_pair(ring0 + slot * kCpBlockBytes, tmap_x, 0, -1, y_in, img, bfull_leader0 + 8u * slot);
                    if (slot == 0) tma_load_4d_pair(ghost0, tmap_x1, 0, -1, y_in, img, bfull_leader0);
                    ++nb;
                }
                if (!ok) break;
                if (new_tenant && !weights_first && !start_weights(c.t, p.models[c.t].layer[layer].w)) { ok = false; break; }
                if (new_tenant && !announce_weights()) { ok = false; break; }
            }
            // the next layer's first weights (they do not depend on this layer's results) go out before the barrier
            first_weights_out = false;
            if (ok && k + 1 < n_stack && s_begin < s_end) {
                const int t0 = s_first[0];
                if (start_weights(t0, p.models[t0].layer[layer + 1].w)) first_weights_out = true; else ok = false;
            }
            }
          }
          __syncwarp();
          if (k + 1 < n_stack) layer_sync(k);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------- MMA issuer (leader CTA; the peer's warp 1
        // only takes part in the layer barriers).  The whole warp walks the loop (addresses and descriptors stay
        // warp-uniform); one elected lane issues.
        const bool leader = elect_one();
            const uint32_t tb = __shfl_sync(0xffffffffu, *tmem_slot, 0);
            constexpr uint32_t idesc64 = make_idesc_bf16(2 * BM, kCpN);
            constexpr uint32_t idesc128 = make_idesc_bf16(2 * BM, 2 * kCpN);
            int g = 0;                      // tiles started so far by this pair; tile g lives in TMEM slot g % kCpSlots
            int bc = 0;                     // load-order number of the block with the current tile's first input rows
            int w_loads = 0;
            bool w_released = false;        // the current weights were handed back at the end of a layer
            bool ok = true;
            const uint32_t w_lo = desc_lo(w_smem);
            const uint32_t ring_lo = desc_lo(ring0);
            constexpr uint32_t kHalfLo = kCpHalfTap >> 4, kFullLo = kCpFullTap >> 4;
            constexpr uint32_t kMidLo = kOffMid >> 4, kPairLo = kOffPair >> 4, kBotLo = kOffBot >> 4, kTopLo = kOffTop >> 4;
            constexpr uint32_t kPixLo = 128 >> 4;                // one pixel (128 bytes) further
            constexpr uint32_t kBlockLo = kCpBlockBytes >> 4;
            // four K steps of one 128-pixel block (of each CTA) against one tap operand
            auto issue = [&](uint32_t a_lo, uint32_t b_lo, uint32_t d_tmem, uint32_t idesc, bool overwrite) {
                if (!leader) return;
                if (overwrite) umma_pair_lohi<false>(d_tmem, a_lo, b_lo, idesc);
                else umma_pair_lohi<true>(d_tmem, a_lo, b_lo, idesc);
                umma_pair_lohi<true>(d_tmem, a_lo + 2, b_lo + 2, idesc);
                umma_pair_lohi<true>(d_tmem, a_lo + 4, b_lo + 4, idesc);
                umma_pair_lohi<true>(d_tmem, a_lo + 6, b_lo + 6, idesc);
            };
            auto bfull_parity = [](int q) { return (uint32_t)((q / kCpRing) & 1); };
            uint32_t block_ready = 0, slot_ready = 0;
        for (int k = 0; k < n_stack; ++k) {
          if (is_leader && ok && !*abort_flag) {
            int t_hi = -1;                  // units [.., t_hi) belong to the current tenant (every layer starts over)
            int in_image = 0;               // index of the current strip inside its image
            block_ready = 0;
            for (int s = s_begin; ok && s < s_end; ++s) {
                const bool new_tenant = (s >= t_hi);
                if (new_tenant) {           // rare: a tenant border (or the first unit)
                    const PairStrip c = locate(s);
                    t_hi = cur_hi;
                    in_image = c.strip_in_image;
                }
                // a segment = the tiles of one image that this pair computes one after the other
                const bool seg_start = !(s > s_begin && in_image > 0);
                const bool seg_end = !(s + 1 < s_end && in_image + 1 < p.strips_per_image);
                if (seg_start) {
                    if (!mbar_wait_spin(bfull_bar(bc & (kCpRing - 1)), bfull_parity(bc), abort_flag, p.status, 55)) { ok = false; break; }
                    block_ready = 0;
                }
                if (new_tenant) {
                    if (w_loads > 0 && !w_released && leader) umma_commit_pair(wempty_bar);   // fires when all MMAs on the old weights are done
                    w_released = false;
                    if (!mbar_wait(wfull_bar, (uint32_t)(w_loads & 1), abort_flag, p.status, 56)) { ok = false; break; }
                    if (!mbar_wait_spin(wpeer_bar, (uint32_t)(w_loads & 1), abort_flag, p.status, 57)) { ok = false; break; }
                    ++w_loads;
                }
                for (int i = 0; i < TS; ++i, ++g, ++bc) {
                    const int slot = g % kCpSlots;
                    // the block under the tile (its tap row 1 runs on into that block's first row)
                    if (!block_ready) {
                        if (!mbar_wait_spin(bfull_bar((bc + 1) & (kCpRing - 1)), bfull_parity(bc + 1), abort_flag, p.status, 59)) { ok = false; break; }
                    }
                    if (!slot_ready) {   // the slot must have been drained by both CTAs' epilogues of tile g - kCpSlots
                        if (!mbar_wait_spin(tempty_bar(slot), (uint32_t)(((g / kCpSlots) & 1) ^ 1), abort_flag, p.status, 54)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t d_this = tb + slot * kCpN;
                    const uint32_t blk = ring_lo + (uint32_t)(bc & (kCpRing - 1)) * kBlockLo;
                    const bool more_in_segment = !(i == TS - 1 && seg_end);
                    // tap row 1 first: these overwrite the fresh accumulator
                    issue(blk + (uint32_t)(Wp + 0) * kPixLo, w_lo + kMidLo + 0 * kHalfLo, d_this, idesc64, true);
                    // look ahead: the answers are consumed after the rest of this tile has been queued
                    const uint32_t poll_slot = mbar_test_wait(tempty_bar((g + 1) % kCpSlots), (uint32_t)((((g + 1) / kCpSlots) & 1) ^ 1));
                    uint32_t poll_block = 0;
                    if (more_in_segment) poll_block = mbar_test_wait(bfull_bar((bc + 2) & (kCpRing - 1)), bfull_parity(bc + 2));
                    issue(blk + (uint32_t)(Wp + 1) * kPixLo, w_lo + kMidLo + 1 * kHalfLo, d_this, idesc64, false);
                    issue(blk + (uint32_t)(Wp + 2) * kPixLo, w_lo + kMidLo + 2 * kHalfLo, d_this, idesc64, false);
                    // the tile's own block: tap row 0 of this tile and tap row 2 of the tile above
                    const bool have_above = (i > 0) || !seg_start;
                    const bool adjacent = slot != 0;                              // slots g-1 and g contiguous in TMEM
                    if (have_above && adjacent) {
#pragma unroll
                        for (int kx = 0; kx < 3; ++kx)
                            issue(blk + kx * kPixLo, w_lo + kPairLo + kx * kFullLo, d_this - kCpN, idesc128, false);
                    } else {
                        for (int kx = 0; kx < 3; ++kx) {
                            if (have_above)
                                issue(blk + kx * kPixLo, w_lo + kBotLo + kx * kHalfLo, tb + ((g - 1) % kCpSlots) * kCpN, idesc64, false);
                            issue(blk + kx * kPixLo, w_lo + kTopLo + kx * kHalfLo, d_this, idesc64, false);
                        }
                    }
                    if (have_above && leader) umma_commit_pair(tfull_bar((g - 1) % kCpSlots));    // tile above is complete
                    slot_ready = poll_slot;
                    block_ready = poll_block;
                }
                if (!ok) break;
                if (seg_end) {
                    // no tile below finishes the segment's last tile: its tap row 2 from the block under it (landed:
                    // the tile waited for it)
                    const uint32_t blk = ring_lo + (uint32_t)(bc & (kCpRing - 1)) * kBlockLo;
                    const int last = (g - 1) % kCpSlots;
                    for (int kx = 0; kx < 3; ++kx)
                        issue(blk + kx * kPixLo, w_lo + kBotLo + kx * kHalfLo, tb + last * kCpN, idesc64, false);
                    if (leader) umma_commit_pair(tfull_bar(last));
                    ++bc;
                    block_ready = 0;
                }
                if (++in_image == p.strips_per_image) in_image = 0;
            }
            // the layer's weights go back to the producer, which requests the next layer's before the barrier
            if (ok && k + 1 < n_stack && s_begin < s_end && w_loads > 0) {
                if (leader) umma_commit_pair(wempty_bar);
                w_released = true;
            }
          }
          __syncwarp();
          if (k + 1 < n_stack) layer_sync(k);
        }
    } else {               // ---------------------------------------------------- epilogue (warps 2..9, both CTAs)
        const int ew = warp - 2;
        const int q4 = warp & 3;                    // TMEM lane quarter this warp may read
        const int half = ew >> 2;                   // which 32 of the 64 output channels
        const int r = q4 * 32 + lane;               // tile-local padded pixel of this thread
        const int yl = r / Wp, x = r - yl * Wp;
        constexpr int rows_per_tile = BM / Wp;
        int g = 0, relu = 0;
        bool ok = true;
        int img_j = 0, y0 = 0, store = 1;
        int rel = 0;                                // blocks released so far (load order), kept by the releasing thread
        const uint32_t tempty_leader0 = map_to_cta(tempty_bar(0), 0);   // the leader's tempty barriers, 8 bytes apart
      for (int k = 0; k < n_stack; ++k) {
        const int layer = p.layer + k;
        const bool pooling = (p.pool_partial != nullptr) && k == n_stack - 1;   // only the stack's last layer feeds the pool
        const CUtensorMap* const tmap_y = &maps.y[k];
        // Identity shortcuts (kSkip only): a thread adds, to its pixel's 32 channels, 64 bytes of the tensor that the
        // layer before read.  The epilogue of this kernel has no slack (the MMAs are bound by operand reads from
        // shared memory and a tile leaves the pipe every 1.4 us), so the obvious form - every thread loads its 64 bytes
        // when the accumulator is ready - took 2.7 x the time of a plain layer.  What this form does instead:
        //  - whole sectors, nothing through shared memory: a thread reads its own 64 bytes as two 32-byte loads (staging
        //    a coalesced load through the warp's shared-memory region took bandwidth from the MMAs' operand reads:
        //    +34 us per layer; an exchange between lanes cost as many instructions as it saved sectors);
        //  - the values of a tile are requested TWO tiles ahead (16 KiB per SM and tile in flight, twice): one tile
        //    ahead the layer's 103 MB could not be in flight often enough to arrive within the layer's 50 us.  That
        //    needs a tile's coordinates long before its record is published, so the epilogue derives them itself (the
        //    same unit -> (tenant, image, row) map as the producer's) and re-reads the tenant's flag and the image's
        //    arrival index only when they change;
        //  - four tiles ahead the same lines are asked into L2 (a prefetch holds no register), so most of those
        //    loads are L2 hits; and the buffers must not spill: a spilled load destination is a wait for the load.
        // On 56 x 56 images a layer with shortcuts now takes 1.65 x a plain one (83 against 50 us), of which a third is
        // the extra instructions, the rest the loads.
        // Tiles alternate between the two register buffers, so a strip must have an even number of tiles (it has two).
        const uint16_t* const skip_k = kSkip ? p.skip[k] : nullptr;
        const int32_t* const skip_perm_k = (kSkip && p.skip_perm[k]) ? (self_bucket ? s_perm : p.skip_perm[k]) : nullptr;
        const bool skip_wide = (reinterpret_cast<uintptr_t>(skip_k) & 31) == 0;      // 32-byte loads need that alignment
        uint4 sk_a[4], sk_b[4];                     // values on their way: even / odd tile of a strip
        bool have_a = false, have_b = false;        // warp-uniform: the buffer holds (or will hold) values to add
        int n1_on = 0, n1_img = 0, n1_y0 = 0;       // strip s + 1: shortcut wanted (and the image real), its image, first row
        int n2_on = 0, n2_img = 0, n2_y0 = 0;       // strip s + 2, looked up while strip s runs
        int d_t = -1, d_resid = 0, d_j = -1, d_img = 0;     // last tenant / image looked up
        auto describe = [&](int s2, int& on, int& img, int& first_row) {
            const PairStrip c = locate(s2);
            if (c.t != d_t) { d_t = c.t; d_resid = p.models[c.t].layer[layer].residual; }
            if (c.j != d_j) { d_j = c.j; d_img = skip_perm_k ? skip_perm_k[c.j] : c.j; }
            on = (skip_k != nullptr && !c.dummy && d_resid) ? 1 : 0;
            first_row = c.y0;
            img = d_img;
        };
        auto request = [&](int on, int img, int yy, uint4 (&dst)[4]) -> bool {      // yy: this thread's image row (warp-uniform)
            if (!on || yy >= p.H) return false;
            if (x < p.W) {
                // written earlier in this launch or by the caller: read past L1
                const uint16_t* sp = skip_k + (((size_t)img * p.H + yy) * p.W + x) * kCpN + half * 32;
                if (skip_wide) {
                    asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                 : "=r"(dst[0].x), "=r"(dst[0].y), "=r"(dst[0].z), "=r"(dst[0].w),
                                   "=r"(dst[1].x), "=r"(dst[1].y), "=r"(dst[1].z), "=r"(dst[1].w) : "l"(sp));
                    asm volatile("ld.global.cg.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                                 : "=r"(dst[2].x), "=r"(dst[2].y), "=r"(dst[2].z), "=r"(dst[2].w),
                                   "=r"(dst[3].x), "=r"(dst[3].y), "=r"(dst[3].z), "=r"(dst[3].w) : "l"(sp + 16));
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) dst[j] = __ldcg(reinterpret_cast<const uint4*>(sp) + j);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) dst[j] = make_uint4(0u, 0u, 0u, 0u);
            }
            return true;
        };
        if (*abort_flag) ok = false;
        if constexpr (kSkip) {
            if (ok && s_begin < s_end) {
                int on, img, first_row;
                describe(s_begin, on, img, first_row);
                have_a = request(on, img, first_row + yl, sk_a);
                if (TS > 1) have_b = request(on, img, first_row + rows_per_tile + yl, sk_b);
                if (s_begin + 1 < s_end) describe(s_begin + 1, n1_on, n1_img, n1_y0);
            }
        }
        float psum[32];
        // One accumulator tile (tile i of strip s); buf / have_buf: the register buffer of the tile's parity.
        auto do_tile = [&](int s, int i, uint4 (&buf)[4], bool& have_buf) -> bool {
            const int slot = g % kCpSlots;
            // tfull is completed by the leader's multicast commit: one lane per warp polls and tells the others
            int got = 1;
            if (lane == 0) got = mbar_wait_spin(tfull_bar(slot), (uint32_t)((g / kCpSlots) & 1), abort_flag, p.status, 58, 32) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) return false;
            if (i == 0) {
                // the strip's record was published (with the strip's data) before any of its MMAs were issued
                const int4 rec = s_rec[(s - s_begin) & (kCpRecords - 1)];
                img_j = rec.y; y0 = rec.z; store = (rec.x & 8) ? 0 : 1;
                // This completion (tile g) follows every read of the block under tile g (by tile g and, if the
                // segment goes on, by the first two tap rows of tile g + 1, which are queued before the commit);
                // the segment's first tile also hands back its own block.
                if (threadIdx.x == 64 && (rec.x & 2)) { mbar_arrive(bempty_bar(rel & (kCpRing - 1))); ++rel; }
                if (rec.x & 1) {                // new tenant: its bias into shared memory, ReLU flag into a register
                    const LayerDev& L = p.models[rec.w].layer[layer];
                    asm volatile("bar.sync 1, %0;" ::"n"(kCpEpiThreads) : "memory");   // everyone done with the old bias
                    if (threadIdx.x - 64 < kCpN) s_bias[threadIdx.x - 64] = L.bias[threadIdx.x - 64];
                    relu = L.relu;
                    asm volatile("bar.sync 1, %0;" ::"n"(kCpEpiThreads) : "memory");
                }
            }
            if (threadIdx.x == 64) { mbar_arrive(bempty_bar(rel & (kCpRing - 1))); ++rel; }
            tc_fence_after();
            uint32_t v[32];
            tmem_ld32(tmem_base + (static_cast<uint32_t>(q4 * 32) << 16) + slot * kCpN + half * 32, v);
            tmem_ld_wait();
            tc_fence_before();
            // values are in registers: the slot can be reused once the eight epilogue warps of both CTAs have said
            // so (one arrival per warp: an arrival that crosses to the other CTA is expensive)
            __syncwarp();
            if (lane == 0) {
                if (is_leader) mbar_arrive(tempty_bar(slot));
                else mbar_arrive_remote_relaxed(tempty_leader0 + 8u * slot);
            }
            const int y = y0 + i * rows_per_tile + yl;
            // bias (+ shortcut) + ReLU in fp32 on this thread's pixel, 32 channels
            float f[32];
            {
                const float4* b4 = reinterpret_cast<const float4*>(s_bias + half * 32);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 b = b4[j];
                    f[4 * j + 0] = __uint_as_float(v[4 * j + 0]) + b.x;
                    f[4 * j + 1] = __uint_as_float(v[4 * j + 1]) + b.y;
                    f[4 * j + 2] = __uint_as_float(v[4 * j + 2]) + b.z;
                    f[4 * j + 3] = __uint_as_float(v[4 * j + 3]) + b.w;
                }
                if constexpr (kSkip) {
                    // this tile's shortcut values were requested two tiles ago; the buffer then takes the request for
                    // the tile of the same parity in the next strip
                    if (have_buf) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t w4[4] = {buf[j].x, buf[j].y, buf[j].z, buf[j].w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {       // two bf16 per word, the lower address in the low half
                                f[8 * j + 2 * e + 0] += __uint_as_float(w4[e] << 16);
                                f[8 * j + 2 * e + 1] += __uint_as_float(w4[e] & 0xffff0000u);
                            }
                        }
                    }
                    have_buf = (s + 1 < s_end) ? request(n1_on, n1_img, n1_y0 + i * rows_per_tile + yl, buf) : false;
                    if (i == 0 && s + 2 < s_end) {
                        describe(s + 2, n2_on, n2_img, n2_y0);
                        // and that strip's lines are asked into L2 now, four tiles ahead (one warp of the two that
                        // share a pixel's 128-byte line does it), so that the loads above mostly find them there
                        if (n2_on && half == 0 && x < p.W) {
#pragma unroll
                            for (int tl = 0; tl < 2; ++tl) {
                                const int yy = n2_y0 + tl * rows_per_tile + yl;
                                if (tl < TS && yy < p.H)
                                    asm volatile("prefetch.global.L2 [%0];" ::"l"(skip_k + (((size_t)n2_img * p.H + yy) * p.W + x) * kCpN));
                            }
                        }
                    }
                }
                if (relu) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) f[e] = fmaxf(f[e], 0.0f);
                }
            }
            if (pooling) {      // the layer feeds a global average pool: only channel sums are kept
                if (store && x < p.W && y < p.H) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) psum[e] += f[e];
                }
            } else {
                // The warp's 32 pixels x 32 channels go to its staging region (64 bytes per pixel, 16-byte chunk c
                // of pixel q at chunk c ^ ((q >> 1) & 3): the 64-byte swizzle of the store's tensor map) and leave
                // as ONE tensor store, which also drops the pad columns and the rows past the image.  A row of
                // per-thread 64-byte global stores would cost the load/store unit 32 separate lines per instruction.
                if (lane == 0) bulk_wait_group_read0();      // the previous tile's store has read the region
                __syncwarp();
                uint8_t* mine = out_stage_ptr + ew * 2048 + lane * 64;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 o;
                    o.x = pack_bf16x2(f[8 * j + 0], f[8 * j + 1]);
                    o.y = pack_bf16x2(f[8 * j + 2], f[8 * j + 3]);
                    o.z = pack_bf16x2(f[8 * j + 4], f[8 * j + 5]);
                    o.w = pack_bf16x2(f[8 * j + 6], f[8 * j + 7]);
                    *reinterpret_cast<uint4*>(mine + ((j ^ ((lane >> 1) & 3)) << 4)) = o;
                }
                fence_proxy_async_smem();
                __syncwarp();
                const int yw = y0 + i * rows_per_tile + (q4 >> 1);       // the warp's image row (warp-uniform)
                if (lane == 0 && store && yw < p.H && (q4 & 1) * 32 < p.W) {
                    tma_store_4d(tmap_y, half * 32, (q4 & 1) * 32, yw, img_j, out_stage0 + ew * 2048);
                    bulk_commit_group();
                }
            }
            __syncwarp();
            ++g;
            return true;
        };
        for (int s = s_begin; ok && s < s_end; ++s) {
#pragma unroll
            for (int e = 0; e < 32; ++e) psum[e] = 0.0f;
            for (int i = 0; ok && i < TS; i += 2) {
                ok = do_tile(s, i, sk_a, have_a);
                if (ok && i + 1 < TS) ok = do_tile(s, i + 1, sk_b, have_b);
            }
            if constexpr (kSkip) { n1_on = n2_on; n1_img = n2_img; n1_y0 = n2_y0; }
            if (pooling && ok) {
                // Channel sums of this strip: a halving butterfly leaves lane c with the warp's total of channel c
                // (31 shuffles), the four lane quarters are then added in a fixed order, and the strip's 64 sums are
                // written to their own slot of pool_partial - no atomics, so the pooled value does not depend on timing.
#pragma unroll
                for (int step = 16; step >= 1; step >>= 1) {
                    const bool upper = (lane & step) != 0;
#pragma unroll
                    for (int e = 0; e < step; ++e) {
                        const float send = upper ? psum[e] : psum[e + step];
                        const float recv = __shfl_xor_sync(0xffffffffu, send, step);
                        psum[e] = (upper ? psum[e + step] : psum[e]) + recv;
                    }
                }
                s_pool[ew * 32 + lane] = psum[0];
                asm volatile("bar.sync 1, %0;" ::"n"(kCpEpiThreads) : "memory");
                const int et = threadIdx.x - 64;                    // 0..255 among the epilogue threads
                if (et < kCpN && store) {
                    const int hf = et >> 5, c = et & 31;
                    const float* q = s_pool + (hf * 4) * 32 + c;     // warps hf*4 .. hf*4+3 hold this half's quarters
                    // quarter order by TMEM lane quarter (ew & 3 maps to q4 = (ew + 2) & 3): sum in pixel order 0,1,2,3
                    const float t = ((q[2 * 32] + q[3 * 32]) + q[0 * 32]) + q[1 * 32];
                    p.pool_partial[((size_t)img_j * p.strips_per_image + y0 / p.R) * kCpN + et] = t;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kCpEpiThreads) : "memory");
            }
        }
        if (k + 1 < n_stack) {
            // this layer's outputs must have reached memory before anyone passes the barrier
            if (lane == 0) {
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                asm volatile("fence.proxy.async;" ::: "memory");
            }
            __syncwarp();
            layer_sync(k);
        }
      }
    }

    // ---- tear-down: every thread of both CTAs gets here, also after an abandoned wait
    bulk_wait_group_read0();     // tensor stores still reading the staging regions
    if (*abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // nobody signals a CTA that has left, and both are done with the pair's TMEM
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc_pair(tmem_base, kCpSlots * kCpN);
    }
}

// Conv weights W[64][3][3][64] -> the two CTAs' weight images of the pair executor (60 KiB each, rank 0 first),
// every tile in the 128-byte-swizzled shared-memory layout: three ky = 1 taps with the CTA's 32 output channels,
// three full 64-channel tiles (rank 0: W(2,kx), rank 1: W(0,kx)), three ky = 2 and three ky = 0 taps with the CTA's
// 32 output channels.
__global__ void pretile_conv_pair_kernel(const uint16_t* __restrict__ w, uint4* __restrict__ out) {
    constexpr int kChunksPerRank = kConvPairWeightBytes / 16;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < 2 * kChunksPerRank; idx += gridDim.x * blockDim.x) {
        const int rank = idx / kChunksPerRank;
        const int off = (idx - rank * kChunksPerRank) * 16;      // byte offset inside the rank's image
        int ky, kx, row0, local;
        if (off < kOffPair) { ky = 1; kx = off / kCpHalfTap; local = off - kx * kCpHalfTap; row0 = 32 * rank; }
        else if (off < kOffBot) { const int o = off - kOffPair; ky = rank == 0 ? 2 : 0; kx = o / kCpFullTap; local = o - kx * kCpFullTap; row0 = 0; }
        else if (off < kOffTop) { const int o = off - kOffBot; ky = 2; kx = o / kCpHalfTap; local = o - kx * kCpHalfTap; row0 = 32 * rank; }
        else { const int o = off - kOffTop; ky = 0; kx = o / kCpHalfTap; local = o - kx * kCpHalfTap; row0 = 32 * rank; }
        const int r = local >> 7, cpos = (local >> 4) & 7;       // row of the tile, physical 16-byte position
        const int c = cpos ^ (r & 7);                            // logical chunk stored there
        out[idx] = *reinterpret_cast<const uint4*>(w + ((size_t)(row0 + r) * 9 + (ky * 3 + kx)) * 64 + c * 8);
    }
}

void launch_pretile_conv_pair(const uint16_t* w, uint16_t* out, cudaStream_t s) {
    pretile_conv_pair_kernel<<<(2 * kConvPairWeightBytes / 16 + 255) / 256, 256, 0, s>>>(w, reinterpret_cast<uint4*>(out));
}

int conv_pair_smem_bytes() { return kCpSmemBytes; }

cudaError_t configure_grouped_conv_pair() {
    cudaError_t e = cudaFuncSetAttribute(grouped_conv3x3_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(grouped_conv3x3_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

// Cluster of two CTAs; grid = an even number of CTAs (one per SM).  a.tile_prefix counts (pair of images, strip) units.
// maps: per layer of the stack (a.n_stack layers from a.layer on) the input as boxes of 64 pixels x 2 rows and x 1 row
// and the output as 32 x 32 store boxes.
cudaError_t launch_grouped_conv_pair(const ConvStackMaps& maps, const ConvArgs& a, int sm_count, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sm_count & ~1);
    cfg.blockDim = dim3(kCpThreads);
    cfg.dynamicSmemBytes = (size_t)kCpSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    ++g_kernel_launches;
    bool any_skip = false;
    for (int k = 0; k < a.n_stack; ++k) any_skip = any_skip || a.skip[k] != nullptr;
    return any_skip ? cudaLaunchKernelEx(&cfg, grouped_conv3x3_pair_kernel<true>, maps, a)
                    : cudaLaunchKernelEx(&cfg, grouped_conv3x3_pair_kernel<false>, maps, a);
}

}  // namespace mt

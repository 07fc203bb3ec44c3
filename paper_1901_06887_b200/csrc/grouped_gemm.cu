// Grouped dense-layer executor: ONE persistent launch evaluates a layer for every tenant of the batch,
//     H_out[seg t] = act(H_in[seg t] . W_t^T + b_t)        (bf16 x bf16 -> fp32, bias + ReLU in fp32)
// where seg t is the contiguous block of bucketed rows of tenant t.  This is the fully-connected layer of
// the paper's primer (Sec. 1.1) applied across co-resident models (Sec. 3); since every tenant has its own
// weights (Sec. 4: "model weights are unique"), the launch walks a device-built list of
// (tenant, row tile, column tile) work items instead of one GEMM.
//
// CTA = 6 warps: warp 0 issues TMA loads (activation tile through a tensor map, each 128-row weight tile as one
// 16 KiB bulk copy of a pre-swizzled image), warp 1 issues tcgen05.mma into one of two TMEM accumulators, warps
// 2..5 drain the other accumulator (tcgen05.ld -> bias -> ReLU -> convert -> 128-bit stores), so the
// epilogue of tile i overlaps the main loop of tile i+1.  Rows of a tile beyond the tenant's segment are
// computed on whatever follows in memory and never stored (rows of a GEMM are independent).  The work list is
// an array of 48-byte records expanded on the device after bucketing; CTA b takes items b, b + grid, ...
#include <type_traits>

#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kGemmThreads = 192;
constexpr int kBarBytes = 256;

// TN = output columns of one work item: 128 (one weight tile per stage) or 256 (two weight tiles per stage, half
// the activation re-reads and half the shared-memory operand traffic per flop; all of TMEM for two accumulators).
template <int TN>
struct GemmCfg {
    static constexpr int kStages = (TN == 256) ? 4 : 6;
    static constexpr int kStageBytes = TILE_BYTES + (TN / BN) * TILE_BYTES;   // A tile + TN/128 weight tiles
    static constexpr int kAccCols = TN;                                       // fp32 columns of one accumulator
    static constexpr int kTmemCols = 2 * TN;                                  // two accumulators: 256 or 512 columns
    static constexpr int kSmem = kStages * kStageBytes + kBarBytes + 1024;    // + slack for 1024-byte alignment
};

// 48-byte work item as three 16-byte loads through the read-only path.
__device__ __forceinline__ WorkItem load_item(const WorkItem* items, int idx) {
    const int4* q = reinterpret_cast<const int4*>(items + idx);
    union { int4 v[3]; WorkItem w; } u;
    u.v[0] = __ldg(q); u.v[1] = __ldg(q + 1); u.v[2] = __ldg(q + 2);
    return u.w;
}

template <int TN>
__global__ void __launch_bounds__(kGemmThreads, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_a32,
                    const GemmArgs p) {
    // Segments of at most kSwapRows requests are computed transposed ("swap-AB"): the 128-row weight tile is the
    // M operand and the requests are the N operand (32 or 64 columns), so only 4 or 8 KiB of activations are
    // fetched per stage instead of a 16 KiB tile that is mostly other tenants' rows.  A 256-column item has two
    // weight tiles, hence two transposed accumulators, 64 TMEM columns apart.
    constexpr bool kSwapOk = true;
    constexpr int kSwapRows = 64;
    constexpr int kStages = GemmCfg<TN>::kStages;
    constexpr int kStageBytes = GemmCfg<TN>::kStageBytes;
    constexpr int kAccCols = GemmCfg<TN>::kAccCols;
    constexpr int kTmemCols = GemmCfg<TN>::kTmemCols;
    constexpr int kWTiles = TN / BN;                  // 128-row weight tiles per stage
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    const uint32_t bar0 = base + kStages * kStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kStages + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_a);
        if (kSwapOk) prefetch_tensormap(&tmap_a32);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    pdl_wait();   // everything above overlapped the previous kernel's tail; its results are needed from here on
    const int total = p.tile_prefix[p.T];

    if (warp == 0 && p.gather_perm) {
        // ---------------------------------------------------------------- TMA producer, rows through the permutation
        // The whole warp walks the loop: lane 0 waits for the stage, announces the bytes and fetches the weights, then
        // lane l fetches rows 4l .. 4l + 3 of the tile with ONE gather of four rows named by perm (32 gathers build
        // the same 16 KiB swizzled image as one 128-row box; a transposed item needs only its 8 or 16).
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        WorkItem cur = {};
        if ((int)blockIdx.x < total) cur = load_item(p.items, blockIdx.x);
        for (int k = 0, item = blockIdx.x; ok && item < total; ++k) {
            const int item_next = dealt_item(k + 1, blockIdx.x, gridDim.x);
            WorkItem nxt = {};
            if (item_next < total) nxt = load_item(p.items, item_next);
            const int kblocks = cur.k_blocks;
            const bool swap = kSwapOk && cur.rows_valid <= kSwapRows;
            const int n_g4 = swap ? ((cur.rows_valid + 31) >> 5) * 8 : 32;       // gathers (= lanes) per stage
            // rows past the segment are computed and never stored: any valid row will do for them
            int rr[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = 4 * lane + j;
                rr[j] = __ldg(p.gather_perm + cur.row0 + (r < cur.rows_valid ? r : 0));
            }
            const uint16_t* wsrc = cur.w + (size_t)cur.n_tile * kWTiles * kblocks * (BN * BK);
            uint32_t wbytes[kWTiles];
            uint32_t wsum = 0;
#pragma unroll
            for (int wt = 0; wt < kWTiles; ++wt) {
                const int rows = min(BN, max(0, cur.N - (cur.n_tile * kWTiles + wt) * BN));
                wbytes[wt] = (uint32_t)((rows + 7) & ~7) * (BK * 2);
                wsum += wbytes[wt];
            }
            for (int kb = 0; kb < kblocks; ++kb) {
                const uint32_t a_dst = base + stage * kStageBytes;
                if (lane == 0) {
                    ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1);
                    if (ok) {
                        mbar_expect_tx(full_bar(stage), (uint32_t)(n_g4 * 512) + wsum);
#pragma unroll
                        for (int wt = 0; wt < kWTiles; ++wt)
                            if (wbytes[wt])
                                bulk_load(a_dst + (1 + wt) * TILE_BYTES, wsrc + ((size_t)wt * kblocks + kb) * (BN * BK),
                                          wbytes[wt], full_bar(stage));
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (lane < n_g4) tma_gather4(a_dst + lane * 512, &tmap_a, kb * BK, rr[0], rr[1], rr[2], rr[3], full_bar(stage));
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
            cur = nxt;
            item = item_next;
        }
    } else if (warp == 0) {
        if (lane == 0) {   // ------------------------------------------------ TMA producer
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            WorkItem cur = {};
            if ((int)blockIdx.x < total) cur = load_item(p.items, blockIdx.x);
            for (int k = 0, item = blockIdx.x; ok && item < total; ++k) {
                const int item_next = dealt_item(k + 1, blockIdx.x, gridDim.x);
                WorkItem nxt = {};
                if (item_next < total) nxt = load_item(p.items, item_next);   // in flight during this item
                const int kblocks = cur.k_blocks;
                const bool swap = kSwapOk && cur.rows_valid <= kSwapRows;
                const int nbox = (cur.rows_valid + 31) >> 5;
                // weight tile (nt, kb) of 128 rows x 64 columns starts at element (nt * kblocks + kb) * 8192
                const uint16_t* wsrc = cur.w + (size_t)cur.n_tile * kWTiles * kblocks * (BN * BK);
                // Only the 8-row groups of a weight tile that hold output features are fetched (a 64-wide last layer
                // would otherwise stream as many zero rows as weights); what stays in the stage from earlier items
                // only reaches accumulator columns (or, transposed, lanes) that are never stored.
                uint32_t wbytes[kWTiles];
                uint32_t wsum = 0;
#pragma unroll
                for (int wt = 0; wt < kWTiles; ++wt) {
                    const int rows = min(BN, max(0, cur.N - (cur.n_tile * kWTiles + wt) * BN));
                    wbytes[wt] = (uint32_t)((rows + 7) & ~7) * (BK * 2);
                    wsum += wbytes[wt];
                }
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
                    const uint32_t a_dst = base + stage * kStageBytes;
                    if (swap) {          // only the 32-row boxes that hold the segment's requests
                        mbar_expect_tx(full_bar(stage), (uint32_t)(nbox * 4096) + wsum);
                        for (int b = 0; b < nbox; ++b)
                            tma_load_2d(a_dst + b * 4096, &tmap_a32, kb * BK, cur.row0 + b * 32, full_bar(stage));
                    } else {
                        mbar_expect_tx(full_bar(stage), (uint32_t)TILE_BYTES + wsum);
                        tma_load_2d(a_dst, &tmap_a, kb * BK, cur.row0, full_bar(stage));
                    }
#pragma unroll
                    for (int wt = 0; wt < kWTiles; ++wt)
                        if (wbytes[wt])
                            bulk_load(a_dst + (1 + wt) * TILE_BYTES, wsrc + ((size_t)wt * kblocks + kb) * (BN * BK),
                                      wbytes[wt], full_bar(stage));
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                cur = nxt;
                item = item_next;
            }
        }
    } else if (warp == 1) {
        {                  // ------------------------------------------------ MMA issuer
            // The whole warp walks the loop, so that addresses and descriptors stay warp-uniform values; one elected
            // lane issues the MMAs and commits.
            const bool leader = elect_one();
            const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
            // This thread alone feeds the tensor pipe, and it issues in order: every instruction it spends on
            // anything else is time the pipe may run dry.  So descriptors are one 32-bit add away from a
            // precomputed base, the next stage's barrier is polled (non-blocking) BEFORE the current stage's MMAs
            // are issued and looked at after them, and the next item's K extent is loaded one item ahead.
            constexpr uint32_t idesc = make_idesc_bf16(BM, TN);
            constexpr uint32_t kStageLo = kStageBytes >> 4;
            const uint32_t a_lo0 = desc_lo(base), b_lo0 = desc_lo(base + TILE_BYTES);
            int stage = 0; uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            int4 head = ((int)blockIdx.x < total) ? __ldg(reinterpret_cast<const int4*>(p.items + blockIdx.x)) : make_int4(0, 0, 0, 0);
            uint32_t ready = 0;
            for (int item = blockIdx.x; ok && item < total; ++it) {
                const int item_next = dealt_item(it + 1, blockIdx.x, gridDim.x);
                const int4 next_head = (item_next < total)
                                           ? __ldg(reinterpret_cast<const int4*>(p.items + item_next)) : make_int4(0, 0, 0, 0);
                const int kblocks = head.w;          // (row0, rows_valid, n_tile, k_blocks)
                const bool swap = kSwapOk && head.y <= kSwapRows;
                // transposed items: M = 128 weight rows, N = 32 or 64 request columns
                const uint32_t idesc_item = swap ? make_idesc_bf16(BM, ((head.y + 31) >> 5) * 32) : idesc;
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 2)) break;
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ready && !mbar_wait(full_bar(stage), phase, abort_flag, p.status, 3)) { ok = false; break; }
                    tc_fence_after();
                    const int next_stage = (stage + 1 == kStages) ? 0 : stage + 1;
                    const uint32_t next_phase = (stage + 1 == kStages) ? (phase ^ 1u) : phase;
                    const uint32_t poll = mbar_test_wait(full_bar(next_stage), next_phase);   // consumed after the MMAs
                    // first operand region of the stage = activations, second = weights; swapped items swap the roles
                    const uint32_t act_lo = a_lo0 + stage * kStageLo, w_lo = b_lo0 + stage * kStageLo;
                    // advancing K by 16 elements = 32 bytes inside the swizzle row: +2 in the address field
                    if (leader) {
                        if (swap) {
#pragma unroll
                            for (int wt = 0; wt < kWTiles; ++wt) {
                                const uint32_t d = d_tmem + wt * kSwapRows, wa = w_lo + wt * (TILE_BYTES >> 4);
                                if (kb == 0) umma_bf16_lohi<false>(d, wa, act_lo, idesc_item);
                                else umma_bf16_lohi<true>(d, wa, act_lo, idesc_item);
                                umma_bf16_lohi<true>(d, wa + 2, act_lo + 2, idesc_item);
                                umma_bf16_lohi<true>(d, wa + 4, act_lo + 4, idesc_item);
                                umma_bf16_lohi<true>(d, wa + 6, act_lo + 6, idesc_item);
                            }
                        } else {
                            if (kb == 0) umma_bf16_lohi<false>(d_tmem, act_lo, w_lo, idesc_item);
                            else umma_bf16_lohi<true>(d_tmem, act_lo, w_lo, idesc_item);
                            umma_bf16_lohi<true>(d_tmem, act_lo + 2, w_lo + 2, idesc_item);
                            umma_bf16_lohi<true>(d_tmem, act_lo + 4, w_lo + 4, idesc_item);
                            umma_bf16_lohi<true>(d_tmem, act_lo + 6, w_lo + 6, idesc_item);
                        }
                        umma_commit(empty_bar(stage));   // frees the stage once these MMAs have read it
                    }
                    stage = next_stage; phase = next_phase;
                    ready = poll;
                }
                if (ok && leader) umma_commit(tfull_bar(acc));
                head = next_head;
                item = item_next;
            }
        }
    } else {               // ---------------------------------------------------- epilogue (warps 2..5)
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int r = q * 32 + lane;            // accumulator row of this thread
        int it = 0;
        WorkItem cur = {};
        if ((int)blockIdx.x < total) cur = load_item(p.items, blockIdx.x);
        const int32_t* const perm = p.perm;
        const bool out_vec_ok = (p.ld_final & 3) == 0 && (reinterpret_cast<uintptr_t>(p.final_out) & 15) == 0;
        if (p.nan_fill) {
            // requests whose id was rejected sort behind every live segment and get no work item: NaN rows
            const int n_valid = p.offsets[p.T], n_all = p.offsets[p.T + 1];
            for (int j = n_valid + blockIdx.x; j < n_all; j += gridDim.x) {
                float* dst = p.final_out + (size_t)perm[j] * p.ld_final;
                for (int e = threadIdx.x - 64; e < p.ld_final; e += 128) dst[e] = __int_as_float(0x7fc00000);
            }
        }
        for (int item = blockIdx.x; item < total; item = dealt_item(++it, blockIdx.x, gridDim.x)) {
            WorkItem nxt = {};
            const int item_next = dealt_item(it + 1, blockIdx.x, gridDim.x);
            if (item_next < total) nxt = load_item(p.items, item_next);
            const WorkItem c = cur;
            cur = nxt;
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            // Everything the drain needs besides the accumulator is fetched BEFORE the wait for it (the item's record
            // is known one item ahead): output rows, through perm for a tenant's last layer, and the bias.  For short
            // items - a few K blocks of a 64-wide layer - the drain is as long as the main loop, so its memory round
            // trips must not come on top of it.
            const int N = c.N, relu = c.relu;
            const bool fin = (c.flags & kItemFinal) != 0;      // this tenant's last layer: fp32 rows to arrival order
            const bool swap_item = kSwapOk && c.rows_valid <= kSwapRows;
            int my_row[2] = {c.row0 + lane, c.row0 + 32 + lane};
            float bias_f[kWTiles];
            size_t grow = (size_t)(c.row0 + r);
            if (swap_item) {
                if (fin) {
                    if (lane < c.rows_valid) my_row[0] = __ldg(perm + c.row0 + lane);
                    if (lane + 32 < c.rows_valid) my_row[1] = __ldg(perm + c.row0 + 32 + lane);
                }
#pragma unroll
                for (int wt = 0; wt < kWTiles; ++wt) {
                    const int f = c.n_tile * TN + wt * BN + r;
                    bias_f[wt] = f < N ? __ldg(c.bias + f) : 0.0f;
                }
            } else if (fin && r < c.rows_valid) {
                grow = (size_t)__ldg(perm + c.row0 + r);
            }
            if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 4)) break;
            tc_fence_after();
            if (swap_item) {
                // Transposed item: this thread owns output feature f, the accumulator columns are the requests.
                // For one request the 32 lanes of a warp write 32 neighbouring features: a 64- or 128-byte run.
                // Requests are taken eight at a time and only as far as the segment goes (most segments of a
                // long-tailed batch hold a handful); the output row of request j is handed round by shuffle.
                const int nbox = (c.rows_valid + 31) >> 5;
                auto store_box = [&](auto fin_c, const uint32_t (&v)[32], const int rows_of_box, const int n_req, const int f,
                                     const float bias) {
                    constexpr bool kFin = decltype(fin_c)::value;
                    const bool f_ok = f < N;
#pragma unroll
                    for (int j0 = 0; j0 < 32; j0 += 8) {
                        if (j0 < n_req) {                       // warp-uniform
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj) {
                                const int j = j0 + jj;
                                const size_t orow = (size_t)__shfl_sync(0xffffffffu, rows_of_box, j);
                                if (f_ok && j < n_req) {
                                    float val = __uint_as_float(v[j]) + bias;
                                    if (relu) val = fmaxf(val, 0.0f);
                                    if (kFin) p.final_out[orow * p.ld_final + f] = val;
                                    else reinterpret_cast<uint16_t*>(p.out)[orow * p.ld_out + f] =
                                             static_cast<uint16_t>(pack_bf16x2(val, 0.0f) & 0xFFFFu);
                                }
                            }
                        }
                    }
                };
#pragma unroll 1
                for (int wt = 0; wt < kWTiles; ++wt) {
                    const int f = c.n_tile * TN + wt * BN + r;
                    for (int b = 0; b < nbox; ++b) {
                        uint32_t v[32];
                        __syncwarp();
                        const int n_req = min(32, c.rows_valid - b * 32);
                        tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccCols + wt * kSwapRows + b * 32, v);
                        tmem_ld_wait();
                        const int rows_of_box = b == 0 ? my_row[0] : my_row[1];
                        const float bias = wt == 0 ? bias_f[0] : bias_f[kWTiles - 1];
                        if (fin) store_box(std::true_type{}, v, rows_of_box, n_req, f, bias);
                        else store_box(std::false_type{}, v, rows_of_box, n_req, f, bias);
                    }
                }
                __syncwarp();
                tc_fence_before();
                mbar_arrive(tempty_bar(acc));
                continue;
            }
            const bool row_ok = r < c.rows_valid;
#pragma unroll 1
            for (int ch = 0; ch < TN / 32; ++ch) {
                uint32_t v[32];
                __syncwarp();   // tcgen05.ld is warp-collective: reconverge after the per-row stores
                tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kAccCols + ch * 32, v);
                tmem_ld_wait();
                const int n0 = c.n_tile * TN + ch * 32;
                if (n0 >= N) break;
                const float4* b4 = reinterpret_cast<const float4*>(c.bias + n0);
                float f[32];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 b = __ldg(b4 + j);
                    f[4 * j + 0] = __uint_as_float(v[4 * j + 0]) + b.x;
                    f[4 * j + 1] = __uint_as_float(v[4 * j + 1]) + b.y;
                    f[4 * j + 2] = __uint_as_float(v[4 * j + 2]) + b.z;
                    f[4 * j + 3] = __uint_as_float(v[4 * j + 3]) + b.w;
                }
                if (relu) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.0f);
                }
                const bool full_chunk = (n0 + 32 <= N);
                if (!row_ok) {
                    // rows past the tenant's segment belong to someone else: never stored
                } else if (fin) {
                    float* dst = p.final_out + grow * p.ld_final + n0;
                    if (full_chunk && out_vec_ok) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            reinterpret_cast<float4*>(dst)[j] = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + j < N) dst[j] = f[j];
                    }
                } else {
                    uint16_t* dst = reinterpret_cast<uint16_t*>(p.out) + grow * p.ld_out + n0;
                    if (full_chunk && (p.ld_out & 7) == 0) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 o;
                            o.x = pack_bf16x2(f[8 * j + 0], f[8 * j + 1]);
                            o.y = pack_bf16x2(f[8 * j + 2], f[8 * j + 3]);
                            o.z = pack_bf16x2(f[8 * j + 4], f[8 * j + 5]);
                            o.w = pack_bf16x2(f[8 * j + 6], f[8 * j + 7]);
                            reinterpret_cast<uint4*>(dst)[j] = o;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + j < N) dst[j] = static_cast<uint16_t>(pack_bf16x2(f[j], 0.0f) & 0xFFFFu);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(acc));
        }
    }

    // ---- tear-down: every thread gets here, also after an abandoned wait
    if (*abort_flag) {   // give copies and MMAs still in flight a bounded time to finish
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------ weight re-layout
__global__ void pretile_dense_kernel(const uint16_t* __restrict__ w, int N, int K, uint4* __restrict__ out,
                                     long long total_chunks) {
    const int kblocks = K / BK;
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total_chunks;
         idx += (long long)gridDim.x * blockDim.x) {
        const long long tile = idx >> 10;            // 1024 chunks of 16 bytes per tile
        const int within = (int)(idx & 1023);
        const int r = within >> 3, cpos = within & 7;
        const int c = cpos ^ (r & 7);                // logical chunk stored at physical position cpos
        const int nt = (int)(tile / kblocks), kb = (int)(tile % kblocks);
        const int row = nt * BN + r;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row < N) val = *reinterpret_cast<const uint4*>(w + (size_t)row * K + kb * BK + c * 8);
        out[idx] = val;
    }
}

void launch_pretile_dense(const uint16_t* w, int N, int K, uint16_t* out, cudaStream_t s) {
    const long long n_tiles = (N + BN - 1) / BN;
    const long long total = n_tiles * (K / BK) * 1024;
    long long blocks = (total + 255) / 256;
    if (blocks > 4096) blocks = 4096;
    pretile_dense_kernel<<<(int)blocks, 256, 0, s>>>(w, N, K, reinterpret_cast<uint4*>(out), total);
}

cudaError_t configure_grouped_gemm() {
    cudaError_t e = cudaFuncSetAttribute(grouped_gemm_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         GemmCfg<128>::kSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(grouped_gemm_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                GemmCfg<256>::kSmem);
}

void launch_grouped_gemm(const CUtensorMap& tmap_a, const CUtensorMap& tmap_a32, const GemmArgs& a, int tile_n,
                         int sm_count, cudaStream_t s) {
    if (tile_n == 256) launch_pdl(grouped_gemm_kernel<256>, dim3(sm_count), dim3(kGemmThreads), GemmCfg<256>::kSmem, s, tmap_a, tmap_a32, a);
    else launch_pdl(grouped_gemm_kernel<128>, dim3(sm_count), dim3(kGemmThreads), GemmCfg<128>::kSmem, s, tmap_a, tmap_a32, a);
}

}  // namespace mt

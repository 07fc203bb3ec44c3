// Grouped dense-layer executor, CTA-pair form, for batches whose tenants have thousands of requests each:
//     H_out[seg t] = act(H_in[seg t] . W_t^T + b_t)        (bf16 x bf16 -> fp32, bias + ReLU in fp32)
// Two CTAs of a cluster (two SMs) share one 256-row x 256-column work item.  Each CTA loads its own 128 activation
// rows and only HALF of the weight columns (one 16 KiB tile per stage instead of two); one thread of the leader CTA
// issues tcgen05.mma.cta_group::2 (M = 256), which reads both CTAs' shared memory and writes both CTAs' TMEM.  Per
// SM that halves the weight traffic from L2 and the shared-memory fill per flop - what the one-CTA form spends its
// power on in the compute-bound regime - and halves the number of MMA instructions issued per SM.
//
// Synchronisation inside the pair:
//   full[s]    in the leader only: the leader's producer announces the bytes of BOTH CTAs' loads, and both CTAs'
//              TMA loads (cta_group::2 form) report their bytes to that one barrier (a software relay from the
//              peer - wait locally, arrive remotely - cost about a microsecond per stage and was dropped);
//   empty[s]   in both CTAs, signalled together by tcgen05.commit ... multicast;
//   tfull[a]   in both CTAs, signalled together by commit multicast: each CTA drains its own 128 accumulator rows;
//   tempty[a]  in the leader: 256 arrivals, 128 local epilogue threads and 128 remote ones.
// Every wait is bounded; the two CTAs meet at a cluster barrier before they exit, so no signal is sent to a CTA
// that has already gone.
//
// The paper's fully-connected layer (Sec. 1.1) across co-resident models (Sec. 3); see grouped_gemm.cu.
#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kPairThreads = 192;
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * TILE_BYTES;              // own activation tile + own half of the weight columns
constexpr int kPairTN = 256;                                 // columns of the pair's tile
constexpr int kPairTmemCols = 2 * kPairTN;                   // two accumulators of 256 columns
constexpr int kPairSmem = kPairStages * kPairStageBytes + 256 + 1024;

// Tiled TMA load whose completion bytes are reported to a barrier of the pair's leader CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(leader_bar)
        : "memory");
}

__device__ __forceinline__ WorkItem load_pair_item(const WorkItem* items, int idx) {
    const int4* q = reinterpret_cast<const int4*>(items + idx);
    union { int4 v[3]; WorkItem w; } u;
    u.v[0] = __ldg(q); u.v[1] = __ldg(q + 1); u.v[2] = __ldg(q + 2);
    return u.w;
}

__global__ void __launch_bounds__(kPairThreads, 1)
grouped_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const GemmArgs p) {
    pdl_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kPairStages * kPairStageBytes);
    const uint32_t bar0 = base + kPairStages * kPairStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kPairStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kPairStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kPairStages + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kPairStages + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader (issues the MMAs), 1 = peer
    const bool is_leader = (rank == 0);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(full_bar(s), 1);                // used in the leader only
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 256);            // used in the leader only: 128 local + 128 remote arrivals
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_a);
    }
    if (warp == 1) {                                  // the same warp of both CTAs
        tmem_alloc_pair(smem_u32(tmem_slot), kPairTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                               // both CTAs' barriers exist before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    const int total = p.tile_prefix[p.T];
    const int n_pairs = gridDim.x >> 1;
    const int pair_id = blockIdx.x >> 1;

    if (warp == 0 && p.gather_perm) {
        // ------------------------------------------------ TMA producer (both CTAs), rows through the permutation: the
        // whole warp walks the loop, lane 0 waits, announces and fetches the weights, lane l gathers rows 4l .. 4l + 3
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        WorkItem cur = {};
        if (pair_id < total) cur = load_pair_item(p.items, pair_id);
        for (int k = 0, item = pair_id; ok && item < total; ++k) {
            const int item_next = dealt_item(k + 1, pair_id, n_pairs);
            WorkItem nxt = {};
            if (item_next < total) nxt = load_pair_item(p.items, item_next);
            const int kblocks = cur.k_blocks;
            const CUtensorMap* wmap = p.wmaps + (size_t)cur.t * MT_MAX_LAYERS + p.layer;
            const int wrow0 = (cur.n_tile * 2 + (int)rank) * kblocks * BN;
            int rr[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = (int)rank * BM + 4 * lane + j;         // rows past the segment: any valid row
                rr[j] = __ldg(p.gather_perm + cur.row0 + (r < cur.rows_valid ? r : 0));
            }
            for (int kb = 0; kb < kblocks; ++kb) {
                const uint32_t a_dst = base + stage * kPairStageBytes;
                const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
                if (lane == 0) {
                    ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 31);
                    if (ok) {
                        if (is_leader) mbar_expect_tx(full_bar(stage), 2 * kPairStageBytes);   // both CTAs' bytes
                        tma_load_2d_pair(a_dst + TILE_BYTES, wmap, 0, wrow0 + kb * BN, leader_full);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                tma_gather4_pair(a_dst + lane * 512, &tmap_a, kb * BK, rr[0], rr[1], rr[2], rr[3], leader_full);
                if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
            }
            cur = nxt;
            item = item_next;
        }
    } else if (warp == 0) {
        if (lane == 0) {   // ------------------------------------------------ TMA producer (both CTAs)
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            WorkItem cur = {};
            if (pair_id < total) cur = load_pair_item(p.items, pair_id);
            for (int k = 0, item = pair_id; ok && item < total; ++k) {
                const int item_next = dealt_item(k + 1, pair_id, n_pairs);
                WorkItem nxt = {};
                if (item_next < total) nxt = load_pair_item(p.items, item_next);
                const int kblocks = cur.k_blocks;
                // this CTA's half of the 256 columns: weight tile 2 * n_tile + rank, rows of the tiled image
                const CUtensorMap* wmap = p.wmaps + (size_t)cur.t * MT_MAX_LAYERS + p.layer;
                const int wrow0 = (cur.n_tile * 2 + (int)rank) * kblocks * BN;
                const int my_row0 = cur.row0 + (int)rank * BM;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 31)) { ok = false; break; }
                    const uint32_t a_dst = base + stage * kPairStageBytes;
                    const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
                    if (is_leader) mbar_expect_tx(full_bar(stage), 2 * kPairStageBytes);   // both CTAs' bytes
                    tma_load_2d_pair(a_dst, &tmap_a, kb * BK, my_row0, leader_full);
                    tma_load_2d_pair(a_dst + TILE_BYTES, wmap, 0, wrow0 + kb * BN, leader_full);
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
                cur = nxt;
                item = item_next;
            }
        }
    } else if (warp == 1) {
        if (is_leader) {   // ------------------------------------------------ MMA issuer (leader CTA)
            const bool leader_lane = elect_one();
            const uint32_t tb = __shfl_sync(0xffffffffu, tmem_base, 0);
            constexpr uint32_t idesc = make_idesc_bf16(2 * BM, kPairTN);
            constexpr uint32_t kStageLo = kPairStageBytes >> 4;
            const uint32_t a_lo0 = desc_lo(base), b_lo0 = desc_lo(base + TILE_BYTES);
            int stage = 0; uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            int kblocks = (pair_id < total) ? __ldg(&p.items[pair_id].k_blocks) : 0;
            uint32_t ready = 0;
            for (int item = pair_id; ok && item < total; ++it) {
                const int item_next = dealt_item(it + 1, pair_id, n_pairs);
                const int next_kblocks = (item_next < total) ? __ldg(&p.items[item_next].k_blocks) : 0;
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 32)) break;
                const uint32_t d_tmem = tb + acc * kPairTN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!ready && !mbar_wait(full_bar(stage), phase, abort_flag, p.status, 33)) { ok = false; break; }
                    tc_fence_after();
                    const int next_stage = (stage + 1 == kPairStages) ? 0 : stage + 1;
                    const uint32_t next_phase = (stage + 1 == kPairStages) ? (phase ^ 1u) : phase;
                    const uint32_t poll = mbar_test_wait(full_bar(next_stage), next_phase);
                    const uint32_t a_lo = a_lo0 + stage * kStageLo, b_lo = b_lo0 + stage * kStageLo;
                    if (leader_lane) {
                        if (kb == 0) umma_pair_lohi<false>(d_tmem, a_lo, b_lo, idesc);
                        else umma_pair_lohi<true>(d_tmem, a_lo, b_lo, idesc);
                        umma_pair_lohi<true>(d_tmem, a_lo + 2, b_lo + 2, idesc);
                        umma_pair_lohi<true>(d_tmem, a_lo + 4, b_lo + 4, idesc);
                        umma_pair_lohi<true>(d_tmem, a_lo + 6, b_lo + 6, idesc);
                        umma_commit_pair(empty_bar(stage));     // frees this stage in both CTAs
                    }
                    stage = next_stage; phase = next_phase;
                    ready = poll;
                }
                if (ok && leader_lane) umma_commit_pair(tfull_bar(acc));   // both CTAs' epilogues may drain
                kblocks = next_kblocks;
                item = item_next;
            }
        }
    } else {               // ---------------------------------------------------- epilogue (warps 2..5, both CTAs)
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int r = q * 32 + lane;            // accumulator row of this thread (row r of this CTA's 128)
        const uint32_t tempty_leader0 = map_to_cta(tempty_bar(0), 0), tempty_leader1 = map_to_cta(tempty_bar(1), 0);
        int it = 0;
        WorkItem cur = {};
        if (pair_id < total) cur = load_pair_item(p.items, pair_id);
        // last layer: rows go straight to their arrival positions in the caller's buffer (see GemmArgs::perm)
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
        for (int item = pair_id; item < total; item = dealt_item(++it, pair_id, n_pairs)) {
            WorkItem nxt = {};
            const int item_next = dealt_item(it + 1, pair_id, n_pairs);
            if (item_next < total) nxt = load_pair_item(p.items, item_next);
            const WorkItem c = cur;
            cur = nxt;
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 35)) break;
            tc_fence_after();
            const int N = c.N, relu = c.relu;
            const bool fin = (c.flags & kItemFinal) != 0;      // this tenant's last layer: fp32 rows to arrival order
            const int my_valid = min(BM, max(0, c.rows_valid - (int)rank * BM));
            const bool row_ok = r < my_valid;
            const size_t grow = (fin && row_ok) ? (size_t)__ldg(perm + c.row0 + (int)rank * BM + r)
                                                 : (size_t)(c.row0 + (int)rank * BM + r);
#pragma unroll 1
            for (int ch = 0; ch < kPairTN / 32; ++ch) {
                uint32_t v[32];
                __syncwarp();   // tcgen05.ld is warp-collective: reconverge after the per-row stores
                tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kPairTN + ch * 32, v);
                tmem_ld_wait();
                const int n0 = c.n_tile * kPairTN + ch * 32;
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
            __syncwarp();
            tc_fence_before();
            // the leader's issuer waits for both CTAs' epilogues before it reuses the accumulator
            if (is_leader) mbar_arrive(tempty_bar(acc));
            else mbar_arrive_remote(acc ? tempty_leader1 : tempty_leader0);
        }
    }

    // ---- tear-down: every thread of both CTAs gets here, also after an abandoned wait
    if (*abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // nobody signals a CTA that has left, and both are done with the pair's TMEM
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc_pair(tmem_base, kPairTmemCols);
    }
}

cudaError_t configure_grouped_gemm_pair() {
    return cudaFuncSetAttribute(grouped_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem);
}

// Cluster of two CTAs per work item; grid = an even number of CTAs (one per SM).
cudaError_t launch_grouped_gemm_pair(const CUtensorMap& tmap_a, const GemmArgs& a, int sm_count, cudaStream_t s) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sm_count & ~1);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = kPairSmem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    ++g_kernel_launches;
    return cudaLaunchKernelEx(&cfg, grouped_gemm_pair_kernel, tmap_a, a);
}

}  // namespace mt

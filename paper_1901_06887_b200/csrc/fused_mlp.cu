// Whole-pass executor for small batches of narrow MLP tenants: ONE launch does the bucketing, every dense layer of
// every tenant and the return to arrival order.
//     out[i] = W_L relu(... relu(W_1 x_i + b_1) ...) + b_L      with the weights of model_ids[i]
// A batch of a few hundred requests against layers at most 256 wide is bound by launch latency, not by bytes or
// flops: the layer-by-layer path spends six launches (bucketing, gather, three layers, un-permute) on a few
// microseconds of work.  Here every CTA repeats the (tiny) stable counting sort in shared memory, then takes work
// units (tenant, tile of up to 128 of its requests) and carries each through all layers without leaving the SM:
// the activations of the unit live in one shared-memory operand buffer (128 rows x 256 features, the swizzled
// K-major image the tensor core reads), each layer's accumulator is drained from TMEM through bias + ReLU straight
// back into that buffer as the next layer's input, and the last layer's fp32 rows go to the caller's buffer at
// their arrival positions.  Weights stream through a four-stage ring of 32 KiB (both 128-row tiles of one K block),
// fetched as bulk copies of the pre-swizzled images written at registration; the producer runs ahead across layers.
//
// Roles: warp 0 producer, warp 1 tcgen05.mma issuer, warps 2..9 gather / epilogue (two warps per TMEM lane quarter,
// which take the accumulator's 32-column chunks in turn: the drain of a layer is on the pass's critical path).
// Same semantics as the layer-by-layer path: the paper's layer-by-layer evaluation of a DNN (Sec. 1.1) for many
// co-resident models (Sec. 3).
#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kFusedThreads = 320;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kFusedEpiThreads = kFusedThreads - 64;   // 256
constexpr int kFusedStages = 4;
constexpr int kFusedStageBytes = 2 * TILE_BYTES;          // weight tiles (0, kb) and (1, kb)
constexpr int kFusedABytes = 4 * TILE_BYTES;              // 128 rows x 256 features, four K blocks
constexpr int kFusedTmemCols = 256;
constexpr int kFusedMisc = 1024;                          // barriers, TMEM slot, abort flag, bias

// Shared memory after the operand buffers: barriers | bias[256] | s_cnt[T+1] | s_off[T+2] | s_uoff[T+1] | s_perm[n]
__host__ __device__ inline size_t fused_smem_bytes(int n, int T) {
    return 1024 + kFusedABytes + kFusedStages * kFusedStageBytes + kFusedMisc + 1024 +
           sizeof(int32_t) * ((size_t)(T + 1) + (T + 2) + (T + 1) + (size_t)n + 8);
}

struct UnitCoord {
    int t, j0, rows;
};

__global__ void __launch_bounds__(kFusedThreads, 1)
fused_mlp_kernel(const FusedArgs p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t a_smem = base;                               // activations (A operand)
    const uint32_t w_smem = base + kFusedABytes;                // weight stages (B operand)
    uint8_t* misc = smem + kFusedABytes + kFusedStages * kFusedStageBytes;
    const uint32_t bar0 = w_smem + kFusedStages * kFusedStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kFusedStages + s); };
    const uint32_t acc_full_bar = bar0 + 8u * (2 * kFusedStages);
    const uint32_t act_ready_bar = acc_full_bar + 8u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 8 * (2 * kFusedStages + 2));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* s_bias = reinterpret_cast<float*>(misc + kFusedMisc);              // 256 floats
    int32_t* s_cnt = reinterpret_cast<int32_t*>(misc + kFusedMisc + 1024);
    const int T = p.T, T1 = p.T + 1, n = p.n;
    int32_t* s_off = s_cnt + T1;          // T + 2 entries
    int32_t* s_uoff = s_off + T1 + 1;     // T + 1 entries: work units before tenant t
    int32_t* s_perm = s_uoff + T1;        // n entries
    int32_t* s_chist = reinterpret_cast<int32_t*>(smem);   // [chunks][T1], borrowed from the activation buffer

    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_chunks = (n + 31) >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kFusedStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(acc_full_bar, 1);
        mbar_init(act_ready_bar, kFusedEpiThreads);
        *abort_flag = 0;
        fence_mbar_init();
    }
    for (int k = threadIdx.x; k < n_chunks * T1; k += kFusedThreads) s_chist[k] = 0;
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kFusedTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    pdl_wait();
    // ---------------------------------------------------------------- stable counting sort, repeated by every CTA
    // chunk c = requests [32c, 32c + 32): rank inside the chunk from the warp's match mask, per-chunk histogram
    constexpr int kMaxOwn = (512 / 32 + kFusedWarps - 1) / kFusedWarps;       // chunks one warp may own (2)
    int own_b[kMaxOwn], own_rank[kMaxOwn];
#pragma unroll
    for (int q = 0; q < kMaxOwn; ++q) {
        own_b[q] = -1; own_rank[q] = 0;
        const int c = warp + kFusedWarps * q;
        const int i = c * 32 + lane;
        if (c < n_chunks && i < n) {
            const int id = p.ids[i];
            const int alive = (id < 0 || id >= T) ? 0 : p.models[id].alive;     // 1 resident, 2 registered but evicted
            const int b = alive == 1 ? id : T;
            if (b == T && blockIdx.x == 0) {
                atomicCAS(&p.status[ST_CODE], MT_OK, alive == 2 ? MT_ERR_NOT_RESIDENT : MT_ERR_BAD_MODEL_ID);
                atomicMin(&p.status[ST_BAD_INDEX], i);
            }
            // (chunks are whole warps up to the batch's ragged end: the lanes with a request are lanes 0 .. n - 32c - 1)
            const unsigned live = (n - c * 32 >= 32) ? 0xffffffffu : ((1u << (n - c * 32)) - 1u);
            const unsigned peers = __match_any_sync(live, b);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            if (rank == 0) s_chist[c * T1 + b] = __popc(peers);
            own_b[q] = b; own_rank[q] = rank;
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < T1; t += kFusedThreads) {       // per bucket: exclusive prefix over the chunks
        int run = 0;
        for (int c = 0; c < n_chunks; ++c) {
            const int v = s_chist[c * T1 + t];
            s_chist[c * T1 + t] = run;
            run += v;
        }
        s_cnt[t] = run;
    }
    __syncthreads();
    if (warp == 0) {                                              // offsets and unit prefixes over the buckets
        const int per = (T1 + 31) >> 5;
        const int lo = min(lane * per, T1), hi = min(lo + per, T1);
        int sum = 0, usum = 0;
        for (int t = lo; t < hi; ++t) { sum += s_cnt[t]; if (t < T) usum += (s_cnt[t] + BM - 1) / BM; }
        int incl = sum, uincl = usum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, incl, d);
            const int uu = __shfl_up_sync(0xffffffffu, uincl, d);
            if (lane >= d) { incl += u; uincl += uu; }
        }
        int run = incl - sum, urun = uincl - usum;
        for (int t = lo; t < hi; ++t) {
            s_off[t] = run; run += s_cnt[t];
            if (t < T) { s_uoff[t] = urun; urun += (s_cnt[t] + BM - 1) / BM; }
        }
        if (lane == 31) { s_off[T1] = incl; s_uoff[T] = uincl; }
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < kMaxOwn; ++q) {
        const int c = warp + kFusedWarps * q;
        const int i = c * 32 + lane;
        if (own_b[q] >= 0) {
            const int pos = s_off[own_b[q]] + s_chist[c * T1 + own_b[q]] + own_rank[q];
            s_perm[pos] = i;
            if (blockIdx.x == 0) { p.perm[pos] = i; p.inv[i] = pos; }
        }
    }
    if (blockIdx.x == 0) {
        for (int t = threadIdx.x; t < T1; t += kFusedThreads) { p.counts[t] = s_cnt[t]; p.offsets[t] = s_off[t]; }
        if (threadIdx.x == 0) p.offsets[T1] = s_off[T1];
    }
    __syncthreads();          // s_chist (the activation buffer) is free from here on

    const int total_units = s_uoff[T];
    auto locate = [&](int u) {
        int lo = 0, hi = T;   // largest t with s_uoff[t] <= u (tenants without requests share their successor's value)
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_uoff[mid] <= u) lo = mid; else hi = mid;
        }
        UnitCoord c;
        c.t = lo;
        const int m = u - s_uoff[lo];
        c.j0 = s_off[lo] + m * BM;
        c.rows = min(BM, s_off[lo + 1] - c.j0);
        return c;
    };
    // (models of one family may differ in depth: every unit runs its own tenant's number of layers)

    if (warp == 0) {
        if (lane == 0) {   // ------------------------------------------------ producer: weight tiles of every layer
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x) {
                const UnitCoord c = locate(u);
                const int L = p.models[c.t].n_layers;
                for (int l = 0; ok && l < L; ++l) {
                    const LayerDev& Ld = p.models[c.t].layer[l];
                    const int kblocks = Ld.k_blocks, N = Ld.N;
                    const uint16_t* w = Ld.w;
                    // only the 8-row groups that hold output features are fetched
                    const uint32_t bytes0 = (uint32_t)((min(N, BN) + 7) & ~7) * 128u;
                    const uint32_t bytes1 = N > BN ? (uint32_t)((N - BN + 7) & ~7) * 128u : 0u;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 41)) { ok = false; break; }
                        const uint32_t dst = w_smem + stage * kFusedStageBytes;
                        mbar_expect_tx(full_bar(stage), bytes0 + bytes1);
                        bulk_load(dst, w + (size_t)kb * (BN * BK), bytes0, full_bar(stage));
                        if (bytes1) bulk_load(dst + TILE_BYTES, w + ((size_t)kblocks + kb) * (BN * BK), bytes1, full_bar(stage));
                        if (++stage == kFusedStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {   // ------------------------------------------------ MMA issuer
        const bool leader = elect_one();
        const uint32_t tmem_acc = __shfl_sync(0xffffffffu, *tmem_slot, 0);
        const uint32_t a_lo0 = desc_lo(a_smem), b_lo0 = desc_lo(w_smem);
        int stage = 0; uint32_t phase = 0;
        uint32_t act_phase = 0;
        bool ok = true;
        for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x) {
            const UnitCoord c = locate(u);
            const int L = p.models[c.t].n_layers;
            for (int l = 0; ok && l < L; ++l) {
                const LayerDev& Ld = p.models[c.t].layer[l];
                const int kblocks = Ld.k_blocks;
                const uint32_t idesc = make_idesc_bf16(BM, (Ld.N + 15) & ~15);
                // the layer's input is in place (gathered rows, or the previous layer's epilogue) and the accumulator
                // has been drained
                if (!mbar_wait(act_ready_bar, act_phase, abort_flag, p.status, 42)) { ok = false; break; }
                act_phase ^= 1u;
                tc_fence_after();
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 43)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + kb * (TILE_BYTES >> 4), b_lo = b_lo0 + stage * (kFusedStageBytes >> 4);
                    if (leader) {
                        if (kb == 0) umma_bf16_lohi<false>(tmem_acc, a_lo, b_lo, idesc);
                        else umma_bf16_lohi<true>(tmem_acc, a_lo, b_lo, idesc);
                        umma_bf16_lohi<true>(tmem_acc, a_lo + 2, b_lo + 2, idesc);
                        umma_bf16_lohi<true>(tmem_acc, a_lo + 4, b_lo + 4, idesc);
                        umma_bf16_lohi<true>(tmem_acc, a_lo + 6, b_lo + 6, idesc);
                        umma_commit(empty_bar(stage));
                    }
                    if (++stage == kFusedStages) { stage = 0; phase ^= 1u; }
                }
                if (ok && leader) umma_commit(acc_full_bar);
            }
        }
    } else {                  // ------------------------------------------------ gather + epilogue (warps 2..9)
        const int et = threadIdx.x - 64;            // 0..255
        const int q = warp & 3;                     // TMEM lane quarter this warp may read
        const int turn = (warp - 2) >> 2;           // which of the quarter's two warps: it takes chunks turn, turn + 2, ...
        const int r = q * 32 + lane;                // accumulator row = request of the unit
        uint32_t acc_phase = 0;
        bool ok = true;
        const bool out_vec_ok = (p.out_elems & 3) == 0 && (reinterpret_cast<uintptr_t>(p.out) & 15) == 0;
        if (blockIdx.x == 0) {
            // requests whose id was rejected sort behind every live segment and belong to no unit: NaN rows
            for (int j = s_off[T]; j < n; ++j) {
                float* dst = p.out + (size_t)s_perm[j] * p.out_elems;
                for (int e = et; e < p.out_elems; e += kFusedEpiThreads) dst[e] = __int_as_float(0x7fc00000);
            }
        }
        const int ld_ch = p.K0 >> 3;                // 16-byte chunks per row of the caller's buffer (the widest input)
        for (int u = blockIdx.x; ok && u < total_units; u += gridDim.x) {
            const UnitCoord c = locate(u);
            const int L = p.models[c.t].n_layers;
            const int cpr = p.models[c.t].layer[0].k_blocks << 3;    // chunks of a row that this tenant's first layer reads
            // gather the unit's rows (arrival order -> bucketed rows) into the operand buffer: row rr, chunk ch of the
            // row goes to K block ch / 8, 16-byte position (ch % 8) ^ (rr % 8) of the 128-byte swizzle row
            const uint4* src = reinterpret_cast<const uint4*>(p.inputs);
            {
                const int total_ch = c.rows * cpr;
                int idx = et;
                for (; idx + 3 * kFusedEpiThreads < total_ch; idx += 4 * kFusedEpiThreads) {   // four loads in flight
                    uint4 v[4];
                    int rr[4], ch[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int e = idx + k * kFusedEpiThreads;
                        rr[k] = e / cpr; ch[k] = e - rr[k] * cpr;
                        v[k] = __ldg(src + (size_t)s_perm[c.j0 + rr[k]] * ld_ch + ch[k]);
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<uint4*>(smem + (ch[k] >> 3) * TILE_BYTES + rr[k] * 128 + (((ch[k] & 7) ^ (rr[k] & 7)) << 4)) = v[k];
                }
                for (; idx < total_ch; idx += kFusedEpiThreads) {
                    const int rr = idx / cpr, ch = idx - rr * cpr;
                    const uint4 v = __ldg(src + (size_t)s_perm[c.j0 + rr] * ld_ch + ch);
                    *reinterpret_cast<uint4*>(smem + (ch >> 3) * TILE_BYTES + rr * 128 + (((ch & 7) ^ (rr & 7)) << 4)) = v;
                }
            }
            fence_proxy_async_smem();
            mbar_arrive(act_ready_bar);
            const bool row_ok = r < c.rows;
            const int arrival = row_ok ? s_perm[c.j0 + r] : 0;
            for (int l = 0; l < L; ++l) {
                const LayerDev& Ld = p.models[c.t].layer[l];
                const int N = Ld.N, relu = Ld.relu;
                const bool last = (l == L - 1);
                // The bias is fetched while the layer's MMAs run and parked in shared memory once the accumulator is
                // complete: by then every epilogue thread has finished with the previous layer's bias (the MMAs could
                // not start before all of them had handed over the layer's input).  The barrier that publishes it
                // also makes the give-up decision of a timed-out wait unanimous.
                const float bias_mine = (et < BN || N > BN) ? Ld.bias[et] : 0.0f;      // padded to whole 128-feature tiles
                const bool got = mbar_wait(acc_full_bar, acc_phase, abort_flag, p.status, 44);
                acc_phase ^= 1u;
                s_bias[et] = bias_mine;
                int any_failed;
                asm volatile(
                    "{\n\t"
                    ".reg .pred pi, po;\n\t"
                    "setp.ne.b32 pi, %1, 0;\n\t"
                    "bar.red.or.pred po, 1, 256, pi;\n\t"
                    "selp.u32 %0, 1, 0, po;\n\t"
                    "}\n"
                    : "=r"(any_failed) : "r"(got ? 0 : 1) : "memory");
                if (any_failed) { ok = false; break; }
                tc_fence_after();
                for (int n0 = turn * 32; n0 < N; n0 += 64) {
                    uint32_t v[32];
                    __syncwarp();
                    tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + n0, v);
                    tmem_ld_wait();
                    const float4* b4 = reinterpret_cast<const float4*>(s_bias + n0);
                    float f[32];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 b = b4[j];
                        f[4 * j + 0] = __uint_as_float(v[4 * j + 0]) + b.x;
                        f[4 * j + 1] = __uint_as_float(v[4 * j + 1]) + b.y;
                        f[4 * j + 2] = __uint_as_float(v[4 * j + 2]) + b.z;
                        f[4 * j + 3] = __uint_as_float(v[4 * j + 3]) + b.w;
                    }
                    if (relu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.0f);
                    }
                    if (!last) {
                        // next layer's input: features n0 .. n0 + 31 of row r, four 16-byte chunks of the swizzled image
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint4 o;
                            o.x = pack_bf16x2(f[8 * j + 0], f[8 * j + 1]);
                            o.y = pack_bf16x2(f[8 * j + 2], f[8 * j + 3]);
                            o.z = pack_bf16x2(f[8 * j + 4], f[8 * j + 5]);
                            o.w = pack_bf16x2(f[8 * j + 6], f[8 * j + 7]);
                            const int ch = (n0 >> 3) + j;
                            *reinterpret_cast<uint4*>(smem + (ch >> 3) * TILE_BYTES + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = o;
                        }
                    } else if (row_ok) {
                        float* dst = p.out + (size_t)arrival * p.out_elems + n0;
                        if (n0 + 32 <= N && out_vec_ok) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                reinterpret_cast<float4*>(dst)[j] = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (n0 + j < N) dst[j] = f[j];
                        }
                    }
                }
                tc_fence_before();
                if (!last) {
                    fence_proxy_async_smem();
                    mbar_arrive(act_ready_bar);
                }
            }
        }
    }

    if (*abort_flag) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, kFusedTmemCols);
    }
}

bool fused_mlp_fits(int n, int T, int max_width) {
    if (n < 1 || n > 512 || max_width > 256) return false;
    const size_t chist = sizeof(int32_t) * (size_t)((n + 31) / 32) * (T + 1);
    return chist <= (size_t)kFusedABytes && fused_smem_bytes(n, T) <= 227 * 1024;
}

cudaError_t configure_fused_mlp() {
    return cudaFuncSetAttribute(fused_mlp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t launch_fused_mlp(const FusedArgs& a, int grid, cudaStream_t s) {
    return launch_pdl(fused_mlp_kernel, dim3(grid), dim3(kFusedThreads), fused_smem_bytes(a.n, a.T), s, a);
}

}  // namespace mt

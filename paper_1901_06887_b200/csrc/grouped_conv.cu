// Grouped 3x3 convolution executor (NHWC, stride 1, zero pad 1, 64 -> 64 channels, bias + ReLU) as an implicit
// GEMM on the tensor cores, ONE persistent launch per layer for all tenants of the batch:
//     Y[r, y, x, o] = act(b_t[o] + sum_{ky,kx,c} X[r, y+ky-1, x+kx-1, c] * W_t[o, ky, kx, c])
//
// Shared-memory picture.  A strip of R output rows of one image is fetched, with its one-pixel halo, by ONE 4-D
// TMA box of (R+2) rows x Wp pixels x 64 channels (128 bytes per pixel, 128-byte swizzle); Wp is W+2 rounded up to
// 32, 64 or 128, and everything outside the image is zero-filled by the copy engine - that IS the zero padding.
// The strip is addressed flat: padded pixel q = yl * Wp + x.  Output pixel q of tap (ky,kx) needs input pixel
// q + ky*Wp + kx, so the A operand of every tap is the SAME strip started (ky*Wp + kx)*128 bytes further on: nine
// shifted matrix descriptors instead of nine copies.  An accumulator tile is 128 consecutive padded pixels
// (= 128/Wp image rows) x 64 output channels; pad columns (x >= W) are computed and never stored.
//
// Tap pairing (Wp == 64, the 56 x 56 workload).  A tcgen05.mma with M = 128 takes as long for N = 64 as for
// N = 128, so 64 output channels alone run the tensor pipe at half rate.  With Wp = 64 a tile is exactly two image
// rows, and the 128-pixel block that starts at an even padded row serves two tiles at once: tap row ky = 2 of the
// tile above it and tap row ky = 0 of the tile that starts there.  Their accumulators are neighbours in TMEM
// (a ring of eight 64-column slots), so ONE N = 128 instruction with B = [W(2,kx) ; W(0,kx)] updates both.  Six of
// the nine taps are issued this way, across strip borders too (the last tile of a strip is completed by the first
// block of the next strip of the same image).  The first instruction into a fresh accumulator must overwrite it,
// which a paired instruction cannot do for one half only, so every tile starts with its (unpaired) ky = 1 taps.
//
// The tenant's nine 64 x 64 tap tiles (72 KiB) stay resident in shared memory while consecutive strips belong to
// the same tenant; CTAs take contiguous ranges of strips, so they change tenant rarely.
//
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 epilogue (two warps per TMEM lane quarter, 32 output
// channels each: tcgen05.ld -> bias (shared memory) -> ReLU -> bf16 -> 128-bit stores).
//
// The paper does not define convolution; it only names a catalogue of standard layers (Sec. 1.1, Sec. 3.1).
#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kConvThreads = 320;
constexpr int kEpiThreads = 256;
constexpr int kCN = 64;                          // output channels
constexpr int kTapBytes = kCN * BK * 2;          // 8 KiB: 64 out channels x 64 in channels
constexpr int kWeightBytes = 9 * kTapBytes;      // 72 KiB, resident per tenant
constexpr int kMaxStages = 4;
constexpr int kSlots = 8;                        // TMEM ring: 8 accumulators of 64 columns = all 512 columns
constexpr int kConvBarBytes = 2048;
constexpr int kRecords = 16;                     // ring of per-strip records (producer -> MMA issuer, epilogue)

// Order of the tap tiles in the executor layout: the three ky = 1 taps, then for every kx the pair
// W(2,kx), W(0,kx) back to back, so that one 128-row B operand covers the pair.
__host__ __device__ constexpr int tap_slot(int ky, int kx) { return ky == 1 ? kx : (3 + 2 * kx + (ky == 0 ? 1 : 0)); }

struct StripCoord {
    int t, j, y0, strip_in_image;
};

// kSkip: the layer has tenants with an identity shortcut (ConvArgs::skip[0]); the plain form carries none of that code.
template <bool kSkip>
__global__ void __launch_bounds__(kConvThreads, 1)
grouped_conv3x3_kernel(const __grid_constant__ CUtensorMap tmap_x, const ConvArgs p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t w_smem = base;
    const uint32_t strip0 = base + kWeightBytes;
    const uint32_t bar0 = strip0 + p.n_stages * p.stage_bytes;
    uint8_t* bar_ptr = smem + kWeightBytes + p.n_stages * p.stage_bytes;
    auto sfull_bar = [&](int s) { return bar0 + 8u * s; };
    auto sempty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + kSlots + a); };
    const uint32_t wfull_bar = bar0 + 8u * (2 * kMaxStages + 2 * kSlots);
    const uint32_t wempty_bar = wfull_bar + 8u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_ptr + 8 * (2 * kMaxStages + 2 * kSlots + 2));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* s_bias = reinterpret_cast<float*>(bar_ptr + 256);          // 64 floats
    // Per-strip record written by the producer before it arms the strip's TMA load (so the mbarrier hand-over
    // publishes it): x = flags (1 new tenant, 2 pair with the tile above, 4 the next strip finishes the last
    // tile), y = image (bucketed index), z = first output row, w = tenant.  The issuing thread must not spend
    // time on index arithmetic: the tensor pipe drains as soon as it stops issuing.
    int4* s_rec = reinterpret_cast<int4*>(bar_ptr + 512);             // kRecords x 16 bytes
    float* s_pool = reinterpret_cast<float*>(bar_ptr + 1024);         // 8 warps x 32 channel sums (fused pooling)

    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(sfull_bar(s), 1); mbar_init(sempty_bar(s), 1); }
        for (int a = 0; a < kSlots; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), kEpiThreads); }
        mbar_init(wfull_bar, 1);
        mbar_init(wempty_bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
    }
    // the last rows of every strip stage are read (for rows that are never stored) but not written by the TMA box
    for (int i = threadIdx.x; i < (p.n_stages * p.stage_bytes) / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(smem + kWeightBytes)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kSlots * kCN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    pdl_wait();   // everything above overlapped the previous kernel's tail; its results are needed from here on
    // contiguous range of strips for this CTA
    const int total = p.tile_prefix[p.T];
    const int s_begin = (int)(((long long)total * blockIdx.x) / gridDim.x);
    const int s_end = (int)(((long long)total * (blockIdx.x + 1)) / gridDim.x);
    const int Wp = p.Wp;
    const int TS = p.tiles_per_strip;
    const bool pairing = (Wp == 64);

    // strip -> (tenant, image, first row); strips of one tenant are consecutive, so the tenant's range is cached
    int cur_t = -1, cur_lo = 0, cur_hi = 0, cur_seg = 0;
    auto locate = [&](int s) {
        if (s < cur_lo || s >= cur_hi) {
            int lo = 0, hi = p.T;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (p.tile_prefix[mid] <= s) lo = mid; else hi = mid;
            }
            cur_t = lo; cur_lo = p.tile_prefix[lo]; cur_hi = p.tile_prefix[lo + 1]; cur_seg = p.offsets[lo];
        }
        StripCoord c;
        const int local = s - cur_lo;
        const int img = local / p.strips_per_image;
        c.t = cur_t;
        c.j = cur_seg + img;
        c.strip_in_image = local - img * p.strips_per_image;
        c.y0 = c.strip_in_image * p.R;
        return c;
    };

    if (warp == 0) {
        if (lane == 0) {   // ------------------------------------------------ TMA producer
            int stage = 0; uint32_t phase = 0;
            int w_loads = 0, w_tenant = -1;
            for (int s = s_begin; s < s_end; ++s) {
                const StripCoord c = locate(s);
                const bool new_tenant = (c.t != w_tenant);
                if (!mbar_wait(sempty_bar(stage), phase ^ 1u, abort_flag, p.status, 22)) break;
                const int img = p.perm ? p.perm[c.j] : c.j;
                const bool pair_top = pairing && s > s_begin && c.strip_in_image > 0;
                const bool defer_bottom = pairing && s + 1 < s_end && c.strip_in_image + 1 < p.strips_per_image;
                s_rec[(s - s_begin) & (kRecords - 1)] =
                    make_int4((new_tenant ? 1 : 0) | (pair_top ? 2 : 0) | (defer_bottom ? 4 : 0), c.j, c.y0, c.t);
                mbar_expect_tx(sfull_bar(stage), p.box_bytes);
                tma_load_4d(strip0 + stage * p.stage_bytes, &tmap_x, 0, -1, c.y0 - 1, img, sfull_bar(stage));
                if (new_tenant) {
                    // This tenant's nine tap tiles.  The issuer learns of the change from the strip's record, i.e.
                    // after the strip has landed, and only then releases the old weights: so the strip goes first.
                    if (w_loads > 0 && !mbar_wait(wempty_bar, (uint32_t)((w_loads - 1) & 1), abort_flag, p.status, 21)) break;
                    mbar_expect_tx(wfull_bar, kWeightBytes);
                    bulk_load(w_smem, p.models[c.t].layer[p.layer].w, kWeightBytes, wfull_bar);
                    w_tenant = c.t;
                    ++w_loads;
                }
                if (++stage == p.n_stages) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        {                  // ------------------------------------------------ MMA issuer
            // The whole warp walks the loop (so that addresses and descriptors stay warp-uniform values); one elected
            // lane issues the MMAs and commits.
            const bool leader = elect_one();
            const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);   // warp-uniform copy
            constexpr uint32_t idesc64 = make_idesc_bf16(BM, kCN);
            constexpr uint32_t idesc128 = make_idesc_bf16(BM, 2 * kCN);
            int stage = 0; uint32_t phase = 0;
            int g = 0;                      // tiles started so far by this CTA; tile g lives in TMEM slot g % kSlots
            int w_loads = 0;
            bool ok = true;
            // Four K steps of one 128-pixel block against one (N = 64) or two stacked (N = 128) tap tiles.  Descriptors
            // are handled as their low words (address >> 4 | constant): stepping costs one add.
            const uint32_t w_lo = desc_lo(w_smem);
            constexpr uint32_t kTapLo = kTapBytes >> 4;          // one tap tile further
            constexpr uint32_t kPixLo = 128 >> 4;                // one pixel (128 bytes) further
            auto issue = [&](uint32_t a_lo, uint32_t b_lo, uint32_t d_tmem, uint32_t idesc, bool overwrite) {
                if (!leader) return;
                if (overwrite) umma_bf16_lohi<false>(d_tmem, a_lo, b_lo, idesc);
                else umma_bf16_lohi<true>(d_tmem, a_lo, b_lo, idesc);
                umma_bf16_lohi<true>(d_tmem, a_lo + 2, b_lo + 2, idesc);
                umma_bf16_lohi<true>(d_tmem, a_lo + 4, b_lo + 4, idesc);
                umma_bf16_lohi<true>(d_tmem, a_lo + 6, b_lo + 6, idesc);
            };
            // This thread is the only feeder of the tensor pipe, and its MMAs, commits and barrier polls go through one
            // in-order queue: an instruction whose result the thread needs (a barrier poll, a shared-memory load)
            // returns only after every MMA before it has been dispatched, and while the thread waits for it nothing
            // new is queued - the pipe runs dry.  So (1) the strip bookkeeping (new tenant? pair with the tile above?
            // leave the last tile to the next strip?) is kept in registers instead of being read from the producer's
            // record, and (2) the barriers of the NEXT tile and strip are polled (non-blocking) a few MMAs into the
            // current tile, and the answers are looked at only after the rest of the tile has been queued.
            int t_hi = -1;                  // strips [.., t_hi) belong to the current tenant
            int in_image = 0;               // index of the current strip inside its image
            uint32_t strip_ready = 0, slot_ready = 0;
            for (int s = s_begin; ok && s < s_end; ++s) {
                const bool new_tenant = (s >= t_hi);
                if (new_tenant) {           // rare: a tenant border (or the first strip)
                    const StripCoord c = locate(s);
                    t_hi = cur_hi;
                    in_image = c.strip_in_image;
                }
                if (!strip_ready) {
                    if (!mbar_wait(sfull_bar(stage), phase, abort_flag, p.status, 25)) break;
                }
                tc_fence_after();
                if (new_tenant) {
                    if (w_loads > 0 && leader) umma_commit(wempty_bar);      // fires when all MMAs on the old weights are done
                    if (!mbar_wait(wfull_bar, (uint32_t)(w_loads & 1), abort_flag, p.status, 23)) break;
                    ++w_loads;
                }
                const bool pair_top = pairing && s > s_begin && in_image > 0;
                const bool defer_bottom = pairing && s + 1 < s_end && in_image + 1 < p.strips_per_image;
                const uint32_t strip_lo = desc_lo(strip0 + stage * p.stage_bytes);
                const int next_stage = (stage + 1 == p.n_stages) ? 0 : stage + 1;
                const uint32_t next_phase = (stage + 1 == p.n_stages) ? (phase ^ 1u) : phase;
                strip_ready = 0;
                for (int i = 0; i < TS; ++i, ++g) {
                    const int slot = g % kSlots;
                    if (!slot_ready) {   // the accumulator slot must have been drained by the epilogue of tile g - kSlots
                        if (!mbar_wait(tempty_bar(slot), (uint32_t)(((g / kSlots) & 1) ^ 1), abort_flag, p.status, 24)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t d_this = tmem_base + slot * kCN;
                    const uint32_t blk = strip_lo + (uint32_t)(i * BM) * kPixLo;     // padded pixel i*128 of the strip
                    const bool last_tile = (i == TS - 1);
                    uint32_t poll_slot = 0, poll_strip = 0;
                    if (pairing) {
                        // ky = 1 first: these overwrite the fresh accumulator
                        issue(blk + (uint32_t)(Wp + 0) * kPixLo, w_lo + tap_slot(1, 0) * kTapLo, d_this, idesc64, true);
                        // look ahead: results are consumed after the rest of this tile has been queued
                        poll_slot = mbar_test_wait(tempty_bar((g + 1) % kSlots), (uint32_t)((((g + 1) / kSlots) & 1) ^ 1));
                        if (last_tile) poll_strip = mbar_test_wait(sfull_bar(next_stage), next_phase);
                        issue(blk + (uint32_t)(Wp + 1) * kPixLo, w_lo + tap_slot(1, 1) * kTapLo, d_this, idesc64, false);
                        issue(blk + (uint32_t)(Wp + 2) * kPixLo, w_lo + tap_slot(1, 2) * kTapLo, d_this, idesc64, false);
                        // block at the tile's first row: ky = 0 of this tile and ky = 2 of the tile above
                        const bool have_above = (i > 0) || pair_top;
                        const bool adjacent = slot != 0;                              // slots g-1 and g contiguous in TMEM
                        if (have_above && adjacent) {
#pragma unroll
                            for (int kx = 0; kx < 3; ++kx)
                                issue(blk + kx * kPixLo, w_lo + tap_slot(2, kx) * kTapLo, d_this - kCN, idesc128, false);
                        } else {
                            for (int kx = 0; kx < 3; ++kx) {
                                if (have_above)
                                    issue(blk + kx * kPixLo, w_lo + tap_slot(2, kx) * kTapLo, tmem_base + ((g - 1) % kSlots) * kCN, idesc64, false);
                                issue(blk + kx * kPixLo, w_lo + tap_slot(0, kx) * kTapLo, d_this, idesc64, false);
                            }
                        }
                        if (have_above && leader) umma_commit(tfull_bar((g - 1) % kSlots));    // tile above is complete
                    } else {
                        for (int tap = 0; tap < 9; ++tap) {
                            const int ky = tap / 3, kx = tap - 3 * ky;
                            issue(blk + (uint32_t)(ky * Wp + kx) * kPixLo, w_lo + tap_slot(ky, kx) * kTapLo, d_this, idesc64, tap == 0);
                            if (tap == 1) {
                                poll_slot = mbar_test_wait(tempty_bar((g + 1) % kSlots), (uint32_t)((((g + 1) / kSlots) & 1) ^ 1));
                                if (last_tile) poll_strip = mbar_test_wait(sfull_bar(next_stage), next_phase);
                            }
                        }
                        if (leader) umma_commit(tfull_bar(slot));
                    }
                    slot_ready = poll_slot;
                    if (last_tile) strip_ready = (s + 1 < s_end) ? poll_strip : 0;
                }
                if (!ok) break;
                if (pairing && !defer_bottom) {
                    // nobody below will finish the strip's last tile: its ky = 2 taps from the block under it
                    const uint32_t blk = strip_lo + (uint32_t)(TS * BM) * kPixLo;
                    const int last = (g - 1) % kSlots;
                    for (int kx = 0; kx < 3; ++kx)
                        issue(blk + kx * kPixLo, w_lo + tap_slot(2, kx) * kTapLo, tmem_base + last * kCN, idesc64, false);
                    if (leader) umma_commit(tfull_bar(last));
                }
                // The strip buffer is released by the epilogue (see there), not by a third commit here: a commit issued
                // while the previous one is still waiting for its MMAs stalls this thread until the queue has drained.
                stage = next_stage; phase = next_phase;
                if (++in_image == p.strips_per_image) in_image = 0;
            }
        }
    } else {               // ---------------------------------------------------- epilogue (warps 2..9)
        const int ew = warp - 2;
        const int q4 = warp & 3;                    // TMEM lane quarter this warp may read
        const int half = ew >> 2;                   // which 32 of the 64 output channels
        const int r = q4 * 32 + lane;               // tile-local padded pixel of this thread
        const int yl = r / Wp, x = r - yl * Wp;
        const int rows_per_tile = BM / Wp;
        int g = 0, relu = 0, resid = 0;
        bool ok = true;
        int img_j = 0, y0 = 0;
        int skip_img = 0;                           // image index of the strip in the tensor a residual layer adds
        const bool pooling = (p.pool_partial != nullptr);
        for (int s = s_begin; ok && s < s_end; ++s) {
            float psum[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) psum[e] = 0.0f;
            for (int i = 0; i < TS; ++i, ++g) {
                const int slot = g % kSlots;
                if (!mbar_wait(tfull_bar(slot), (uint32_t)((g / kSlots) & 1), abort_flag, p.status, 26)) { ok = false; break; }
                // The completion of a strip's last tile is signalled after every MMA that reads the strip's buffer (by
                // the strip's own last instruction, or by the next strip when the tile was left to it): release it.
                if (i == TS - 1 && threadIdx.x == 64) mbar_arrive(sempty_bar((s - s_begin) % p.n_stages));
                if (i == 0) {
                    // the strip's record was published (with the strip's data) before any of its MMAs were issued
                    const int4 rec = s_rec[(s - s_begin) & (kRecords - 1)];
                    img_j = rec.y; y0 = rec.z;
                    if (rec.x & 1) {                // new tenant: its bias into shared memory, ReLU flag into a register
                        const LayerDev& L = p.models[rec.w].layer[p.layer];
                        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // everyone done with the old bias
                        if (threadIdx.x - 64 < kCN) s_bias[threadIdx.x - 64] = L.bias[threadIdx.x - 64];
                        relu = L.relu;
                        if constexpr (kSkip) resid = (L.residual && p.skip[0] != nullptr) ? 1 : 0;
                        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                    }
                    if constexpr (kSkip) {
                        if (resid) skip_img = p.skip_perm[0] ? p.skip_perm[0][img_j] : img_j;
                    }
                }
                tc_fence_after();
                uint32_t v[32];
                tmem_ld32(tmem_base + (static_cast<uint32_t>(q4 * 32) << 16) + slot * kCN + half * 32, v);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(tempty_bar(slot));      // values are in registers: the slot can be reused
                const int y = y0 + i * rows_per_tile + yl;
                if (x < p.W && y < p.H) {
                    uint16_t* dst = p.out + (((size_t)img_j * p.H + y) * p.W + x) * kCN + half * 32;
                    const float4* b4 = reinterpret_cast<const float4*>(s_bias + half * 32);
                    // identity shortcut: this thread's pixel of the block's input, 32 channels = 64 bytes
                    uint4 sk[4];
                    if constexpr (kSkip) if (resid) {
                        const uint4* sp = reinterpret_cast<const uint4*>(
                            p.skip[0] + (((size_t)skip_img * p.H + y) * p.W + x) * kCN + half * 32);
#pragma unroll
                        for (int j = 0; j < 4; ++j) sk[j] = __ldcg(sp + j);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float f[8];
#pragma unroll
                        for (int h2 = 0; h2 < 2; ++h2) {
                            const float4 b = b4[2 * j + h2];
                            f[4 * h2 + 0] = __uint_as_float(v[8 * j + 4 * h2 + 0]) + b.x;
                            f[4 * h2 + 1] = __uint_as_float(v[8 * j + 4 * h2 + 1]) + b.y;
                            f[4 * h2 + 2] = __uint_as_float(v[8 * j + 4 * h2 + 2]) + b.z;
                            f[4 * h2 + 3] = __uint_as_float(v[8 * j + 4 * h2 + 3]) + b.w;
                        }
                        if constexpr (kSkip) if (resid) {
                            const uint32_t w4[4] = {sk[j].x, sk[j].y, sk[j].z, sk[j].w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {       // two bf16 per word, the lower address in the low half
                                f[2 * e + 0] += __uint_as_float(w4[e] << 16);
                                f[2 * e + 1] += __uint_as_float(w4[e] & 0xffff0000u);
                            }
                        }
                        if (relu) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) f[e] = fmaxf(f[e], 0.0f);
                        }
                        if (pooling) {      // the layer feeds a global average pool: only channel sums are kept
#pragma unroll
                            for (int e = 0; e < 8; ++e) psum[8 * j + e] += f[e];
                        } else {
                            uint4 o;
                            o.x = pack_bf16x2(f[0], f[1]);
                            o.y = pack_bf16x2(f[2], f[3]);
                            o.z = pack_bf16x2(f[4], f[5]);
                            o.w = pack_bf16x2(f[6], f[7]);
                            reinterpret_cast<uint4*>(dst)[j] = o;
                        }
                    }
                }
                __syncwarp();
            }
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
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                const int et = threadIdx.x - 64;                    // 0..255 among the epilogue threads
                if (et < kCN) {
                    const int hf = et >> 5, c = et & 31;
                    const float* q = s_pool + (hf * 4) * 32 + c;     // warps hf*4 .. hf*4+3 hold this half's quarters
                    // quarter order by TMEM lane quarter (ew & 3 maps to q4 = (ew + 2) & 3): sum in pixel order 0,1,2,3
                    const float t = ((q[2 * 32] + q[3 * 32]) + q[0 * 32]) + q[1 * 32];
                    p.pool_partial[((size_t)img_j * p.strips_per_image + y0 / p.R) * kCN + et] = t;
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
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
        tmem_dealloc(tmem_base, kSlots * kCN);
    }
}

// Strip geometry for an H x W image (W <= 126).
bool plan_conv(int H, int W, ConvPlan* plan) {
    if (W < 1 || H < 1 || W + 2 > 128) return false;
    const int Wp = (W + 2 <= 32) ? 32 : (W + 2 <= 64) ? 64 : 128;
    const int rows_per_tile = BM / Wp;
    const int TS = 2;                                         // accumulator tiles per strip
    const int R = TS * rows_per_tile;
    if (R + 2 > 256) return false;
    const int box = (R + 2) * Wp * 128;
    const int stage = box + 1024;                             // taps shifted by up to 2 pixels read past the box
    int stages = (227 * 1024 - kWeightBytes - kConvBarBytes - 1024) / stage;
    if (stages < 2) return false;
    if (stages > kMaxStages) stages = kMaxStages;
    plan->Wp = Wp; plan->R = R; plan->tiles_per_strip = TS; plan->stage_bytes = stage; plan->n_stages = stages;
    plan->strips_per_image = (H + R - 1) / R;
    plan->box_bytes = box;
    plan->smem_bytes = kWeightBytes + stages * stage + kConvBarBytes + 1024;
    return true;
}

// Conv weights W[64][3][3][64] -> nine tap tiles of 64 rows (out channel) x 64 columns (in channel), each the
// 8 KiB swizzled shared-memory image; tile order given by tap_slot().
__global__ void pretile_conv_kernel(const uint16_t* __restrict__ w, int C_out, int C_in, uint4* __restrict__ out,
                                    int total_chunks) {
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total_chunks; idx += gridDim.x * blockDim.x) {
        const int tap = idx / (C_out * 8);                   // natural tap index ky * 3 + kx
        const int within = idx % (C_out * 8);
        const int r = within >> 3, cpos = within & 7;
        const int c = cpos ^ (r & 7);
        const int ky = tap / 3, kx = tap - 3 * ky;
        out[tap_slot(ky, kx) * (C_out * 8) + within] =
            *reinterpret_cast<const uint4*>(w + ((size_t)r * 9 + tap) * C_in + c * 8);
    }
}

void launch_pretile_conv(const uint16_t* w, int C_out, int C_in, uint16_t* out, cudaStream_t s) {
    const int total = 9 * C_out * 8;
    pretile_conv_kernel<<<(total + 255) / 256, 256, 0, s>>>(w, C_out, C_in, reinterpret_cast<uint4*>(out), total);
}

// g[j][c] = (1 / HW) * sum over the image's strips of pool_partial[j][strip][c] (fixed order), rounded to bf16.
__global__ void pool_finalize_kernel(const float* __restrict__ partial, int n, int strips, int C, float inv_hw,
                                     uint16_t* __restrict__ out, int ld_out, unsigned* grid_bar) {
    pdl_launch_dependents();
    pdl_wait();
    if (grid_bar && blockIdx.x == 0 && threadIdx.x < 8) grid_bar[threadIdx.x] = 0u;   // the conv launches are done with them
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n * C) return;
    const int j = idx / C, c = idx - j * C;
    float s = 0.f;
    for (int k = 0; k < strips; ++k) s += partial[((size_t)j * strips + k) * C + c];
    out[(size_t)j * ld_out + c] = static_cast<uint16_t>(pack_bf16x2(s * inv_hw, 0.0f) & 0xFFFFu);
}

void launch_pool_finalize(const float* partial, int n, int strips, int C, int HW, uint16_t* out, int ld_out,
                          unsigned* grid_bar, cudaStream_t s) {
    launch_pdl(pool_finalize_kernel, dim3((n * C + 255) / 256), dim3(256), 0, s, partial, n, strips, C, 1.0f / (float)HW, out, ld_out,
               grid_bar);
}

// Pool + narrow head in one launch: for every image, finish the global average pool (sum the strips' channel sums in
// a fixed order, divide by H*W, round to bf16 - exactly what pool_finalize hands to a dense layer) and apply the
// model's last dense layer (64 -> at most 64 outputs, fp32 accumulate, bias, optional ReLU), writing the fp32 row to
// the request's arrival position.  One warp per image: lane c holds channels c and c + 32.  Rows of rejected requests
// (bucketed rows at and after offsets[T]) become NaN.  The head's weights are read from the executor's tiled image
// (128 rows x 64 columns per tile, 16-byte chunk c of row r at chunk c ^ (r & 7)); K = 64 is one tile column.
__global__ void __launch_bounds__(256)
pool_head_kernel(const float* __restrict__ partial, int n, int strips, float inv_hw, const ModelDev* __restrict__ models,
                 int layer, const int32_t* __restrict__ offsets, int T, const int32_t* __restrict__ perm,
                 float* __restrict__ out, int out_elems, unsigned* grid_bar) {
    pdl_launch_dependents();
    pdl_wait();
    if (grid_bar && blockIdx.x == 0 && threadIdx.x < 8) grid_bar[threadIdx.x] = 0u;   // the conv launches are done with them
    const int lane = threadIdx.x & 31;
    const int j = blockIdx.x * 8 + (threadIdx.x >> 5);          // bucketed row = image
    if (j >= n) return;
    float* dst = out + (size_t)perm[j] * out_elems;
    if (j >= offsets[T]) {                                       // rejected id: no model
        for (int o = lane; o < out_elems; o += 32) dst[o] = __int_as_float(0x7fc00000);
        return;
    }
    int lo = 0, hi = T;                                          // tenant of row j: largest t with offsets[t] <= j
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (offsets[mid] <= j) lo = mid; else hi = mid;
    }
    const LayerDev& L = models[lo].layer[layer];
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 4
    for (int k = 0; k < strips; ++k) {      // fixed order: the pooled value does not depend on timing
        const float* q = partial + ((size_t)j * strips + k) * 64;
        s0 += __ldg(q + lane);
        s1 += __ldg(q + lane + 32);
    }
    // the pooled activation as the dense executor would see it: rounded to bf16
    const float p0 = __uint_as_float(pack_bf16x2(0.0f, s0 * inv_hw) & 0xFFFF0000u);
    const float p1 = __uint_as_float(pack_bf16x2(0.0f, s1 * inv_hw) & 0xFFFF0000u);
    const uint16_t* w = L.w;
    const float* bias = L.bias;
    const int N = L.N, relu = L.relu;
    const int c0 = lane, c1 = lane + 32;
    for (int o0 = 0; o0 < N; o0 += 8) {
        // W[o][c] in the tiled image: row o of tile 0, chunk (c / 8) ^ (o & 7), element c % 8.  Eight outputs at a
        // time, their weights fetched before any of the reductions.
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int o = min(o0 + e, N - 1);
            const float w0 = __uint_as_float((uint32_t)__ldg(w + o * 64 + (((c0 >> 3) ^ (o & 7)) << 3) + (c0 & 7)) << 16);
            const float w1 = __uint_as_float((uint32_t)__ldg(w + o * 64 + (((c1 >> 3) ^ (o & 7)) << 3) + (c1 & 7)) << 16);
            acc[e] = p0 * w0 + p1 * w1;
        }
        const float b = (o0 + (lane & 7) < N) ? __ldg(bias + o0 + (lane & 7)) : 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], d);
        }
        // lane e (< 8) writes output o0 + e
        float mine = acc[0];
#pragma unroll
        for (int e = 1; e < 8; ++e) mine = ((lane & 7) == e) ? acc[e] : mine;
        if (lane < 8 && o0 + lane < N) {
            float v = mine + b;
            if (relu) v = fmaxf(v, 0.0f);
            dst[o0 + lane] = v;
        }
    }
}

void launch_pool_head(const float* partial, int n, int strips, int HW, const ModelDev* models, int layer,
                      const int32_t* offsets, int T, const int32_t* perm, float* out, int out_elems, unsigned* grid_bar,
                      cudaStream_t s) {
    launch_pdl(pool_head_kernel, dim3((n + 7) / 8), dim3(256), 0, s, partial, n, strips, 1.0f / (float)HW, models, layer,
               offsets, T, perm, out, out_elems, grid_bar);
}

cudaError_t configure_grouped_conv() {
    cudaError_t e = cudaFuncSetAttribute(grouped_conv3x3_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(grouped_conv3x3_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

void launch_grouped_conv(const CUtensorMap& tmap_x, const ConvArgs& a, int smem_bytes, int sm_count, cudaStream_t s) {
    if (a.skip[0]) launch_pdl(grouped_conv3x3_kernel<true>, dim3(sm_count), dim3(kConvThreads), (size_t)smem_bytes, s, tmap_x, a);
    else launch_pdl(grouped_conv3x3_kernel<false>, dim3(sm_count), dim3(kConvThreads), (size_t)smem_bytes, s, tmap_x, a);
}

}  // namespace mt

// Grouped 3x3 convolution executor (NHWC, stride 1, zero pad 1, 64 -> 64 channels, bias + ReLU) as an
// implicit GEMM on the tensor cores, one persistent launch per layer for all tenants of the batch:
//     Y[r, y, x, o] = act(b_t[o] + sum_{ky,kx,c} X[r, y+ky-1, x+kx-1, c] * W_t[o, ky, kx, c])
// GEMM view per work item: M = one strip of `rows_per_tile` image rows (rows_per_tile * W <= 128 pixels),
// N = 64 output channels, K = 9 taps x 64 input channels.  One pipeline stage = one tap: the strip shifted
// by (ky-1, kx-1) is fetched by a 4-D TMA box whose out-of-image part is zero-filled by the hardware (that
// IS the zero padding), and the tap's 64 x 64 weight tile arrives as an 8 KiB bulk copy of a pre-swizzled
// image.  Images are addressed by index, so the first layer reads the caller's buffer through the bucketing
// permutation and no image is ever moved to group requests.
//
// The paper does not define convolution; it only names a catalogue of standard layers (Sec. 1.1, Sec. 3.1).
#include "mt_device.cuh"
#include "mt_host.h"

namespace mt {

constexpr int kConvStages = 6;
constexpr int kConvN = 64;
constexpr int kTapBytes = kConvN * BK * 2;                       // 8 KiB: 64 out channels x 64 in channels
constexpr int kConvStageBytes = TILE_BYTES + kTapBytes;          // strip (<= 16 KiB) + tap weights
constexpr int kConvThreads = 192;
constexpr int kConvTmemCols = 128;                               // two 64-column accumulators
constexpr int kConvSmem = kConvStages * kConvStageBytes + 256 + 1024;

struct ConvTile {
    int t, j, y0;
};

__device__ __forceinline__ ConvTile decode_conv_tile(int item, const ConvArgs& p) {
    int lo = 0, hi = p.T;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (p.tile_prefix[mid] <= item) lo = mid; else hi = mid;
    }
    const int local = item - p.tile_prefix[lo];
    const int img = local / p.tiles_per_image;
    ConvTile c;
    c.t = lo;
    c.j = p.offsets[lo] + img;
    c.y0 = (local - img * p.tiles_per_image) * p.rows_per_tile;
    return c;
}

__global__ void __launch_bounds__(kConvThreads, 1)
grouped_conv3x3_kernel(const __grid_constant__ CUtensorMap tmap_x, const ConvArgs p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kConvStages * kConvStageBytes);
    const uint32_t bar0 = base + kConvStages * kConvStageBytes;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kConvStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kConvStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kConvStages + 2 + a); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kConvStages + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kConvStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 128); }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmap_x);
    }
    // rows of the strip buffer that no TMA box ever writes (W * rows_per_tile .. 127) must not hold NaN
    // patterns forever: clear all stage buffers once (their accumulator rows are never stored anyway)
    for (int i = threadIdx.x; i < kConvStages * kConvStageBytes / 16; i += blockDim.x)
        reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async_smem();
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kConvTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int total = p.tile_prefix[p.T];
    const int strip_pixels = p.rows_per_tile * p.W;
    const uint32_t strip_bytes = (uint32_t)strip_pixels * 128u;

    if (warp == 0) {
        if (lane == 0) {   // ------------------------------------------------ TMA producer
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < total; item += gridDim.x) {
                const ConvTile c = decode_conv_tile(item, p);
                const uint16_t* wsrc = p.models[c.t].layer[p.layer].w;
                const int img = p.perm ? p.perm[c.j] : c.j;
                for (int tap = 0; tap < 9; ++tap) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, 11)) { ok = false; break; }
                    const int ky = tap / 3, kx = tap - 3 * ky;
                    const uint32_t a_dst = base + stage * kConvStageBytes;
                    mbar_expect_tx(full_bar(stage), strip_bytes + kTapBytes);
                    tma_load_4d(a_dst, &tmap_x, 0, kx - 1, c.y0 + ky - 1, img, full_bar(stage));
                    bulk_load(a_dst + TILE_BYTES, wsrc + (size_t)tap * (kConvN * BK), kTapBytes, full_bar(stage));
                    if (++stage == kConvStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {   // ------------------------------------------------ MMA issuer
            constexpr uint32_t idesc = make_idesc_bf16(BM, kConvN);
            int stage = 0; uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < total; item += gridDim.x, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status, 12)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kConvN;
                for (int tap = 0; tap < 9; ++tap) {
                    if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status, 13)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = base + stage * kConvStageBytes;
                    const uint64_t a_desc = make_kmajor_sw128_desc(a_src, 1024);
                    const uint64_t b_desc = make_kmajor_sw128_desc(a_src + TILE_BYTES, 1024);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k)
                        umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (tap | k) != 0);
                    umma_commit(empty_bar(stage));
                    if (++stage == kConvStages) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar(acc));
            }
        }
    } else {               // ---------------------------------------------------- epilogue (warps 2..5)
        const int q = warp & 3;
        const int r = q * 32 + lane;            // pixel of the strip handled by this thread
        int it = 0;
        for (int item = blockIdx.x; item < total; item += gridDim.x, ++it) {
            const ConvTile c = decode_conv_tile(item, p);
            const LayerDev& L = p.models[c.t].layer[p.layer];
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status, 14)) break;
            tc_fence_after();
            const bool row_ok = (r < strip_pixels) && (c.y0 + r / p.W < p.H);
            uint16_t* dst = p.out + (((size_t)c.j * p.H + c.y0) * p.W + r) * kConvN;
            const int relu = L.relu;
#pragma unroll 1
            for (int ch = 0; ch < kConvN / 32; ++ch) {
                uint32_t v[32];
                __syncwarp();
                tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * kConvN + ch * 32, v);
                tmem_ld_wait();
                const float4* b4 = reinterpret_cast<const float4*>(L.bias + ch * 32);
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
                if (row_ok) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 o;
                        o.x = pack_bf16x2(f[8 * j + 0], f[8 * j + 1]);
                        o.y = pack_bf16x2(f[8 * j + 2], f[8 * j + 3]);
                        o.z = pack_bf16x2(f[8 * j + 4], f[8 * j + 5]);
                        o.w = pack_bf16x2(f[8 * j + 6], f[8 * j + 7]);
                        reinterpret_cast<uint4*>(dst + ch * 32)[j] = o;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(tempty_bar(acc));
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
        tmem_dealloc(tmem_base, kConvTmemCols);
    }
}

// g[j][c] = (1 / HW) * sum_p x[j][p][c]; one CTA per image, 8 channels (16 bytes) per thread per pixel.
constexpr int kPoolThreads = 256;

__global__ void __launch_bounds__(kPoolThreads)
global_avg_pool_kernel(const uint16_t* __restrict__ x, int HW, int C, uint16_t* __restrict__ out, int ld_out) {
    extern __shared__ float s_part[];   // [groups][C]
    const int vec_per_pixel = C / 8;
    const int groups = kPoolThreads / vec_per_pixel;      // pixels processed per iteration
    const int g_id = threadIdx.x / vec_per_pixel, v = threadIdx.x % vec_per_pixel;
    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)blockIdx.x * HW * C);
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (g_id < groups) {
        for (int pix = g_id; pix < HW; pix += groups) {
            const uint4 q = __ldg(&src[(size_t)pix * vec_per_pixel + v]);
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k + 0] += __uint_as_float(w[k] << 16);
                acc[2 * k + 1] += __uint_as_float(w[k] & 0xFFFF0000u);
            }
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) s_part[g_id * C + v * 8 + k] = acc[k];
    }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        float s = 0.f;
        for (int gi = 0; gi < groups; ++gi) s += s_part[gi * C + c];
        const float m = s / (float)HW;
        out[(size_t)blockIdx.x * ld_out + c] = static_cast<uint16_t>(pack_bf16x2(m, 0.0f) & 0xFFFFu);
    }
}

cudaError_t configure_grouped_conv() {
    return cudaFuncSetAttribute(grouped_conv3x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kConvSmem);
}

void launch_grouped_conv(const CUtensorMap& tmap_x, const ConvArgs& a, int sm_count, cudaStream_t s) {
    grouped_conv3x3_kernel<<<sm_count, kConvThreads, kConvSmem, s>>>(tmap_x, a);
}

void launch_global_avg_pool(const uint16_t* x, int n, int HW, int C, uint16_t* out, int ld_out, int /*sm_count*/,
                            cudaStream_t s) {
    const int groups = kPoolThreads / (C / 8);
    global_avg_pool_kernel<<<n, kPoolThreads, sizeof(float) * groups * C, s>>>(x, HW, C, out, ld_out);
}

}  // namespace mt

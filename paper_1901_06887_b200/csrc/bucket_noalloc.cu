// Bucketing for callers that cannot allocate device memory.
//
// mt_infer keeps its bucketing scratch (per-block histograms) in a workspace it allocates with cudaMalloc
// and grows on demand.  Some callers may not do that: code running inside a framework's memory-pool
// callback or allocator hook, a real-time serving loop that has frozen its memory map after start-up, a
// process whose device memory is entirely owned by another allocator, or a library called while the CUDA
// context's allocator lock must not be taken.  mt_bucket_noalloc gives them the same stable counting sort
// (counts, offsets, perm, inv) with the scratch held in a fixed array that is part of the library image:
// every GPU that loads the library carries kScratchInts * 4 = 1,057,804 bytes (1.01 MiB) until the process exits.
// The FIRST call on a device may still allocate inside the driver: with lazy module loading that call loads this
// file's kernels and places the scratch array.  Make it once at start-up (n = 0 is enough), outside any allocator
// hook or frozen-memory phase; every later call on that device allocates nothing.
//
// The kernels below are separate copies of the bucketing passes, without the model table: an id is valid iff
// it lies in [0, n_models).
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/mt.h"

namespace {

constexpr int kChunk = 256;                                   // requests per CTA
constexpr int kMaxBatch = MT_NOALLOC_MAX_BATCH;
constexpr int kMaxModels = MT_NOALLOC_MAX_MODELS;
constexpr int kMaxBlocks = (kMaxBatch + kChunk - 1) / kChunk;
constexpr int kHistInts = kMaxBlocks * (kMaxModels + 1);      // per-block histograms, one extra bucket for bad ids
constexpr int kOffsetInts = kMaxModels + 2;                   // offsets incl. the extra bucket and the total
constexpr int kCountInts = kMaxModels + 1;
constexpr int kScratchInts = kHistInts + kOffsetInts + kCountInts;
constexpr int kScanThreads = 1024;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; it is not a device
// address and must never be passed to a kernel.
static __device__ __align__(256) int32_t g_noalloc_scratch[kScratchInts];

__device__ __forceinline__ int bucket_of(int id, int T) { return (id < 0 || id >= T) ? T : id; }

__global__ void __launch_bounds__(kChunk)
na_block_hist(const int32_t* __restrict__ ids, int n, int T, int32_t* __restrict__ block_hist) {
    extern __shared__ int32_t s_hist[];
    const int T1 = T + 1;
    for (int t = threadIdx.x; t < T1; t += blockDim.x) s_hist[t] = 0;
    __syncthreads();
    const int i = blockIdx.x * kChunk + threadIdx.x;
    if (i < n) {
        const int b = bucket_of(ids[i], T);
        const unsigned peers = __match_any_sync(__activemask(), b);
        if ((__ffs(peers) - 1) == (threadIdx.x & 31)) atomicAdd(&s_hist[b], __popc(peers));
    }
    __syncthreads();
    // every entry that the later passes read is written here, so stale contents of the shared scratch from an
    // earlier call are never observed and nothing has to be cleared between calls
    for (int t = threadIdx.x; t < T1; t += blockDim.x) block_hist[(size_t)blockIdx.x * T1 + t] = s_hist[t];
}

__global__ void __launch_bounds__(kScanThreads)
na_scan(int n_blocks, int T, int32_t* __restrict__ block_hist, int32_t* __restrict__ counts_s,
        int32_t* __restrict__ offsets_s, int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out) {
    __shared__ int32_t s_tmp[kScanThreads];
    const int T1 = T + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int t = warp; t < T1; t += kScanThreads / 32) {      // per bucket: total, and exclusive prefix over blocks
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
        if (lane == 0) counts_s[t] = carry;
    }
    __syncthreads();
    // exclusive scan of the T + 1 bucket totals (T + 1 <= 1025: at most two items per thread)
    const int tid = threadIdx.x;
    const int per = (T1 + kScanThreads - 1) / kScanThreads;
    const int lo = min(tid * per, T1), hi = min(lo + per, T1);
    int sum = 0;
    for (int j = lo; j < hi; ++j) sum += counts_s[j];
    s_tmp[tid] = sum;
    __syncthreads();
    for (int d = 1; d < kScanThreads; d <<= 1) {
        const int v = (tid >= d) ? s_tmp[tid - d] : 0;
        __syncthreads();
        s_tmp[tid] += v;
        __syncthreads();
    }
    int run = s_tmp[tid] - sum;
    for (int j = lo; j < hi; ++j) {
        offsets_s[j] = run;
        if (j <= T) offsets_out[j] = run;
        if (j < T) counts_out[j] = counts_s[j];
        run += counts_s[j];
    }
    if (tid == kScanThreads - 1) offsets_s[T1] = s_tmp[tid];
}

__global__ void __launch_bounds__(kChunk)
na_scatter(const int32_t* __restrict__ ids, int n, int T, const int32_t* __restrict__ block_hist,
           const int32_t* __restrict__ offsets_s, int32_t* __restrict__ perm, int32_t* __restrict__ inv) {
    extern __shared__ int32_t s_next[];
    const int T1 = T + 1;
    for (int t = threadIdx.x; t < T1; t += blockDim.x)
        s_next[t] = offsets_s[t] + block_hist[(size_t)blockIdx.x * T1 + t];
    __syncthreads();
    const int i = blockIdx.x * kChunk + threadIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = (i < n) ? bucket_of(ids[i], T) : -1;
    // lanes that hold a request, agreed on by the whole warp before the divergent branch (the ranks are only right
    // if every such lane takes part in the match)
    const unsigned live = __ballot_sync(0xffffffffu, i < n);
    for (int w = 0; w < kChunk / 32; ++w) {                   // warps take turns, so the sort is stable
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

std::mutex g_setup_mu;
int32_t* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device; resolved once per device.
mt_status scratch_for_current_device(int32_t** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MT_ERR_CUDA;
    std::lock_guard<std::mutex> lk(g_setup_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return MT_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_scratch_ptr[dev];
    return MT_OK;
}

}  // namespace

extern "C" mt_status mt_bucket_noalloc(const int32_t* model_ids, int32_t n, int32_t n_models, int32_t* counts_out,
                                       int32_t* offsets_out, int32_t* perm_out, int32_t* inv_out, void* stream) {
    if (n < 0 || n_models < 1) return MT_ERR_INVALID_ARG;
    if (n > kMaxBatch || n_models > kMaxModels) return MT_ERR_UNSUPPORTED;   // beyond the fixed scratch
    if (!counts_out || !offsets_out) return MT_ERR_INVALID_ARG;
    if (n > 0 && (!model_ids || !perm_out || !inv_out)) return MT_ERR_INVALID_ARG;
    int32_t* scratch = nullptr;
    const mt_status st = scratch_for_current_device(&scratch);
    if (st != MT_OK) return st;
    int32_t* block_hist = scratch;
    int32_t* offsets_s = scratch + kHistInts;
    int32_t* counts_s = offsets_s + kOffsetInts;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n_blocks = (n + kChunk - 1) / kChunk;           // 0 for an empty batch: the scan then writes zeros
    const size_t smem = sizeof(int32_t) * (size_t)(n_models + 1);
    if (n_blocks > 0) na_block_hist<<<n_blocks, kChunk, smem, s>>>(model_ids, n, n_models, block_hist);
    na_scan<<<1, kScanThreads, 0, s>>>(n_blocks, n_models, block_hist, counts_s, offsets_s, counts_out, offsets_out);
    if (n_blocks > 0)
        na_scatter<<<n_blocks, kChunk, smem, s>>>(model_ids, n, n_models, block_hist, offsets_s, perm_out, inv_out);
    return cudaGetLastError() == cudaSuccess ? MT_OK : MT_ERR_CUDA;
}

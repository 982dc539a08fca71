// Top-k selection (Algorithm 1, the top-k step) with a total order: score descending, then
// index ascending. Each score becomes a 64-bit key whose high word is the bitwise complement of an
// order-preserving integer image of the float and whose low word is the row index; every key is
// distinct, so an ascending LSD radix sort of the keys (8-bit digits, stable scatter) puts the rows in
// exactly that order and the first k low words are the answer. Integer work only: results are exact.
#include <cstdio>
#include <mutex>

#include "sage_internal.h"

namespace sage {
namespace {

constexpr int kThreads = 256;
constexpr int kItems = 16;
constexpr int kTile = kThreads * kItems;   // keys per block
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ uint32_t ordered_bits(float f) {
    if (f != f) return 0u;                                   // NaN ranks below everything
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);       // larger float <-> larger integer
}

__global__ void __launch_bounds__(kThreads) k_make_keys(const float* __restrict__ scores, int64_t N,
                                                        unsigned long long* __restrict__ keys) {
    const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i >= N) return;
    float s = scores[i];
    if (s == 0.f) s = 0.f;                                   // -0 and +0 compare equal: give them one key
    keys[i] = ((unsigned long long)(~ordered_bits(s)) << 32) | (unsigned long long)(uint32_t)i;
}

__global__ void __launch_bounds__(kThreads) k_histogram(const unsigned long long* __restrict__ keys, int64_t N, int shift,
                                                        unsigned* __restrict__ hist, int nblocks) {
    __shared__ unsigned h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kTile;
#pragma unroll
    for (int s = 0; s < kItems; ++s) {
        const int64_t i = base + s * kThreads + threadIdx.x;
        if (i < N) atomicAdd(&h[(unsigned)(keys[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    hist[(int64_t)threadIdx.x * nblocks + blockIdx.x] = h[threadIdx.x];
}

// Exclusive scan of hist in (digit-major, block-minor) order, in place. One block.
__global__ void __launch_bounds__(1024) k_scan(unsigned* __restrict__ hist, int64_t total) {
    __shared__ unsigned warp_sums[32];
    __shared__ unsigned carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < total; base += 1024) {
        const int64_t i = base + tid;
        const unsigned v = (i < total) ? hist[i] : 0u;
        unsigned x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            unsigned w = warp_sums[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += y;
            }
            warp_sums[lane] = w;
        }
        __syncthreads();
        const unsigned before = carry + (warp > 0 ? warp_sums[warp - 1] : 0u) + (x - v);
        if (i < total) hist[i] = before;
        __syncthreads();
        if (tid == 1023) carry = before + v;
        __syncthreads();
    }
}

// Stable scatter: warp w of a block owns the contiguous keys [w*512, (w+1)*512) of the tile, walked in
// 16 slots of 32 consecutive keys, so (warp, slot, lane) order is index order.
__global__ void __launch_bounds__(kThreads) k_scatter(const unsigned long long* __restrict__ in, int64_t N, int shift,
                                                      const unsigned* __restrict__ offsets, int nblocks,
                                                      unsigned long long* __restrict__ out) {
    __shared__ unsigned cnt[kWarps][256];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int e = tid; e < kWarps * 256; e += kThreads) (&cnt[0][0])[e] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kTile + (int64_t)warp * (kItems * 32);
    unsigned long long key[kItems];
    unsigned short pos[kItems];
#pragma unroll
    for (int s = 0; s < kItems; ++s) {
        const int64_t i = base + s * 32 + lane;
        const bool live = i < N;
        key[s] = live ? in[i] : 0ull;
        const unsigned d = live ? ((unsigned)(key[s] >> shift) & 255u) : 256u;
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        const unsigned rank = __popc(peers & ((1u << lane) - 1u));
        unsigned before = 0;
        if (live) before = cnt[warp][d];
        __syncwarp();
        if (live && rank == 0) cnt[warp][d] = before + __popc(peers);
        __syncwarp();
        pos[s] = (unsigned short)(before + rank);
    }
    __syncthreads();
    {   // thread d: turn per-warp counts of digit d into start offsets
        unsigned off = offsets[(int64_t)tid * nblocks + blockIdx.x];
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const unsigned c = cnt[w][tid];
            cnt[w][tid] = off;
            off += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int s = 0; s < kItems; ++s) {
        const int64_t i = base + s * 32 + lane;
        if (i < N) {
            const unsigned d = (unsigned)(key[s] >> shift) & 255u;
            out[cnt[warp][d] + pos[s]] = key[s];
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_emit(const unsigned long long* __restrict__ keys, int64_t k,
                                                   int64_t* __restrict__ idx) {
    const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (i < k) idx[i] = (int64_t)(keys[i] & 0xffffffffull);
}

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace

cudaError_t select_scratch_bytes(int64_t N, size_t* bytes) {
    const int64_t nblocks = (N + kTile - 1) / kTile;
    *bytes = 2 * align256((size_t)N * 8) + align256((size_t)nblocks * 256 * 4) + 256;
    return cudaSuccess;
}

cudaError_t launch_select(const float* scores, int64_t N, int64_t k, int64_t* idx, void* scratch, cudaStream_t st) {
    if (N <= 0 || k <= 0) return cudaSuccess;
    const int nblocks = (int)((N + kTile - 1) / kTile);
    char* p = static_cast<char*>(scratch);
    unsigned long long* a = reinterpret_cast<unsigned long long*>(p);
    unsigned long long* b = reinterpret_cast<unsigned long long*>(p + align256((size_t)N * 8));
    unsigned* hist = reinterpret_cast<unsigned*>(p + 2 * align256((size_t)N * 8));
    k_make_keys<<<(unsigned)((N + kThreads - 1) / kThreads), kThreads, 0, st>>>(scores, N, a);
    int idx_bits = 1;
    while (idx_bits < 32 && (1ll << idx_bits) < N) ++idx_bits;
    for (int shift = 0; shift < 64; shift += 8) {
        if (shift < 32 && shift >= idx_bits) continue;       // index digits that are all zero
        k_histogram<<<nblocks, kThreads, 0, st>>>(a, N, shift, hist, nblocks);
        k_scan<<<1, 1024, 0, st>>>(hist, (int64_t)nblocks * 256);
        k_scatter<<<nblocks, kThreads, 0, st>>>(a, N, shift, hist, nblocks, b);
        unsigned long long* t = a; a = b; b = t;
    }
    k_emit<<<(unsigned)((k + kThreads - 1) / kThreads), kThreads, 0, st>>>(a, k, idx);
    return cudaGetLastError();
}

}  // namespace sage

// ------------------------------------------------------------------------------------------------
// sage_select_static: the same selection for callers that must not allocate.
//
// Some callers run where device allocation is off the table: inside a serving or training loop whose
// memory is handed out once at start-up by a pool they do not own, in a process whose remaining device
// memory is deliberately zero, or on a thread that may not take the allocator's locks. sage_select asks
// the stream-ordered allocator for its O(N) scratch on every call; this variant keeps that scratch in
// the library image instead, in the array below, which every device that loads the library holds
// until the process exits.
//
// The array's name is only a host-side stand-in in host code, so its device address is looked up once
// per device (with that device current) and that address is what the kernels get.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int64_t kStaticMaxN = 262144;    // largest N served without allocating
constexpr size_t kStaticKeyBytes = (size_t)kStaticMaxN * 8;                          // one key array
constexpr size_t kStaticHistBytes = (size_t)((kStaticMaxN + sage::kTile - 1) / sage::kTile) * 256 * 4;
constexpr size_t kStaticScratchBytes = 2 * kStaticKeyBytes + kStaticHistBytes + 256;  // about 4.06 MiB

static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};    // device address of g_select_scratch, per device ordinal
std::mutex g_scratch_mutex;

}  // namespace

extern "C" sage_status_t sage_select_static(const float* scores, int64_t N, double keep_rate, int64_t* idx, int64_t* k_out,
                                            void* cuda_stream) {
    if (N < 0 || !(keep_rate == keep_rate) || (N > 0 && !scores)) {
        sage::set_error_message("sage_select_static: bad argument (negative N, NaN keep_rate or null scores)");
        return SAGE_ERR_INVALID_ARG;
    }
    if (N > kStaticMaxN) {
        char msg[200];
        snprintf(msg, sizeof msg, "sage_select_static: N=%lld exceeds the built-in scratch (at most %lld scores); use sage_select",
                 (long long)N, (long long)kStaticMaxN);
        sage::set_error_message(msg);
        return SAGE_ERR_UNSUPPORTED;
    }
    const int64_t k = sage_select_count(N, keep_rate);
    if (k > 0 && !idx) {
        sage::set_error_message("sage_select_static: null idx");
        return SAGE_ERR_INVALID_ARG;
    }
    if (k > 0) {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
            sage::set_error_message("sage_select_static: no current CUDA device (or ordinal above 63)");
            return SAGE_ERR_CUDA;
        }
        void* scratch = nullptr;
        {
            std::lock_guard<std::mutex> lock(g_scratch_mutex);
            if (!g_scratch_addr[dev]) {       // first call on this device: resolve the array's device address
                void* p = nullptr;
                e = cudaGetSymbolAddress(&p, g_select_scratch);
                if (e != cudaSuccess || !p) {
                    char msg[200];
                    snprintf(msg, sizeof msg, "sage_select_static: cudaGetSymbolAddress failed on device %d: %s", dev,
                             cudaGetErrorString(e));
                    sage::set_error_message(msg);
                    return SAGE_ERR_CUDA;
                }
                g_scratch_addr[dev] = p;
            }
            scratch = g_scratch_addr[dev];
        }
        // Nothing in the scratch has to start at zero: the key arrays are written for every i < N before
        // they are read and each radix pass rewrites the whole histogram it scans.
        e = sage::launch_select(scores, N, k, idx, scratch, static_cast<cudaStream_t>(cuda_stream));
        if (e != cudaSuccess) {
            char msg[200];
            snprintf(msg, sizeof msg, "sage_select_static: launch failed: %s", cudaGetErrorString(e));
            sage::set_error_message(msg);
            return SAGE_ERR_CUDA;
        }
        int idx_bits = 1;
        while (idx_bits < 32 && (1ll << idx_bits) < N) ++idx_bits;
        sage::count_launches(2 + 3 * (4 + (idx_bits + 7) / 8));
    }
    if (k_out) *k_out = k;
    return SAGE_OK;
}

// fp32-faithful tensor-core contraction C[z] = A_z * B_z^T for fp32 operands (both contiguous along the
// contraction index): the Gram matrix K = B B^T of the sketch buffer (Method, first paragraph: the SVD of
// the buffer is taken through the eigen-decomposition of B B^T) and the pass-2 projection of fp32 rows.
//
// Two things keep fp32 fidelity on tensor cores:
//   * tcgen05 kind::tf32 reads an fp32 word by ignoring its low 13 bits (11 significant bits), so every value x
//     counts as hi = x with those bits cleared, and the workers write the remainder lo = x - hi (exact, then rounded
//     to 11 bits) into a second buffer; the MMAs accumulate hi*hi + hi*lo + lo*hi. The dropped lo*lo term is below
//     2^-20 relative (3e-7 on average on a Gram diagonal). The raw tile itself is the hi operand: nothing is written
//     back over it, which saves a third of the workers' shared-memory stores;
//   * the TMEM accumulator rounds toward zero at every accumulation, which biases long sums of like-signed
//     terms (measured about 0.45 * 2^-24 per MMA step), so the accumulator is drained every kChunk K
//     tiles into fp32 registers with round-to-nearest additions and restarted from zero.
//
// One CTA owns a 128 x (<=128) output tile and one K slice:
//   warp 0    TMA producer (raw fp32 tiles, 128-byte swizzle),
//   warp 1    TMEM allocation and MMA issue into a ring of four accumulators,
//   warps 2-9 write the lo part of each landed stage into its second buffer. The stage slots are dealt to G groups of
//             8 / G warps (G = the number of stages where that is at most 8: one warp per slot), so as many
//             wait -> load -> remainder -> store -> fence -> arrive chains are in flight as there are slots (measured on the
//             128 x 11.2 M Gram matrix: two groups of four warps 1.64 ms, six groups of one 1.54 ms, seven stages with seven
//             groups 1.46 ms). Every kChunk stages each warp also drains its lanes and columns of the accumulator
//             that was finished ring / 2 chunks earlier (its MMAs are long done, so the drain hardly waits) into
//             registers, and stores them at the end. Warp w drains TMEM lanes 32 * (w % 4), columns 64 * ((w - 2) / 4).
// The producer and the MMA thread keep running stage / phase / chunk counters and advance the operand descriptors by a
// constant per stage: with integer divisions and freshly built descriptors in its loop the single MMA-issuing thread took
// 1,500 cycles per K tile and was what bounded the kernel (now about 600).
// On the diagonal tiles of a Gram matrix only one operand tile is loaded and used on both sides. A Gram matrix
// of at most 128 rows (sym mode) needs ONE 256-wide MMA per K step: the hi tile and the lo tile lie back to back
// in the stage and serve as one 256-row B operand, so the accumulator holds hi*hi^T | hi*lo^T side by side; the drain
// forms T = hi*hi^T + 2*hi*lo^T (the doubling is exact), which satisfies (T + T^T)/2 = hi*hi^T + hi*lo^T + lo*hi^T,
// formed by the split reduction. (A 128 x 128 x 8 tf32 MMA executes in about 70 cycles, less than issuing it costs
// the issuing thread: narrow MMAs leave the tensor pipe idle, wide ones do not.)
// The projection of fp32 rows onto a sketch of at most 64 rows (proj mode, sym = 2) uses the same wide form with the
// operands' roles exchanged: the sketch, split once into [hi (64 rows) ; lo (64 rows)] when it was frozen, is the
// 128-row A operand and needs no work per stage; the tile of 128 data rows is split by the workers into hi | lo and
// serves as one 256-row B operand. One MMA per K step leaves S_hi (G_hi | G_lo) on TMEM lanes 0-63 and
// S_lo (G_hi | G_lo) on lanes 64-127; the drain adds the two column halves, and the lane halves are stored as two
// partial planes of the (transposed) output, which the split reduction sums with the K slices.
#include "sage_internal.h"
#include "tc05.cuh"

namespace sage {
namespace tc {
namespace {

constexpr int kThreads = 320;
constexpr int kWorkers = 256;               // warps 2-9
constexpr int kTileM = 128;
constexpr int kTileN = 128;
constexpr int kTileBytes = 128 * 128;       // 128 rows of 128 bytes
constexpr int BK = 32;                      // fp32 elements per 128-byte K tile
constexpr int kChunkTiles = 8;              // K tiles accumulated in TMEM between drains (32 MMA steps: bias below 1e-6; 4 -> 8 gave 8 %, 16 no more)
constexpr int kAccs = 4;                    // accumulators in TMEM (4 x 128 columns)

// The tensor cores read an fp32 word as tf32 by ignoring its low 13 bits, so the raw tile already is the hi operand
// (hi = x with those bits cleared) and only the remainder has to be written: lo = x - hi, exact, then rounded to 11
// significant bits so that the hardware's truncation of lo finds nothing to cut (a truncated lo would bias sums of
// like-signed products).
__device__ __forceinline__ uint32_t lo_of(uint32_t x) {
    const float l = __uint_as_float(x) - __uint_as_float(x & 0xffffe000u);
    return (__float_as_uint(l) + 0x1000u) & 0xffffe000u;
}
__device__ __forceinline__ uint4 lo4(const uint4 v) { return make_uint4(lo_of(v.x), lo_of(v.y), lo_of(v.z), lo_of(v.w)); }

__global__ void __launch_bounds__(kThreads, 1)
k_tc_gemm_nt_x3(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, int M, int N, int gram,
                int b_box_rows, int sym, long long K, long long k_per_split, int a_shared, float* __restrict__ C, long long ldc,
                long long split_stride, int stages, int stage_bytes, int G, int direct_new, int direct_box, int* __restrict__ err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int m0 = blockIdx.x * kTileM, n0 = blockIdx.y * kTileN;
    if (gram && m0 > n0) return;                          // a Gram matrix is symmetric: the reduction mirrors the upper tiles
    const bool proj = sym == 2;
    const bool wide = sym != 0;                           // one 256-wide MMA per K step
    const bool diag = gram && m0 == n0;                   // A tile == B tile: load once
    // stage layout: [hi: A | B][lo: A | B]; on diagonal tiles there is no separate B; proj: [hi: rows][lo: rows][sketch]
    const int half_bytes = (diag || proj) ? kTileBytes : kTileBytes + b_box_rows * 128;
    // direct_new > 0 (a symmetric Gram matrix of at most 128 rows whose last direct_new rows are still bfloat16 rows in the
    // caller's memory): tmA covers the first M - direct_new + 1 buffer rows (the last of them is a placeholder), tmB the
    // caller's rows (boxes of direct_box rows x 64 bytes, no swizzle) which land behind the two tiles of the stage; the
    // workers convert them and put them where rows M - direct_new ... M - 1 of the operand tile belong (128-byte swizzle:
    // 16-byte chunk j of row r sits in slot j ^ (r & 7)). Their remainders are zero (bfloat16 has 8 significant bits):
    // the remainder tiles are cleared once and only rows below M - direct_new are ever written.
    const int old_rows = direct_new ? M - direct_new : 0;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
    uint64_t* split_done = full + stages;
    uint64_t* empty = split_done + stages;
    uint64_t* acc_full = empty + stages;                   // [kAccs]
    uint64_t* acc_empty = acc_full + kAccs;                // [kAccs]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + kAccs);
    volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long k_begin = (long long)blockIdx.z * k_per_split;
    const long long k_end = K < k_begin + k_per_split ? K : k_begin + k_per_split;
    const int nkt = k_end > k_begin ? (int)((k_end - k_begin + BK - 1) / BK) : 0;
    const int kChunk = kChunkTiles;
    const int nchunks = (nkt + kChunk - 1) / kChunk;
    const int acc_cols = wide ? 2 * kTileN : kTileN;      // sym: P and 2Q side by side; proj: hi and lo columns of the rows
    const int ring = (kAccs * kTileN) / acc_cols;         // accumulators in flight: 4, or 2 in sym mode
    int n_pad = N - n0 < kTileN ? N - n0 : kTileN;        // MMA width of this tile, a multiple of 16
    n_pad = ((n_pad + 15) / 16) * 16;
    if (proj) n_pad = kTileN;                             // accumulator columns are the 128 data rows of the tile

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&split_done[s], 8 / G);                           // one arrival per warp of the group that owns the slot
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < kAccs; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], kWorkers / 32);
        }
        *abort = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (direct_new) {
        for (int s = 0; s < stages; ++s) {
            uint4* lo = reinterpret_cast<uint4*>(smem + (size_t)s * stage_bytes + kTileBytes);
            for (int c = threadIdx.x; c < kTileBytes / 16; c += kThreads) lo[c] = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc(tmem_slot, kAccs * kTileN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            int s = 0;
            uint32_t ph = 1;                                    // parity of the empty-barrier phase to wait for
            int x = (int)k_begin, xa = a_shared ? 0 : (int)k_begin;   // class slices: the same columns of A for every slice
            uint8_t* st = smem;
            const uint32_t tx_bytes = direct_new ? (uint32_t)((old_rows + 1) * 128 + direct_box * 64) : (uint32_t)(proj ? 2 * kTileBytes : half_bytes);
            for (int kt = 0; kt < nkt; ++kt) {
                if (!mbar_wait(&empty[s], ph, abort)) break;
                mbar_expect_tx(&full[s], tx_bytes);
                tma_load_2d(st, &tmA, &full[s], xa, m0);
                if (proj || direct_new) tma_load_2d(st + 2 * kTileBytes, &tmB, &full[s], x, 0);
                else if (!diag) tma_load_2d(st + kTileBytes, &tmB, &full[s], x, n0);
                issued = kt + 1;
                x += BK;
                xa += BK;
                if (++s == stages) { s = 0; ph ^= 1u; st = smem; } else { st += stage_bytes; }
            }
            if (*abort) {
                for (int kt = issued > stages ? issued - stages : 0; kt < issued; ++kt)
                    mbar_wait_quiet(&full[kt % stages], (uint32_t)(kt / stages) & 1u, 20000000ll);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(2, kTileM, wide ? 2 * kTileN : n_pad, 0, 0);
            // everything but the start address of an operand descriptor (see smem_desc_k_sw128); the addresses advance by
            // stage_bytes per stage
            const uint64_t desc_hi = smem_desc_k_sw128(0);
            const uint32_t st0 = smem_u32(smem);
            const uint32_t a_hi_off = proj ? 2 * kTileBytes : 0, a_lo_off = half_bytes;   // proj: A = the split sketch
            const uint32_t b_hi_off = (diag || proj) ? 0 : kTileBytes, b_lo_off = b_hi_off + half_bytes;
            int s = 0, in_chunk = 0, b = 0;
            uint32_t ph = 0, acc_par = 1;
            uint32_t st = st0;
            for (int kt = 0; kt < nkt; ++kt) {
                if (in_chunk == 0 && !mbar_wait(&acc_empty[b], acc_par, abort)) break;
                if (!mbar_wait(&split_done[s], ph, abort)) break;
                tc_fence_after();
                const uint64_t d_ahi = desc_hi | ((st + a_hi_off) >> 4), d_bhi = desc_hi | ((st + b_hi_off) >> 4);
                const uint32_t acc = tmem_base + (uint32_t)(b * acc_cols);
                if (wide) {                                 // sym: B = [hi ; lo] (the drain doubles the lo half), proj: [hi ; lo]
                    mma_tf32(acc, d_ahi, d_bhi, idesc, in_chunk != 0);
                    mma_tf32(acc, d_ahi + 2, d_bhi + 2, idesc, 1);       // 4 x 8 tf32 elements per 128-byte row
                    mma_tf32(acc, d_ahi + 4, d_bhi + 4, idesc, 1);
                    mma_tf32(acc, d_ahi + 6, d_bhi + 6, idesc, 1);
                } else {
                    const uint64_t d_alo = desc_hi | ((st + a_lo_off) >> 4), d_blo = desc_hi | ((st + b_lo_off) >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        mma_tf32(acc, d_ahi + 2 * k, d_bhi + 2 * k, idesc, (in_chunk | k) != 0);
                        mma_tf32(acc, d_ahi + 2 * k, d_blo + 2 * k, idesc, 1);
                        mma_tf32(acc, d_alo + 2 * k, d_bhi + 2 * k, idesc, 1);
                    }
                }
                mma_commit(&empty[s]);
                if (in_chunk == kChunk - 1 || kt == nkt - 1) {
                    mma_commit(&acc_full[b]);
                    in_chunk = 0;
                    if (++b == ring) { b = 0; acc_par ^= 1u; }
                } else {
                    ++in_chunk;
                }
                if (++s == stages) { s = 0; ph ^= 1u; st = st0; } else { st += (uint32_t)stage_bytes; }
            }
        }
    } else {
        // ---- workers: write the lo part of landed stages; drain finished accumulators ----
        const int t = threadIdx.x - 64;                 // 0..255
        const int chunks16 = direct_new ? old_rows * 8 : half_bytes / 16;     // direct: remainders of the buffer rows only
        const float lo_scale = sym == 1 ? 2.f : 1.f;          // sym: the lo half of the accumulator counts twice (folded into the drain)
        const int quarter = warp & 3, chalf = (warp - 2) >> 2;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + (uint32_t)(chalf * 64);
        float acc[64];
#pragma unroll
        for (int j = 0; j < 64; ++j) acc[j] = 0.f;
        bool ok = true;
        auto drain = [&](int c) {
            const int b = c % ring;
            bool w = mbar_wait(&acc_full[b], ((uint32_t)c / ring) & 1u, abort);
            w = __all_sync(0xffffffffu, w);
            if (!w) { ok = false; return; }
            tc_fence_after();
            // two TMEM loads in flight per wait (a wait after every load made the drain a third of the workers' time)
            if (wide) {                                      // columns c and kTileN + c belong together
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (chalf * 64 + 16 * q < n_pad) {
                        uint32_t v0[16], v1[16];
                        tmem_ld16_issue(lane_base + (uint32_t)(b * acc_cols + 16 * q), v0);
                        tmem_ld16_issue(lane_base + (uint32_t)(b * acc_cols + kTileN + 16 * q), v1);
                        tmem_ld_wait();
                        tmem_ld_use(v0);
                        tmem_ld_use(v1);
#pragma unroll
                        for (int j = 0; j < 16; ++j) acc[16 * q + j] += fmaf(lo_scale, __uint_as_float(v1[j]), __uint_as_float(v0[j]));
                    }
                }
            } else {
#pragma unroll
                for (int q = 0; q < 4; q += 2) {
                    const bool on0 = chalf * 64 + 16 * q < n_pad, on1 = chalf * 64 + 16 * (q + 1) < n_pad;
                    uint32_t v0[16], v1[16];
                    if (on0) tmem_ld16_issue(lane_base + (uint32_t)(b * acc_cols + 16 * q), v0);
                    if (on1) tmem_ld16_issue(lane_base + (uint32_t)(b * acc_cols + 16 * (q + 1)), v1);
                    tmem_ld_wait();
                    if (on0) {
                        tmem_ld_use(v0);
#pragma unroll
                        for (int j = 0; j < 16; ++j) acc[16 * q + j] += __uint_as_float(v0[j]);
                    }
                    if (on1) {
                        tmem_ld_use(v1);
#pragma unroll
                        for (int j = 0; j < 16; ++j) acc[16 * (q + 1) + j] += __uint_as_float(v1[j]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[b]);
        };
        // The stage slots are dealt to G groups of 8 / G warps: group g takes the K tiles kt = g, g + G, ... A slot then
        // always belongs to the same group (stages is a multiple of G), which sees every phase of its barrier in turn: a
        // group that skipped a phase could not tell "two phases back" from "done" with a parity wait. Warps beyond
        // G * (8 / G) only drain.
        int drained = 0;                                // chunks drained so far
        const int wpg = 8 / G, ww = warp - 2;
        const int grp = ww / wpg, tg = (ww - grp * wpg) * 32 + lane;      // group, thread index within it
        const int kGroup = 32 * wpg, kstep = G;
        int s = grp % stages;
        uint32_t ph = (uint32_t)(grp / stages) & 1u;
        for (int kt = ww < wpg * G ? grp : nkt; kt < nkt && ok; kt += kstep) {
            bool landed = mbar_wait(&full[s], ph, abort);
            landed = __all_sync(0xffffffffu, landed);
            if (!landed) { ok = false; break; }
            uint4* hi = reinterpret_cast<uint4*>(smem + (size_t)s * stage_bytes);
            uint4* lo = reinterpret_cast<uint4*>(smem + (size_t)s * stage_bytes + half_bytes);
            const int s_now = s;
            s += kstep;                                 // the slot and phase of this group's next K tile
            while (s >= stages) { s -= stages; ph ^= 1u; }
            for (int c = tg; c < chunks16; c += 4 * kGroup) {      // four independent 16-byte pieces in flight (eight: slower)
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (c + u * kGroup < chunks16) v[u] = hi[c + u * kGroup];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (c + u * kGroup < chunks16) lo[c + u * kGroup] = lo4(v[u]);
            }
            if (direct_new) {
                // the caller's bfloat16 rows: 4 x 16 bytes (32 values) per row and K tile -> 8 chunks of 4 floats in the operand tile
                const uint4* src = reinterpret_cast<const uint4*>(smem + (size_t)s_now * stage_bytes + 2 * kTileBytes);
                for (int i = tg; i < direct_new * 4; i += kGroup) {
                    const int row = i >> 2, q = i & 3, R = old_rows + row;
                    const uint4 v = src[i];
                    const uint4 a = make_uint4(v.x << 16, v.x & 0xffff0000u, v.y << 16, v.y & 0xffff0000u);
                    const uint4 b = make_uint4(v.z << 16, v.z & 0xffff0000u, v.w << 16, v.w & 0xffff0000u);
                    hi[R * 8 + ((2 * q) ^ (R & 7))] = a;
                    hi[R * 8 + ((2 * q + 1) ^ (R & 7))] = b;
                }
            }
            fence_proxy_async_smem();                   // the tensor cores read these writes
            __syncwarp();                               // one arrival per warp
            if (lane == 0) mbar_arrive(&split_done[s_now]);
            // a chunk is folded into the registers once the stages of the following ring / 2 chunks have been handled
            // (its MMAs are long done by then); every warp drains its own lanes and columns of every chunk
            while (ok && drained < nchunks && (drained + 1 + ring / 2) * kChunk - kstep <= kt) drain(drained++);
        }
        while (ok && drained < nchunks) drain(drained++);
        const int row = m0 + quarter * 32 + lane;
        if (proj) {
            // lane = sketch row (0-63: hi part, 64-127: lo part), register c = data row chalf * 64 + c of the tile:
            // the output is stored transposed, 32 consecutive sketch rows of one data row per warp instruction
            const int mrow = quarter * 32 + lane, plane = mrow >> 6, j = mrow & 63;
            float* cbase = C + (2ll * blockIdx.z + plane) * split_stride + j;
            if (j < N) {
#pragma unroll
                for (int c = 0; c < 64; ++c) {
                    const int r = m0 + chalf * 64 + c;
                    if (r < M) cbase[(long long)r * ldc] = acc[c];
                }
            }
        } else if (row < M) {
            float* crow = C + (long long)blockIdx.z * split_stride + (long long)row * ldc + n0 + chalf * 64;
            const bool vec = (ldc % 4 == 0) && ((reinterpret_cast<uintptr_t>(C) & 15u) == 0) && (split_stride % 4 == 0);
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 4) {
                const int col = n0 + chalf * 64 + c0;
                if (col + 4 <= N && vec) {
                    *reinterpret_cast<float4*>(crow + c0) = make_float4(acc[c0], acc[c0 + 1], acc[c0 + 2], acc[c0 + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (col + j < N) crow[c0 + j] = acc[c0 + j];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        // no MMA may be in flight when TMEM is freed: the last chunk's commit covers every MMA issued
        if (nchunks > 0 && !*abort)
            mbar_wait_quiet(&acc_full[(nchunks - 1) % ring], ((uint32_t)(nchunks - 1) / ring) & 1u, kWaitLimitCycles);
        tc_fence_after();
        tmem_dealloc(tmem_base, kAccs * kTileN);
    }
    if (threadIdx.x == 0 && *abort) atomicExch(err, 1);
}

}  // namespace
}  // namespace tc

cudaError_t launch_tc_gemm_nt_x3(const float* A, int64_t lda, const float* Bm, int64_t ldb, int M, int N, int64_t K, int splits,
                                 float* C, int64_t ldc, int64_t split_stride, int sym, int* err, cudaStream_t st, int64_t class_F) {
    if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
    if (splits < 1 || splits > 65535) return cudaErrorNotSupported;
    const int gram = (A == Bm && lda == ldb && M == N) ? 1 : 0;
    const bool proj = sym == 2;       // Bm: the sketch split into [hi (64 rows) ; lo (64 rows)], 128 rows of pitch ldb; N <= 64
    if (sym == 1 && !(gram && M <= tc::kTileM)) return cudaErrorInvalidValue;
    if (proj && (N > 64 || gram)) return cudaErrorInvalidValue;
    // class slices: see launch_tc_gemm_nt
    if (class_F > 0 && (gram || class_F % 4 != 0 || (int64_t)splits * class_F != K)) return cudaErrorNotSupported;
    CUtensorMap tmA, tmB;
    if (!tc::make_tmap_2d(&tmA, A, 4, (uint64_t)M, (uint64_t)(class_F > 0 ? class_F : K), (uint64_t)lda, tc::kTileM)) return cudaErrorNotSupported;
    const int b_box_rows = proj ? tc::kTileN : (N >= tc::kTileN ? tc::kTileN : ((N + 15) / 16) * 16);
    if (!tc::make_tmap_2d(&tmB, Bm, 4, (uint64_t)(proj ? 128 : N), (uint64_t)K, (uint64_t)ldb, (uint32_t)b_box_rows)) return cudaErrorNotSupported;
    int64_t kps = (K + splits - 1) / splits;
    kps = ((kps + tc::BK - 1) / tc::BK) * tc::BK;
    if (class_F > 0) kps = class_F;
    // a trailing slice may be empty after rounding to whole K tiles: its CTAs store zeros
    // a Gram matrix of at most 128 rows has diagonal tiles only: one operand per stage
    const int stage_bytes = proj ? 3 * tc::kTileBytes : 2 * ((gram && M <= tc::kTileM) ? tc::kTileBytes : tc::kTileBytes + b_box_rows * 128);
    // Long K slices of the one-MMA-per-step forms (16 KB of remainders per stage): as many stages as fit the 227 KB a block
    // may have (7 of 32 KB, 4 of 48 KB), each slot with a worker group of its own (8 / stages warps), so that many
    // remainder chains overlap. Short slices, and the three-MMA form (32 KB of remainders per stage, 3 stages): the
    // eight warps work on a stage together (odd number of stages) or as two groups of four on alternate stages, which
    // finishes a single stage sooner.
    const bool deep = sym != 0 && kps / tc::BK >= 64;
    int stages = ((deep ? 227 * 1024 - 1536 : 200 * 1024)) / stage_bytes;
    if (stages > 8) stages = 8;
    if (stages < 2) return cudaErrorNotSupported;
    const int G = deep ? stages : ((stages & 1) ? 1 : 2);
    const size_t smem = (size_t)stages * stage_bytes + 1024 + (3 * stages + 2 * tc::kAccs) * 8 + 16;
    dim3 grid((unsigned)((M + tc::kTileM - 1) / tc::kTileM), proj ? 1u : (unsigned)((N + tc::kTileN - 1) / tc::kTileN), (unsigned)splits);
    cudaError_t e = cudaFuncSetAttribute(tc::k_tc_gemm_nt_x3, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    tc::k_tc_gemm_nt_x3<<<grid, tc::kThreads, smem, st>>>(tmA, tmB, M, N, gram, b_box_rows, sym, K, kps, class_F > 0 ? 1 : 0, C, ldc, split_stride, stages,
                                                                 stage_bytes, G, 0, 0, err);
    return cudaGetLastError();
}

// See sage_internal.h.
cudaError_t launch_tc_gram_direct(const float* Bold, int64_t pitch, int old_rows, const void* src, int64_t ld_src, int n_new, int64_t D,
                                  int splits, float* C, int64_t ldc, int64_t split_stride, int* err, cudaStream_t st) {
    const int M = old_rows + n_new;
    if (old_rows < 1 || n_new < 1 || M > tc::kTileM || D <= 0 || splits < 1 || splits > 65535) return cudaErrorNotSupported;
    const int old_box = old_rows + 1;                         // one placeholder row, overwritten by the first new row
    const int src_box = ((n_new + 7) / 8) * 8;
    if ((old_box & 7) || src_box > 128) return cudaErrorNotSupported;
    CUtensorMap tmA, tmB;
    if (!tc::make_tmap_2d(&tmA, Bold, 4, (uint64_t)old_box, (uint64_t)D, (uint64_t)pitch, (uint32_t)old_box)) return cudaErrorNotSupported;
    if (!tc::make_tmap_2d_plain(&tmB, src, 2, (uint64_t)n_new, (uint64_t)D, (uint64_t)ld_src, 32, (uint32_t)src_box)) return cudaErrorNotSupported;
    int64_t kps = (D + splits - 1) / splits;
    kps = ((kps + tc::BK - 1) / tc::BK) * tc::BK;
    const int stage_bytes = 2 * tc::kTileBytes + ((src_box * 64 + 1023) / 1024) * 1024;
    const bool deep = kps / tc::BK >= 64;
    int stages = ((deep ? 227 * 1024 - 1536 : 200 * 1024)) / stage_bytes;
    if (stages > 8) stages = 8;
    if (stages < 2) return cudaErrorNotSupported;
    const int G = deep ? stages : ((stages & 1) ? 1 : 2);
    const size_t smem = (size_t)stages * stage_bytes + 1024 + (3 * stages + 2 * tc::kAccs) * 8 + 16;
    dim3 grid(1u, 1u, (unsigned)splits);
    cudaError_t e = cudaFuncSetAttribute(tc::k_tc_gemm_nt_x3, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    tc::k_tc_gemm_nt_x3<<<grid, tc::kThreads, smem, st>>>(tmA, tmB, M, M, 1, 0, 1, D, kps, 0, C, ldc, split_stride, stages, stage_bytes, G, n_new,
                                                         src_box, err);
    return cudaGetLastError();
}

}  // namespace sage

// Tensor-core rebuild of the sketch buffer (Method, first paragraph: the sketch is rebuilt from the shrunk singular values and the right factor).
// With B B^T = U Lambda U^T, Sigma' V^T = diag(sigma'_j / sigma_j) U^T B, i.e.
//     out[j][d] = sum_i W[j][i] * B[i][d],   W[j][i] = U[i][j] * sqrt(max(1 - delta/lambda_j, 0)).
// The buffer is the streamed operand: a CTA walks 128-column tiles of it, and for each tile accumulates over
// chunks of 32 buffer rows   D[d][j] += B[i][d] * W[j][i]   with d on the 128 TMEM lanes (the buffer tile is the
// "A" operand, stored with d contiguous = MN-major), so the epilogue writes out[j][d0..d0+127] as full lines.
//
// fp32 fidelity as in the Gram kernel: the tensor cores read a buffer value as hi (its low 13 bits ignored),
// the split warps write lo = x - hi into a second buffer; W arrives already split from global memory as two stacked operands [W_hi; W_lo],
// so one MMA of width 2*j_pad gives hi*W_hi and hi*W_lo side by side and a second one adds lo*W_hi; the
// epilogue adds the two halves. One TMEM accumulator takes at most 8 chunks (256 buffer rows); with more buffer rows
// (up to 512) a tile uses both accumulators, one per half of the rows, and the epilogue adds them in registers (the
// tiles then no longer alternate between the accumulators, so a tile's MMAs start after the previous tile's epilogue).
//
//   warp 0    TMA producer: per chunk 4 boxes of [32 rows][32 columns] of the buffer (128-byte swizzle with
//             32-byte atoms, the only layout the tensor cores take for 32-bit MN-major operands) and one box of W; where
//             all chunk boxes of W fit 64 KB (up to 128 buffer rows onto 64 output rows) they are loaded once and stay,
//   warp 1    TMEM allocation, MMA issue into two ping-pong accumulators (one per column tile),
//   warps 2-5 write the lo part of the buffer tile of each landed stage,
//   warps 6-9 epilogue: TMEM -> registers -> out.
#include "sage_internal.h"
#include "tc05.cuh"

namespace sage {
namespace tc {
namespace {

constexpr int kThreads = 320;
constexpr int kSplitThreads = 128;
constexpr int kEpiThreads = 128;
constexpr int kTileD = 128;                 // buffer columns per tile (MMA M)
constexpr int kChunkRows = 32;              // buffer rows per stage (MMA K = 4 x 8)
constexpr int kBufBytes = kChunkRows * kTileD * 4;   // 16 KB: 4 spans of [32 rows][128 bytes]
constexpr int kSpanBytes = kChunkRows * 128;         // 4 KB

__global__ void __launch_bounds__(kThreads, 1)
k_tc_rebuild(const __grid_constant__ CUtensorMap tmBuf, const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmSrc,
             const __grid_constant__ CUtensorMap tmSrc1, int direct_new, int r, int keep, int j_pad,
             long long pitch, long long num_tiles, float* __restrict__ out, int stages, int w_res, int* __restrict__ err) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    // stage layout: [buffer hi 16 KB][buffer lo 16 KB][W_hi ; W_lo: 2*j_pad rows of 128 bytes]; w_res: the W boxes of all
    // chunks are loaded once and stay behind the ring (W does not depend on the column tile), the stages hold buffer data only
    const int w_bytes = 2 * j_pad * 128;
    // direct_new > 0 (needs w_res): the last direct_new of the r rows are bfloat16 rows in the caller's memory. Rows
    // 0 .. r - direct_new - 1 come from the buffer as usual; r - direct_new is the last row of its chunk of 32 (cb), so that
    // chunk gets one bfloat16 row (tmSrc1) and the chunks after it 32 each (tmSrc) into an 8 KB staging area behind the two
    // buffer tiles; the split warps convert them into the operand layout (32-byte atoms: chunk j of k row rr sits in slot
    // ((j >> 1) ^ (rr & 3)) * 2 + (j & 1) of its 128-byte span row). Their remainders are zero, so chunks after cb take one
    // MMA per K step instead of two.
    const int stage_bytes = (w_res ? 2 * kBufBytes : 2 * kBufBytes + w_bytes) + (direct_new ? 8192 : 0);
    const int cb = direct_new ? (r - direct_new) / kChunkRows : 1 << 30;
    const int nchunk = (r + kChunkRows - 1) / kChunkRows;
    uint8_t* wres = smem + (size_t)stages * stage_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(wres + (w_res ? (size_t)nchunk * w_bytes : 0));
    uint64_t* split_done = full + stages;
    uint64_t* empty = split_done + stages;
    uint64_t* acc_full = empty + stages;                   // [2]
    uint64_t* acc_empty = acc_full + 2;                    // [2]
    uint64_t* w_full = acc_empty + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(w_full + 1);
    volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_mma = 2 * j_pad;                           // <= 256
    const bool two = nchunk > 8;                           // both accumulators serve one tile
    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)(2 * n_mma)) tmem_cols <<= 1;
    // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
    const long long my_tiles = num_tiles > blockIdx.x ? (num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&split_done[s], kSplitThreads);
            mbar_init(&empty[s], 1);
        }
        mbar_init(w_full, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], kEpiThreads);
        }
        *abort = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmBuf);
        tma_prefetch_desc(&tmW);
    }
    if (warp == 1) tmem_alloc(tmem_slot, tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            long long issued = 0;
            bool alive = true;
            int s = 0;
            uint32_t ph = 1;                                // parity of the empty-barrier phase to wait for
            uint8_t* st = smem;
            const uint32_t tx_bytes = (uint32_t)(w_res ? kBufBytes : kBufBytes + w_bytes);
            if (w_res) {
                mbar_expect_tx(w_full, (uint32_t)(nchunk * w_bytes));
                for (int c = 0; c < nchunk; ++c) tma_load_2d(wres + (size_t)c * w_bytes, &tmW, w_full, c * kChunkRows, 0);
            }
            for (long long lt = 0; lt < my_tiles && alive; ++lt) {
                const int d0 = (int)((blockIdx.x + lt * gridDim.x) * kTileD);
                for (int c = 0; c < nchunk; ++c) {
                    if (!mbar_wait(&empty[s], ph, abort)) { alive = false; break; }
                    if (c > cb) {                               // caller's rows only
                        mbar_expect_tx(&full[s], 8192u);
                        tma_load_2d(st + 2 * kBufBytes, &tmSrc, &full[s], d0, 1 + (c - cb - 1) * kChunkRows);
                    } else {
                        mbar_expect_tx(&full[s], c == cb ? tx_bytes + 256u : tx_bytes);
#pragma unroll
                        for (int sp = 0; sp < 4; ++sp) tma_load_2d(st + sp * kSpanBytes, &tmBuf, &full[s], d0 + 32 * sp, c * kChunkRows);
                        if (c == cb) tma_load_2d(st + 2 * kBufBytes, &tmSrc1, &full[s], d0, 0);
                        if (!w_res) tma_load_2d(st + 2 * kBufBytes, &tmW, &full[s], c * kChunkRows, 0);
                    }
                    ++issued;
                    if (++s == stages) { s = 0; ph ^= 1u; st = smem; } else { st += stage_bytes; }
                }
            }
            if (*abort) {
                if (w_res) mbar_wait_quiet(w_full, 0, 20000000ll);
                for (long long k = issued > stages ? issued - stages : 0; k < issued; ++k)
                    mbar_wait_quiet(&full[k % stages], (uint32_t)(k / stages) & 1u, 20000000ll);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc_fold = instr_desc(2, kTileD, n_mma, 1, 0);   // A (buffer) MN-major, B (W) K-major
            const uint32_t idesc_half = instr_desc(2, kTileD, j_pad, 1, 0);
            // running stage / phase counters and descriptors advanced by a constant per stage: the loop of the single issuing
            // thread bounds the kernel, so it holds no division and builds no descriptor from scratch
            const uint64_t desc_w = smem_desc_k_sw128(0), desc_buf = smem_desc_mn_sw128_atom32(0, kSpanBytes);
            const uint32_t st0 = smem_u32(smem);
            bool alive = true;
            int s = 0;
            uint32_t ph = 0, st = st0;
            const uint32_t wres0 = smem_u32(wres);
            if (w_res) alive = mbar_wait(w_full, 0, abort);
            for (long long lt = 0; lt < my_tiles && alive; ++lt) {
                const int b = two ? 0 : (int)(lt & 1);
                const uint32_t par = two ? (uint32_t)lt : (uint32_t)(lt >> 1);
                alive = mbar_wait(&acc_empty[b], (par & 1u) ^ 1u, abort);
                if (!alive) break;
                for (int c = 0; c < nchunk; ++c) {
                    const uint32_t acc = tmem_base + (uint32_t)((two ? (c >> 3) : b) * n_mma);
                    const int c_in = two ? (c & 7) : c;       // position within this accumulator's run
                    if (!mbar_wait(&split_done[s], ph, abort)) { alive = false; break; }
                    tc_fence_after();
                    const uint64_t d_w = desc_w | ((w_res ? wres0 + (uint32_t)(c * w_bytes) : st + 2 * kBufBytes) >> 4);
                    const uint64_t d_hi = desc_buf | (st >> 4), d_lo = desc_buf | ((st + kBufBytes) >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {          // 8 buffer rows per MMA: one 1024-byte row group (64 descriptor units)
                        mma_tf32(acc, d_hi + 64 * k, d_w + 2 * k, idesc_fold, (c_in | k) != 0);   // hi*W_hi | hi*W_lo
                        if (c <= cb) mma_tf32(acc, d_lo + 64 * k, d_w + 2 * k, idesc_half, 1);     // + lo*W_hi (zero for bfloat16 rows)
                    }
                    mma_commit(&empty[s]);
                    if (++s == stages) { s = 0; ph ^= 1u; st = st0; } else { st += (uint32_t)stage_bytes; }
                }
                if (alive) mma_commit(&acc_full[b]);
            }
        }
    } else if (warp < 6) {
        const int t = threadIdx.x - 64;
        const long long total = my_tiles * nchunk;
        int s = 0, c = 0;                               // stage slot and chunk (32 buffer rows) of the current tile
        uint32_t ph = 0;
        for (long long q = 0; q < total; ++q) {
            if (!mbar_wait(&full[s], ph, abort)) break;
            uint4* hi = reinterpret_cast<uint4*>(smem + (size_t)s * stage_bytes);
            uint4* lo = reinterpret_cast<uint4*>(smem + (size_t)s * stage_bytes + kBufBytes);
            if (c <= cb) {
#pragma unroll
                for (int cc = 0; cc < kBufBytes / 16 / kSplitThreads; ++cc) {
                    const int idx = t + cc * kSplitThreads;
                    // the tensor cores ignore the low 13 bits of an fp32 word, so the raw tile is the hi operand as it stands;
                    // lo = x - hi (exact), rounded to 11 significant bits so that the same truncation cuts nothing from it
                    const uint4 v = hi[idx];
                    uint4 l;
                    l.x = (__float_as_uint(__uint_as_float(v.x) - __uint_as_float(v.x & 0xffffe000u)) + 0x1000u) & 0xffffe000u;
                    l.y = (__float_as_uint(__uint_as_float(v.y) - __uint_as_float(v.y & 0xffffe000u)) + 0x1000u) & 0xffffe000u;
                    l.z = (__float_as_uint(__uint_as_float(v.z) - __uint_as_float(v.z & 0xffffe000u)) + 0x1000u) & 0xffffe000u;
                    l.w = (__float_as_uint(__uint_as_float(v.w) - __uint_as_float(v.w & 0xffffe000u)) + 0x1000u) & 0xffffe000u;
                    // the last row of chunk cb is a placeholder for the caller's first row (a bfloat16 row: remainder zero)
                    if (c == cb && ((idx >> 3) & 31) == kChunkRows - 1) l = make_uint4(0u, 0u, 0u, 0u);
                    lo[idx] = l;
                }
            }
            if (c >= cb) {
                // bfloat16 rows from the staging area (256 bytes = 128 columns per row): 8 values -> two chunks of 4 floats
                const uint4* src = reinterpret_cast<const uint4*>(smem + (size_t)s * stage_bytes + 2 * kBufBytes);
                const int n_in = c == cb ? 16 : kChunkRows * 16;
                for (int i = t; i < n_in; i += kSplitThreads) {
                    const int rr = c == cb ? kChunkRows - 1 : i >> 4, q8 = i & 15;     // k row within the chunk, group of 8 columns
                    const uint4 v = src[i];
                    const uint4 a = make_uint4(v.x << 16, v.x & 0xffff0000u, v.y << 16, v.y & 0xffff0000u);
                    const uint4 b = make_uint4(v.z << 16, v.z & 0xffff0000u, v.w << 16, v.w & 0xffff0000u);
                    const int span = q8 >> 2, j = (q8 & 3) * 2;                          // 32-column span, 16-byte chunk within its row
                    uint4* row = hi + span * (kSpanBytes / 16) + rr * 8;
                    row[(((j >> 1) ^ (rr & 3)) << 1) | (j & 1)] = a;
                    row[((((j + 1) >> 1) ^ (rr & 3)) << 1) | ((j + 1) & 1)] = b;
                }
            }
            if (++c == nchunk) c = 0;
            fence_proxy_async_smem();
            mbar_arrive(&split_done[s]);
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
    } else {
        const int quarter = warp & 3;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        for (long long lt = 0; lt < my_tiles; ++lt) {
            const int b = two ? 0 : (int)(lt & 1);
            const uint32_t par = two ? (uint32_t)lt : (uint32_t)(lt >> 1);
            bool ok = mbar_wait(&acc_full[b], par & 1u, abort);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const long long d = (blockIdx.x + lt * gridDim.x) * kTileD + quarter * 32 + lane;
            const uint32_t acc = lane_base + (uint32_t)(b * n_mma);
            for (int j0 = 0; j0 < j_pad; j0 += 32) {
                // four TMEM loads in flight per wait (hi*W_hi | hi*W_lo halves of two groups of 16 output rows)
                const bool second = j0 + 16 < j_pad;
                uint32_t v0[16], w0[16], v1[16], w1[16];
                tmem_ld16_issue(acc + (uint32_t)j0, v0);
                tmem_ld16_issue(acc + (uint32_t)(j_pad + j0), w0);
                if (second) {
                    tmem_ld16_issue(acc + (uint32_t)(j0 + 16), v1);
                    tmem_ld16_issue(acc + (uint32_t)(j_pad + j0 + 16), w1);
                }
                tmem_ld_wait();
                tmem_ld_use(v0);
                tmem_ld_use(w0);
                float a0[16], a1[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) a0[j] = __uint_as_float(v0[j]) + __uint_as_float(w0[j]);
                if (second) {
                    tmem_ld_use(v1);
                    tmem_ld_use(w1);
#pragma unroll
                    for (int j = 0; j < 16; ++j) a1[j] = __uint_as_float(v1[j]) + __uint_as_float(w1[j]);
                }
                if (two) {                                  // the second half of the buffer rows, from the other accumulator
                    tmem_ld16_issue(acc + (uint32_t)(n_mma + j0), v0);
                    tmem_ld16_issue(acc + (uint32_t)(n_mma + j_pad + j0), w0);
                    if (second) {
                        tmem_ld16_issue(acc + (uint32_t)(n_mma + j0 + 16), v1);
                        tmem_ld16_issue(acc + (uint32_t)(n_mma + j_pad + j0 + 16), w1);
                    }
                    tmem_ld_wait();
                    tmem_ld_use(v0);
                    tmem_ld_use(w0);
#pragma unroll
                    for (int j = 0; j < 16; ++j) a0[j] += __uint_as_float(v0[j]) + __uint_as_float(w0[j]);
                    if (second) {
                        tmem_ld_use(v1);
                        tmem_ld_use(w1);
#pragma unroll
                        for (int j = 0; j < 16; ++j) a1[j] += __uint_as_float(v1[j]) + __uint_as_float(w1[j]);
                    }
                }
                if (d < pitch) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (j0 + j < keep) out[(long long)(j0 + j) * pitch + d] = a0[j];
                    if (second) {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (j0 + 16 + j < keep) out[(long long)(j0 + 16 + j) * pitch + d] = a1[j];
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&acc_empty[b]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (my_tiles > 0 && !*abort)
            mbar_wait_quiet(&acc_full[two ? 0 : (my_tiles - 1) & 1], (uint32_t)(two ? my_tiles - 1 : (my_tiles - 1) >> 1) & 1u, kWaitLimitCycles);
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && *abort) atomicExch(err, 1);
}

}  // namespace
}  // namespace tc

// See sage_internal.h.
static cudaError_t launch_tc_rebuild_part(const float* Wsplit, int ldw, int j_pad, const float* Bsrc, float* Bdst, int64_t pitch, int r,
                                          int keep, int* err, cudaStream_t st, const void* src = nullptr, int64_t ld_src = 0, int n_new = 0,
                                          int64_t D = 0) {
    if (keep <= 0 || r <= 0) return cudaSuccess;
    if (j_pad < 16 || j_pad > 128 || (j_pad & 15) || keep > j_pad || r > 512) return cudaErrorNotSupported;
    CUtensorMap tmBuf, tmW;
    // buffer: columns beyond D up to the pitch are zero and are rebuilt as zero, so the map spans the pitch
    // direct form (src != nullptr): only the rows that are in the buffer, plus the placeholder row, are addressable
    if (!tc::make_tmap_2d(&tmBuf, Bsrc, 4, (uint64_t)(src ? r - n_new + 1 : r), (uint64_t)pitch, (uint64_t)pitch, tc::kChunkRows, 1))
        return cudaErrorNotSupported;
    const int kcols = ((r + tc::kChunkRows - 1) / tc::kChunkRows) * tc::kChunkRows;
    if (kcols > ldw) return cudaErrorNotSupported;
    if (!tc::make_tmap_2d(&tmW, Wsplit, 4, (uint64_t)(2 * j_pad), (uint64_t)kcols, (uint64_t)ldw, (uint32_t)(2 * j_pad)))
        return cudaErrorNotSupported;
    // W resident in shared memory when all its chunk boxes take at most 64 KB (up to 128 buffer rows onto 64 output rows)
    const int nchunk = (r + tc::kChunkRows - 1) / tc::kChunkRows;
    const size_t w_all = (size_t)nchunk * 2 * j_pad * 128;
    const int w_res = w_all <= 64 * 1024 ? 1 : 0;
    CUtensorMap tmSrc = tmW, tmSrc1 = tmW;
    if (src) {
        if (!w_res || n_new < 2 || n_new >= r || (r - n_new + 1) % tc::kChunkRows != 0 || r % tc::kChunkRows != 0) return cudaErrorNotSupported;
        if (!tc::make_tmap_2d_plain(&tmSrc, src, 2, (uint64_t)n_new, (uint64_t)D, (uint64_t)ld_src, 128, (uint32_t)tc::kChunkRows) ||
            !tc::make_tmap_2d_plain(&tmSrc1, src, 2, (uint64_t)n_new, (uint64_t)D, (uint64_t)ld_src, 128, 1))
            return cudaErrorNotSupported;
    }
    const int stage_bytes = (w_res ? 2 * tc::kBufBytes : 2 * tc::kBufBytes + 2 * j_pad * 128) + (src ? 8192 : 0);
    int stages = (int)((227 * 1024 - 1536 - (w_res ? w_all : 0)) / stage_bytes);
    if (stages > 8) stages = 8;
    if (stages < 2) return cudaErrorNotSupported;
    const size_t smem = (size_t)stages * stage_bytes + (w_res ? w_all : 0) + 1024 + (3 * stages + 5) * 8 + 16;
    const long long num_tiles = (pitch + tc::kTileD - 1) / tc::kTileD;
    const int grid = (int)(num_tiles < 148 ? num_tiles : 148);
    cudaError_t e = cudaFuncSetAttribute(tc::k_tc_rebuild, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    tc::k_tc_rebuild<<<grid, tc::kThreads, smem, st>>>(tmBuf, tmW, tmSrc, tmSrc1, src ? n_new : 0, r, keep, j_pad, pitch, num_tiles, Bdst, stages,
                                                       w_res, err);
    return cudaGetLastError();
}

// See sage_internal.h. One launch takes at most 128 output rows (accumulator width) of up to 512 buffer rows; 129 to 256
// output rows (ell = 256: 255 rows out of 512) run as two launches over the same buffer rows.
cudaError_t launch_tc_rebuild(const float* Wsplit, int ldw, int j_pad, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D, int r,
                              int keep, int* err, cudaStream_t st) {
    (void)D;
    if (keep <= 0 || r <= 0) return cudaSuccess;
    if (j_pad < 16 || j_pad > 256 || (j_pad & 15) || keep > j_pad || r > 512) return cudaErrorNotSupported;
    const int jparts = j_pad > 128 ? 2 : 1;
    for (int jh = 0; jh < jparts; ++jh) {
        const int jp = jparts == 2 ? 128 : j_pad;
        const int keep_h = keep - jh * 128 < jp ? keep - jh * 128 : jp;
        if (keep_h <= 0) continue;
        const float* Wb = Wsplit + (size_t)(jparts == 2 ? jh * 256 : 0) * ldw;
        cudaError_t e = launch_tc_rebuild_part(Wb, ldw, jp, Bsrc, Bdst + (size_t)jh * 128 * pitch, pitch, r, keep_h, err, st);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// See sage_internal.h.
cudaError_t launch_tc_rebuild_direct(const float* Wsplit, int ldw, int j_pad, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D,
                                     int r, int keep, const void* src, int64_t ld_src, int n_new, int* err, cudaStream_t st) {
    if (keep <= 0 || r <= 0 || !src) return cudaErrorNotSupported;
    if (j_pad < 16 || j_pad > 128 || (j_pad & 15) || keep > j_pad || r > 128) return cudaErrorNotSupported;
    return launch_tc_rebuild_part(Wsplit, ldw, j_pad, Bsrc, Bdst, pitch, r, keep, err, st, src, ld_src, n_new, D);
}

}  // namespace sage

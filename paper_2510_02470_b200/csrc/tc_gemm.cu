// Tensor-core contraction C[z] = A_z * B_z^T over slices z of the contraction index, both operands
// contiguous along that index ("K-major"): the pass-2 projection Z = G S^T (Method, paragraph on two-pass scoring:
// z_i = S g_i) with G streamed from HBM exactly once.
//
// One CTA owns mt (1, 2 or 4) consecutive 128-row tiles of A, all N rows of B and one K slice; the B tile of
// a stage is shared by the mt row tiles, so B crosses L2 -> SM once per mt * 128 rows:
//   warp 0   TMA producer: 128-byte-wide K tiles of A (mt x 128 rows) and B (N rows) into a ring of stages,
//   warp 1   allocates TMEM and issues tcgen05.mma (M = 128, N, K = 32 bytes per instruction) into mt accumulators,
//   warps 2-5 read the fp32 accumulators out of TMEM (one row per thread) and store the partial result.
// Rows and K elements outside the matrices are zero-filled by TMA, so no tail code exists. Split-K
// partials are summed by a separate kernel in a fixed order.
#include "sage_internal.h"
#include "tc05.cuh"

namespace sage {
namespace tc {

bool make_tmap_2d(CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                  uint32_t box_rows, int atom32) {
    using Fn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                            const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                            CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Fn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<Fn>(fn);
    }();
    if (!encode) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((ld * (uint64_t)elem_bytes) & 15u) || rows == 0 || cols == 0) return false;
    if (box_rows == 0 || box_rows > 256 || cols >= (1ull << 32) || rows >= (1ull << 32)) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes), box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    return encode(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_2d_plain(CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                        uint32_t box_cols, uint32_t box_rows) {
    using Fn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                            const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                            CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Fn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<Fn>(fn);
    }();
    if (!encode) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((ld * (uint64_t)elem_bytes) & 15u) || rows == 0 || cols == 0) return false;
    if (box_rows == 0 || box_rows > 256 || box_cols == 0 || box_cols > 256 || ((box_cols * elem_bytes) & 15u) || cols >= (1ull << 32) ||
        rows >= (1ull << 32))
        return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * (uint64_t)elem_bytes};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    return encode(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tmap_4d_ktiles(CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols, uint64_t ld,
                         uint32_t box_rows, uint32_t kt) {
    using Fn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                            const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                            CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Fn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<Fn>(fn);
    }();
    if (!encode) return false;
    const uint64_t per_tile = 128 / elem_bytes, ktiles = cols / per_tile;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) || ((ld * (uint64_t)elem_bytes) & 15u) || rows == 0 || (rows & 7u) || ktiles == 0) return false;
    if (box_rows == 0 || box_rows > 256 || (box_rows & 7u) || kt == 0 || kt > 8 || rows >= (1ull << 32)) return false;
    const cuuint64_t dims[4] = {per_tile, 8, ktiles, rows / 8};
    const cuuint64_t strides[3] = {ld * (uint64_t)elem_bytes, 128, 8 * ld * (uint64_t)elem_bytes};
    const cuuint32_t box[4] = {static_cast<cuuint32_t>(per_tile), 8, kt, box_rows / 8};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    return encode(out, dt, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

constexpr int kThreads = 192;
constexpr int kTileM = 128;
constexpr int kATileBytes = kTileM * 128;

// kFmt: 1 = bf16 operands (64 elements per 128-byte K tile), 2 = fp32 operands read as tf32 (32 elements).
template <int kFmt>
__global__ void __launch_bounds__(kThreads, 1)
k_tc_gemm_nt(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmA4,
             const __grid_constant__ CUtensorMap tmB4, int kt2, int M, int N, int n_pad, int fold, int mt, long long K,
             long long k_per_split, int a_shared, float* __restrict__ C, long long ldc, long long split_stride, int stages,
             uint32_t tmem_cols, int* __restrict__ err) {
    constexpr int BK = kFmt == 1 ? 64 : 32;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_mma = fold ? 2 * n_pad : n_pad;         // folded: B holds two stacked operands whose products are added
    // kt2 (rows megabytes apart): a stage holds TWO K tiles, fetched by one 4-D box per operand tile so that every row
    // visit reads 256 consecutive bytes (see make_tmap_4d_ktiles); the two tiles lie interleaved by groups of 8 rows. A
    // slice's last odd or ragged K tiles go through the 2-D maps (zero fill) into the front of a stage.
    const int ktn = kt2 ? 2 : 1;
    const int a_tile_bytes = ktn * kATileBytes;
    const int a_bytes = mt * a_tile_bytes;
    const int stage_bytes = a_bytes + ktn * n_mma * 128;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
    uint64_t* empty = full + stages;
    uint64_t* tmem_full = empty + stages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_full + 1);
    volatile int* abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kTileM * mt;
    const long long k_begin = (long long)blockIdx.y * k_per_split;
    const long long k_end = K < k_begin + k_per_split ? K : k_begin + k_per_split;
    const int nkt = k_end > k_begin ? (int)((k_end - k_begin + BK - 1) / BK) : 0;
    const int npairs = kt2 && k_end > k_begin ? (int)((k_end - k_begin) / BK) / 2 : 0;   // pairs of whole K tiles
    const int nsteps = npairs + (nkt - 2 * npairs);                                     // stages filled by this CTA

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(tmem_full, 1);
        *abort = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) tmem_alloc(tmem_slot, tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int issued = 0;
            int s = 0;
            uint32_t ph = 1;                                    // parity of the empty-barrier phase to wait for
            uint8_t* st = smem;
            const int kt_b0 = (int)(k_begin / BK), kt_a0 = a_shared ? 0 : kt_b0;   // class slices: every slice reads the same columns of A
            for (int i = 0; i < nsteps; ++i) {
                if (!mbar_wait(&empty[s], ph, abort)) break;
                if (i < npairs) {
                    mbar_expect_tx(&full[s], (uint32_t)stage_bytes);
                    for (int t = 0; t < mt; ++t)     // row groups past the end of A are zero-filled by TMA
                        tma_load_4d(st + (size_t)t * a_tile_bytes, &tmA4, &full[s], 0, 0, kt_a0 + 2 * i, (m0 + t * kTileM) / 8);
                    tma_load_4d(st + a_bytes, &tmB4, &full[s], 0, 0, kt_b0 + 2 * i, 0);
                } else {
                    const int kt = 2 * npairs + (i - npairs);
                    mbar_expect_tx(&full[s], (uint32_t)(mt * kATileBytes + n_mma * 128));
                    const int x = (int)(k_begin + (long long)kt * BK);
                    const int xa = a_shared ? kt * BK : x;
                    for (int t = 0; t < mt; ++t)     // row tiles past the end of A are zero-filled by TMA
                        tma_load_2d(st + (size_t)t * a_tile_bytes, &tmA, &full[s], xa, m0 + t * kTileM);
                    tma_load_2d(st + a_bytes, &tmB, &full[s], x, 0);
                }
                issued = i + 1;
                if (++s == stages) { s = 0; ph ^= 1u; st = smem; } else { st += stage_bytes; }
            }
            if (*abort) {   // give copies already in flight a bounded time to land before the block goes away
                for (int kt = issued > stages ? issued - stages : 0; kt < issued; ++kt)
                    mbar_wait_quiet(&full[kt % stages], (uint32_t)(kt / stages) & 1u, 20000000ll);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(kFmt, kTileM, n_mma, 0, 0);
            const uint32_t st0 = smem_u32(smem);
            int s = 0;
            uint32_t ph = 0, st = st0;
            bool first = true;                         // the first MMA of every accumulator overwrites it
            for (int i = 0; i < nsteps; ++i) {
                if (!mbar_wait(&full[s], ph, abort)) break;
                tc_fence_after();
                const bool pair = i < npairs;
                const uint32_t group_stride = pair ? 2048u : 1024u;
                for (int kk = 0; kk < (pair ? 2 : 1); ++kk) {
                    const uint64_t bdesc = smem_desc_k_sw128(st + a_bytes + kk * 1024, group_stride);
                    for (int t = 0; t < mt; ++t) {
                        const uint64_t adesc = smem_desc_k_sw128(st + t * a_tile_bytes + kk * 1024, group_stride);
                        const uint32_t acc = tmem_base + (uint32_t)(t * n_mma);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {      // 4 x 32 bytes of K per 128-byte row
                            if constexpr (kFmt == 1) mma_bf16(acc, adesc + 2 * k, bdesc + 2 * k, idesc, !(first && k == 0));
                            else mma_tf32(acc, adesc + 2 * k, bdesc + 2 * k, idesc, !(first && k == 0));
                        }
                    }
                    first = false;
                }
                mma_commit(&empty[s]);                 // the stage is free once these MMAs have read it
                if (++s == stages) { s = 0; ph ^= 1u; st = st0; } else { st += (uint32_t)stage_bytes; }
            }
            mma_commit(tmem_full);
        }
    } else {
        const int quarter = warp & 3;                  // TMEM lanes this warp may read: 32 * (warp % 4) ...
        bool ok = true;
        if (nkt > 0) ok = mbar_wait(tmem_full, 0, abort);
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        const bool vec = (ldc % 4 == 0) && ((reinterpret_cast<uintptr_t>(C) & 15u) == 0) && (split_stride % 4 == 0);
        for (int t = 0; t < mt; ++t) {
            const int row = m0 + t * kTileM + quarter * 32 + lane;
            float* crow = C + (long long)blockIdx.y * split_stride + (long long)row * ldc;
            const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + (uint32_t)(t * n_mma);
            for (int c0 = 0; c0 < n_pad; c0 += 16) {
                float v[16];
                if (nkt > 0 && ok) {
                    tmem_ld16(lane_base + (uint32_t)c0, v);
                    if (fold) {
                        float w[16];
                        tmem_ld16(lane_base + (uint32_t)(n_pad + c0), w);
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] += w[j];
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = 0.f;
                }
                if (row < M) {
                    if (vec && c0 + 16 <= N) {
#pragma unroll
                        for (int j = 0; j < 16; j += 4) *reinterpret_cast<float4*>(crow + c0 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c0 + j < N) crow[c0 + j] = v[j];
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (nkt > 0) mbar_wait_quiet(tmem_full, 0, kWaitLimitCycles);   // no MMA in flight when TMEM is freed
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && *abort) atomicExch(err, 1);
}

}  // namespace
}  // namespace tc

cudaError_t launch_tc_gemm_nt(const void* A, sage_dtype_t dt, int64_t lda, const void* Bm, int64_t ldb, int M, int N, int fold,
                              int mt, int64_t K, int splits, float* C, int64_t ldc, int64_t split_stride, int* err, cudaStream_t st,
                              int64_t class_F) {
    if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
    const int es = dt == SAGE_F32 ? 4 : 2;
    const int BK = 128 / es;
    const int n_pad = ((N + 15) / 16) * 16;
    const int n_mma = fold ? 2 * n_pad : n_pad;
    if (n_mma > 256 || splits < 1 || splits > 65535) return cudaErrorNotSupported;
    if ((mt != 1 && mt != 2 && mt != 4) || mt * n_mma > 512) return cudaErrorNotSupported;
    CUtensorMap tmA, tmB;
    // class slices: A has class_F columns, slice c contracts them with columns [c class_F, (c + 1) class_F) of Bm. A slice
    // starts at a multiple of class_F, which TMA wants on a 16-byte boundary; its last K tile may reach into the next
    // slice's columns of Bm, where A reads as zero (beyond its extent).
    if (class_F > 0 && ((class_F * es) % 16 != 0 || (int64_t)splits * class_F != K)) return cudaErrorNotSupported;
    if (!tc::make_tmap_2d(&tmA, A, es, (uint64_t)M, (uint64_t)(class_F > 0 ? class_F : K), (uint64_t)lda, tc::kTileM)) return cudaErrorNotSupported;
    if (!tc::make_tmap_2d(&tmB, Bm, es, (uint64_t)(fold ? n_pad + N : N), (uint64_t)K, (uint64_t)ldb, (uint32_t)n_mma))
        return cudaErrorNotSupported;
    int64_t kps = (K + splits - 1) / splits;
    kps = ((kps + BK - 1) / BK) * BK;
    if (class_F > 0) kps = class_F;
    const int a_shared = class_F > 0 ? 1 : 0;
    // a trailing slice may be empty after rounding to whole K tiles: its CTAs store zeros
    // Rows at least a page (2 MB) apart: two K tiles per stage through 4-D boxes (256 bytes per row visit), where the
    // shapes allow it (whole groups of 8 rows in both operands, slices that start on a K tile) and two such stages fit.
    CUtensorMap tmA4 = tmA, tmB4 = tmB;
    const uint64_t b_rows = (uint64_t)(fold ? n_pad + N : N);
    int kt2 = (lda * es >= (2 << 20) && M % 8 == 0 && b_rows % 8 == 0 && (class_F == 0 || class_F % BK == 0) &&
               2 * (2 * mt * tc::kATileBytes + 2 * n_mma * 128) + 2048 <= 227 * 1024)
                  ? 1 : 0;
    if (kt2 && !(tc::make_tmap_4d_ktiles(&tmA4, A, es, (uint64_t)M, (uint64_t)(class_F > 0 ? class_F : K), (uint64_t)lda, tc::kTileM, 2) &&
                 tc::make_tmap_4d_ktiles(&tmB4, Bm, es, b_rows, (uint64_t)K, (uint64_t)ldb, (uint32_t)n_mma, 2)))
        kt2 = 0;
    const int stage_bytes = (kt2 ? 2 : 1) * (mt * tc::kATileBytes + n_mma * 128);
    int stages = ((kt2 ? 227 * 1024 - 2048 : 200 * 1024)) / stage_bytes;
    if (stages > 8) stages = 8;
    if (stages < 2) return cudaErrorNotSupported;
    const size_t smem = (size_t)stages * stage_bytes + 1024 + (2 * stages + 1) * 8 + 16;
    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)(mt * n_mma)) tmem_cols <<= 1;
    const int tiles = (M + tc::kTileM - 1) / tc::kTileM;
    dim3 grid((unsigned)((tiles + mt - 1) / mt), (unsigned)splits);
    cudaError_t e;
    if (dt == SAGE_BF16) {
        e = cudaFuncSetAttribute(tc::k_tc_gemm_nt<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        tc::k_tc_gemm_nt<1><<<grid, tc::kThreads, smem, st>>>(tmA, tmB, tmA4, tmB4, kt2, M, N, n_pad, fold, mt, K, kps, a_shared, C, ldc, split_stride, stages,
                                                              tmem_cols, err);
    } else {
        e = cudaFuncSetAttribute(tc::k_tc_gemm_nt<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        tc::k_tc_gemm_nt<2><<<grid, tc::kThreads, smem, st>>>(tmA, tmB, tmA4, tmB4, kt2, M, N, n_pad, fold, mt, K, kps, a_shared, C, ldc, split_stride, stages,
                                                              tmem_cols, err);
    }
    return cudaGetLastError();
}

}  // namespace sage

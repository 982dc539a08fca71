// Generic (alignment-free) CUDA-core kernels of the sketch path: row append, Gram / projection
// contraction, split reduction and the rebuild. They accept any pitch and any D; the tensor-core
// kernels take over where their alignment rules hold.
#include "sage_internal.h"

namespace sage {
namespace {

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// ------------------------------------------------------------------------------------------------
// Append (Algorithm 1, Phase I, the row insertion): copy / convert rows into free buffer rows.
// One block row of threads walks a row with 16-byte accesses where the addresses allow it.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) k_append(const T* __restrict__ rows, int64_t n, int64_t ld, int64_t D,
                                                float* __restrict__ B, int64_t pitch, int dst_row0) {
    constexpr int V = 16 / sizeof(T);   // elements per 16-byte load
    const int64_t row = blockIdx.y;
    const T* src = rows + row * ld;
    float* dst = B + (int64_t)(dst_row0 + row) * pitch;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(src) & 15) == 0);
    const int64_t chunk0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * V;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x * V;
    for (int64_t c = chunk0; c < pitch; c += stride) {
        float v[V];
        if (vec_ok && c + V <= D) {
            const uint4 raw = *reinterpret_cast<const uint4*>(src + c);
            const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
            for (int i = 0; i < V; ++i) v[i] = to_f32(e[i]);
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) v[i] = (c + i < D) ? to_f32(src[c + i]) : 0.0f;
        }
        if (c + V <= pitch) {   // pitch is a multiple of 4 floats and dst rows are 16-byte aligned
#pragma unroll
            for (int i = 0; i < V; i += 4) *reinterpret_cast<float4*>(dst + c + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i)
                if (c + i < pitch) dst[c + i] = v[i];
        }
    }
}

// Append of structured last-layer rows (the per-example gradient of a softmax head, Method section): row i is
// [vec_rowmajor(q_i h_i^T) ; q_i] with q_i (C values) = softmax - onehot and h_i (F values) the features; it is formed here
// from the two factors and written straight into the destination rows, so the C F + C values never exist in the caller's
// memory. Products are taken in fp32 (exact for bf16 factors). Columns from C F + C up to the pitch are zeroed.
template <typename T>
__global__ void __launch_bounds__(256) k_append_outer(const T* __restrict__ q, int64_t ldq, const T* __restrict__ feat, int64_t ldf, int C,
                                                      int F, float* __restrict__ B, int64_t pitch, int dst_row0) {
    const int64_t row = blockIdx.y;
    const T* qr = q + row * ldq;
    const T* hr = feat + row * ldf;
    float* dst = B + (int64_t)(dst_row0 + row) * pitch;
    const int64_t CF = (int64_t)C * F, D = CF + C;
    const int64_t c0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x * 4;
    for (int64_t d = c0; d < pitch; d += stride) {          // the pitch is a multiple of 4 elements, rows are 16-byte aligned
        float v[4];
        const int c0q = (int)(d / F);
        const int f0 = (int)(d - (int64_t)c0q * F);
        if (d + 3 < CF && f0 + 3 < F) {              // the four columns belong to one class: one factor, four features
            const float qc = to_f32(qr[c0q]);
#pragma unroll
            for (int i = 0; i < 4; ++i) v[i] = qc * to_f32(hr[f0 + i]);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int64_t e = d + i;
                if (e < CF) {
                    const int c = (int)(e / F), f = (int)(e - (int64_t)c * F);
                    v[i] = to_f32(qr[c]) * to_f32(hr[f]);
                } else {
                    v[i] = e < D ? to_f32(qr[e - CF]) : 0.f;
                }
            }
        }
        *reinterpret_cast<float4*>(dst + d) = make_float4(v[0], v[1], v[2], v[3]);
    }
}

// ------------------------------------------------------------------------------------------------
// C[z] = A_z * Bm_z^T over the z-th slice of the contraction index (both operands k-contiguous).
// 64 x 64 output tile, 32-deep k tiles, 256 threads with 4 x 4 register tiles. The register
// accumulators are folded into a second set every kFold k-tiles to bound fp32 summation error on
// very long contractions.
// ------------------------------------------------------------------------------------------------
constexpr int BM = 64, BN = 64, BK = 32, PAD = 4, kFold = 64;

template <typename T>
__device__ __forceinline__ void load4(const T* p, bool vec, int64_t k, int64_t k_end, float out[4]) {
    if (vec && k + 4 <= k_end) {
        if constexpr (sizeof(T) == 4) {
            const float4 v = *reinterpret_cast<const float4*>(p + k);
            out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
        } else {
            const uint2 raw = *reinterpret_cast<const uint2*>(p + k);
            const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) out[i] = to_f32(e[i]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = (k + i < k_end) ? to_f32(p[k + i]) : 0.0f;
    }
}

template <typename T>
__global__ void __launch_bounds__(256) k_gemm_nt(const T* __restrict__ A, int64_t lda, const float* __restrict__ Bm,
                                                 int64_t ldb, int M, int N, int64_t K, int64_t k_per_split, int a_shared,
                                                 float* __restrict__ C, int64_t ldc, int64_t split_stride) {
    __shared__ float As[BK][BM + PAD];
    __shared__ float Bs[BK][BN + PAD];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int64_t k_begin = (int64_t)blockIdx.z * k_per_split;
    const int64_t k_end = min(K, k_begin + k_per_split);
    const int lrow = tid >> 3;          // 0..31
    const int lk = (tid & 7) * 4;       // 0,4,..,28
    const int ty = tid >> 4, tx = tid & 15;
    // class slices (a_shared): slice z contracts columns [0, k_per_split) of A with columns [k_begin, k_end) of Bm
    const int64_t a_back = a_shared ? k_begin : 0;
    const bool a_vec = (lda * sizeof(T)) % (4 * sizeof(T)) == 0 && (reinterpret_cast<uintptr_t>(A) % (4 * sizeof(T))) == 0 &&
                       (lda % 4 == 0) && ((k_begin - a_back) % 4 == 0);
    const bool b_vec = (ldb % 4 == 0) && (reinterpret_cast<uintptr_t>(Bm) % 16 == 0) && (k_begin % 4 == 0);

    float acc[4][4] = {}, tot[4][4] = {};
    int fold = 0;
    for (int64_t k0 = k_begin; k0 < k_end; k0 += BK) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = lrow + h * 32;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (m0 + r < M) load4(A + (int64_t)(m0 + r) * lda, a_vec, k0 + lk - a_back, k_end - a_back, v);
#pragma unroll
            for (int i = 0; i < 4; ++i) As[lk + i][r] = v[i];
            float w[4] = {0.f, 0.f, 0.f, 0.f};
            if (n0 + r < N) load4(Bm + (int64_t)(n0 + r) * ldb, b_vec, k0 + lk, k_end, w);
#pragma unroll
            for (int i = 0; i < 4; ++i) Bs[lk + i][r] = w[i];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
        if (++fold == kFold) {
            fold = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) { tot[i][j] += acc[i][j]; acc[i][j] = 0.f; }
        }
    }
    float* Cz = C + (int64_t)blockIdx.z * split_stride;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = m0 + ty * 4 + i;
        if (r >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = n0 + tx * 4 + j;
            if (c < N) Cz[(int64_t)r * ldc + c] = tot[i][j] + acc[i][j];
        }
    }
}

__global__ void __launch_bounds__(256) k_to_bf16(const float* __restrict__ src, int64_t lds, int64_t cols, __nv_bfloat16* __restrict__ hi,
                                                  __nv_bfloat16* __restrict__ lo, int64_t ldd) {
    const float* s = src + (int64_t)blockIdx.y * lds;
    __nv_bfloat16* dh = hi + (int64_t)blockIdx.y * ldd;
    __nv_bfloat16* dl = lo ? lo + (int64_t)blockIdx.y * ldd : nullptr;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < cols; c += (int64_t)gridDim.x * blockDim.x) {
        const float x = s[c];
        const __nv_bfloat16 h = __float2bfloat16_rn(x);
        dh[c] = h;
        if (dl) dl[c] = __float2bfloat16_rn(x - __bfloat162float(h));
    }
}

// The frozen sketch split once for the tf32 tensor cores: hi = 11 significant bits, lo = the exact remainder.
__global__ void __launch_bounds__(256) k_split_tf32(const float* __restrict__ src, int64_t lds, int64_t cols, float* __restrict__ out,
                                                     int64_t ldo) {
    const float* s = src + (int64_t)blockIdx.y * lds;
    float* dh = out + (int64_t)blockIdx.y * ldo;
    float* dl = out + (int64_t)(64 + blockIdx.y) * ldo;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < cols; c += (int64_t)gridDim.x * blockDim.x) {
        const float x = s[c];
        const float h = __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
        dh[c] = h;
        dl[c] = x - h;
    }
}

// mirror != 0 (a symmetric matrix of which only the 128 x 128 tiles on and above the diagonal were computed): elements of
// the tiles below the diagonal are read from their mirror image.
__global__ void __launch_bounds__(256) k_split_reduce(const float* __restrict__ parts, int splits, int64_t split_stride,
                                                      int M, int N, int64_t ldp, float* __restrict__ out, int64_t ldo, int mirror) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (int64_t)M * N) return;
    const int i = (int)(e / N), j = (int)(e % N);
    const bool below = mirror && (i >> 7) > (j >> 7);
    const float* src = parts + (below ? (int64_t)j * ldp + i : (int64_t)i * ldp + j);
    double s = 0.0;
    for (int z = 0; z < splits; ++z) s += (double)src[(int64_t)z * split_stride];
    out[(int64_t)i * ldo + j] = (float)s;
}

// Split reduction of a Gram matrix computed in the symmetric form: slice z left T_z = hi*hi^T + 2*hi*lo^T at
// parts + z*stride; K = sum_z (T_z + T_z^T) / 2 in fp64. One block of 16 x 16 x 4 threads per 16 x 16 tile (I, J): thread
// (ty, tx) of layer tz sums T[I+ty][J+tx] and T[J+ty][I+tx] (both read along rows) over the slices z = tz, tz+4, ...;
// the four layers are added in a fixed order and the second sum is transposed through shared memory.
__global__ void __launch_bounds__(1024) k_gram_sym_reduce(const float* __restrict__ parts, int splits, int64_t stride, int r,
                                                          int64_t ldp, float* __restrict__ out, int64_t ldo) {
    // 16 x 16 outputs per block; the four z-layers of the block each sum a quarter of the partial matrices
    // (several loads in flight per thread: the kernel is bound by load latency, not by bytes).
    __shared__ double sa[4][16][17], sb[4][16][17];
    const int tx = threadIdx.x, ty = threadIdx.y, tz = threadIdx.z;
    const int i = blockIdx.y * 16 + ty, j = blockIdx.x * 16 + tx;          // direct element (i, j)
    const int ti = blockIdx.x * 16 + ty, tj = blockIdx.y * 16 + tx;        // element (ti, tj) of the mirrored tile
    double a = 0.0, b = 0.0;
    const bool in_a = i < r && j < r, in_b = ti < r && tj < r;
    const float* pa = parts + (in_a ? (int64_t)i * ldp + j : 0);
    const float* pb = parts + (in_b ? (int64_t)ti * ldp + tj : 0);
#pragma unroll 4
    for (int z = tz; z < splits; z += 4) {
        const float va = pa[(int64_t)z * stride], vb = pb[(int64_t)z * stride];
        a += (double)va;
        b += (double)vb;
    }
    sa[tz][ty][tx] = a;
    sb[tz][ty][tx] = b;                                                    // belongs to out[I + tx'][J + ty'] after the transpose
    __syncthreads();
    if (tz == 0 && in_a) {
        const double sum_a = (sa[0][ty][tx] + sa[1][ty][tx]) + (sa[2][ty][tx] + sa[3][ty][tx]);
        const double sum_b = (sb[0][tx][ty] + sb[1][tx][ty]) + (sb[2][tx][ty] + sb[3][tx][ty]);
        out[(int64_t)i * ldo + j] = (float)(0.5 * (sum_a + sum_b));
    }
}

// ------------------------------------------------------------------------------------------------
// Rebuild (Method, first paragraph: the sketch is rebuilt from the shrunk singular values and the right factor): with B B^T = U Lambda U^T,
// Sigma' V^T = diag(sigma'_j / sigma_j) U^T B, so out[j][:] = sum_i Ur[i][j] B[i][:] where Ur already
// carries the factor sqrt(max(1 - delta/lambda_j, 0)). Source and destination are different buffers.
// Block tile: 64 output rows x 128 columns, contraction over the r buffer rows in steps of 16.
// ------------------------------------------------------------------------------------------------
constexpr int RM = 64, RN = 128, RK = 16;

__global__ void __launch_bounds__(256) k_rebuild(const float* __restrict__ Ur, int ldu, const float* __restrict__ Bsrc,
                                                 float* __restrict__ Bdst, int64_t pitch, int r, int keep, int m_total) {
    __shared__ float Us[RK][RM];
    __shared__ float Bs[RK][RN];
    const int tid = threadIdx.x;
    const int64_t d0 = (int64_t)blockIdx.x * RN;
    const int j0 = blockIdx.y * RM;
    const int ty = tid >> 5, tx = tid & 31;     // 8 x 32 threads -> 8 rows x 4 cols each
    if (j0 >= keep) {                           // rows beyond keep: zero fill
        for (int j = j0 + ty; j < min(j0 + RM, m_total); j += 8)
            for (int c = tx * 4; c < RN; c += 128)
                if (d0 + c < pitch) *reinterpret_cast<float4*>(Bdst + (int64_t)j * pitch + d0 + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    float acc[8][4] = {};
    for (int i0 = 0; i0 < r; i0 += RK) {
        for (int e = tid; e < RK * RM; e += 256) {
            const int kk = e / RM, jj = e % RM;
            Us[kk][jj] = (i0 + kk < r && j0 + jj < keep) ? Ur[(int64_t)(i0 + kk) * ldu + j0 + jj] : 0.f;
        }
        for (int e = tid; e < RK * RN / 4; e += 256) {
            const int kk = e / (RN / 4), cc = (e % (RN / 4)) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i0 + kk < r && d0 + cc < pitch) v = *reinterpret_cast<const float4*>(Bsrc + (int64_t)(i0 + kk) * pitch + d0 + cc);
            *reinterpret_cast<float4*>(&Bs[kk][cc]) = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < RK; ++kk) {
            const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float u = Us[kk][ty * 8 + i];
                acc[i][0] = fmaf(u, b.x, acc[i][0]);
                acc[i][1] = fmaf(u, b.y, acc[i][1]);
                acc[i][2] = fmaf(u, b.z, acc[i][2]);
                acc[i][3] = fmaf(u, b.w, acc[i][3]);
            }
        }
        __syncthreads();
    }
    if (d0 + tx * 4 >= pitch) return;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int j = j0 + ty * 8 + i;
        if (j >= m_total) continue;
        float4 v = (j < keep) ? make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]) : make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(Bdst + (int64_t)j * pitch + d0 + tx * 4) = v;
    }
}

}  // namespace

cudaError_t launch_append(const void* rows, sage_dtype_t dt, int64_t n, int64_t ld, int64_t D, float* B, int64_t pitch,
                          int dst_row0, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const int V = dt == SAGE_F32 ? 4 : 8;
    int64_t bx = (pitch / V + 255) / 256;
    if (bx > 592) bx = 592;
    if (bx < 1) bx = 1;
    dim3 grid((unsigned)bx, (unsigned)n);
    if (dt == SAGE_F32)
        k_append<float><<<grid, 256, 0, st>>>(static_cast<const float*>(rows), n, ld, D, B, pitch, dst_row0);
    else
        k_append<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(rows), n, ld, D, B, pitch, dst_row0);
    return cudaGetLastError();
}

cudaError_t launch_append_outer(const void* q, int64_t ldq, const void* feat, int64_t ldf, sage_dtype_t dt, int64_t n, int C, int F,
                                float* B, int64_t pitch, int dst_row0, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    if (pitch & 3) return cudaErrorInvalidValue;
    int64_t bx = (pitch / 4 + 255) / 256;
    if (bx > 592) bx = 592;
    if (bx < 1) bx = 1;
    dim3 grid((unsigned)bx, (unsigned)n);
    if (dt == SAGE_F32)
        k_append_outer<float><<<grid, 256, 0, st>>>(static_cast<const float*>(q), ldq, static_cast<const float*>(feat), ldf, C, F, B, pitch,
                                                    dst_row0);
    else
        k_append_outer<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(q), ldq, static_cast<const __nv_bfloat16*>(feat),
                                                            ldf, C, F, B, pitch, dst_row0);
    return cudaGetLastError();
}

cudaError_t launch_gemm_nt(const void* A, sage_dtype_t dt, int64_t lda, const float* Bm, int64_t ldb, int M, int N,
                           int64_t K, int splits, float* C, int64_t ldc, int64_t split_stride, cudaStream_t st, int64_t class_F) {
    if (M <= 0 || N <= 0) return cudaSuccess;
    if (class_F > 0 && (int64_t)splits * class_F != K) return cudaErrorInvalidValue;
    int64_t kps = (K + splits - 1) / splits;
    kps = ((kps + BK - 1) / BK) * BK;
    if (class_F > 0) kps = class_F;
    const int a_shared = class_F > 0 ? 1 : 0;
    dim3 grid((M + BM - 1) / BM, (N + BN - 1) / BN, splits);
    if (dt == SAGE_F32)
        k_gemm_nt<float><<<grid, 256, 0, st>>>(static_cast<const float*>(A), lda, Bm, ldb, M, N, K, kps, a_shared, C, ldc, split_stride);
    else
        k_gemm_nt<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(A), lda, Bm, ldb, M, N, K, kps, a_shared, C,
                                                       ldc, split_stride);
    return cudaGetLastError();
}

cudaError_t launch_to_bf16(const float* src, int64_t lds, int rows, int64_t cols, __nv_bfloat16* hi, __nv_bfloat16* lo, int64_t ldd,
                           cudaStream_t st) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    int64_t bx = (cols + 255) / 256;
    if (bx > 1184) bx = 1184;
    k_to_bf16<<<dim3((unsigned)bx, (unsigned)rows), 256, 0, st>>>(src, lds, cols, hi, lo, ldd);
    return cudaGetLastError();
}

cudaError_t launch_split_tf32(const float* src, int64_t lds, int rows, int64_t cols, float* out, int64_t ldo, cudaStream_t st) {
    if (rows <= 0 || cols <= 0) return cudaSuccess;
    if (rows > 64) return cudaErrorInvalidValue;
    int64_t bx = (cols + 255) / 256;
    if (bx > 1184) bx = 1184;
    k_split_tf32<<<dim3((unsigned)bx, (unsigned)rows), 256, 0, st>>>(src, lds, cols, out, ldo);
    return cudaGetLastError();
}

cudaError_t launch_split_reduce(const float* parts, int splits, int64_t split_stride, int M, int N, int64_t ldp, float* out,
                                int64_t ldo, cudaStream_t st, int mirror) {
    const int64_t total = (int64_t)M * N;
    if (total <= 0) return cudaSuccess;
    k_split_reduce<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(parts, splits, split_stride, M, N, ldp, out, ldo, mirror);
    return cudaGetLastError();
}

cudaError_t launch_gram_sym_reduce(const float* parts, int splits, int64_t stride, int r, int64_t ldp, float* out, int64_t ldo,
                                   cudaStream_t st) {
    if (r <= 0) return cudaSuccess;
    const unsigned t = (unsigned)((r + 15) / 16);
    k_gram_sym_reduce<<<dim3(t, t), dim3(16, 16, 4), 0, st>>>(parts, splits, stride, r, ldp, out, ldo);
    return cudaGetLastError();
}

cudaError_t launch_rebuild(const float* Ur, int ldu, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D, int r, int keep,
                           int m_total, cudaStream_t st) {
    (void)D;
    dim3 grid((unsigned)((pitch + RN - 1) / RN), (unsigned)((m_total + RM - 1) / RM));
    k_rebuild<<<grid, 256, 0, st>>>(Ur, ldu, Bsrc, Bdst, pitch, r, keep, m_total);
    return cudaGetLastError();
}

}  // namespace sage

// Phase II after the projection (Method, paragraph on two-pass scoring; Algorithm 1, Phase II):
// row normalisation zhat_i = z_i/||z_i|| (0 when z_i = 0), the consensus sum over all rows, the unit
// consensus u and the agreement scores alpha_i = <zhat_i, u>. All reductions run in a fixed order, so
// a given sequence of calls gives bit-identical results every time.
#include "sage_internal.h"

namespace sage {
namespace {

constexpr int kRowsPerBlock = 64;   // rows whose zhat are summed into one partial
constexpr int kMaxPerLane = 8;      // ell <= 256

// One warp per row, 8 warps per block, each warp walks rows w, w+8, ... of the block's 64 rows.
// planes > 1: the projections arrive as that many partial planes (K slices of the projection, `plane_stride` floats apart),
// which are summed here in ascending plane order with fp64 accumulation before the row is normalised.
__global__ void __launch_bounds__(256) k_normalise(const float* __restrict__ Z, int planes, int64_t plane_stride, int64_t ldz, int64_t n,
                                                   int ell, float* __restrict__ zhat, float* __restrict__ znorm,
                                                   float* __restrict__ partials, unsigned* __restrict__ flags) {
    __shared__ float part[8][256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row0 = (int64_t)blockIdx.x * kRowsPerBlock;
    float sum[kMaxPerLane];
#pragma unroll
    for (int t = 0; t < kMaxPerLane; ++t) sum[t] = 0.f;
    bool bad = false;
    for (int rr = warp; rr < kRowsPerBlock; rr += 8) {
        const int64_t row = row0 + rr;
        if (row >= n) break;
        float z[kMaxPerLane];
        float amax = 0.f;
        bool finite = true;
#pragma unroll
        for (int t = 0; t < kMaxPerLane; ++t) {
            const int j = lane + 32 * t;
            if (j >= ell) {
                z[t] = 0.f;
            } else if (planes == 1) {
                z[t] = Z[row * ldz + j];
            } else {
                const float* src = Z + row * ldz + j;
                double acc = 0.0;
                int pz = 0;
                for (; pz + 4 <= planes; pz += 4) {      // four loads in flight, added in plane order
                    const float a0 = src[(int64_t)pz * plane_stride], a1 = src[(int64_t)(pz + 1) * plane_stride];
                    const float a2 = src[(int64_t)(pz + 2) * plane_stride], a3 = src[(int64_t)(pz + 3) * plane_stride];
                    acc += (double)a0;
                    acc += (double)a1;
                    acc += (double)a2;
                    acc += (double)a3;
                }
                for (; pz < planes; ++pz) acc += (double)src[(int64_t)pz * plane_stride];
                z[t] = (float)acc;
            }
            finite = finite && (fabsf(z[t]) <= 3.0e38f);   // false for NaN and Inf
            amax = fmaxf(amax, fabsf(z[t]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        finite = __all_sync(0xffffffffu, finite);
        float nrm = 0.f, scale = 0.f;
        if (finite && amax > 0.f) {
            const float inv = 1.f / amax;
            float s = 0.f;
#pragma unroll
            for (int t = 0; t < kMaxPerLane; ++t) {
                z[t] *= inv;
                s = fmaf(z[t], z[t], s);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            const float rs = sqrtf(s);
            nrm = amax * rs;
            scale = 1.f / rs;
        }
        if (!finite) bad = true;
#pragma unroll
        for (int t = 0; t < kMaxPerLane; ++t) {
            const int j = lane + 32 * t;
            const float v = z[t] * scale;       // scale = 0 for zero / non-finite rows
            if (j < ell) zhat[row * ell + j] = (scale > 0.f) ? v : 0.f;
            sum[t] += (scale > 0.f) ? v : 0.f;
        }
        if (lane == 0) znorm[row] = nrm;
    }
#pragma unroll
    for (int t = 0; t < kMaxPerLane; ++t) part[warp][lane + 32 * t] = sum[t];
    __syncthreads();
    if (threadIdx.x < ell) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += part[w][threadIdx.x];
        partials[(int64_t)blockIdx.x * ell + threadIdx.x] = s;
    }
    if (bad && lane == 0) atomicOr(flags, kFlagNonFinite);
}

// zsum[j] += sum over blocks b of partials[b][j], in a fixed order: the 1024 threads form 1024 / jw groups (jw = ell rounded up to
// a power of two, at least 32); group g adds the partials of blocks g, g + G, g + 2G, ... in ascending order in fp64, and the
// groups' sums are then added in ascending g.
__global__ void __launch_bounds__(1024) k_accumulate(const float* __restrict__ partials, int nblocks, int ell, int jw,
                                                     double* __restrict__ zsum) {
    __shared__ double sh[1024];
    const int G = 1024 / jw;
    const int j = threadIdx.x % jw, g = threadIdx.x / jw;
    double s = 0.0;
    if (j < ell)
        for (int b = g; b < nblocks; b += G) s += (double)partials[(int64_t)b * ell + j];
    sh[threadIdx.x] = s;
    __syncthreads();
    if (g == 0 && j < ell) {
        double t = zsum[j];
        for (int q = 0; q < G; ++q) t += sh[q * jw + j];
        zsum[j] = t;
    }
}

// u = zsum/||zsum|| (the 1/N of the mean cancels); alpha_i = <zhat_i, u>. One warp per row.
__global__ void __launch_bounds__(256) k_consensus_score(const double* __restrict__ zsum, const float* __restrict__ zhat,
                                                         int64_t N, int ell, float* __restrict__ u_out,
                                                         float* __restrict__ scores) {
    __shared__ float u[256];
    __shared__ double red[8];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double v = (tid < ell) ? zsum[tid] : 0.0;
    double sq = v * v;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) red[warp] = sq;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    const double nrm = sqrt(tot);
    u[tid] = (nrm > 0.0 && tid < ell) ? (float)(v / nrm) : 0.f;
    if (blockIdx.x == 0 && tid < ell) u_out[tid] = u[tid];
    __syncthreads();
    const int64_t row = (int64_t)blockIdx.x * 8 + warp;
    if (row >= N) return;
    float acc = 0.f;
    for (int j = lane; j < ell; j += 32) acc = fmaf(zhat[row * ell + j], u[j], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) scores[row] = fminf(1.f, fmaxf(-1.f, acc));
}


// Structured rows: the projection z_i = sum_c q_ic (S_c h_i + b_c), b_c = column c of the bias block of the sketch, from the
// per-class planes T_c = H S_c^T. A thread owns four consecutive columns of one row of Z and walks the classes in ascending
// order (fp32), four classes' loads in flight at a time. biasT is the bias block transposed (C x ell, by k_bias_transpose), so
// that its reads are contiguous and shared by all rows. Needs ell a multiple of 4 and 16-byte aligned planes.
template <typename T>
__global__ void __launch_bounds__(256) k_outer_combine(const T* __restrict__ q, int64_t ldq, int C, const float* __restrict__ planes, int pp,
                                                       int64_t plane_stride, const float* __restrict__ biasT, int64_t total4, int ell,
                                                       float* __restrict__ Z) {
    const int64_t e4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e4 >= total4) return;
    const int ell4 = ell >> 2;
    const int64_t i = e4 / ell4;
    const int j = (int)(e4 - i * ell4) * 4;
    const T* qr = q + i * ldq;
    const float* t = planes + i * ell + j;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int cb = 0; cb < C; cb += 4) {
        float4 v[4];
        float qc[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = cb + u;
            qc[u] = c < C ? (float)qr[c] : 0.f;
            v[u] = c < C ? __ldg(reinterpret_cast<const float4*>(biasT + (int64_t)c * ell + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int p = 0; p < pp; ++p) {
            float4 w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                w[u] = cb + u < C ? __ldcs(reinterpret_cast<const float4*>(t + ((int64_t)(cb + u) * pp + p) * plane_stride))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 4; ++u) { v[u].x += w[u].x; v[u].y += w[u].y; v[u].z += w[u].z; v[u].w += w[u].w; }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            acc.x = fmaf(qc[u], v[u].x, acc.x);
            acc.y = fmaf(qc[u], v[u].y, acc.y);
            acc.z = fmaf(qc[u], v[u].z, acc.z);
            acc.w = fmaf(qc[u], v[u].w, acc.w);
        }
    }
    *reinterpret_cast<float4*>(Z + i * ell + j) = acc;
}

// biasT[c][j] = Sb[j][c] (Sb: ell rows of pitch lds)
__global__ void __launch_bounds__(256) k_bias_transpose(const float* __restrict__ Sb, int64_t lds, int C, int ell, float* __restrict__ biasT) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= C * ell) return;
    const int j = x / C, c = x - j * C;
    biasT[(int64_t)c * ell + j] = Sb[(int64_t)j * lds + c];
}

// any ell: one thread per element
template <typename T>
__global__ void __launch_bounds__(256) k_outer_combine_scalar(const T* __restrict__ q, int64_t ldq, int C, const float* __restrict__ planes,
                                                              int pp, int64_t plane_stride, const float* __restrict__ biasT,
                                                              int64_t total, int ell, float* __restrict__ Z) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const int64_t i = e / ell;
    const int j = (int)(e - i * ell);
    const T* qr = q + i * ldq;
    const float* t = planes + e;
    float acc = 0.f;
    for (int c = 0; c < C; ++c) {
        float v = __ldg(biasT + (int64_t)c * ell + j);
        for (int p = 0; p < pp; ++p) v += t[((int64_t)c * pp + p) * plane_stride];
        acc = fmaf((float)qr[c], v, acc);
    }
    Z[e] = acc;
}

}  // namespace

cudaError_t launch_normalise(const float* Z, int planes, int64_t plane_stride, int64_t ldz, int64_t n, int ell, float* zhat,
                             float* znorm, float* partials, double* zsum, unsigned* flags, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const int nblocks = (int)((n + kRowsPerBlock - 1) / kRowsPerBlock);
    k_normalise<<<nblocks, 256, 0, st>>>(Z, planes, plane_stride, ldz, n, ell, zhat, znorm, partials, flags);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || !zsum) return e;
    int jw = 32;
    while (jw < ell) jw <<= 1;
    k_accumulate<<<1, 1024, 0, st>>>(partials, nblocks, ell, jw, zsum);
    return cudaGetLastError();
}

cudaError_t launch_outer_combine(const void* q, int64_t ldq, sage_dtype_t dt, int C, const float* planes, int pp, int64_t plane_stride,
                                 const float* Sb, int64_t lds, float* biasT, int64_t n, int ell, float* Z, cudaStream_t st) {
    const int64_t total = n * ell;
    if (total <= 0 || C <= 0) return cudaSuccess;
    k_bias_transpose<<<(unsigned)(((int64_t)C * ell + 255) / 256), 256, 0, st>>>(Sb, lds, C, ell, biasT);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const bool vec = ell % 4 == 0 && plane_stride % 4 == 0 && (reinterpret_cast<uintptr_t>(planes) & 15u) == 0 &&
                     (reinterpret_cast<uintptr_t>(Z) & 15u) == 0 && (reinterpret_cast<uintptr_t>(biasT) & 15u) == 0;
    if (vec) {
        const int64_t total4 = total / 4;
        const unsigned blocks = (unsigned)((total4 + 255) / 256);
        if (dt == SAGE_F32)
            k_outer_combine<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(q), ldq, C, planes, pp, plane_stride, biasT, total4, ell, Z);
        else
            k_outer_combine<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(q), ldq, C, planes, pp, plane_stride,
                                                                   biasT, total4, ell, Z);
        return cudaGetLastError();
    }
    const unsigned blocks = (unsigned)((total + 255) / 256);
    if (dt == SAGE_F32)
        k_outer_combine_scalar<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(q), ldq, C, planes, pp, plane_stride, biasT, total, ell, Z);
    else
        k_outer_combine_scalar<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(q), ldq, C, planes, pp, plane_stride,
                                                                      biasT, total, ell, Z);
    return cudaGetLastError();
}

cudaError_t launch_consensus_score(const double* zsum, const float* zhat, int64_t N, int ell, float* u, float* scores,
                                   cudaStream_t st) {
    const int64_t blocks = N > 0 ? (N + 7) / 8 : 1;
    k_consensus_score<<<(unsigned)blocks, 256, 0, st>>>(zsum, zhat, N, ell, u, scores);
    return cudaGetLastError();
}

}  // namespace sage

// Class-balanced variant (Algorithm 1, the class-balanced branch; section on agreement scoring and selection):
// per-class unit centroids u_c of the stored normalised projections, scores <zhat_i, u_c(i)>, and the top-k_c
// examples of every class. All reductions run in a fixed order (ascending example index), so results are
// reproducible bit for bit.
#include "sage_internal.h"

namespace sage {
namespace {

// Block c: sum over the examples of class c of zhat (fp64, ascending index), its unit vector, the class size.
// The mean's 1/|I_c| cancels in the unit vector. Thread j owns component j (ell <= 256).
__global__ void __launch_bounds__(256) k_class_centroids(const float* __restrict__ zhat, const int* __restrict__ labels,
                                                         int64_t N, int ell, float* __restrict__ U, int* __restrict__ counts) {
    __shared__ int sl[256];
    __shared__ double red[8];
    const int c = blockIdx.x, j = threadIdx.x;
    double acc = 0.0;
    int cnt = 0;
    for (int64_t base = 0; base < N; base += 256) {
        sl[j] = (base + j < N) ? labels[base + j] : -1;
        __syncthreads();
        const int m = (int)((N - base < 256) ? N - base : 256);
        for (int t = 0; t < m; ++t) {
            if (sl[t] == c) {                                   // same decision in every thread
                if (j < ell) acc += (double)zhat[(base + t) * ell + j];
                ++cnt;
            }
        }
        __syncthreads();
    }
    double sq = (j < ell) ? acc * acc : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if ((j & 31) == 0) red[j >> 5] = sq;
    __syncthreads();
    double tot = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    if (j < ell) U[(int64_t)c * ell + j] = tot > 0.0 ? (float)(acc / sqrt(tot)) : 0.f;
    if (j == 0) counts[c] = cnt;
}

// One warp per example: score = <zhat_i, u_label(i)>; examples without a class in [0, C) score 0.
__global__ void __launch_bounds__(256) k_class_scores(const float* __restrict__ zhat, const int* __restrict__ labels, int64_t N,
                                                      int ell, int C, const float* __restrict__ U, float* __restrict__ scores) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= N) return;
    const int lab = labels[row];
    float acc = 0.f;
    if (lab >= 0 && lab < C)
        for (int j = lane; j < ell; j += 32) acc = fmaf(zhat[row * ell + j], U[(int64_t)lab * ell + j], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) scores[row] = fminf(1.f, fmaxf(-1.f, acc));
}

__global__ void __launch_bounds__(256) k_class_count(const int* __restrict__ labels, int64_t N, int C, int* __restrict__ counts) {
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= N) return;
    const int lab = labels[i];
    if (lab >= 0 && lab < C) atomicAdd(&counts[lab], 1);       // integer counts: the result does not depend on order
}

// Block c walks the globally sorted examples (score descending, index ascending) and keeps the first kc[c] of its class.
__global__ void __launch_bounds__(256) k_class_pick(const int64_t* __restrict__ sorted, const int* __restrict__ labels, int64_t N,
                                                    const long long* __restrict__ kc, const long long* __restrict__ offs,
                                                    int64_t* __restrict__ out) {
    __shared__ int wsum[8];
    const int c = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long want = kc[c];
    long long got = 0;
    for (int64_t base = 0; base < N && got < want; base += 256) {
        const int64_t i = base + tid;
        int64_t ex = -1;
        bool flag = false;
        if (i < N) {
            ex = sorted[i];
            flag = labels[ex] == c;
        }
        const unsigned b = __ballot_sync(0xffffffffu, flag);
        if (lane == 0) wsum[warp] = __popc(b);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            if (w < warp) before += wsum[w];
            total += wsum[w];
        }
        const long long rank = got + before + __popc(b & ((1u << lane) - 1u));
        if (flag && rank < want) out[offs[c] + rank] = ex;
        got += total;
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_class_scores(const float* zhat, const int* labels, int64_t N, int ell, int C, float* U, int* counts, float* scores,
                                cudaStream_t st) {
    if (C <= 0) return cudaSuccess;
    k_class_centroids<<<C, 256, 0, st>>>(zhat, labels, N, ell, U, counts);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || N <= 0) return e;
    k_class_scores<<<(unsigned)((N + 7) / 8), 256, 0, st>>>(zhat, labels, N, ell, C, U, scores);
    return cudaGetLastError();
}

cudaError_t launch_class_count(const int* labels, int64_t N, int C, int* counts, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(counts, 0, (size_t)C * sizeof(int), st);
    if (e != cudaSuccess || N <= 0) return e;
    k_class_count<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(labels, N, C, counts);
    return cudaGetLastError();
}

cudaError_t launch_class_pick(const int64_t* sorted, const int* labels, int64_t N, int C, const long long* kc, const long long* offs,
                              int64_t* out, cudaStream_t st) {
    if (C <= 0 || N <= 0) return cudaSuccess;
    k_class_pick<<<C, 256, 0, st>>>(sorted, labels, N, kc, offs, out);
    return cudaGetLastError();
}

}  // namespace sage

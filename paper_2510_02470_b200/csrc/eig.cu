// Eigen-decomposition of the buffer's Gram matrix and the Frequent-Directions shrink factors
// (Method, first paragraph: "compute a thin SVD S = U Sigma V^T, set delta = sigma_ell^2, shrink
// Sigma'_jj = sqrt(max(sigma_j^2 - delta, 0))"). With K = B B^T = U Sigma^2 U^T the left factor U and
// sigma^2 come from the symmetric eigen-problem of K, and Sigma' V^T = diag(sigma'/sigma) U^T B.
//
// Method: implicit (one-sided) cyclic Jacobi on a Cholesky factor. K is factored with diagonal
// pivoting, P^T K P = L L^T (stopping at the numerical rank), then plane rotations are applied to
// column pairs of L from the right until all columns are mutually orthogonal: L V = U Sigma. The
// columns of the result are sigma_j u_j, so U needs no separate accumulation and small eigenvalues
// keep their relative accuracy. One thread block does the whole solve; the matrix lives in shared
// memory when it fits (n <= 232) and in global scratch (L2-resident) otherwise. All loops are bounded;
// hitting the sweep limit sets a flag instead of spinning.
#include "sage_internal.h"

namespace sage {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

struct ArgMax {
    float v;
    int i;
};

__device__ __forceinline__ ArgMax better(ArgMax a, ArgMax b) {
    // larger value wins; ties (and NaN on the right) keep the smaller index
    if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
    return a;
}

// Round-robin pairing: n_even players, rounds 0..n_even-2, slots 0..n_even/2-1 give disjoint pairs.
__device__ __forceinline__ void rr_pair(int n_even, int round, int slot, int& p, int& q) {
    const int nm1 = n_even - 1;
    int a, b;
    if (slot == 0) {
        a = nm1;
        b = round % nm1;
    } else {
        a = (round + slot) % nm1;
        b = (round + nm1 - slot) % nm1;
    }
    p = min(a, b);
    q = max(a, b);
}

// ------------------------------------------------------------------------------------------------
// Shared-memory solver for n <= 192 (the common case: n = 2*ell <= 128, and partly filled buffers at
// the freeze). Same mathematics as k_eig_shrink below, restructured for latency:
//   * Cholesky with diagonal pivoting but WITHOUT data movement: the pivot column stays where it is,
//     a per-index pivot order replaces the row/column swaps, every warp keeps the running diagonal in
//     registers and finds the pivot redundantly, so a step costs one block barrier;
//   * one-sided Jacobi with one pair per HALF-warp: 16 lanes hold both columns in registers (float4
//     accesses, conflict-free), reduce the three dot products with 4 shuffle steps and rotate;
//   * a sweep whose largest pre-rotation cosine is below 3e-4 ends the iteration (the next sweep
//     would find cosines near 1e-7, below the rotation threshold).
// X is column-major with a row pitch of LD = 64*T floats; column c of the factor stays at the physical
// position of the c-th pivot, so the rows of U come out in the original buffer order.
// ------------------------------------------------------------------------------------------------
constexpr int kHalfWarps = kThreads / 16;
constexpr int kMaxFast = 192;

template <int T>
__global__ void __launch_bounds__(kThreads, 1)
k_eig_shrink_fast(const float* __restrict__ K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* __restrict__ Ur,
                  int ldu, float* __restrict__ sigma_out, int n_sigma, int max_sweeps, EigInfo* __restrict__ info) {
    constexpr int LD = 64 * T;
    constexpr int R = 2 * T;            // rows per lane when a warp spans a column (32 lanes)
    extern __shared__ __align__(16) float smem[];
    float* X = smem;                                    // LD x LD
    float* lam = X + LD * LD;                           // kMaxFast each from here on
    float* fac = lam + kMaxFast;
    float* scl = fac + kMaxFast;
    int* ord = reinterpret_cast<int*>(scl + kMaxFast);  // physical index -> pivot step (-1: never pivoted)
    int* perm = ord + kMaxFast;                         // pivot step -> physical index
    int* order = perm + kMaxFast;                       // sorted position -> pivot step
    float* sh_f = reinterpret_cast<float*>(order + kMaxFast);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int e = tid; e < n * LD; e += kThreads) {
        const int c = e / LD, i = e - c * LD;
        X[e] = (i < n) ? K[(size_t)c * ldk + i] : 0.f;  // K is symmetric: row c serves as column c
    }
    if (tid < kMaxFast) ord[tid] = -1;
    // running diagonal and liveness of the rows this lane owns (rows lane + 32 t), one copy per warp
    float dg[R];
    bool alive[R];
    bool bad = false;
#pragma unroll
    for (int t = 0; t < R; ++t) {
        const int i = lane + 32 * t;
        dg[t] = (i < n) ? K[(size_t)i * ldk + i] : -1.f;
        alive[t] = i < n;
        if (alive[t] && !(fabsf(dg[t]) <= 3.0e38f)) { bad = true; alive[t] = false; }
    }
    if (warp == 0 && bad) atomicOr(&info->flags, kFlagNonFinite);
    __syncthreads();

    // ---- pivoted Cholesky without swaps ----
    float tol = 0.f;
    int rank = n;
    for (int k = 0; k < n; ++k) {
        ArgMax am{-1.f, 0x7fffffff};
#pragma unroll
        for (int t = 0; t < R; ++t)
            if (alive[t]) am = better(am, ArgMax{dg[t], lane + 32 * t});
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ArgMax other{__shfl_xor_sync(0xffffffffu, am.v, o), __shfl_xor_sync(0xffffffffu, am.i, o)};
            am = better(am, other);
        }
        const float d = am.v;
        const int p = am.i;
        if (k == 0) tol = fmaxf(d * 1e-7f, 1e-37f);
        if (!(d > tol) || p >= n) { rank = k; break; }            // identical in every warp
        const float inv = 1.f / sqrtf(d);
        const float* Xp = X + p * LD;
        float li[R];
#pragma unroll
        for (int t = 0; t < R; ++t) {
            const int i = lane + 32 * t;
            if (i == p) alive[t] = false;
            li[t] = alive[t] ? Xp[i] * inv : 0.f;
            dg[t] = fmaf(-li[t], li[t], dg[t]);
        }
        for (int j = warp; j < n; j += kWarps) {
            if (j == p) continue;
            if (ord[j] >= 0) continue;                            // ord[p] is written below but never read here
            const float lj = Xp[j] * inv;
            float* col = X + j * LD;
#pragma unroll
            for (int t = 0; t < R; ++t) {
                const int i = lane + 32 * t;
                col[i] = fmaf(-li[t], lj, col[i]);
            }
        }
        if (tid == 0) { ord[p] = k; perm[k] = p; scl[k] = inv; }
        __syncthreads();
    }
    __syncthreads();
    // ---- scale the pivot columns into the factor L (zero above the pivot order, zero unpivoted columns) ----
    for (int e = tid; e < n * LD; e += kThreads) {
        const int c = e / LD, i = e - c * LD;
        const int kc = ord[c];
        float v = 0.f;
        if (kc >= 0 && i < n) {
            const int ki = ord[i];
            if (!(ki >= 0 && ki < kc)) v = X[e] * scl[kc];
        }
        X[e] = v;
    }
    __syncthreads();

    // ---- one-sided cyclic Jacobi on the rank pivot columns, one pair per half-warp ----
    const int hw = tid >> 4, l16 = tid & 15;
    const float jtol = 1e-6f;
    int sweeps = 0;
    float worst = 0.f;
    if (rank >= 2) {
        const int ne = rank + (rank & 1), nm1 = ne - 1, half = ne >> 1;
        for (; sweeps < max_sweeps;) {
            int rotated = 0;
            worst = 0.f;
            for (int round = 0; round < nm1; ++round) {
                for (int base = 0; base < half; base += kHalfWarps) {
                    const int slot = base + hw;
                    int p = 0, q = ne;
                    if (slot < half) {
                        int a, b;
                        if (slot == 0) { a = nm1; b = round; }
                        else {
                            a = round + slot; if (a >= nm1) a -= nm1;
                            b = round + nm1 - slot; if (b >= nm1) b -= nm1;
                        }
                        p = min(a, b); q = max(a, b);
                    }
                    const bool valid = q < rank;
                    float4* xp = reinterpret_cast<float4*>(X + (valid ? perm[p] : 0) * LD) + l16;
                    float4* xq = reinterpret_cast<float4*>(X + (valid ? perm[q] : 0) * LD) + l16;
                    float4 x[T], y[T];
                    float a = 0.f, b = 0.f, g = 0.f;
#pragma unroll
                    for (int t = 0; t < T; ++t) {
                        x[t] = xp[16 * t];
                        y[t] = xq[16 * t];
                        a = fmaf(x[t].x, x[t].x, a); a = fmaf(x[t].y, x[t].y, a); a = fmaf(x[t].z, x[t].z, a); a = fmaf(x[t].w, x[t].w, a);
                        b = fmaf(y[t].x, y[t].x, b); b = fmaf(y[t].y, y[t].y, b); b = fmaf(y[t].z, y[t].z, b); b = fmaf(y[t].w, y[t].w, b);
                        g = fmaf(x[t].x, y[t].x, g); g = fmaf(x[t].y, y[t].y, g); g = fmaf(x[t].z, y[t].z, g); g = fmaf(x[t].w, y[t].w, g);
                    }
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) {
                        a += __shfl_xor_sync(0xffffffffu, a, o);
                        b += __shfl_xor_sync(0xffffffffu, b, o);
                        g += __shfl_xor_sync(0xffffffffu, g, o);
                    }
                    const float lim = sqrtf(a) * sqrtf(b);
                    const float ag = fabsf(g);
                    if (valid && lim > 0.f && ag > jtol * lim) {
                        worst = fmaxf(worst, ag / lim);
                        const float zeta = (b - a) / (2.f * g);
                        const float tt = copysignf(1.f, zeta) / (fabsf(zeta) + sqrtf(fmaf(zeta, zeta, 1.f)));
                        const float c = rsqrtf(fmaf(tt, tt, 1.f));
                        const float s = c * tt;
#pragma unroll
                        for (int t = 0; t < T; ++t) {
                            float4 nx, ny;
                            nx.x = c * x[t].x - s * y[t].x; ny.x = fmaf(s, x[t].x, c * y[t].x);
                            nx.y = c * x[t].y - s * y[t].y; ny.y = fmaf(s, x[t].y, c * y[t].y);
                            nx.z = c * x[t].z - s * y[t].z; ny.z = fmaf(s, x[t].z, c * y[t].z);
                            nx.w = c * x[t].w - s * y[t].w; ny.w = fmaf(s, x[t].w, c * y[t].w);
                            xp[16 * t] = nx;
                            xq[16 * t] = ny;
                        }
                        rotated = 1;
                    }
                }
                __syncthreads();
            }
            ++sweeps;
            (void)rotated;
            if (!__syncthreads_or(worst > 3e-4f)) break;   // every cosine of this sweep was small: converged after it
        }
    }
    const int not_converged = __syncthreads_or(sweeps >= max_sweeps && worst > 1e-4f);

    // ---- eigenvalues = squared column norms (pivot-step order); sort descending, stable ----
    for (int k = warp; k < n; k += kWarps) {
        float a = 0.f;
        if (k < rank) {
            const float* x = X + perm[k] * LD;
#pragma unroll
            for (int t = 0; t < R; ++t) a = fmaf(x[lane + 32 * t], x[lane + 32 * t], a);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        }
        if (lane == 0) lam[k] = a;
    }
    __syncthreads();
    if (tid < n) {
        const float mine = lam[tid];
        int pos = 0;
        for (int i = 0; i < n; ++i) {
            const float o = lam[i];
            pos += (o > mine) || (o == mine && i < tid);
        }
        order[pos] = tid;
    }
    __syncthreads();
    if (tid == 0) {
        float delta = 0.f;
        if (do_shrink && delta_rank - 1 < n) delta = lam[order[delta_rank - 1]];
        sh_f[0] = delta;
        info->delta = delta;
        info->sweeps = sweeps;
        if (sweeps > info->max_sweeps) info->max_sweeps = sweeps;
        info->rank = rank;
        if (not_converged) info->flags |= kFlagNotConverged;
        if (do_shrink) {
            info->sum_delta += (double)delta;
            info->shrinks += 1;
        }
    }
    __syncthreads();
    const float delta = sh_f[0];
    if (tid < n) {
        const float l = lam[order[tid]];
        float f = 0.f, sp = 0.f;
        if (l > 0.f && tid < keep) {
            const float kept = fmaxf(l - delta, 0.f);
            sp = sqrtf(kept);
            f = sqrtf(kept / l) * rsqrtf(l);
        }
        fac[tid] = f;
        if (tid < n_sigma) sigma_out[tid] = sp;
    }
    for (int j = n + tid; j < n_sigma; j += kThreads) sigma_out[j] = 0.f;
    __syncthreads();
    for (int e = tid; e < n * keep; e += kThreads) {
        const int j = e / n, i = e - j * n;
        float v = 0.f;
        if (j < n) {
            const int k = order[j];
            if (k < rank) v = X[perm[k] * LD + i] * fac[j];
        }
        Ur[(size_t)i * ldu + j] = v;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
k_eig_shrink(const float* __restrict__ K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* __restrict__ Ur,
             int ldu, float* __restrict__ sigma_out, int n_sigma, float* __restrict__ work, int use_smem, int max_sweeps,
             EigInfo* __restrict__ info) {
    extern __shared__ __align__(16) float smem[];
    float* lam = smem;                 // n   eigenvalues (unsorted), later reused
    float* fac = lam + 512;            // n   per sorted position: r_j / sigma_j
    int* perm = reinterpret_cast<int*>(fac + 512);   // n   physical row -> original buffer row
    int* order = perm + 512;           // n   sorted position -> column
    float* red_v = reinterpret_cast<float*>(order + 512);   // kWarps
    int* red_i = reinterpret_cast<int*>(red_v + kWarps);    // kWarps
    int* sh_int = red_i + kWarps;      // [0] pivot index, [1] rank
    float* sh_f = reinterpret_cast<float*>(sh_int + 4);     // [0] pivot value, [1] delta
    float* X = use_smem ? (sh_f + 4) : work;
    const int ldx = n;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- load K (full symmetric storage, column-major X[c*ldx + i] = K[i][c]) ----
    for (int e = tid; e < n * n; e += kThreads) {
        const int i = e / n, c = e % n;
        X[(size_t)c * ldx + i] = K[(size_t)i * ldk + c];
    }
    if (tid < n) perm[tid] = tid;
    if (tid == 0) sh_int[1] = n;
    __syncthreads();

    // ---- pivoted Cholesky, right-looking, in place ----
    float tol = 0.f;
    int rank = n;
    for (int k = 0; k < n; ++k) {
        ArgMax am{-1.f, 0x7fffffff};
        if (tid >= k && tid < n) {
            const float d = X[(size_t)tid * ldx + tid];
            if (fabsf(d) <= 3.0e38f) am = ArgMax{d, tid};
            else if (k == 0) atomicOr(&info->flags, kFlagNonFinite);    // NaN/Inf rows reached the buffer
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ArgMax other{__shfl_xor_sync(0xffffffffu, am.v, o), __shfl_xor_sync(0xffffffffu, am.i, o)};
            am = better(am, other);
        }
        if (lane == 0) { red_v[warp] = am.v; red_i[warp] = am.i; }
        __syncthreads();
        if (warp == 0) {
            ArgMax a{red_v[lane], red_i[lane]};
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                ArgMax other{__shfl_xor_sync(0xffffffffu, a.v, o), __shfl_xor_sync(0xffffffffu, a.i, o)};
                a = better(a, other);
            }
            if (lane == 0) { sh_f[0] = a.v; sh_int[0] = a.i; }
        }
        __syncthreads();
        const float d = sh_f[0];
        const int p = sh_int[0];
        if (k == 0) tol = fmaxf(d * 1e-7f, 1e-37f);
        if (!(d > tol) || p >= n) { rank = k; break; }     // uniform across the block
        if (p != k) {
            // swap rows k and p in every column, then columns k and p for rows >= k
            for (int c = tid; c < n; c += kThreads) {
                const float a = X[(size_t)c * ldx + k], b = X[(size_t)c * ldx + p];
                X[(size_t)c * ldx + k] = b;
                X[(size_t)c * ldx + p] = a;
            }
            __syncthreads();
            for (int i = k + tid; i < n; i += kThreads) {
                const float a = X[(size_t)k * ldx + i], b = X[(size_t)p * ldx + i];
                X[(size_t)k * ldx + i] = b;
                X[(size_t)p * ldx + i] = a;
            }
            if (tid == 0) { const int t = perm[k]; perm[k] = perm[p]; perm[p] = t; }
            __syncthreads();
        }
        const float lkk = sqrtf(d), inv = 1.f / lkk;
        for (int i = tid; i < n; i += kThreads) {
            float v = X[(size_t)k * ldx + i];
            v = (i < k) ? 0.f : (i == k ? lkk : v * inv);
            X[(size_t)k * ldx + i] = v;
        }
        __syncthreads();
        {   // trailing update S[i][j] -= L[i][k] L[j][k], rows along lanes
            const float* Lk = X + (size_t)k * ldx;
            for (int j = k + 1 + warp; j < n; j += kWarps) {
                const float lj = Lk[j];
                float* col = X + (size_t)j * ldx;
                for (int i = k + 1 + lane; i < n; i += 32) col[i] = fmaf(-Lk[i], lj, col[i]);
            }
        }
        __syncthreads();
    }
    // columns >= rank do not take part; zero them so that later norms are exact zeros
    for (int e = tid; e < (n - rank) * n; e += kThreads) X[(size_t)rank * ldx + e] = 0.f;
    __syncthreads();

    // ---- one-sided cyclic Jacobi on columns 0..rank-1 ----
    const float jtol = 1e-6f;
    int sweeps = 0;
    float worst = 0.f;
    if (rank >= 2) {
        const int ne = rank + (rank & 1);
        for (; sweeps < max_sweeps; ++sweeps) {
            int rotated = 0;
            worst = 0.f;
            for (int round = 0; round < ne - 1; ++round) {
                for (int slot = warp; slot < ne / 2; slot += kWarps) {
                    int p, q;
                    rr_pair(ne, round, slot, p, q);
                    if (q >= rank) continue;
                    float* xp = X + (size_t)p * ldx;
                    float* xq = X + (size_t)q * ldx;
                    float a = 0.f, b = 0.f, g = 0.f;
                    for (int i = lane; i < n; i += 32) {
                        const float x = xp[i], y = xq[i];
                        a = fmaf(x, x, a);
                        b = fmaf(y, y, b);
                        g = fmaf(x, y, g);
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        a += __shfl_xor_sync(0xffffffffu, a, o);
                        b += __shfl_xor_sync(0xffffffffu, b, o);
                        g += __shfl_xor_sync(0xffffffffu, g, o);
                    }
                    const float lim = sqrtf(a) * sqrtf(b);
                    const float ag = fabsf(g);
                    if (!(lim > 0.f) || !(ag > jtol * lim)) continue;
                    worst = fmaxf(worst, ag / lim);
                    const float zeta = (b - a) / (2.f * g);
                    const float t = copysignf(1.f, zeta) / (fabsf(zeta) + sqrtf(fmaf(zeta, zeta, 1.f)));
                    const float c = rsqrtf(fmaf(t, t, 1.f));
                    const float s = c * t;
                    for (int i = lane; i < n; i += 32) {
                        const float x = xp[i], y = xq[i];
                        xp[i] = c * x - s * y;
                        xq[i] = fmaf(s, x, c * y);
                    }
                    rotated = 1;
                }
                __syncthreads();
            }
            if (!__syncthreads_or(rotated)) break;
        }
    }
    // a run that stopped at the sweep limit while still rotating by a visible amount did not converge
    const int not_converged = __syncthreads_or(sweeps >= max_sweeps && worst > 1e-4f);

    // ---- eigenvalues = squared column norms; sort descending (stable by column index) ----
    for (int c = warp; c < n; c += kWarps) {
        float a = 0.f;
        if (c < rank) {
            const float* x = X + (size_t)c * ldx;
            for (int i = lane; i < n; i += 32) a = fmaf(x[i], x[i], a);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        }
        if (lane == 0) lam[c] = a;
    }
    __syncthreads();
    if (tid < n) {
        const float mine = lam[tid];
        int pos = 0;
        for (int i = 0; i < n; ++i) {
            const float o = lam[i];
            pos += (o > mine) || (o == mine && i < tid);
        }
        order[pos] = tid;
    }
    __syncthreads();
    if (tid == 0) {
        float delta = 0.f;
        if (do_shrink && delta_rank - 1 < n) delta = lam[order[delta_rank - 1]];
        sh_f[1] = delta;
        info->delta = delta;
        info->sweeps = sweeps;
        if (sweeps > info->max_sweeps) info->max_sweeps = sweeps;
        info->rank = rank;
        if (not_converged) info->flags |= kFlagNotConverged;
        if (do_shrink) {
            info->sum_delta += (double)delta;
            info->shrinks += 1;
        }
    }
    __syncthreads();
    const float delta = sh_f[1];
    if (tid < n) {
        const float l = lam[order[tid]];
        float f = 0.f, sp = 0.f;
        if (l > 0.f && tid < keep) {
            const float kept = fmaxf(l - delta, 0.f);
            sp = sqrtf(kept);
            f = sqrtf(kept / l) * rsqrtf(l);       // (sigma'/sigma) / sigma : scales the column sigma_j u_j
        }
        fac[tid] = f;
        if (tid < n_sigma) sigma_out[tid] = sp;
    }
    for (int j = n + tid; j < n_sigma; j += kThreads) sigma_out[j] = 0.f;
    __syncthreads();

    // ---- Ur[orig_row][j] = u_j[orig_row] * sigma'_j / sigma_j ----
    for (int e = tid; e < n * keep; e += kThreads) {
        const int j = e / n, i = e % n;      // i fastest: conflict-free reads of X
        float v = 0.f;
        if (j < n) v = X[(size_t)order[j] * ldx + i] * fac[j];
        Ur[(size_t)perm[i] * ldu + j] = v;
    }
}

}  // namespace

cudaError_t launch_eig_shrink(const float* K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* Ur, int ldu,
                              float* sigma_out, int n_sigma, float* work, int max_sweeps, EigInfo* info, cudaStream_t st) {
    if (n <= 0 || n > 512) return cudaErrorInvalidValue;
    if (n <= kMaxFast) {
        const int T = (n + 63) / 64;
        const size_t bytes = ((size_t)(64 * T) * (64 * T) + 3 * kMaxFast) * sizeof(float) + 3 * kMaxFast * sizeof(int) + 16;
        cudaError_t e;
#define SAGE_EIG_FAST(TT)                                                                                              \
    e = cudaFuncSetAttribute(k_eig_shrink_fast<TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);          \
    if (e != cudaSuccess) return e;                                                                                    \
    k_eig_shrink_fast<TT><<<1, kThreads, bytes, st>>>(K, ldk, n, do_shrink, delta_rank, keep, Ur, ldu, sigma_out, n_sigma, \
                                                      max_sweeps, info);
        if (T == 1) { SAGE_EIG_FAST(1) } else if (T == 2) { SAGE_EIG_FAST(2) } else { SAGE_EIG_FAST(3) }
#undef SAGE_EIG_FAST
        return cudaGetLastError();
    }
    const size_t aux = (4 * 512 + 2 * kWarps + 8) * sizeof(float);
    const size_t xbytes = (size_t)n * n * sizeof(float);
    static int max_optin = -1;
    if (max_optin < 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    }
    const int use_smem = (aux + xbytes + 64 <= (size_t)max_optin) ? 1 : 0;
    const size_t smem = aux + (use_smem ? xbytes : 0) + 64;
    cudaError_t e = cudaFuncSetAttribute(k_eig_shrink, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_eig_shrink<<<1, kThreads, smem, st>>>(K, ldk, n, do_shrink, delta_rank, keep, Ur, ldu, sigma_out, n_sigma, work, use_smem,
                                            max_sweeps, info);
    return cudaGetLastError();
}

}  // namespace sage

// Eigen-decomposition of the buffer's Gram matrix and the Frequent-Directions shrink factors (Method, first
// paragraph: the buffer's thin SVD is taken, delta is the squared ell-th singular value, and every squared singular
// value is reduced by delta and clamped at zero). With K = B B^T = U Sigma^2 U^T the left factor U and sigma^2 come
// from the symmetric eigen-problem of K, and Sigma' V^T = diag(sigma'/sigma) U^T B.
//
// Method: implicit (one-sided) cyclic Jacobi on a Cholesky factor. K is factored with diagonal pivoting,
// P^T K P = L L^T (stopping at the numerical rank), then plane rotations are applied to column pairs of L from the
// right until all columns are mutually orthogonal: L V = U Sigma. The columns of the result are sigma_j u_j, so U
// needs no separate accumulation and small eigenvalues keep their relative accuracy. Three kernel families follow:
// one thread block with the factor in shared memory (buffers of up to 192 rows), a cluster of 8 thread blocks with
// the factor in L2, and a cluster of 8 with Cholesky and Jacobi columns in distributed shared memory (the default
// above 64 rows). All loops and waits are bounded; hitting the sweep limit sets a flag instead of spinning.
#include <cooperative_groups.h>

#include "sage_internal.h"

namespace sage {
namespace {

namespace cg = cooperative_groups;

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

// Row of the split rebuild factors [W_hi ; W_lo] that holds output row j: stacked as two blocks of j_pad rows, or, when
// more than 128 output rows are kept, as one such pair per 128 output rows (the rebuild kernel takes 128 at a time).
__device__ __forceinline__ size_t wsplit_row(int j, int j_pad, bool lo) {
    if (j_pad <= 128) return (size_t)(lo ? j_pad + j : j);
    return (size_t)(j >> 7) * 256 + (size_t)(j & 127) + (lo ? 128 : 0);
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

// Rotation that orthogonalises two columns with squared norms a, b and inner product g:
// tan 2theta = 2g / (b - a), cos 2theta = |b - a| / r, c = sqrt((1 + cos 2theta) / 2), s = sin 2theta / (2c), from two
// approximate reciprocal square roots, followed by one Newton step towards c^2 + s^2 = 1 taken from the residual
// itself: scaling by 1.5 - 0.5 (c^2 + s^2) would be lost to the coarser float grid above 1 whenever c^2 + s^2 < 1,
// a one-sided correction that shrinks every column a little at every rotation (measured 1e-5 relative on the
// singular values after a few thousand rotations; with the residual form they agree with fp64 to 1e-7).
__device__ __forceinline__ void jacobi_rotation(float a, float b, float g, float& c, float& s) {
    const float tau = b - a, gam = 2.f * g;
    const float inv_r = rsqrtf(fmaf(tau, tau, gam * gam));
    const float c2 = fmaf(0.5f * fabsf(tau), inv_r, 0.5f);
    const float invc = rsqrtf(c2);
    c = c2 * invc;
    s = copysignf(0.5f, tau) * gam * inv_r * invc;
    const float half_res = 0.5f * fmaf(-s, s, fmaf(-c, c, 1.f));
    c = fmaf(c, half_res, c);
    s = fmaf(s, half_res, s);
}

// ------------------------------------------------------------------------------------------------
// Shared-memory solver for n <= 192 (the common case: n = 2*ell <= 128, and partly filled buffers at
// the freeze). Same mathematics as k_eig_shrink below, restructured for instruction count and latency:
//   * K is scaled by 1/max(diag) on load, so every intermediate is O(1) and fast reciprocal / rsqrt
//     intrinsics are safe; eigenvalues are scaled back at the end;
//   * Cholesky with diagonal pivoting but WITHOUT data movement: the pivot column stays where it is and
//     a per-index pivot order replaces the row/column swaps; every warp keeps the running diagonal in
//     registers and finds the pivot redundantly with one warp-wide integer max, so a step costs one
//     block barrier;
//   * one-sided Jacobi with one pair per QUARTER-warp: 8 lanes hold both columns in registers (float4
//     accesses, conflict-free), reduce the three dot products with 3 shuffle steps and rotate; warps
//     without a pair only take part in the barrier;
//   * a sweep whose largest pre-rotation cosine is below 1e-3 ends the iteration (the next sweep
//     would find cosines near 1e-6, the rotation threshold).
// X is column-major with a row pitch of LD = 64*T floats; column c of the factor stays at the physical
// position of the c-th pivot, so the rows of U come out in the original buffer order.
// ------------------------------------------------------------------------------------------------
constexpr int kMaxFast = 192;      // largest n whose matrix fits in shared memory
constexpr int kMaxN = 256;         // largest n of this kernel (above kMaxFast the matrix stays in global memory, i.e. L2)

template <int T, int NT, bool G>
__global__ void __launch_bounds__(NT, 1)
k_eig_shrink_fast(const float* __restrict__ K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* __restrict__ Ur,
                  int ldu, float* __restrict__ sigma_out, int n_sigma, int max_sweeps, EigInfo* __restrict__ info,
                  float* __restrict__ Wsplit, int ldw, int j_pad, float* __restrict__ gwork) {
    constexpr int LD = 64 * T;
    constexpr int NW = NT / 32;
    constexpr int R = 2 * T;            // rows per lane when 32 lanes span a column
    constexpr int Q = 2 * T;            // float4 per lane when 8 lanes span a column
    extern __shared__ __align__(16) float smem[];
    float* X = G ? gwork : smem;                        // LD x LD (global scratch when it does not fit on chip)
    float* lam = G ? smem : smem + LD * LD;             // kMaxN each from here on
    float* fac = lam + kMaxN;
    float* scl = fac + kMaxN;
    int* ord = reinterpret_cast<int*>(scl + kMaxN);     // physical index -> pivot step (-1: never pivoted)
    int* perm = ord + kMaxN;                            // pivot step -> physical index
    int* order = perm + kMaxN;                          // sorted position -> pivot step
    float* sh_f = reinterpret_cast<float*>(order + kMaxN);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // running diagonal and liveness of the rows this lane owns (rows lane + 32 t), one copy per warp
    float dg[R];
    bool alive[R];
    bool bad = false;
    float dmax = 0.f;
#pragma unroll
    for (int t = 0; t < R; ++t) {
        const int i = lane + 32 * t;
        dg[t] = (i < n) ? K[(size_t)i * ldk + i] : -1.f;
        alive[t] = i < n;
        if (alive[t] && !(fabsf(dg[t]) <= 3.0e38f)) { bad = true; alive[t] = false; }
        if (alive[t]) dmax = fmaxf(dmax, dg[t]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
    if (warp == 0 && bad) atomicOr(&info->flags, kFlagNonFinite);
    const bool empty = !(dmax >= 1e-30f);              // nothing to factor: rank 0
    const float kscale = empty ? 0.f : 1.f / dmax;
    for (int e = tid; e < n * LD; e += NT) {
        const int c = e / LD, i = e - c * LD;
        X[e] = (i < n) ? K[(size_t)c * ldk + i] * kscale : 0.f;  // K is symmetric: row c serves as column c
    }
#pragma unroll
    for (int t = 0; t < R; ++t) dg[t] *= kscale;
    for (int i = tid; i < kMaxN; i += NT) ord[i] = -1;
    __syncthreads();

    // ---- pivoted Cholesky without swaps (scaled matrix: diagonal <= 1) ----
    constexpr int CW = (LD + NW - 1) / NW;                     // columns a warp owns: warp + NW u
    unsigned colmask = 0u;                                     // bit u: column warp + 32 u is still unpivoted
#pragma unroll
    for (int u = 0; u < CW; ++u)
        if (warp + NW * u < n) colmask |= 1u << u;
    const float tol = 1e-7f;
    int rank = empty ? 0 : n;
    for (int k = 0; k < rank; ++k) {
        unsigned key = 0u;
#pragma unroll
        for (int t = 0; t < R; ++t)
            if (alive[t]) key = max(key, (__float_as_uint(fmaxf(dg[t], 0.f)) & 0xffffff00u) | (unsigned)(255 - (lane + 32 * t)));
        key = __reduce_max_sync(0xffffffffu, key);                // largest diagonal (24 significant bits), smaller index on ties
        const int p = 255 - (int)(key & 255u);
        if (key == 0u || p >= n) { rank = k; break; }             // identical in every warp
        const float* Xp = X + p * LD;
        const float d = Xp[p];
        if (!(d > tol)) { rank = k; break; }
        const float inv = rsqrtf(d);
        if ((p & (NW - 1)) == warp) colmask &= ~(1u << (p / NW));
        float li[R];
#pragma unroll
        for (int t = 0; t < R; ++t) {
            const int i = lane + 32 * t;
            if (i == p) alive[t] = false;
            li[t] = alive[t] ? Xp[i] * inv : 0.f;
            dg[t] = fmaf(-li[t], li[t], dg[t]);
        }
#pragma unroll
        for (int u0 = 0; u0 < CW; u0 += 2) {                      // two columns at a time: loads first, then stores
            const bool on0 = (colmask >> u0) & 1u, on1 = (u0 + 1 < CW) && ((colmask >> (u0 + 1)) & 1u);
            if (!on0 && !on1) continue;
            float* c0 = X + (warp + NW * u0) * LD;
            float* c1 = X + (warp + NW * (u0 + 1)) * LD;
            const float l0 = on0 ? Xp[warp + NW * u0] * inv : 0.f;
            const float l1 = on1 ? Xp[warp + NW * (u0 + 1)] * inv : 0.f;
            float v0[R], v1[R];
#pragma unroll
            for (int t = 0; t < R; ++t) {
                v0[t] = on0 ? c0[lane + 32 * t] : 0.f;
                v1[t] = on1 ? c1[lane + 32 * t] : 0.f;
            }
#pragma unroll
            for (int t = 0; t < R; ++t) {
                if (on0) c0[lane + 32 * t] = fmaf(-li[t], l0, v0[t]);
                if (on1) c1[lane + 32 * t] = fmaf(-li[t], l1, v1[t]);
            }
        }
        if (tid == 0) { ord[p] = k; perm[k] = p; scl[k] = inv; }
        __syncthreads();
    }
    __syncthreads();
    // ---- scale the pivot columns into the factor L (zero above the pivot order, zero unpivoted columns) ----
    for (int e = tid; e < n * LD; e += NT) {
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

    // ---- one-sided cyclic Jacobi on the rank pivot columns ----
    // Columns (in pivot order) form blocks of 4. A block round pairs the blocks round-robin, one block
    // pair per warp; the warp rotates the 16 cross pairs of its two blocks in 4 local rounds (one pair per
    // quarter-warp, synchronised inside the warp only), and in the first block round of a sweep also the
    // pairs inside each block. Only the warps that own a block pair take part, on a named barrier.
    const int l8 = tid & 7, qd = lane >> 3;
    int sweeps = 0;
    float worst2 = 0.f;                 // largest squared cosine met in the current sweep
    int* sh_flag = reinterpret_cast<int*>(sh_f + 2);
    if (tid < 2) sh_flag[tid] = 0;
    __syncthreads();
    if (rank >= 2) {
        const int nb = (rank + 3) >> 2, nbe = nb + (nb & 1), nbm1 = nbe - 1, nact = nbe >> 1;   // block pairs per round
        const int nwork = nact < NW ? nact : NW;                  // warps that take part; each owns slots w, w + nwork, ...
        if (warp < nwork) {
            const int nthreads = nwork * 32;
            auto pair_step = [&](int p, int q) {                  // p, q: pivot-order columns, q >= rank means no pair
                const bool valid = p < rank && q < rank;
                float4* xp = reinterpret_cast<float4*>(X + (valid ? perm[p] : 0) * LD) + l8;
                float4* xq = reinterpret_cast<float4*>(X + (valid ? perm[q] : 0) * LD) + l8;
                float4 x[Q], y[Q];
                float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll
                for (int t = 0; t < Q; ++t) {
                    x[t] = xp[8 * t];
                    y[t] = xq[8 * t];
                    a0 = fmaf(x[t].x, x[t].x, a0); a1 = fmaf(x[t].y, x[t].y, a1); a0 = fmaf(x[t].z, x[t].z, a0); a1 = fmaf(x[t].w, x[t].w, a1);
                    b0 = fmaf(y[t].x, y[t].x, b0); b1 = fmaf(y[t].y, y[t].y, b1); b0 = fmaf(y[t].z, y[t].z, b0); b1 = fmaf(y[t].w, y[t].w, b1);
                    g0 = fmaf(x[t].x, y[t].x, g0); g1 = fmaf(x[t].y, y[t].y, g1); g0 = fmaf(x[t].z, y[t].z, g0); g1 = fmaf(x[t].w, y[t].w, g1);
                }
                float a = a0 + a1, b = b0 + b1, g = g0 + g1;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) {
                    a += __shfl_xor_sync(0xffffffffu, a, o);
                    b += __shfl_xor_sync(0xffffffffu, b, o);
                    g += __shfl_xor_sync(0xffffffffu, g, o);
                }
                const float ab = a * b, g2 = g * g;
                if (valid && ab > 0.f && g2 > 1e-12f * ab) {
                    worst2 = fmaxf(worst2, __fdividef(g2, ab));
                    float c, s;
                    jacobi_rotation(a, b, g, c, s);
#pragma unroll
                    for (int t = 0; t < Q; ++t) {
                        float4 nx, ny;
                        nx.x = fmaf(-s, y[t].x, c * x[t].x); ny.x = fmaf(s, x[t].x, c * y[t].x);
                        nx.y = fmaf(-s, y[t].y, c * x[t].y); ny.y = fmaf(s, x[t].y, c * y[t].y);
                        nx.z = fmaf(-s, y[t].z, c * x[t].z); ny.z = fmaf(s, x[t].z, c * y[t].z);
                        nx.w = fmaf(-s, y[t].w, c * x[t].w); ny.w = fmaf(s, x[t].w, c * y[t].w);
                        xp[8 * t] = nx;
                        xq[8 * t] = ny;
                    }
                }
                __syncwarp();
            };
            int more = 0;
            while (sweeps < max_sweeps) {
                worst2 = 0.f;
                for (int br = 0; br < nbm1; ++br) {
                  for (int slot = warp; slot < nact; slot += nwork) {
                    int ba, bb;                                   // the two blocks of this slot in this block round
                    if (slot == 0) { ba = nbm1; bb = br; }
                    else {
                        ba = br + slot; if (ba >= nbm1) ba -= nbm1;
                        bb = br + nbm1 - slot; if (bb >= nbm1) bb -= nbm1;
                    }
                    if (br == 0) {                                // pairs inside each block: quarters 0,1 -> ba, 2,3 -> bb
                        const int base = 4 * ((qd < 2) ? ba : bb), h = qd & 1;
                        pair_step(base + (h ? 2 : 0), base + (h ? 3 : 1));
                        pair_step(base + (h ? 1 : 0), base + (h ? 3 : 2));
                        pair_step(base + (h ? 1 : 0), base + (h ? 2 : 3));
                    }
                    const int lo = min(ba, bb), hi = max(ba, bb);
                    {   // the 16 cross pairs, columns held in registers: quarter qd keeps column qd of block lo and
                        // the columns of block hi travel from quarter to quarter by shuffles between the 4 rounds
                        const int pa = 4 * lo + qd, pb = 4 * hi + qd;
                        const bool va = pa < rank, vb0 = pb < rank;
                        float4* xa = reinterpret_cast<float4*>(X + (va ? perm[pa] : 0) * LD) + l8;
                        float4* xb = reinterpret_cast<float4*>(X + (vb0 ? perm[pb] : 0) * LD) + l8;
                        float4 x[Q], y[Q];
#pragma unroll
                        for (int t = 0; t < Q; ++t) {
                            x[t] = va ? xa[8 * t] : make_float4(0.f, 0.f, 0.f, 0.f);
                            y[t] = vb0 ? xb[8 * t] : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const bool valid = va && (4 * hi + ((qd + r) & 3) < rank);
                            float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll
                            for (int t = 0; t < Q; ++t) {
                                a0 = fmaf(x[t].x, x[t].x, a0); a1 = fmaf(x[t].y, x[t].y, a1); a0 = fmaf(x[t].z, x[t].z, a0); a1 = fmaf(x[t].w, x[t].w, a1);
                                b0 = fmaf(y[t].x, y[t].x, b0); b1 = fmaf(y[t].y, y[t].y, b1); b0 = fmaf(y[t].z, y[t].z, b0); b1 = fmaf(y[t].w, y[t].w, b1);
                                g0 = fmaf(x[t].x, y[t].x, g0); g1 = fmaf(x[t].y, y[t].y, g1); g0 = fmaf(x[t].z, y[t].z, g0); g1 = fmaf(x[t].w, y[t].w, g1);
                            }
                            float a = a0 + a1, b = b0 + b1, g = g0 + g1;
#pragma unroll
                            for (int o = 4; o > 0; o >>= 1) {
                                a += __shfl_xor_sync(0xffffffffu, a, o);
                                b += __shfl_xor_sync(0xffffffffu, b, o);
                                g += __shfl_xor_sync(0xffffffffu, g, o);
                            }
                            const float ab = a * b, g2 = g * g;
                            if (valid && ab > 0.f && g2 > 1e-12f * ab) {
                                worst2 = fmaxf(worst2, __fdividef(g2, ab));
                                float c, s;
                                jacobi_rotation(a, b, g, c, s);
#pragma unroll
                                for (int t = 0; t < Q; ++t) {
                                    float4 nx, ny;
                                    nx.x = fmaf(-s, y[t].x, c * x[t].x); ny.x = fmaf(s, x[t].x, c * y[t].x);
                                    nx.y = fmaf(-s, y[t].y, c * x[t].y); ny.y = fmaf(s, x[t].y, c * y[t].y);
                                    nx.z = fmaf(-s, y[t].z, c * x[t].z); ny.z = fmaf(s, x[t].z, c * y[t].z);
                                    nx.w = fmaf(-s, y[t].w, c * x[t].w); ny.w = fmaf(s, x[t].w, c * y[t].w);
                                    x[t] = nx;
                                    y[t] = ny;
                                }
                            }
                            if (r < 3) {                          // quarter qd takes over the column quarter qd + 1 holds
                                const int src = (lane + 8) & 31;
#pragma unroll
                                for (int t = 0; t < Q; ++t) {
                                    y[t].x = __shfl_sync(0xffffffffu, y[t].x, src);
                                    y[t].y = __shfl_sync(0xffffffffu, y[t].y, src);
                                    y[t].z = __shfl_sync(0xffffffffu, y[t].z, src);
                                    y[t].w = __shfl_sync(0xffffffffu, y[t].w, src);
                                }
                            }
                        }
                        const int pl = 4 * hi + ((qd + 3) & 3);   // the hi column this quarter ends up with
                        if (va) {
#pragma unroll
                            for (int t = 0; t < Q; ++t) xa[8 * t] = x[t];
                        }
                        if (pl < rank) {
                            float4* xl = reinterpret_cast<float4*>(X + perm[pl] * LD) + l8;
#pragma unroll
                            for (int t = 0; t < Q; ++t) xl[8 * t] = y[t];
                        }
                        __syncwarp();
                    }
                  }
                    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
                }
                ++sweeps;
                const int par = sweeps & 1;
                if (__any_sync(0xffffffffu, worst2 > 1e-6f) && lane == 0) atomicOr(&sh_flag[par], 1);
                if (tid == 0) sh_flag[par ^ 1] = 0;
                asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
                more = sh_flag[par];
                if (!more) break;               // every cosine of this sweep was below 1e-3: converged after it
            }
            if (tid == 0) { sh_f[1] = (float)sweeps; sh_f[4] = more ? 1.f : 0.f; }
        }
    }
    __syncthreads();
    sweeps = rank >= 2 ? (int)sh_f[1] : 0;
    const int not_converged = rank >= 2 && sh_f[4] != 0.f;     // stopped at the sweep limit while still rotating visibly

    // ---- eigenvalues = squared column norms (pivot-step order), scaled back; sort descending, stable ----
    for (int k = warp; k < n; k += NW) {
        float a = 0.f;
        if (k < rank) {
            const float* x = X + perm[k] * LD;
#pragma unroll
            for (int t = 0; t < R; ++t) a = fmaf(x[lane + 32 * t], x[lane + 32 * t], a);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        }
        if (lane == 0) lam[k] = a * dmax;
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
    const float back = sqrtf(dmax);     // columns of X are sigma_j u_j / sqrt(dmax)
    if (tid < n) {
        const float l = lam[order[tid]];
        float f = 0.f, sp = 0.f;
        if (l > 0.f && tid < keep) {
            const float kept = fmaxf(l - delta, 0.f);
            sp = sqrtf(kept);
            f = sqrtf(kept / l) * rsqrtf(l) * back;   // (sigma'/sigma) / sigma, for the unscaled column
        }
        fac[tid] = f;
        if (tid < n_sigma) sigma_out[tid] = sp;
    }
    for (int j = n + tid; j < n_sigma; j += NT) sigma_out[j] = 0.f;
    __syncthreads();
    for (int e = tid; e < n * keep; e += NT) {
        const int j = e / n, i = e - j * n;
        float v = 0.f;
        if (j < n) {
            const int k = order[j];
            if (k < rank) v = X[perm[k] * LD + i] * fac[j];
        }
        Ur[(size_t)i * ldu + j] = v;
    }
    if (Wsplit) {   // the same factors transposed and split for the tensor-core rebuild: [W_hi ; W_lo], zero padded
        for (int e = tid; e < j_pad * ldw; e += NT) {
            const int j = e / ldw, i = e - j * ldw;
            float v = 0.f;
            if (j < keep && j < n && i < n) {
                const int k = order[j];
                if (k < rank) v = X[perm[k] * LD + i] * fac[j];
            }
            const float hi = __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xffffe000u);
            Wsplit[wsplit_row(j, j_pad, false) * ldw + i] = hi;
            Wsplit[wsplit_row(j, j_pad, true) * ldw + i] = v - hi;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Cluster solver for 192 < n <= 512: the same algorithm as k_eig_shrink_fast, run by a thread-block cluster
// (8 CTAs of 256 threads on 8 SMs) with the matrix in global memory (L2-resident) and a hardware cluster
// barrier where the one-CTA kernel has a block barrier. Every warp of the cluster owns Cholesky columns and one
// Jacobi block pair, so a block round costs one L2 round trip for its 8 columns, 4 register-resident local rounds
// and one cluster barrier, instead of several passes over 16 warps on one SM. Control flow is identical in
// every CTA (pivot search and convergence flag are computed from identical data), so every thread of the cluster
// reaches every barrier; the small tables (pivot order, eigenvalues, factors) are kept per CTA.
// ------------------------------------------------------------------------------------------------
template <int T>
__global__ void __launch_bounds__(256, 1)
k_eig_shrink_cluster(const float* __restrict__ K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* __restrict__ Ur,
                  int ldu, float* __restrict__ sigma_out, int n_sigma, int max_sweeps, EigInfo* __restrict__ info,
                  float* __restrict__ Wsplit, int ldw, int j_pad, float* __restrict__ gwork) {
    constexpr int LD = 64 * T;
    constexpr int NT = 256;                              // threads per CTA
    constexpr int kMaxN = 512;                           // shadows the namespace constant: this kernel serves n <= 512
    cg::cluster_group cluster = cg::this_cluster();
    const int csize = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
    const int NW = 8 * csize;                            // warps of the whole cluster
    const int GT = NT * csize;                           // threads of the whole cluster
    constexpr int R = 2 * T;            // rows per lane when 32 lanes span a column
    constexpr int Q = 2 * T;            // float4 per lane when 8 lanes span a column
    extern __shared__ __align__(16) float smem[];
    float* X = gwork;                                   // LD x LD in global memory (L2), shared by the cluster
    int* gflag = reinterpret_cast<int*>(gwork + (size_t)LD * LD);   // two convergence words after the matrix
    float* lam = smem;                                  // kMaxN each from here on (one copy per CTA)
    float* fac = lam + kMaxN;
    float* scl = fac + kMaxN;
    int* ord = reinterpret_cast<int*>(scl + kMaxN);     // physical index -> pivot step (-1: never pivoted)
    int* perm = ord + kMaxN;                            // pivot step -> physical index
    int* order = perm + kMaxN;                          // sorted position -> pivot step
    float* sh_f = reinterpret_cast<float*>(order + kMaxN);

    const int tid = threadIdx.x, lane = tid & 31, lwarp = tid >> 5;
    const int warp = crank * 8 + lwarp;                  // warp index within the cluster
    const int gtid = crank * NT + tid;

    // running diagonal and liveness of the rows this lane owns (rows lane + 32 t), one copy per warp
    float dg[R];
    bool alive[R];
    bool bad = false;
    float dmax = 0.f;
#pragma unroll
    for (int t = 0; t < R; ++t) {
        const int i = lane + 32 * t;
        dg[t] = (i < n) ? K[(size_t)i * ldk + i] : -1.f;
        alive[t] = i < n;
        if (alive[t] && !(fabsf(dg[t]) <= 3.0e38f)) { bad = true; alive[t] = false; }
        if (alive[t]) dmax = fmaxf(dmax, dg[t]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
    if (warp == 0 && bad) atomicOr(&info->flags, kFlagNonFinite);
    const bool empty = !(dmax >= 1e-30f);              // nothing to factor: rank 0
    const float kscale = empty ? 0.f : 1.f / dmax;
    for (int e = gtid; e < n * LD; e += GT) {
        const int c = e / LD, i = e - c * LD;
        X[e] = (i < n) ? K[(size_t)c * ldk + i] * kscale : 0.f;  // K is symmetric: row c serves as column c
    }
    if (gtid < 2) gflag[gtid] = 0;
#pragma unroll
    for (int t = 0; t < R; ++t) dg[t] *= kscale;
    for (int i = tid; i < kMaxN; i += NT) ord[i] = -1;
    cluster.sync();

    // ---- pivoted Cholesky without swaps (scaled matrix: diagonal <= 1) ----
    constexpr int CW = (LD + 63) / 64 * 2;                     // upper bound of columns a warp owns (warp + NW u) for NW >= 32
    unsigned colmask = 0u;                                     // bit u: column warp + 32 u is still unpivoted
#pragma unroll
    for (int u = 0; u < CW; ++u)
        if (warp + NW * u < n) colmask |= 1u << u;
    const float tol = 1e-7f;
    int rank = empty ? 0 : n;
    for (int k = 0; k < rank; ++k) {
        unsigned key = 0u;
#pragma unroll
        for (int t = 0; t < R; ++t)
            if (alive[t]) key = max(key, (__float_as_uint(fmaxf(dg[t], 0.f)) & 0xfffffe00u) | (unsigned)(511 - (lane + 32 * t)));
        key = __reduce_max_sync(0xffffffffu, key);                // largest diagonal (24 significant bits), smaller index on ties
        const int p = 511 - (int)(key & 511u);
        if (key == 0u || p >= n) { rank = k; break; }             // identical in every warp
        const float* Xp = X + p * LD;
        const float d = __ldcg(Xp + p);
        if (!(d > tol)) { rank = k; break; }
        const float inv = rsqrtf(d);
        if ((p % NW) == warp) colmask &= ~(1u << (p / NW));
        float li[R];
#pragma unroll
        for (int t = 0; t < R; ++t) {
            const int i = lane + 32 * t;
            if (i == p) alive[t] = false;
            li[t] = alive[t] ? __ldcg(Xp + i) * inv : 0.f;
            dg[t] = fmaf(-li[t], li[t], dg[t]);
        }
#pragma unroll
        for (int u0 = 0; u0 < CW; u0 += 2) {                      // two columns at a time: loads first, then stores
            const bool on0 = (colmask >> u0) & 1u, on1 = (u0 + 1 < CW) && ((colmask >> (u0 + 1)) & 1u);
            if (!on0 && !on1) continue;
            float* c0 = X + (warp + NW * u0) * LD;
            float* c1 = X + (warp + NW * (u0 + 1)) * LD;
            const float l0 = on0 ? __ldcg(Xp + warp + NW * u0) * inv : 0.f;
            const float l1 = on1 ? __ldcg(Xp + warp + NW * (u0 + 1)) * inv : 0.f;
            float v0[R], v1[R];
#pragma unroll
            for (int t = 0; t < R; ++t) {
                v0[t] = on0 ? __ldcg(c0 + lane + 32 * t) : 0.f;
                v1[t] = on1 ? __ldcg(c1 + lane + 32 * t) : 0.f;
            }
#pragma unroll
            for (int t = 0; t < R; ++t) {
                if (on0) c0[lane + 32 * t] = fmaf(-li[t], l0, v0[t]);
                if (on1) c1[lane + 32 * t] = fmaf(-li[t], l1, v1[t]);
            }
        }
        if (tid == 0) { ord[p] = k; perm[k] = p; scl[k] = inv; }   // every CTA keeps its own copy of the tables
        cluster.sync();
    }
    cluster.sync();
    // ---- scale the pivot columns into the factor L (zero above the pivot order, zero unpivoted columns) ----
    for (int e = gtid; e < n * LD; e += GT) {
        const int c = e / LD, i = e - c * LD;
        const int kc = ord[c];
        float v = 0.f;
        if (kc >= 0 && i < n) {
            const int ki = ord[i];
            if (!(ki >= 0 && ki < kc)) v = __ldcg(X + e) * scl[kc];
        }
        X[e] = v;
    }
    cluster.sync();

    // ---- one-sided cyclic Jacobi on the rank pivot columns ----
    // Columns (in pivot order) form blocks of 4. A block round pairs the blocks round-robin, one block
    // pair per warp; the warp rotates the 16 cross pairs of its two blocks in 4 local rounds (one pair per
    // quarter-warp, synchronised inside the warp only), and in the first block round of a sweep also the
    // pairs inside each block. Only the warps that own a block pair take part, on a named barrier.
    const int l8 = tid & 7, qd = lane >> 3;
    int sweeps = 0;
    float worst2 = 0.f;                 // largest squared cosine met in the current sweep
    if (rank >= 2) {
        const int nb = (rank + 3) >> 2, nbe = nb + (nb & 1), nbm1 = nbe - 1, nact = nbe >> 1;   // block pairs per round
        const int nwork = nact < NW ? nact : NW;                  // warps that take part; each owns slots w, w + nwork, ...
        {
            const bool active = warp < nwork;                     // the other warps only take part in the cluster barriers
            auto pair_step = [&](int p, int q) {                  // p, q: pivot-order columns, q >= rank means no pair
                const bool valid = p < rank && q < rank;
                float4* xp = reinterpret_cast<float4*>(X + (valid ? perm[p] : 0) * LD) + l8;
                float4* xq = reinterpret_cast<float4*>(X + (valid ? perm[q] : 0) * LD) + l8;
                float4 x[Q], y[Q];
                float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll
                for (int t = 0; t < Q; ++t) {
                    x[t] = __ldcg(xp + 8 * t);
                    y[t] = __ldcg(xq + 8 * t);
                    a0 = fmaf(x[t].x, x[t].x, a0); a1 = fmaf(x[t].y, x[t].y, a1); a0 = fmaf(x[t].z, x[t].z, a0); a1 = fmaf(x[t].w, x[t].w, a1);
                    b0 = fmaf(y[t].x, y[t].x, b0); b1 = fmaf(y[t].y, y[t].y, b1); b0 = fmaf(y[t].z, y[t].z, b0); b1 = fmaf(y[t].w, y[t].w, b1);
                    g0 = fmaf(x[t].x, y[t].x, g0); g1 = fmaf(x[t].y, y[t].y, g1); g0 = fmaf(x[t].z, y[t].z, g0); g1 = fmaf(x[t].w, y[t].w, g1);
                }
                float a = a0 + a1, b = b0 + b1, g = g0 + g1;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) {
                    a += __shfl_xor_sync(0xffffffffu, a, o);
                    b += __shfl_xor_sync(0xffffffffu, b, o);
                    g += __shfl_xor_sync(0xffffffffu, g, o);
                }
                const float ab = a * b, g2 = g * g;
                if (valid && ab > 0.f && g2 > 1e-12f * ab) {
                    worst2 = fmaxf(worst2, __fdividef(g2, ab));
                    float c, s;
                    jacobi_rotation(a, b, g, c, s);
#pragma unroll
                    for (int t = 0; t < Q; ++t) {
                        float4 nx, ny;
                        nx.x = fmaf(-s, y[t].x, c * x[t].x); ny.x = fmaf(s, x[t].x, c * y[t].x);
                        nx.y = fmaf(-s, y[t].y, c * x[t].y); ny.y = fmaf(s, x[t].y, c * y[t].y);
                        nx.z = fmaf(-s, y[t].z, c * x[t].z); ny.z = fmaf(s, x[t].z, c * y[t].z);
                        nx.w = fmaf(-s, y[t].w, c * x[t].w); ny.w = fmaf(s, x[t].w, c * y[t].w);
                        xp[8 * t] = nx;
                        xq[8 * t] = ny;
                    }
                }
                __syncwarp();
            };
            int more = 0;
            while (sweeps < max_sweeps) {
                worst2 = 0.f;
                for (int br = 0; br < nbm1; ++br) {
                  for (int slot = active ? warp : nact; slot < nact; slot += nwork) {
                    int ba, bb;                                   // the two blocks of this slot in this block round
                    if (slot == 0) { ba = nbm1; bb = br; }
                    else {
                        ba = br + slot; if (ba >= nbm1) ba -= nbm1;
                        bb = br + nbm1 - slot; if (bb >= nbm1) bb -= nbm1;
                    }
                    if (br == 0) {                                // pairs inside each block: quarters 0,1 -> ba, 2,3 -> bb
                        const int base = 4 * ((qd < 2) ? ba : bb), h = qd & 1;
                        pair_step(base + (h ? 2 : 0), base + (h ? 3 : 1));
                        pair_step(base + (h ? 1 : 0), base + (h ? 3 : 2));
                        pair_step(base + (h ? 1 : 0), base + (h ? 2 : 3));
                    }
                    const int lo = min(ba, bb), hi = max(ba, bb);
                    {   // the 16 cross pairs, columns held in registers: quarter qd keeps column qd of block lo and
                        // the columns of block hi travel from quarter to quarter by shuffles between the 4 rounds
                        const int pa = 4 * lo + qd, pb = 4 * hi + qd;
                        const bool va = pa < rank, vb0 = pb < rank;
                        float4* xa = reinterpret_cast<float4*>(X + (va ? perm[pa] : 0) * LD) + l8;
                        float4* xb = reinterpret_cast<float4*>(X + (vb0 ? perm[pb] : 0) * LD) + l8;
                        float4 x[Q], y[Q];
#pragma unroll
                        for (int t = 0; t < Q; ++t) {
                            x[t] = va ? __ldcg(xa + 8 * t) : make_float4(0.f, 0.f, 0.f, 0.f);
                            y[t] = vb0 ? __ldcg(xb + 8 * t) : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int r = 0; r < 4; ++r) {
                            const bool valid = va && (4 * hi + ((qd + r) & 3) < rank);
                            float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll
                            for (int t = 0; t < Q; ++t) {
                                a0 = fmaf(x[t].x, x[t].x, a0); a1 = fmaf(x[t].y, x[t].y, a1); a0 = fmaf(x[t].z, x[t].z, a0); a1 = fmaf(x[t].w, x[t].w, a1);
                                b0 = fmaf(y[t].x, y[t].x, b0); b1 = fmaf(y[t].y, y[t].y, b1); b0 = fmaf(y[t].z, y[t].z, b0); b1 = fmaf(y[t].w, y[t].w, b1);
                                g0 = fmaf(x[t].x, y[t].x, g0); g1 = fmaf(x[t].y, y[t].y, g1); g0 = fmaf(x[t].z, y[t].z, g0); g1 = fmaf(x[t].w, y[t].w, g1);
                            }
                            float a = a0 + a1, b = b0 + b1, g = g0 + g1;
#pragma unroll
                            for (int o = 4; o > 0; o >>= 1) {
                                a += __shfl_xor_sync(0xffffffffu, a, o);
                                b += __shfl_xor_sync(0xffffffffu, b, o);
                                g += __shfl_xor_sync(0xffffffffu, g, o);
                            }
                            const float ab = a * b, g2 = g * g;
                            if (valid && ab > 0.f && g2 > 1e-12f * ab) {
                                worst2 = fmaxf(worst2, __fdividef(g2, ab));
                                float c, s;
                                jacobi_rotation(a, b, g, c, s);
#pragma unroll
                                for (int t = 0; t < Q; ++t) {
                                    float4 nx, ny;
                                    nx.x = fmaf(-s, y[t].x, c * x[t].x); ny.x = fmaf(s, x[t].x, c * y[t].x);
                                    nx.y = fmaf(-s, y[t].y, c * x[t].y); ny.y = fmaf(s, x[t].y, c * y[t].y);
                                    nx.z = fmaf(-s, y[t].z, c * x[t].z); ny.z = fmaf(s, x[t].z, c * y[t].z);
                                    nx.w = fmaf(-s, y[t].w, c * x[t].w); ny.w = fmaf(s, x[t].w, c * y[t].w);
                                    x[t] = nx;
                                    y[t] = ny;
                                }
                            }
                            if (r < 3) {                          // quarter qd takes over the column quarter qd + 1 holds
                                const int src = (lane + 8) & 31;
#pragma unroll
                                for (int t = 0; t < Q; ++t) {
                                    y[t].x = __shfl_sync(0xffffffffu, y[t].x, src);
                                    y[t].y = __shfl_sync(0xffffffffu, y[t].y, src);
                                    y[t].z = __shfl_sync(0xffffffffu, y[t].z, src);
                                    y[t].w = __shfl_sync(0xffffffffu, y[t].w, src);
                                }
                            }
                        }
                        const int pl = 4 * hi + ((qd + 3) & 3);   // the hi column this quarter ends up with
                        if (va) {
#pragma unroll
                            for (int t = 0; t < Q; ++t) xa[8 * t] = x[t];
                        }
                        if (pl < rank) {
                            float4* xl = reinterpret_cast<float4*>(X + perm[pl] * LD) + l8;
#pragma unroll
                            for (int t = 0; t < Q; ++t) xl[8 * t] = y[t];
                        }
                        __syncwarp();
                    }
                  }
                    cluster.sync();
                }
                ++sweeps;
                const int par = sweeps & 1;
                if (__any_sync(0xffffffffu, worst2 > 1e-6f) && lane == 0) atomicOr(&gflag[par], 1);
                if (gtid == 0) gflag[par ^ 1] = 0;
                cluster.sync();
                more = __ldcg(&gflag[par]);
                if (!more) break;               // every cosine of this sweep was below 1e-3: converged after it
            }
            if (tid == 0) { sh_f[1] = (float)sweeps; sh_f[4] = more ? 1.f : 0.f; }
        }
    }
    __syncthreads();
    sweeps = rank >= 2 ? (int)sh_f[1] : 0;
    const int not_converged = rank >= 2 && sh_f[4] != 0.f;     // stopped at the sweep limit while still rotating visibly

    // ---- eigenvalues = squared column norms (pivot-step order), scaled back; sort descending, stable ----
    for (int k = lwarp; k < n; k += 8) {                          // every CTA forms all eigenvalues for its own tables
        float a = 0.f;
        if (k < rank) {
            const float* x = X + perm[k] * LD;
#pragma unroll
            for (int t = 0; t < R; ++t) { const float xv = __ldcg(x + lane + 32 * t); a = fmaf(xv, xv, a); }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        }
        if (lane == 0) lam[k] = a * dmax;
    }
    __syncthreads();
    for (int t = tid; t < n; t += NT) {
        const float mine = lam[t];
        int pos = 0;
        for (int i = 0; i < n; ++i) {
            const float o = lam[i];
            pos += (o > mine) || (o == mine && i < t);
        }
        order[pos] = t;
    }
    __syncthreads();
    if (tid == 0) {
        float delta = 0.f;
        if (do_shrink && delta_rank - 1 < n) delta = lam[order[delta_rank - 1]];
        sh_f[0] = delta;
        if (crank == 0) {
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
    }
    __syncthreads();
    const float delta = sh_f[0];
    const float back = sqrtf(dmax);     // columns of X are sigma_j u_j / sqrt(dmax)
    for (int t = tid; t < n; t += NT) {
        const float l = lam[order[t]];
        float f = 0.f, sp = 0.f;
        if (l > 0.f && t < keep) {
            const float kept = fmaxf(l - delta, 0.f);
            sp = sqrtf(kept);
            f = sqrtf(kept / l) * rsqrtf(l) * back;   // (sigma'/sigma) / sigma, for the unscaled column
        }
        fac[t] = f;
        if (t < n_sigma && crank == 0) sigma_out[t] = sp;
    }
    if (crank == 0)
        for (int j = n + tid; j < n_sigma; j += NT) sigma_out[j] = 0.f;
    __syncthreads();
    for (int e = gtid; e < n * keep; e += GT) {
        const int j = e / n, i = e - j * n;
        float v = 0.f;
        if (j < n) {
            const int k = order[j];
            if (k < rank) v = __ldcg(X + perm[k] * LD + i) * fac[j];
        }
        Ur[(size_t)i * ldu + j] = v;
    }
    if (Wsplit) {   // the same factors transposed and split for the tensor-core rebuild: [W_hi ; W_lo], zero padded
        for (int e = gtid; e < j_pad * ldw; e += GT) {
            const int j = e / ldw, i = e - j * ldw;
            float v = 0.f;
            if (j < keep && j < n && i < n) {
                const int k = order[j];
                if (k < rank) v = __ldcg(X + perm[k] * LD + i) * fac[j];
            }
            const float hi = __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xffffe000u);
            Wsplit[wsplit_row(j, j_pad, false) * ldw + i] = hi;
            Wsplit[wsplit_row(j, j_pad, true) * ldw + i] = v - hi;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Distributed-shared-memory solver, all n <= 512: the same algorithm again, with the Jacobi phase spread over a
// thread-block cluster of 8 CTAs and its columns kept ON CHIP. The one-CTA kernel is bound by instruction issue
// (16 block pairs share four schedulers); here every block pair has a warp of its own on one of 8 SMs, so a local
// round costs its dependent-latency chain only.
//   * Round-robin slots are dealt to the CTAs in runs (slot s -> CTA s / SPC, warp s % SPC). Each warp owns a slot
//     buffer of 2 blocks x 4 columns in its CTA's shared memory. A block round: load the 8 columns into registers,
//     rotate the 16 cross pairs in 4 local rounds (as in the one-CTA kernel), then store every column straight
//     into the slot buffer of the warp that needs it next (a remote shared-memory store when that warp sits in
//     another CTA; the tournament moves a block to a neighbouring slot, so most stores stay local).
//   * Exchange, n <= 192: two buffer sets per slot, used by alternate block rounds, and one mbarrier per slot and
//     set. A warp sends its columns into the reader's other set with asynchronous stores (st.async) that count
//     their bytes on the reader's barrier as they land: one-way latency, no fence or round trip on the writer's
//     side (a plain remote store followed by a releasing arrival, or by a cluster barrier, cost the writer about
//     900 cycles per block round); the reader announces the 8 columns it expects and waits for the phase. A set
//     is overwritten two rounds after it was read: the writer could only finish the round in between after the
//     reader had finished the round before that (the tournament makes every slot's readers also its suppliers), so
//     no write overtakes a read. Waits are bounded; one that runs out raises a cluster-wide word, every warp stops
//     exchanging and the solve ends with an error flag. One cluster barrier per sweep, for the convergence word.
//   * Exchange, n > 192 (asynchronous stores of 16 bytes become the bottleneck: 16 and more per lane and round
//     measured slower than plain remote stores; above 256 only one set fits anyway): two cluster barriers per block round, "everyone has loaded" (its wait
//     is hidden behind the local rounds) before the stores, "everyone has stored" before the next loads.
//   * All threads of the cluster execute the same number of cluster barriers: trip counts depend only on the rank,
//     the sweep limit and words that all read from global memory after a barrier.
//   * Cholesky: the columns are dealt to the 8 CTAs and stay in their shared memory; the pivot column of a step
//     reaches every CTA by asynchronous stores (see the comment at the loop). The factor is handed to the Jacobi
//     phase through global memory (L2), so both phases can use the same shared memory.
// `gwork`: LD*LD floats (factor), then 2 convergence words, a spare word and the give-up word.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void cl_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cl_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// The two blocks slot `slot` holds in block round `br` (half 0: ba, half 1: bb).
__device__ __forceinline__ void rr_blocks(int slot, int br, int nbm1, int& ba, int& bb) {
    if (slot == 0) { ba = nbm1; bb = br; }
    else {
        ba = br + slot; if (ba >= nbm1) ba -= nbm1;
        bb = br + nbm1 - slot; if (bb >= nbm1) bb -= nbm1;
    }
}
// Inverse: slot and half that hold block b in block round br.
__device__ __forceinline__ void rr_slot_of(int b, int br, int nbm1, int nact, int& slot, int& half) {
    if (b == nbm1) { slot = 0; half = 0; return; }
    int d = b - br;
    if (d < 0) d += nbm1;
    if (d == 0) { slot = 0; half = 1; }
    else if (d < nact) { slot = d; half = 0; }
    else { slot = nbm1 - d; half = 1; }
}

// ---- pieces of the cluster exchange: cluster-scope shared-memory addresses, mbarrier operations, async stores ----
__device__ __forceinline__ uint32_t smem_addr_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t mapa_u32(uint32_t local_addr, uint32_t cta_rank) {   // same offset in another CTA of the cluster
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(cta_rank));
    return r;
}
__device__ __forceinline__ void mbar_init_cluster(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_local(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {   // a barrier of any CTA of the cluster
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The reader's own arrival for the current phase, announcing how many bytes asynchronous stores will deliver.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr_u32(bar)), "r"(bytes) : "memory");
}
// 16 bytes into the shared memory of a CTA of the cluster; the store itself counts its bytes on the barrier (same
// CTA as the data) when it has landed, so the writer needs neither a fence nor a round trip.
__device__ __forceinline__ void st_async_v4(uint32_t cluster_addr, const float4& v, uint32_t cluster_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(cluster_addr),
                 "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(cluster_bar)
                 : "memory");
}
constexpr long long kExchangeWaitCycles = 400000000ll;   // about 0.2 s
// Waits for the phase with the given parity of a barrier in this CTA's shared memory. Bounded: gives up (false) after
// kExchangeWaitCycles or as soon as another warp of the cluster has given up (*gabort != 0).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, const int* gabort) {
    const uint32_t a = smem_addr_u32(bar);
    const long long t0 = clock64();
    for (int it = 0;; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(ok)
            : "r"(a), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((it & 63) == 63 && (clock64() - t0 > kExchangeWaitCycles || __ldcg(gabort) != 0)) return false;
    }
}

// One column pair held in shared memory, 8 lanes per pair (Q float4 per lane and column).
template <int Q>
__device__ __forceinline__ void jacobi_pair_in_smem(float* cp, float* cq, bool valid, int l8, float& worst2) {
    float4* xp = reinterpret_cast<float4*>(cp) + l8;
    float4* xq = reinterpret_cast<float4*>(cq) + l8;
    float4 x[Q], y[Q];
    float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll
    for (int t = 0; t < Q; ++t) {
        x[t] = xp[8 * t];
        y[t] = xq[8 * t];
        a0 = fmaf(x[t].x, x[t].x, a0); a1 = fmaf(x[t].y, x[t].y, a1); a0 = fmaf(x[t].z, x[t].z, a0); a1 = fmaf(x[t].w, x[t].w, a1);
        b0 = fmaf(y[t].x, y[t].x, b0); b1 = fmaf(y[t].y, y[t].y, b1); b0 = fmaf(y[t].z, y[t].z, b0); b1 = fmaf(y[t].w, y[t].w, b1);
        g0 = fmaf(x[t].x, y[t].x, g0); g1 = fmaf(x[t].y, y[t].y, g1); g0 = fmaf(x[t].z, y[t].z, g0); g1 = fmaf(x[t].w, y[t].w, g1);
    }
    float a = a0 + a1, b = b0 + b1, g = g0 + g1;
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        b += __shfl_xor_sync(0xffffffffu, b, o);
        g += __shfl_xor_sync(0xffffffffu, g, o);
    }
    const float ab = a * b, g2 = g * g;
    if (valid && ab > 0.f && g2 > 1e-12f * ab) {
        worst2 = fmaxf(worst2, __fdividef(g2, ab));
        float c, s;
        jacobi_rotation(a, b, g, c, s);
#pragma unroll
        for (int t = 0; t < Q; ++t) {
            float4 nx, ny;
            nx.x = fmaf(-s, y[t].x, c * x[t].x); ny.x = fmaf(s, x[t].x, c * y[t].x);
            nx.y = fmaf(-s, y[t].y, c * x[t].y); ny.y = fmaf(s, x[t].y, c * y[t].y);
            nx.z = fmaf(-s, y[t].z, c * x[t].z); ny.z = fmaf(s, x[t].z, c * y[t].z);
            nx.w = fmaf(-s, y[t].w, c * x[t].w); ny.w = fmaf(s, x[t].w, c * y[t].w);
            xp[8 * t] = nx;
            xq[8 * t] = ny;
        }
    }
    __syncwarp();
}

// The 16 cross pairs of two blocks of 4 columns, columns in registers: quarter qd of the warp keeps column qd of the
// lower block (x) and meets the 4 columns of the higher block (y) in 4 rounds; between rounds the y columns move to
// the next quarter by shuffles. Afterwards quarter qd holds column (qd + 3) % 4 of the higher block.
template <int Q>
__device__ __forceinline__ void jacobi_cross_rounds(float4 (&x)[Q], float4 (&y)[Q], bool va, int hi, int rank, int qd, int lane,
                                                    float& worst2) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const bool valid = va && (4 * hi + ((qd + r) & 3) < rank);
        float a0 = 0.f, a1 = 0.f, b0 = 0.f, b1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll
        for (int t = 0; t < Q; ++t) {
            a0 = fmaf(x[t].x, x[t].x, a0); a1 = fmaf(x[t].y, x[t].y, a1); a0 = fmaf(x[t].z, x[t].z, a0); a1 = fmaf(x[t].w, x[t].w, a1);
            b0 = fmaf(y[t].x, y[t].x, b0); b1 = fmaf(y[t].y, y[t].y, b1); b0 = fmaf(y[t].z, y[t].z, b0); b1 = fmaf(y[t].w, y[t].w, b1);
            g0 = fmaf(x[t].x, y[t].x, g0); g1 = fmaf(x[t].y, y[t].y, g1); g0 = fmaf(x[t].z, y[t].z, g0); g1 = fmaf(x[t].w, y[t].w, g1);
        }
        float a = a0 + a1, b = b0 + b1, g = g0 + g1;
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
            a += __shfl_xor_sync(0xffffffffu, a, o);
            b += __shfl_xor_sync(0xffffffffu, b, o);
            g += __shfl_xor_sync(0xffffffffu, g, o);
        }
        const float ab = a * b, g2 = g * g;
        if (valid && ab > 0.f && g2 > 1e-12f * ab) {
            worst2 = fmaxf(worst2, __fdividef(g2, ab));
            float c, s;
            jacobi_rotation(a, b, g, c, s);
#pragma unroll
            for (int t = 0; t < Q; ++t) {
                float4 nx, ny;
                nx.x = fmaf(-s, y[t].x, c * x[t].x); ny.x = fmaf(s, x[t].x, c * y[t].x);
                nx.y = fmaf(-s, y[t].y, c * x[t].y); ny.y = fmaf(s, x[t].y, c * y[t].y);
                nx.z = fmaf(-s, y[t].z, c * x[t].z); ny.z = fmaf(s, x[t].z, c * y[t].z);
                nx.w = fmaf(-s, y[t].w, c * x[t].w); ny.w = fmaf(s, x[t].w, c * y[t].w);
                x[t] = nx;
                y[t] = ny;
            }
        }
        if (r < 3) {                              // quarter qd takes over the column quarter qd + 1 holds
            const int src = (lane + 8) & 31;
#pragma unroll
            for (int t = 0; t < Q; ++t) {
                y[t].x = __shfl_sync(0xffffffffu, y[t].x, src);
                y[t].y = __shfl_sync(0xffffffffu, y[t].y, src);
                y[t].z = __shfl_sync(0xffffffffu, y[t].z, src);
                y[t].w = __shfl_sync(0xffffffffu, y[t].w, src);
            }
        }
    }
}

template <int T, int NT>
__global__ void __launch_bounds__(NT, 1)
k_eig_shrink_dsm(const float* __restrict__ K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* __restrict__ Ur,
                 int ldu, float* __restrict__ sigma_out, int n_sigma, int max_sweeps, EigInfo* __restrict__ info,
                 float* __restrict__ Wsplit, int ldw, int j_pad, float* __restrict__ gwork) {
    constexpr int LD = 64 * T;
    constexpr int kMaxN = 512;                           // shadows the namespace constant
    constexpr int WPC = NT / 32;                         // warps per CTA
    constexpr bool kP2P = T <= 3;                        // exchange by asynchronous stores, per-slot barriers and two buffer sets
    constexpr int R = 2 * T;            // rows per lane when 32 lanes span a column
    constexpr int Q = 2 * T;            // float4 per lane when 8 lanes span a column
    cg::cluster_group cluster = cg::this_cluster();
    const int csize = (int)cluster.num_blocks(), crank = (int)cluster.block_rank();
    const int GT = NT * csize;
    extern __shared__ __align__(16) float smem[];
    float* X = gwork;                                   // LD x LD factor in global memory (L2)
    int* gflag = reinterpret_cast<int*>(gwork + (size_t)LD * LD);   // [0],[1] convergence words, [2] rank
    float* lam = smem;                                  // kMaxN each from here on (one copy per CTA)
    float* fac = lam + kMaxN;
    float* scl = fac + kMaxN;
    int* ord = reinterpret_cast<int*>(scl + kMaxN);     // physical index -> pivot step (-1: never pivoted)
    int* perm = ord + kMaxN;                            // pivot step -> physical index
    int* order = perm + kMaxN;                          // sorted position -> pivot step
    float* sh_f = reinterpret_cast<float*>(order + kMaxN);
    uint64_t* mbar = reinterpret_cast<uint64_t*>(sh_f + 8);   // [2 sets][8 slots] exchange barriers (kP2P)
    uint64_t* pbar = mbar + 16;                         // Cholesky phase: [3] pivot column landed (bytes), then
    uint64_t* cdone = mbar + 19;                        // [3] every warp of this CTA has finished the step, and
    uint64_t* alldone = mbar + 22;                      // [3] every CTA of the cluster has
    uint32_t* sched = reinterpret_cast<uint32_t*>(mbar + 32);   // [T slots][128 block rounds] packed exchange schedule
    float* pbuf = reinterpret_cast<float*>(sched + T * 128);    // [3][LD] pivot columns of the Cholesky phase
    float* sbuf = pbuf + 3 * LD;                        // slot buffers: [kSets][T slots][2 halves][4 columns][LD]

    const int tid = threadIdx.x, lane = tid & 31, lwarp = tid >> 5;
    const int gtid = crank * NT + tid;

    // running diagonal and liveness of the rows this lane owns (rows lane + 32 t), one copy per warp
    float dg[R];
    bool alive[R];
    bool bad = false;
    float dmax = 0.f;
#pragma unroll
    for (int t = 0; t < R; ++t) {
        const int i = lane + 32 * t;
        dg[t] = (i < n) ? K[(size_t)i * ldk + i] : -1.f;
        alive[t] = i < n;
        if (alive[t] && !(fabsf(dg[t]) <= 3.0e38f)) { bad = true; alive[t] = false; }
        if (alive[t]) dmax = fmaxf(dmax, dg[t]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
    if (gtid < 32 && bad) atomicOr(&info->flags, kFlagNonFinite);
    const bool empty = !(dmax >= 1e-30f);              // nothing to factor: rank 0
    const float kscale = empty ? 0.f : 1.f / dmax;
#pragma unroll
    for (int t = 0; t < R; ++t) dg[t] *= kscale;
    for (int i = tid; i < kMaxN; i += NT) { ord[i] = -1; perm[i] = 0; }
    if (gtid < 4) gflag[gtid] = 0;
    if (tid < 19) mbar_init_cluster(&mbar[tid], 1);     // the reader's own arrival; the stores count bytes
    if (tid >= 19 && tid < 22) mbar_init_cluster(&mbar[tid], WPC);
    if (tid >= 22 && tid < 25) mbar_init_cluster(&mbar[tid], 8);
    if (tid == 0) asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const float tol = 1e-7f;
    int rank = empty ? 0 : n;

    // ---- pivoted Cholesky without swaps, columns dealt to the 8 CTAs (physical column j lives in CTA j % 8) ----
    // Every warp of the cluster finds the pivot from its own copy of the running diagonal (identical everywhere).
    // The warp that owns the pivot column sends it to all 8 CTAs with asynchronous stores that count their bytes
    // on a barrier in each CTA; every warp waits for that, refreshes its diagonal and updates the columns it owns
    // in its CTA's shared memory: a step costs one one-way trip instead of a cluster barrier plus L2 round trips,
    // and the trailing update has the shared-memory bandwidth of 8 SMs. The owner of the NEXT pivot column (known as
    // soon as the diagonal is refreshed) updates that column first and sends it at once, so the trip overlaps the rest
    // of the step. Three pivot buffers rotate; before a warp overwrites the buffer of step k - 3 it waits until every
    // CTA has reported that step finished (each warp
    // arrives on its CTA's `cdone` barrier at the end of a step; warp 0 of each CTA waits for that and arrives on
    // the `alldone` barrier of all 8 CTAs: a whole step of slack, so the sender rarely waits). Every wait is bounded;
    // one that runs out raises the cluster-wide give-up word, which ends all other waits, and every warp leaves the
    // loop for the same barriers below.
    constexpr int CPC = LD / 8;                          // local columns per CTA
    constexpr int CW = (CPC + WPC - 1) / WPC;            // local columns a warp owns: lwarp + WPC u
    float* Xc = sbuf;                                    // [CPC][LD], reuses the slot buffers (the hand-over goes through L2)
    const bool geometry_ok = csize == 8;                 // the layout above assumes the cluster this kernel is launched with
    if (!geometry_ok) rank = 0;
    unsigned colmask = 0u;                               // bit u: local column lwarp + WPC u is still unpivoted
#pragma unroll
    for (int u = 0; u < CW; ++u) {
        const int jl = lwarp + WPC * u, j = jl * 8 + crank;
        if (jl < CPC && j < n && geometry_ok) {
            colmask |= 1u << u;
#pragma unroll
            for (int t = 0; t < R; ++t) {
                const int i = lane + 32 * t;
                Xc[jl * LD + i] = (i < n) ? K[(size_t)j * ldk + i] * kscale : 0.f;   // K is symmetric: row j serves as column j
            }
        }
    }
    __syncwarp();
    cluster.sync();                                      // barriers initialised everywhere before the first remote store
    bool chol_failed = false;
    auto find_pivot = [&]() -> int {                              // largest remaining diagonal entry; -1: none left
        unsigned key = 0u;
#pragma unroll
        for (int t = 0; t < R; ++t)
            if (alive[t]) key = max(key, (__float_as_uint(fmaxf(dg[t], 0.f)) & 0xfffffe00u) | (unsigned)(511 - (lane + 32 * t)));
        key = __reduce_max_sync(0xffffffffu, key);                // 23 significant bits, smaller index on ties
        const int p = 511 - (int)(key & 511u);
        return (key == 0u || p >= n) ? -1 : p;                    // identical in every warp of the cluster
    };
    // The warp that owns column p sends it to all 8 CTAs as the pivot column of step k (buffer and barrier k % 3), once
    // every CTA has reported step k - 3 finished. Returns false if that wait ran out.
    auto send_pivot = [&](int p, int k) -> bool {
        const int ojl = p >> 3, set = k % 3;
        if ((p & 7) != crank || (ojl % WPC) != lwarp) return true;
        if (k >= 3) {
            bool free_ = mbar_wait_cluster(&alldone[set], (uint32_t)(k / 3 - 1) & 1u, &gflag[3]);
            free_ = __all_sync(0xffffffffu, free_);
            if (!free_) {
                if (lane == 0) atomicOr(&gflag[3], 1);
                return false;
            }
        }
        const float4* src = reinterpret_cast<const float4*>(Xc + ojl * LD);
        const uint32_t dst0 = smem_addr_u32(pbuf + set * LD), bar0 = smem_addr_u32(&pbar[set]);
        for (int q = lane; q < LD / 4; q += 32) {
            const float4 v = src[q];
#pragma unroll
            for (int c = 0; c < 8; ++c) st_async_v4(mapa_u32(dst0 + 16u * q, (uint32_t)c), v, mapa_u32(bar0, (uint32_t)c));
        }
        colmask &= ~(1u << (ojl / WPC));
        return true;
    };
    int p = rank > 0 ? find_pivot() : -1;
    if (p >= 0 && !send_pivot(p, 0)) chol_failed = true;
    if (tid == 0) mbar_arrive_expect_tx(&pbar[0], (uint32_t)(LD * sizeof(float)));   // this CTA expects the column of step 0
    for (int k = 0; k < rank && !chol_failed; ++k) {
        if (p < 0) { rank = k; break; }                           // identical in every warp of the cluster
        const int set = k % 3;
        const float* pb = pbuf + set * LD;
        bool ok = mbar_wait_cluster(&pbar[set], (uint32_t)(k / 3) & 1u, &gflag[3]);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
            if (lane == 0) atomicOr(&gflag[3], 1);
            chol_failed = true;
            break;
        }
        // announce the next step's column now (its barrier finished its previous use three steps ago), so that the
        // other warps of this CTA never wait for warp 0, which has the reporting below to do
        if (tid == 0) mbar_arrive_expect_tx(&pbar[(k + 1) % 3], (uint32_t)(LD * sizeof(float)));
        const float d = pb[p];
        if (!(d > tol)) { rank = k; break; }                      // identical everywhere: all read the same column
        const float inv = rsqrtf(d);
        float li[R];
#pragma unroll
        for (int t = 0; t < R; ++t) {
            const int i = lane + 32 * t;
            if (i == p) alive[t] = false;
            li[t] = alive[t] ? pb[i] * inv : 0.f;
            dg[t] = fmaf(-li[t], li[t], dg[t]);
        }
        // Look-ahead: the refreshed diagonal already names the next pivot; its owner brings that column up to date first
        // and sends it, so that its trip to the other CTAs overlaps the rest of this step's update.
        const int p_next = (k + 1 < rank) ? find_pivot() : -1;
        auto update_column = [&](int u) {
            const int jl = lwarp + WPC * u;
            float* col = Xc + jl * LD;
            const float l = pb[jl * 8 + crank] * inv;
#pragma unroll
            for (int t = 0; t < R; ++t) col[lane + 32 * t] = fmaf(-li[t], l, col[lane + 32 * t]);
        };
        if (p_next >= 0 && (p_next & 7) == crank && ((p_next >> 3) % WPC) == lwarp) {
            update_column((p_next >> 3) / WPC);
            __syncwarp();                                         // the send reads whole float4s of what the lanes updated
            if (!send_pivot(p_next, k + 1)) { chol_failed = true; break; }
        }
#pragma unroll
        for (int u = 0; u < CW; ++u)
            if ((colmask >> u) & 1u) update_column(u);
        if (tid == 0) { ord[p] = k; perm[k] = p; scl[k] = inv; }   // every CTA keeps its own copy of the tables
        if (lane == 0) mbar_arrive_local(&cdone[set]);            // this warp has finished step k
        if (lwarp == 0) {                                         // warp 0 reports the whole CTA to all 8 CTAs
            bool fin = mbar_wait_cluster(&cdone[set], (uint32_t)(k / 3) & 1u, &gflag[3]);
            fin = __all_sync(0xffffffffu, fin);
            if (!fin) {
                if (lane == 0) atomicOr(&gflag[3], 1);
                chol_failed = true;
                break;
            }
            if (lane < 8) mbar_arrive_remote(mapa_u32(smem_addr_u32(&alldone[set]), (uint32_t)lane));
        }
        p = p_next;
    }
    __syncthreads();
    // ---- scale the pivot columns into the factor L (zero above the pivot order, zero unpivoted columns), into L2 ----
    if (!chol_failed) {
#pragma unroll
        for (int u = 0; u < CW; ++u) {
            const int jl = lwarp + WPC * u, j = jl * 8 + crank;
            if (jl < CPC && j < n && geometry_ok) {
                const int kc = ord[j];
#pragma unroll
                for (int t = 0; t < R; ++t) {
                    const int i = lane + 32 * t;
                    float v = 0.f;
                    if (kc >= 0 && i < n) {
                        const int ki = ord[i];
                        if (!(ki >= 0 && ki < kc)) v = Xc[jl * LD + i] * scl[kc];
                    }
                    X[(size_t)j * LD + i] = v;
                }
            }
        }
    }
    cluster.sync();
    if (__ldcg(&gflag[3]) != 0 || !geometry_ok) rank = 0;         // a wait ran out somewhere: no Jacobi, flagged below
    __syncthreads();

    // ---- one-sided cyclic Jacobi on the rank pivot columns, columns in distributed shared memory ----
    const int l8 = lane & 7, qd = lane >> 3;
    int sweeps = 0, more = 0;
    float worst2 = 0.f;                 // largest squared cosine met in the current sweep
    if (rank >= 2) {
        const int nb = (rank + 3) >> 2, nbe = nb + (nb & 1), nbm1 = nbe - 1, nact = nbe >> 1;   // block pairs per round
        const int SPC = (nact + csize - 1) / csize;               // slots per CTA
        const unsigned spc_inv = (65536u + (unsigned)SPC - 1u) / (unsigned)SPC;   // s / SPC = (s * spc_inv) >> 16 for s < 64
        const int slot = crank * SPC + lwarp;
        const bool fits = SPC <= T && SPC <= WPC;                 // holds for a cluster of 8; otherwise report, do not run
        const bool active = fits && lwarp < SPC && slot < nact;   // the other warps only take part in the barriers
        const int myslot = lwarp < T ? lwarp : 0;
        float* mybuf = sbuf + (size_t)myslot * 8 * LD;            // set 0
        if (active) {                                             // columns of block round 0 from the factor in L2
            int ba, bb;
            rr_blocks(slot, 0, nbm1, ba, bb);
            for (int hc = 0; hc < 8; hc += 2) {                  // two columns' loads in flight (each is an L2 round trip)
                const int p0 = 4 * (hc < 4 ? ba : bb) + (hc & 3), p1 = p0 + 1;
                const float* s0 = X + (size_t)perm[p0 < rank ? p0 : 0] * LD;
                const float* s1 = X + (size_t)perm[p1 < rank ? p1 : 0] * LD;
                float v0[R], v1[R];
#pragma unroll
                for (int t = 0; t < R; ++t) {
                    v0[t] = (p0 < rank) ? __ldcg(s0 + lane + 32 * t) : 0.f;
                    v1[t] = (p1 < rank) ? __ldcg(s1 + lane + 32 * t) : 0.f;
                }
#pragma unroll
                for (int t = 0; t < R; ++t) {
                    mybuf[hc * LD + lane + 32 * t] = v0[t];
                    mybuf[(hc + 1) * LD + lane + 32 * t] = v1[t];
                }
            }
        }
        // The tournament repeats every sweep: block pair and destinations of every block round, packed into one word
        // per round (a warp alone on its scheduler pays full latency for every dependent index instruction, so the
        // schedule is worked out once, a round per lane, instead of in every round).
        uint32_t* mysched = sched + myslot * 128;
        if (active) {
            for (int br = lane; br < nbm1; br += 32) {
                int ba, bb;
                rr_blocks(slot, br, nbm1, ba, bb);
                const int lo = min(ba, bb), hi = max(ba, bb);
                const int brn = (br + 1 == nbm1) ? 0 : br + 1;
                int s_lo, h_lo, s_hi, h_hi;
                rr_slot_of(lo, brn, nbm1, nact, s_lo, h_lo);
                rr_slot_of(hi, brn, nbm1, nact, s_hi, h_hi);
                const int c_lo = (int)(((unsigned)s_lo * spc_inv) >> 16), c_hi = (int)(((unsigned)s_hi * spc_inv) >> 16);
                const int l_lo = s_lo - c_lo * SPC, l_hi = s_hi - c_hi * SPC;
                mysched[br] = (uint32_t)ba | ((uint32_t)bb << 8) | ((uint32_t)c_lo << 16) | ((uint32_t)l_lo << 19) | ((uint32_t)h_lo << 22) |
                              ((uint32_t)c_hi << 23) | ((uint32_t)l_hi << 26) | ((uint32_t)h_hi << 29);
            }
        }
        __syncwarp();
        int g = 0;                                                // block rounds done so far, over all sweeps
        bool failed = false;                                      // an exchange wait ran out (kP2P only)
        while (sweeps < max_sweeps) {
            worst2 = 0.f;
            for (int br = 0; br < nbm1; ++br, ++g) {
                float4 x[Q], y[Q];
                int hi = 0;
                bool va = false;
                float4 *o_lo = nullptr, *o_hi = nullptr;                // !kP2P: generic pointers into the readers' buffers
                uint32_t a_lo = 0, a_hi = 0, bar_lo = 0, bar_hi = 0;   // kP2P: cluster addresses of data and barriers
                const bool work = active && !failed;
                bool loaded = false;
                if (work) {
                    float* cur = kP2P ? sbuf + (size_t)((g & 1) * T + myslot) * 8 * LD : mybuf;
                    // Everything that does not depend on the incoming columns first (it runs while they are in flight):
                    // the block pair of this round and where the next block round reads the columns this quarter ends with
                    const uint32_t sc = mysched[br];
                    const int ba = (int)(sc & 255u), bb = (int)((sc >> 8) & 255u);
                    const int lo = min(ba, bb);
                    hi = max(ba, bb);
                    const int half_lo = (ba < bb) ? 0 : 1;
                    va = 4 * lo + qd < rank;
                    {
                        const int c_lo = (int)((sc >> 16) & 7u), l_lo = (int)((sc >> 19) & 7u), h_lo = (int)((sc >> 22) & 1u);
                        const int c_hi = (int)((sc >> 23) & 7u), l_hi = (int)((sc >> 26) & 7u), h_hi = (int)((sc >> 29) & 1u);
                        const int nset = kP2P ? ((g + 1) & 1) : 0;
                        float* d_lo = sbuf + ((size_t)(nset * T + l_lo) * 8 + h_lo * 4 + qd) * LD + 4 * l8;                // in CTA c_lo
                        float* d_hi = sbuf + ((size_t)(nset * T + l_hi) * 8 + h_hi * 4 + ((qd + 3) & 3)) * LD + 4 * l8;    // in CTA c_hi
                        if (kP2P) {
                            a_lo = mapa_u32(smem_addr_u32(d_lo), (uint32_t)c_lo);
                            a_hi = mapa_u32(smem_addr_u32(d_hi), (uint32_t)c_hi);
                            bar_lo = mapa_u32(smem_addr_u32(&mbar[nset * 8 + l_lo]), (uint32_t)c_lo);
                            bar_hi = mapa_u32(smem_addr_u32(&mbar[nset * 8 + l_hi]), (uint32_t)c_hi);
                        } else {
                            o_lo = reinterpret_cast<float4*>(cluster.map_shared_rank(d_lo, c_lo));
                            o_hi = reinterpret_cast<float4*>(cluster.map_shared_rank(d_hi, c_hi));
                        }
                    }
                    bool ok = true;
                    if (kP2P && g > 0) {                          // both blocks of this round have landed in this set
                        if (lane == 0) mbar_arrive_expect_tx(&mbar[(g & 1) * 8 + myslot], 8u * LD * sizeof(float));
                        ok = mbar_wait_cluster(&mbar[(g & 1) * 8 + myslot], (uint32_t)((g - 1) >> 1) & 1u, &gflag[3]);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) {
                            failed = true;
                            if (lane == 0) atomicOr(&gflag[3], 1);
                        }
                    }
                    if (ok) {
                        loaded = true;
                        if (br == 0) {                            // pairs inside each block: quarters 0,1 -> ba, 2,3 -> bb
                            const int half = (qd < 2) ? 0 : 1, base = 4 * (half ? bb : ba), h = qd & 1;
                            float* blk = cur + half * 4 * LD;
                            const int c0 = h ? 2 : 0, c1 = h ? 3 : 1, c2 = h ? 1 : 0, c3 = h ? 3 : 2, c4 = h ? 1 : 0, c5 = h ? 2 : 3;
                            jacobi_pair_in_smem<Q>(blk + c0 * LD, blk + c1 * LD, base + c0 < rank && base + c1 < rank, l8, worst2);
                            jacobi_pair_in_smem<Q>(blk + c2 * LD, blk + c3 * LD, base + c2 < rank && base + c3 < rank, l8, worst2);
                            jacobi_pair_in_smem<Q>(blk + c4 * LD, blk + c5 * LD, base + c4 < rank && base + c5 < rank, l8, worst2);
                        }
                        // quarter qd keeps column qd of block lo; the columns of block hi travel between quarters
                        const float4* xa = reinterpret_cast<const float4*>(cur + (half_lo * 4 + qd) * LD) + l8;
                        const float4* xb = reinterpret_cast<const float4*>(cur + ((1 - half_lo) * 4 + qd) * LD) + l8;
#pragma unroll
                        for (int t = 0; t < Q; ++t) {
                            x[t] = xa[8 * t];
                            y[t] = xb[8 * t];
                        }
                    }
                }
                if (!kP2P) cl_arrive();                            // "loaded": completes while the local rounds run
                if (loaded) jacobi_cross_rounds<Q>(x, y, va, hi, rank, qd, lane, worst2);
                if (!kP2P) cl_wait();                              // every warp of the cluster holds its columns in registers
                if (loaded) {                                      // send each column to where the next block round reads it
                    if (kP2P) {                                    // asynchronous stores that count their bytes on the reader's barrier
#pragma unroll
                        for (int t = 0; t < Q; ++t) {
                            st_async_v4(a_lo + 128u * t, x[t], bar_lo);
                            st_async_v4(a_hi + 128u * t, y[t], bar_hi);
                        }
                    } else {
#pragma unroll
                        for (int t = 0; t < Q; ++t) {
                            o_lo[8 * t] = x[t];
                            o_hi[8 * t] = y[t];
                        }
                    }
                }
                if (br == nbm1 - 1) {                              // end of a sweep: publish whether anything still rotated
                    const int par = (sweeps + 1) & 1;
                    if (__any_sync(0xffffffffu, worst2 > 1e-6f) && lane == 0) atomicOr(&gflag[par], 1);
                    if (gtid == 0) gflag[par ^ 1] = 0;
                }
                if (!kP2P || br == nbm1 - 1) {
                    cl_arrive();
                    cl_wait();                                     // "stored" (kP2P: once per sweep, for the convergence word)
                }
            }
            ++sweeps;
            more = fits ? __ldcg(&gflag[sweeps & 1]) : 1;
            if (kP2P && __ldcg(&gflag[3])) { more = 2; break; }    // an exchange wait ran out somewhere: stop everywhere
            if (!more) break;               // every cosine of this sweep was below 1e-3: converged after it
            if (!fits) break;
        }
        if (kP2P && active && more != 2 && g > 0) {               // the last round's columns: wait for them like any round's
            if (lane == 0) mbar_arrive_expect_tx(&mbar[(g & 1) * 8 + myslot], 8u * LD * sizeof(float));
            bool ok = mbar_wait_cluster(&mbar[(g & 1) * 8 + myslot], (uint32_t)((g - 1) >> 1) & 1u, &gflag[3]);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                failed = true;
                if (lane == 0) atomicOr(&gflag[3], 1);
            }
        }
        if (active && more != 2 && !failed) {                     // back to the factor in L2, for the final phase
            const float* cur = kP2P ? sbuf + (size_t)((g & 1) * T + myslot) * 8 * LD : mybuf;
            int ba, bb;
            rr_blocks(slot, 0, nbm1, ba, bb);
            for (int hc = 0; hc < 8; ++hc) {
                const int p = 4 * (hc < 4 ? ba : bb) + (hc & 3);
                if (p < rank) {
                    float* dst = X + (size_t)perm[p] * LD;
#pragma unroll
                    for (int t = 0; t < R; ++t) dst[lane + 32 * t] = cur[hc * LD + lane + 32 * t];
                }
            }
        }
    }
    cluster.sync();
    if (__ldcg(&gflag[3])) more = 2;                           // a bounded wait ran out in either phase
    if (more == 2 && gtid == 0) atomicOr(&info->flags, kFlagExchangeTimeout);
    const int not_converged = rank >= 2 && more != 0;          // stopped at the sweep limit while still rotating visibly
    // ---- eigenvalues = squared column norms (pivot-step order), scaled back; sort descending, stable ----
    for (int k0 = lwarp; k0 < n; k0 += 4 * WPC) {                  // every CTA forms all eigenvalues for its own tables;
        float a[4] = {0.f, 0.f, 0.f, 0.f};                          // four columns' loads in flight (each is an L2 round trip)
        float xv[4][R];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int k = k0 + u * WPC;
            const float* x = X + perm[k < rank ? k : 0] * LD;
#pragma unroll
            for (int t = 0; t < R; ++t) xv[u][t] = (k < rank) ? __ldcg(x + lane + 32 * t) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int t = 0; t < R; ++t) a[u] = fmaf(xv[u][t], xv[u][t], a[u]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) a[u] += __shfl_xor_sync(0xffffffffu, a[u], o);
            const int k = k0 + u * WPC;
            if (lane == 0 && k < n) lam[k] = a[u] * dmax;
        }
    }
    __syncthreads();
    for (int t = tid; t < n; t += NT) {
        const float mine = lam[t];
        int pos = 0;
        for (int i = 0; i < n; ++i) {
            const float o = lam[i];
            pos += (o > mine) || (o == mine && i < t);
        }
        order[pos] = t;
    }
    __syncthreads();
    if (tid == 0) {
        float delta = 0.f;
        if (do_shrink && delta_rank - 1 < n) delta = lam[order[delta_rank - 1]];
        sh_f[0] = delta;
        if (crank == 0) {
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
    }
    __syncthreads();
    const float delta = sh_f[0];
    const float back = sqrtf(dmax);     // columns of X are sigma_j u_j / sqrt(dmax)
    for (int t = tid; t < n; t += NT) {
        const float l = lam[order[t]];
        float f = 0.f, sp = 0.f;
        if (l > 0.f && t < keep) {
            const float kept = fmaxf(l - delta, 0.f);
            sp = sqrtf(kept);
            f = sqrtf(kept / l) * rsqrtf(l) * back;   // (sigma'/sigma) / sigma, for the unscaled column
        }
        fac[t] = f;
        if (t < n_sigma && crank == 0) sigma_out[t] = sp;
    }
    if (crank == 0)
        for (int j = n + tid; j < n_sigma; j += NT) sigma_out[j] = 0.f;
    __syncthreads();
    for (int e = gtid; e < n * keep; e += GT) {
        const int j = e / n, i = e - j * n;
        float v = 0.f;
        if (j < n) {
            const int k = order[j];
            if (k < rank) v = __ldcg(X + perm[k] * LD + i) * fac[j];
        }
        Ur[(size_t)i * ldu + j] = v;
    }
    if (Wsplit) {   // the same factors transposed and split for the tensor-core rebuild: [W_hi ; W_lo], zero padded
        for (int e = gtid; e < j_pad * ldw; e += GT) {
            const int j = e / ldw, i = e - j * ldw;
            float v = 0.f;
            if (j < keep && j < n && i < n) {
                const int k = order[j];
                if (k < rank) v = __ldcg(X + perm[k] * LD + i) * fac[j];
            }
            const float hi = __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xffffe000u);
            Wsplit[wsplit_row(j, j_pad, false) * ldw + i] = hi;
            Wsplit[wsplit_row(j, j_pad, true) * ldw + i] = v - hi;
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1)
k_eig_shrink(const float* __restrict__ K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* __restrict__ Ur,
             int ldu, float* __restrict__ sigma_out, int n_sigma, float* __restrict__ work, int use_smem, int max_sweeps,
             EigInfo* __restrict__ info, float* __restrict__ Wsplit, int ldw, int j_pad) {
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
    if (Wsplit) {
        for (int e = tid; e < j_pad * ldw; e += kThreads) {
            const int j = e / ldw, c = e - j * ldw;
            Wsplit[wsplit_row(j, j_pad, false) * ldw + c] = 0.f;
            Wsplit[wsplit_row(j, j_pad, true) * ldw + c] = 0.f;
        }
        __syncthreads();
        for (int e = tid; e < n * keep; e += kThreads) {
            const int j = e / n, i = e % n;
            if (j >= n || j >= j_pad) continue;
            const float v = X[(size_t)order[j] * ldx + i] * fac[j];
            const float hi = __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xffffe000u);
            Wsplit[wsplit_row(j, j_pad, false) * ldw + perm[i]] = hi;
            Wsplit[wsplit_row(j, j_pad, true) * ldw + perm[i]] = v - hi;
        }
    }
}

}  // namespace

cudaError_t launch_eig_shrink(const float* K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* Ur, int ldu,
                              float* sigma_out, int n_sigma, float* work, int max_sweeps, EigInfo* info, float* Wsplit, int ldw,
                              int j_pad, int variant, cudaStream_t st) {
    if (n <= 0 || n > 512) return cudaErrorInvalidValue;
    if (variant == 0 && n > 64) {   // cluster of 8 CTAs, Jacobi columns in distributed shared memory (n <= 64: one CTA is as fast)
        const int T = n <= 128 ? 2 : n <= 192 ? 3 : n <= 256 ? 4 : 8;
        const int LD = 64 * T;
        const size_t bytes = 3 * 512 * sizeof(float) + 3 * 512 * sizeof(int) + 32 + 32 * sizeof(uint64_t) + (size_t)T * 128 * sizeof(uint32_t) +
                             3 * (size_t)LD * sizeof(float) + (size_t)(T <= 3 ? 2 : 1) * T * 8 * LD * sizeof(float);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(8);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = bytes;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 8;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        cudaError_t e = cudaSuccess;
#define SAGE_EIG_DSM(TT, NTT)                                                                                                 \
    e = cudaFuncSetAttribute(k_eig_shrink_dsm<TT, NTT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);              \
    if (e == cudaSuccess)                                                                                                      \
        e = cudaLaunchKernelEx(&cfg, k_eig_shrink_dsm<TT, NTT>, K, ldk, n, do_shrink, delta_rank, keep, Ur, ldu, sigma_out, n_sigma, \
                               max_sweeps, info, Wsplit, ldw, j_pad, work);
        if (T == 2) { SAGE_EIG_DSM(2, 256) } else if (T == 3) { SAGE_EIG_DSM(3, 256) }
        else if (T == 4) { SAGE_EIG_DSM(4, 256) } else { SAGE_EIG_DSM(8, 256) }
#undef SAGE_EIG_DSM
        if (e == cudaSuccess) return cudaGetLastError();
        (void)cudaGetLastError();          // no cluster launch on this device: the kernels below serve every n <= 512
    }
    if (n <= kMaxFast) {
        const int T = (n + 63) / 64;
        const size_t aux_bytes = 3 * kMaxN * sizeof(float) + 3 * kMaxN * sizeof(int) + 32;
        const size_t bytes = (size_t)(64 * T) * (64 * T) * sizeof(float) + aux_bytes;
        cudaError_t e;
#define SAGE_EIG_FAST(TT)                                                                                              \
    e = cudaFuncSetAttribute(k_eig_shrink_fast<TT, 1024, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes); \
    if (e != cudaSuccess) return e;                                                                                    \
    k_eig_shrink_fast<TT, 1024, false><<<1, 1024, bytes, st>>>(K, ldk, n, do_shrink, delta_rank, keep, Ur, ldu, sigma_out,  \
                                                               n_sigma, max_sweeps, info, Wsplit, ldw, j_pad, work);
        if (T == 1) { SAGE_EIG_FAST(1) } else if (T == 2) { SAGE_EIG_FAST(2) } else { SAGE_EIG_FAST(3) }
#undef SAGE_EIG_FAST
        return cudaGetLastError();
    }
    {   // thread-block cluster, matrix in `work` (>= 512*512 + 64 floats when n > 256, else >= 256*256 + 64)
        const size_t bytes = 3 * 512 * sizeof(float) + 3 * 512 * sizeof(int) + 32;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(8);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = bytes;
        cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 8;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        cudaError_t e = n <= 256 ? cudaLaunchKernelEx(&cfg, k_eig_shrink_cluster<4>, K, ldk, n, do_shrink, delta_rank, keep, Ur, ldu,
                                                      sigma_out, n_sigma, max_sweeps, info, Wsplit, ldw, j_pad, work)
                                 : cudaLaunchKernelEx(&cfg, k_eig_shrink_cluster<8>, K, ldk, n, do_shrink, delta_rank, keep, Ur, ldu,
                                                      sigma_out, n_sigma, max_sweeps, info, Wsplit, ldw, j_pad, work);
        if (e == cudaSuccess) return cudaGetLastError();
        (void)cudaGetLastError();          // no cluster launch on this device: the one-CTA kernel below serves n <= 512
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
                                            max_sweeps, info, Wsplit, ldw, j_pad);
    return cudaGetLastError();
}

}  // namespace sage

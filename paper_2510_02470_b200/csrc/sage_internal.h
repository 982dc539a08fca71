// Internal declarations shared by the host orchestration and the kernel translation units.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sage.h"

namespace sage {

// Device-side flags accumulated in the handle's status word.
constexpr uint32_t kFlagNotConverged = 1u;
constexpr uint32_t kFlagNonFinite = 2u;

// Results of one eigen-solve, written by the eigen kernel and read by later kernels / stats.
struct EigInfo {
    double sum_delta;   // running sum of delta over shrinks
    float delta;        // delta of the most recent shrink
    int sweeps;         // sweeps of the most recent solve
    int max_sweeps;
    int rank;           // numerical rank of the most recent Gram matrix
    unsigned flags;     // kFlag*
    long long shrinks;  // shrinks applied so far
};

// ---- launchers (each enqueues on `st` and returns cudaGetLastError()) -----------------------------

// B[dst_row0 + i, 0:D] = float(rows[i, 0:D]) for i < n; columns D..pitch-1 of those rows are zeroed.
cudaError_t launch_append(const void* rows, sage_dtype_t dt, int64_t n, int64_t ld, int64_t D, float* B,
                          int64_t pitch, int dst_row0, cudaStream_t st);

// C[z][i][j] = sum over the z-th K-slice of A[i][k] * Bm[j][k]   (both operands contiguous along k).
// A is M x K (element type dt, pitch lda), Bm is N x K fp32 (pitch ldb). splits >= 1 slices of k.
cudaError_t launch_gemm_nt(const void* A, sage_dtype_t dt, int64_t lda, const float* Bm, int64_t ldb, int M, int N,
                           int64_t K, int splits, float* C, int64_t ldc, int64_t split_stride, cudaStream_t st);

// out[i][j] = sum_z parts[z][i][j] in ascending z with fp64 accumulation. (M x N, pitches ldp / ldo.)
cudaError_t launch_split_reduce(const float* parts, int splits, int64_t split_stride, int M, int N, int64_t ldp,
                                float* out, int64_t ldo, cudaStream_t st);

// out[j][d] = sum_{i<r} Ur[i*ldu + j] * Bsrc[i*pitch + d] for j < keep; rows keep..m_total-1 of out are zeroed.
cudaError_t launch_rebuild(const float* Ur, int ldu, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D, int r,
                           int keep, int m_total, cudaStream_t st);

// Eigen-decomposition of the symmetric positive semi-definite n x n matrix K (pitch ldk) and the
// Frequent-Directions shrink factors. do_shrink != 0: delta = lambda at 1-indexed rank delta_rank (0 if the
// matrix has fewer eigenvalues), keep = delta_rank-1 columns. do_shrink == 0: delta = 0, keep columns.
// Writes Ur[i*ldu + j] = U[i][j] * sqrt(max(1 - delta/lambda_j, 0)) for j < keep (eigenvalues descending),
// sigma_out[j] = sqrt(max(lambda_j - delta, 0)) for j < n_sigma, and updates *info.
// `work` is scratch of at least n*n floats (used when the matrix does not fit in shared memory).
cudaError_t launch_eig_shrink(const float* K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* Ur,
                              int ldu, float* sigma_out, int n_sigma, float* work, int max_sweeps, EigInfo* info,
                              cudaStream_t st);

// Z (n x ell, pitch ldz, already reduced over splits) -> zhat rows, ||z|| and per-block partial sums of zhat.
// zsum (ell doubles) += the partial sums in ascending block order (done by a second, single-block kernel).
cudaError_t launch_normalise(const float* Z, int64_t ldz, int64_t n, int ell, float* zhat, float* znorm,
                             float* partials, double* zsum, unsigned* flags, cudaStream_t st);

// u = zsum/||zsum|| (0 if zsum = 0); scores[i] = <zhat_i, u>.
cudaError_t launch_consensus_score(const double* zsum, const float* zhat, int64_t N, int ell, float* u, float* scores,
                                   cudaStream_t st);

// Top-k by (score desc, index asc). keys/vals scratch: see select.cu. Returns through idx (device).
cudaError_t select_scratch_bytes(int64_t N, size_t* bytes);
cudaError_t launch_select(const float* scores, int64_t N, int64_t k, int64_t* idx, void* scratch, cudaStream_t st);

// Hooks into the C ABI's bookkeeping for entry points defined outside api.cu.
void set_error_message(const char* msg);   // becomes the calling thread's sage_last_error()
void count_launches(int k);                // adds to sage_launch_count()

int launches_append();
int launches_gemm_nt(int splits);

}  // namespace sage

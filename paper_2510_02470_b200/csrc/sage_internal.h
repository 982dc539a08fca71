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
constexpr uint32_t kFlagExchangeTimeout = 8u;   // a bounded wait between thread blocks of the eigen-solve ran out (4: tensor-core waits)

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

// Structured last-layer rows: B[dst_row0 + i, :] = [vec_rowmajor(q_i feat_i^T) ; q_i] for i < n, with q n x C (pitch ldq) and feat
// n x F (pitch ldf) of element type dt; products in fp32 (exact for bf16 factors); columns C F + C .. pitch-1 zeroed. pitch
// must be a multiple of 4.
cudaError_t launch_append_outer(const void* q, int64_t ldq, const void* feat, int64_t ldf, sage_dtype_t dt, int64_t n, int C, int F,
                                float* B, int64_t pitch, int dst_row0, cudaStream_t st);

// Projection of structured rows from per-class planes: with T[c] = feat * S_c^T (n x ell, the sum of pp consecutive planes of
// `planes`, plane_stride floats apart, n x ell each with pitch ell) and S_c the columns [c F, c F + F) of the sketch,
//     Z[i][j] = sum_c q[i][c] * (T[c][i][j] + Sb[j][c]),      Sb = S + C F (the bias columns of the sketch, pitch lds).
// Classes are added in ascending order in fp32. q is n x C of element type dt (pitch ldq); Z is n x ell, pitch ell. biasT:
// scratch of C x ell floats (receives Sb transposed). Two launches.
cudaError_t launch_outer_combine(const void* q, int64_t ldq, sage_dtype_t dt, int C, const float* planes, int pp, int64_t plane_stride,
                                 const float* Sb, int64_t lds, float* biasT, int64_t n, int ell, float* Z, cudaStream_t st);

// C[z][i][j] = sum over the z-th K-slice of A[i][k] * Bm[j][k]   (both operands contiguous along k).
// A is M x K (element type dt, pitch lda), Bm is N x K fp32 (pitch ldb). splits >= 1 slices of k.
// class_F > 0 ("class slices", needs splits * class_F == K): A is M x class_F and slice z contracts ALL of it with the columns
// [z class_F, (z + 1) class_F) of Bm, so C[z] = A * Bm_z^T: the per-class projections of structured rows in one launch.
cudaError_t launch_gemm_nt(const void* A, sage_dtype_t dt, int64_t lda, const float* Bm, int64_t ldb, int M, int N,
                           int64_t K, int splits, float* C, int64_t ldc, int64_t split_stride, cudaStream_t st, int64_t class_F = 0);

// Tensor-core version of launch_gemm_nt (tcgen05 + TMA). Both operands have element type dt (fp32 operands are
// read as tf32) and must satisfy TMA's rules: 16-byte aligned base, pitch a multiple of 16 bytes.
// Returns cudaErrorNotSupported when they do not, so that the caller can take launch_gemm_nt instead.
// fold != 0: Bm holds two stacked operands, rows [0, N) and rows [n_pad, n_pad + N) with n_pad = N rounded up to
// 16, and C receives the sum of both products (a two-term representation of a more precise B); needs 2 n_pad <= 256.
// Without fold N <= 256. *err (device) is set to 1 if a bounded wait inside the kernel ran out.
// mt (1, 2 or 4) row tiles of 128 share each B tile inside one CTA; needs mt * (fold ? 2 n_pad : n_pad) <= 512.
cudaError_t launch_tc_gemm_nt(const void* A, sage_dtype_t dt, int64_t lda, const void* Bm, int64_t ldb, int M, int N, int fold,
                              int mt, int64_t K, int splits, float* C, int64_t ldc, int64_t split_stride, int* err, cudaStream_t st,
                              int64_t class_F = 0);   // class slices as in launch_gemm_nt; needs class_F * element size a multiple of 16

// fp32-faithful tensor-core C[z] = A_z * Bm_z^T for fp32 operands (three tf32 MMAs on hi/lo halves split in shared
// memory, accumulator drained into registers every few K tiles). Same alignment rules and return convention as
// launch_tc_gemm_nt; any N. When A == Bm (a Gram matrix) the diagonal tiles load one operand only and the 128 x 128
// tiles below the diagonal are NOT computed (their part of C is left untouched): reduce with mirror = 1.
// sym != 0 (only for a Gram matrix of at most 128 rows): two MMAs per K step instead of three; slice z then stores
// T_z = hi*hi^T + 2*hi*lo^T and the Gram matrix is sum_z (T_z + T_z^T)/2: see launch_gram_sym_reduce.
// sym == 2 (projection onto at most 64 sketch rows): Bm is the sketch already split by launch_split_tf32 (128 rows);
// one MMA per K step; C receives 2 * splits partial planes (split_stride apart) whose sum is A * S^T (M x N).
cudaError_t launch_tc_gemm_nt_x3(const float* A, int64_t lda, const float* Bm, int64_t ldb, int M, int N, int64_t K, int splits,
                                 float* C, int64_t ldc, int64_t split_stride, int sym, int* err, cudaStream_t st,
                                 int64_t class_F = 0);   // class slices as in launch_gemm_nt; needs class_F a multiple of 4
// The symmetric form of launch_tc_gemm_nt_x3 (sym = 1) for a buffer whose last n_new rows have not been appended: rows
// 0 .. old_rows - 1 come from Bold (fp32, pitch elements; one more row must be readable), the n_new rows after them are
// bfloat16 rows at src (pitch ld_src). old_rows + n_new <= 128, old_rows + 1 a multiple of 8. Same output as the appended form.
cudaError_t launch_tc_gram_direct(const float* Bold, int64_t pitch, int old_rows, const void* src, int64_t ld_src, int n_new, int64_t D,
                                  int splits, float* C, int64_t ldc, int64_t split_stride, int* err, cudaStream_t st);
cudaError_t launch_gram_sym_reduce(const float* parts, int splits, int64_t stride, int r, int64_t ldp, float* out, int64_t ldo,
                                   cudaStream_t st);

// Tensor-core rebuild: Bdst[j][d] = sum_{i<r} W[j][i] * Bsrc[i][d] for j < keep, d < pitch (fp32-faithful, see
// tc_rebuild.cu). Wsplit holds W already split for tf32: rows [0, j_pad) = W rounded to 11 significant bits, rows
// [j_pad, 2 j_pad) = the remainder; row pitch ldw floats, columns i >= r and rows j >= keep zero (rows the eigen-solve
// does not write, up to the next multiple of 128, are read by the MMA and must be finite: the caller zeroes the array
// once). Needs j_pad a multiple of 16 with keep <= j_pad <= 256 (one launch per 128 output rows) and r <= 512;
// returns cudaErrorNotSupported otherwise.
cudaError_t launch_tc_rebuild(const float* Wsplit, int ldw, int j_pad, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D, int r,
                              int keep, int* err, cudaStream_t st);
// The same rebuild for a buffer whose last n_new rows have not been appended: rows 0 .. r - n_new - 1 come from Bsrc (one
// more row must be readable), the n_new rows after them are bfloat16 rows at src (pitch ld_src, D columns). Needs r <= 128,
// r and r - n_new + 1 multiples of 32, and the factors resident (at most 64 output rows); cudaErrorNotSupported otherwise.
cudaError_t launch_tc_rebuild_direct(const float* Wsplit, int ldw, int j_pad, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D,
                                     int r, int keep, const void* src, int64_t ld_src, int n_new, int* err, cudaStream_t st);

// hi[i][0:cols] = bf16(src[i][0:cols]) (round to nearest even) for i < rows; when lo != nullptr also
// lo[i][:] = bf16(src - float(hi)), so that hi + lo carries 16 significant bits of src.
cudaError_t launch_to_bf16(const float* src, int64_t lds, int rows, int64_t cols, __nv_bfloat16* hi, __nv_bfloat16* lo, int64_t ldd,
                           cudaStream_t st);

// out[i][j] = sum_z parts[z][i][j] in ascending z with fp64 accumulation. (M x N, pitches ldp / ldo.)
// out (128 rows, pitch ldo): row j = src row j rounded to 11 significant bits, row 64 + j = the remainder, for
// j < rows <= 64; the other rows are left as they are (zero from allocation).
cudaError_t launch_split_tf32(const float* src, int64_t lds, int rows, int64_t cols, float* out, int64_t ldo, cudaStream_t st);

cudaError_t launch_split_reduce(const float* parts, int splits, int64_t split_stride, int M, int N, int64_t ldp,
                                float* out, int64_t ldo, cudaStream_t st, int mirror = 0);

// out[j][d] = sum_{i<r} Ur[i*ldu + j] * Bsrc[i*pitch + d] for j < keep; rows keep..m_total-1 of out are zeroed.
cudaError_t launch_rebuild(const float* Ur, int ldu, const float* Bsrc, float* Bdst, int64_t pitch, int64_t D, int r,
                           int keep, int m_total, cudaStream_t st);

// Eigen-decomposition of the symmetric positive semi-definite n x n matrix K (pitch ldk) and the
// Frequent-Directions shrink factors. do_shrink != 0: delta = lambda at 1-indexed rank delta_rank (0 if the
// matrix has fewer eigenvalues), keep = delta_rank-1 columns. do_shrink == 0: delta = 0, keep columns.
// Writes Ur[i*ldu + j] = U[i][j] * sqrt(max(1 - delta/lambda_j, 0)) for j < keep (eigenvalues descending),
// sigma_out[j] = sqrt(max(lambda_j - delta, 0)) for j < n_sigma, and updates *info.
// `work` is scratch of at least 256*256 + 64 floats (512*512 + 64 when n > 256), used when the matrix does not fit in
// shared memory.
// Wsplit != nullptr: also writes the factors transposed and split for launch_tc_rebuild, rows [0, j_pad) =
// W rounded to 11 significant bits and rows [j_pad, 2 j_pad) = the remainders, W[j][i] = Ur[i][j], pitch ldw >= n,
// zero outside j < keep, i < n.
cudaError_t launch_eig_shrink(const float* K, int ldk, int n, int do_shrink, int delta_rank, int keep, float* Ur,
                              int ldu, float* sigma_out, int n_sigma, float* work, int max_sweeps, EigInfo* info,
                              float* Wsplit, int ldw, int j_pad, int variant, cudaStream_t st);

// Z (n x ell, pitch ldz; planes > 1: that many partial planes plane_stride floats apart, summed in plane order with fp64
// accumulation) -> zhat rows, ||z|| and per-block partial sums of zhat. zsum (ell doubles, may be null) += the partial sums in
// a fixed order (done by a second, single-block kernel).
cudaError_t launch_normalise(const float* Z, int planes, int64_t plane_stride, int64_t ldz, int64_t n, int ell, float* zhat,
                             float* znorm, float* partials, double* zsum, unsigned* flags, cudaStream_t st);

// u = zsum/||zsum|| (0 if zsum = 0); scores[i] = <zhat_i, u>.
cudaError_t launch_consensus_score(const double* zsum, const float* zhat, int64_t N, int ell, float* u, float* scores,
                                   cudaStream_t st);

// Class-balanced variant. U (C x ell) receives the unit centroids, counts (C) the class sizes, scores (N) the
// per-class agreement scores; labels outside [0, C) score 0.
cudaError_t launch_class_scores(const float* zhat, const int* labels, int64_t N, int ell, int C, float* U, int* counts, float* scores,
                                cudaStream_t st);
cudaError_t launch_class_count(const int* labels, int64_t N, int C, int* counts, cudaStream_t st);
// out[offs[c] + r] = the r-th example of class c in the order of `sorted` (all N examples, best first), r < kc[c].
cudaError_t launch_class_pick(const int64_t* sorted, const int* labels, int64_t N, int C, const long long* kc, const long long* offs,
                              int64_t* out, cudaStream_t st);

// Top-k by (score desc, index asc). keys/vals scratch: see select.cu. Returns through idx (device).
cudaError_t select_scratch_bytes(int64_t N, size_t* bytes);
cudaError_t launch_select(const float* scores, int64_t N, int64_t k, int64_t* idx, void* scratch, cudaStream_t st);

// Hooks into the C ABI's bookkeeping for entry points defined outside api.cu.
void set_error_message(const char* msg);   // becomes the calling thread's sage_last_error()
void count_launches(int k);                // adds to sage_launch_count()

int launches_append();
int launches_gemm_nt(int splits);

}  // namespace sage

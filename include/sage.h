/*
 * sage.h -- C ABI of the B200 (sm_100a) implementation of SAGE's two-pass selection hot path.
 *
 * The path (paper: Method section and Algorithm 1):
 *   pass 1  stream per-example gradient rows into a Frequent-Directions sketch
 *           (Algorithm 1, Phase I; Method, first paragraph),
 *   freeze  the ell x D sketch S (Algorithm 1, the freeze step),
 *   pass 2  z_i = S g_i, zhat_i = z_i/||z_i||, consensus u, agreement score alpha_i = <zhat_i, u>
 *           (Method, paragraph on two-pass scoring; Algorithm 1, Phase II),
 *   select  the top-k examples by alpha (Algorithm 1, the top-k step).
 *
 * Conventions shared by every entry point
 *   - Every function returns a sage_status_t; nothing throws or aborts. Out-parameters are written only
 *     on SAGE_OK. sage_last_error() returns a thread-local, human-readable message for the last failure.
 *   - Pointers named rows / scores / idx are DEVICE pointers owned by the caller unless the parameter
 *     says "host". The library never frees them and does not use them after the stream work it
 *     enqueued has finished.
 *   - Rows are row-major with a pitch `ld` counted in elements (ld >= D). Element type is the handle's
 *     row dtype (float32, or bfloat16 stored as 16-bit words).
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Work is
 *     enqueued asynchronously on it unless the entry point documents a synchronisation.
 *   - A handle belongs to one device and one host thread at a time. Calls on one handle must be issued
 *     on one stream (or on streams the caller has ordered).
 *   - Rows are consumed strictly in the order given: the sketch depends on row order.
 *   - There is no CPU fallback: without a usable CUDA device every compute entry point fails with
 *     SAGE_ERR_CUDA.
 */
#ifndef SAGE_B200_H_
#define SAGE_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sage_fd sage_fd_t; /* opaque, library-owned */

typedef enum {
    SAGE_OK = 0,
    SAGE_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, ld < D, keep_rate not finite, ... */
    SAGE_ERR_BAD_STATE = 2,     /* call order violates the state machine below */
    SAGE_ERR_ALLOC = 3,         /* device or host allocation failed */
    SAGE_ERR_CUDA = 4,          /* a CUDA runtime call failed (see sage_last_error) */
    SAGE_ERR_UNSUPPORTED = 5,   /* size outside the supported range */
    SAGE_ERR_NOT_CONVERGED = 6, /* the eigen-solver hit its sweep limit (results were still produced) */
    SAGE_ERR_NONFINITE = 7      /* a NaN/Inf was met in the input rows (such rows score 0) */
} sage_status_t;

typedef enum { SAGE_F32 = 0, SAGE_BF16 = 1 } sage_dtype_t;

/* State machine of a handle:
 *   create -> SKETCHING --update*--> SKETCHING --finalize--> FROZEN
 *   FROZEN --score_begin--> SCORING --score_chunk*--> SCORING --score_end--> FROZEN
 *   sage_score() = score_begin + one score_chunk + score_end.  sage_fd_reset() returns to SKETCHING.
 */

/* Frequent-Directions sketch state for rows of dimension D with sketch size ell (Method, first
 * paragraph; Algorithm 1, the initialisation step). The library keeps a buffer of 2*ell rows in fp32: rows
 * are appended into free rows and the buffer is shrunk when all 2*ell rows are in use.
 *   out        receives the handle (host pointer).
 *   D          row dimension, 1 <= D.
 *   ell        sketch size, 2 <= ell <= 256.
 *   row_dtype  element type of every rows pointer later given to this handle.
 *   device     CUDA device ordinal; all later calls must be made with pointers of this device.
 * Allocates about 2 * (2*ell) * D * 4 bytes of device memory. Synchronous. */
sage_status_t sage_fd_create(sage_fd_t** out, int64_t D, int32_t ell, sage_dtype_t row_dtype, int device);

/* Releases everything the handle owns (synchronises the device first). NULL is allowed. */
void sage_fd_destroy(sage_fd_t* h);

/* Forget all rows and return to SKETCHING, keeping the allocations. Synchronous. */
sage_status_t sage_fd_reset(sage_fd_t* h);

/* Algorithm 1, Phase I, for n rows: append each row to the buffer; whenever the buffer is full,
 * factor it (SVD through the eigen-decomposition of the 2ell x 2ell Gram matrix), set
 * delta = sigma_ell^2, Sigma'_jj = sqrt(max(sigma_j^2 - delta, 0)) and rebuild S <- Sigma' V^T
 * (Method, first paragraph). ell-1 rows survive a shrink, so after the first 2*ell rows a shrink
 * happens every ell+1 rows.
 *   rows  device, n x ld elements of the handle's dtype; n == 0 is a no-op. The library only reads them, by work
 *         enqueued on cuda_stream (or ordered before what the caller enqueues there next): they may be changed by
 *         later work on that stream, not before it. Rows that do not fill the buffer are copied into it; a shrink
 *         whose new rows all come from this call may read them in place instead (option 9 of sage_fd_set_option).
 * Asynchronous on the stream: the shrink schedule depends only on counts, so no device->host
 * synchronisation happens here. Device-side problems are reported by sage_fd_finalize. */
sage_status_t sage_fd_update(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, void* cuda_stream);

/* Makes cuda_stream wait (on the device, without blocking the host) for everything this handle has enqueued on streams
 * of its own: the merged form of pass 1 (option 6) runs its sketches on internal streams, and sage_fd_update only makes
 * the caller's stream wait until the rows have been copied out of `rows`. sage_fd_finalize joins by itself; this call
 * is for callers that want the handle's work ordered before other work of theirs (a benchmark that times what it
 * enqueues next). The paper has no counterpart. */
sage_status_t sage_fd_join(sage_fd_t* h, void* cuda_stream);

/* Algorithm 1, the freeze step: orthogonalise what the buffer holds, apply the shrink only if
 * more than ell rows are in use (so N <= ell is exact), keep the first ell rows as S.
 * Synchronises the stream once and returns SAGE_ERR_NOT_CONVERGED / SAGE_ERR_NONFINITE if the device
 * recorded such an event during pass 1 (the sketch is still usable). */
sage_status_t sage_fd_finalize(sage_fd_t* h, void* cuda_stream);

/* Borrowed pointers to the frozen sketch: S is ell x D fp32 on the device with pitch *pitch
 * elements, sigma holds its ell row norms sigma'_j (device, fp32). Valid until reset/destroy.
 * Requires FROZEN or later. Any out-pointer may be NULL. */
sage_status_t sage_fd_sketch(const sage_fd_t* h, const float** S, int64_t* pitch, const float** sigma);

/* Replace the frozen sketch by caller data (ell x D fp32, device, pitch ld): scoring with a sketch
 * computed elsewhere. Moves the handle to FROZEN. Asynchronous on the stream. */
sage_status_t sage_fd_load_sketch(sage_fd_t* h, const float* S, int64_t ld, void* cuda_stream);

/* Algorithm 1, Phase II on n resident rows: z_i = S g_i, zhat_i, u, alpha_i = <zhat_i, u>.
 *   scores  device, n floats. Rows whose projection is exactly zero (or non-finite) score 0; if the
 *           consensus is zero every score is 0.
 * Asynchronous on the stream. */
sage_status_t sage_score(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, float* scores, void* cuda_stream);

/* Streamed form of Phase II for row sets that are not resident: announce the total row count, feed
 * chunks (each read once), then finish. row_offset is the index of the chunk's first row in
 * [0, N_total); chunks must tile [0, N_total) without overlap and be given in ascending order.
 * The library keeps the N_total x ell normalised projections between chunk and end, because the
 * consensus direction is only known once every row has been seen.
 * sage_score / sage_score_end return as soon as the work is enqueued, so they cannot report what the device meets
 * while it runs: after synchronising the stream, sage_fd_stats().device_flags tells whether a row was non-finite
 * (bit 1; such rows score 0) or a kernel gave up a bounded wait (bits 2, 3; scores invalid). The synchronous
 * sage_select_from_host checks those words itself and returns SAGE_ERR_NONFINITE / SAGE_ERR_CUDA. */
sage_status_t sage_score_begin(sage_fd_t* h, int64_t N_total, void* cuda_stream);
sage_status_t sage_score_chunk(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, int64_t row_offset,
                               void* cuda_stream);
sage_status_t sage_score_end(sage_fd_t* h, float* scores, void* cuda_stream);

/* Structured last-layer rows (Method, the definition of the per-example gradient; Limitations, on last-layer gradients).
 * For a softmax head with C classes on F features the per-example gradient with respect to (weights, bias) is the outer
 * product q_i (x) [h_i ; 1], q_i = softmax - onehot(label): row i is [vec_rowmajor(q_i h_i^T) (C x F) ; q_i (C)], D = C F + C.
 * These entry points take the two factors instead of the row, so the N x D matrix is never formed, neither in the caller's
 * memory nor in the library's: pass 1 writes each row straight into the sketch buffer (products in fp32, exact for bfloat16
 * factors); pass 2 uses z_i = S g_i = sum_c q_ic (S_c h_i + b_c), with S_c the columns [c F, c F + F) of the sketch and b_c
 * column c of its last C columns: one launch of the projection kernel of the dense path contracts the features with every
 * class block (the classes take the place of its K slices), a second kernel folds the per-class planes with the factors
 * q_ic. The planes of a sub-chunk of rows are scratch of the library's own (C x ell floats per row, at most 1 GiB at a time).
 * Results are those of sage_fd_update / sage_score_chunk / sage_score on the materialised rows up to rounding. Both kinds of
 * call may be mixed on one handle.
 *   q     device, n x ldq elements of the handle's row dtype, C values used per row (ldq >= C).
 *   feat  device, n x ldf elements of the handle's row dtype, F values used per row (ldf >= F).
 * C F + C must equal the handle's D. Stream semantics, state machine and errors are those of the dense calls. */
sage_status_t sage_fd_update_outer(sage_fd_t* h, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n, int32_t C, int32_t F,
                                   void* cuda_stream);
sage_status_t sage_score_chunk_outer(sage_fd_t* h, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n, int32_t C,
                                     int32_t F, int64_t row_offset, void* cuda_stream);
sage_status_t sage_score_outer(sage_fd_t* h, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n, int32_t C, int32_t F,
                               float* scores, void* cuda_stream);

/* Strict-memory form of Phase II (Method, the complexity paragraph and the abstract: memory O(ell D), independent of N).
 * The default keeps the N x ell normalised projections between the scoring pass and its end, because alpha_i needs the
 * consensus u, which needs every row. With option 8 set to 1 nothing of size N is kept: sage_score_begin / _chunk / _end
 * then only form u (sage_score_end accepts scores == NULL), holding the normalised projections of one sub-chunk at a
 * time, and a third pass over the rows produces the scores:
 *   sage_score_apply  alpha_i = <zhat_i, u> for the n given rows (any subset, any order, any chunking) against the u of
 *                     the finished pass; scores: device, n floats. The rows are projected again, so this pass costs as much
 *                     as the scoring pass; results equal the default's up to the rounding order of the consensus sum.
 * Requires a pass finished in this mode; sage_score_intermediates and sage_score_classes need the default mode.
 * Asynchronous on the stream. */
sage_status_t sage_score_apply(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, float* scores, void* cuda_stream);

/* Borrowed device pointers to the last scoring pass's intermediates (for checks of the lemma in
 * "Energy preservation"): zhat N x ell fp32, znorm N fp32 (||z_i||), u ell fp32. Any may be NULL. */
sage_status_t sage_score_intermediates(const sage_fd_t* h, const float** zhat, const float** znorm, const float** u);

/* Number of indices sage_select returns for N scores: floor(keep_rate*N + 0.5) clamped to [0, N]. */
int64_t sage_select_count(int64_t N, double keep_rate);

/* Algorithm 1, the top-k step: the k = sage_select_count(N, keep_rate) largest scores,
 * ordered by (score descending, index ascending); equal scores go to the smaller index. NaN scores
 * rank below every number.
 *   scores  device, N floats.         idx    device, capacity >= k int64 values.
 *   k_out   host, receives k (may be NULL).
 * Allocates and frees O(N) scratch on the device; asynchronous on the stream apart from that. */
sage_status_t sage_select(const float* scores, int64_t N, double keep_rate, int64_t* idx, int64_t* k_out,
                          void* cuda_stream);

/* Class-balanced variant (Algorithm 1, the class-balanced branch; section on agreement scoring and selection): after a
 * finished scoring pass on this handle (sage_score or sage_score_end over N rows), replace the consensus u by the
 * per-class unit centroids u_c = zbar_c / ||zbar_c||, zbar_c the mean of zhat_i over the examples of class c (u_c = 0
 * when that mean is zero), and score every example against the centroid of its own class.
 *   labels       device, N int32 class ids of the rows of that pass, in the same order; ids outside
 *                [0, num_classes) take no part: such examples score 0.
 *   num_classes  1 .. 65535.
 *   scores       device, N floats.
 * Asynchronous on the stream (the first call with a larger num_classes allocates and synchronises). */
sage_status_t sage_score_classes(sage_fd_t* h, const int32_t* labels, int32_t num_classes, float* scores, void* cuda_stream);

/* Borrowed device pointers to the result of the last sage_score_classes: U num_classes x ell fp32 unit centroids,
 * counts num_classes int32 class sizes. Any out-pointer may be NULL. */
sage_status_t sage_score_class_centroids(const sage_fd_t* h, const float** U, const int32_t** counts, int32_t* num_classes);

/* Algorithm 1, the per-class top-k step of the class-balanced variant (the k_c sum to k). The paper fixes only the sum; here
 * k = sage_select_count(N_valid, keep_rate) with N_valid the number of examples whose label lies in [0, num_classes),
 * and k_c is proportional to the class size n_c with largest-remainder rounding: k_c = floor(k n_c / N_valid), the
 * k - sum floor(.) classes with the largest remainders (ties: smaller class id) get one more. Inside a class the order
 * is (score descending, index ascending); idx lists the picks of class 0, then class 1, ...
 *   scores, labels  device, N floats / N int32.      idx  device, capacity >= k int64.
 *   k_per_class     host, num_classes values (may be NULL).      k_out  host (may be NULL).
 * Synchronises the stream (class sizes are read back to derive k_c); allocates O(N) scratch from the stream-ordered pool. */
sage_status_t sage_select_classes(const float* scores, const int32_t* labels, int64_t N, int32_t num_classes, double keep_rate,
                                  int64_t* idx, int64_t* k_per_class, int64_t* k_out, void* cuda_stream);

/* Selection without any allocation (the paper has no counterpart; this is a packaging variant of
 * sage_select with identical results). For callers that cannot allocate device memory at call time:
 * code running inside a loop whose memory was handed out once at start-up by a pool it does not own,
 * processes that leave no free device memory, threads that must not block on the allocator. The O(N)
 * scratch that sage_select obtains per call lives here in a fixed array inside the library image
 * (about 4.06 MiB, held by every device that loads the library until the process exits), so
 *   N <= 262,144 scores; larger N returns SAGE_ERR_UNSUPPORTED with a message naming the limit.
 * Arguments, ordering, tie rule and k_out are those of sage_select; it runs on the CURRENT device.
 * The first call on each device looks up the array's device address (a synchronous query, no
 * allocation); make that first call before starting any stream capture. All calls on a device share the
 * one array: nothing in it needs clearing between calls (every word is written before it is read), but
 * two calls whose kernels can overlap on the GPU (different streams, no ordering) race on it and give
 * undefined results. Calls neither allocate nor free: no cudaMalloc, cudaFree or stream-ordered pool. */
sage_status_t sage_select_static(const float* scores, int64_t N, double keep_rate, int64_t* idx, int64_t* k_out,
                                 void* cuda_stream);

/* The whole path for rows that live in HOST memory (pinned memory gives overlap of copies and
 * kernels): streams the rows to the device in chunks for pass 1, freezes, streams them again for
 * pass 2, selects, and copies scores (N floats, may be NULL) and indices back to the host.
 * Synchronous. chunk_rows <= 0 picks a default. */
sage_status_t sage_select_from_host(const void* rows_host, int64_t N, int64_t D, int64_t ld, int32_t ell,
                                    sage_dtype_t row_dtype, double keep_rate, int64_t chunk_rows, int device,
                                    float* scores_host, int64_t* idx_host, int64_t* k_out);

/* Checkpoint of the sketch (Method, first paragraph and the complexity paragraph: the whole state of pass 1 is the buffer
 * and a few counters, O(ell D) whatever N is). sage_fd_export writes it to HOST memory, sage_fd_import restores it into
 * a handle created with the same D, ell and row type; a stream of rows can so be sketched in several sessions, or a frozen
 * sketch kept for later scoring. Allowed while sketching (between updates) and when frozen, not during a scoring pass.
 * A restored handle continues exactly where the exported one stood: feeding the remaining rows gives the same sketch,
 * bit for bit, as the uninterrupted run. The merged form (option 6) is exported with all its sketches.
 *   sage_fd_export_size  bytes the checkpoint needs now (it grows and shrinks with the rows in the buffer).
 *   sage_fd_export       dst_host: host memory of `capacity` bytes; *written (may be NULL) receives the size. Synchronises
 *                        the device.
 *   sage_fd_import       src_host / bytes: a checkpoint; the handle is reset first and takes the checkpoint's options 1, 6
 *                        and 7. SAGE_ERR_INVALID_ARG (handle untouched) if the data is not a checkpoint of this shape.
 *                        Synchronises the device. */
sage_status_t sage_fd_export_size(const sage_fd_t* h, size_t* bytes);
sage_status_t sage_fd_export(sage_fd_t* h, void* dst_host, size_t capacity, size_t* written);
sage_status_t sage_fd_import(sage_fd_t* h, const void* src_host, size_t bytes, void* cuda_stream);

typedef struct {
    int64_t rows_seen;      /* rows given to sage_fd_update since create/reset */
    int64_t shrinks;        /* shrinks applied (including the one in finalize, if any) */
    double sum_delta;       /* sum of delta over shrinks: an upper bound on ||G^T G - S^T S||_2 */
    int32_t last_sweeps;    /* Jacobi sweeps of the most recent eigen-solve */
    int32_t max_sweeps;     /* largest sweep count seen */
    int32_t last_rank;      /* numerical rank found by the most recent factorisation */
    uint32_t device_flags;  /* bit 0: eigen-solver not converged, bit 1: non-finite input seen,
                               bit 2: a tensor-core kernel gave up a bounded wait (results invalid),
                               bit 3: the cluster eigen-solve gave up a bounded wait (results invalid) */
    int64_t kernel_launches;/* kernels this handle has launched since create/reset */
    int64_t tensor_core_launches; /* how many of them were tensor-core (tcgen05) kernels: Gram, rebuild, projection */
    int64_t rows_in_place;  /* rows of sage_fd_update that whole shrink cycles read where the caller held them (option 9) */
} sage_stats_t;

/* Synchronises the device and reads the counters back. */
sage_status_t sage_fd_stats(sage_fd_t* h, sage_stats_t* out);

/* Options. Before the first update: key 1 = delta rank (which singular value, 1-indexed, defines
 * delta; default ell), key 2 = maximum Jacobi sweeps (default 30). At any time: key 3 = bit mask of
 * kernel classes to time with CUDA events on the launching stream (see sage_fd_profile; default 0); key 4 =
 * 1 (default) to use the tensor-core kernels wherever the operands meet their alignment rules (16-byte
 * aligned base, row pitch a multiple of 16 bytes), 0 to use the CUDA-core kernels everywhere; key 5 = which
 * kernels run the eigen-solve: 0 (default) a cluster of 8 thread blocks with the Jacobi columns in distributed
 * shared memory, 1 the single-block kernel (buffers of up to 192 rows) or the cluster kernel that keeps the
 * matrix in L2. Same algorithm either way; results agree up to rounding order.
 * Before the first update: key 6 = P, the number of sketches of the merged form of pass 1 (1 .. 64, default 1 = the
 * paper's single sequential sketch); key 7 = rows per dealt block (default ell + 1). With P > 1 the row stream is cut into
 * blocks of that many consecutive rows, block b (counted from the first row ever given, across calls) goes to sketch
 * b mod P, and each sketch is a sequential Frequent-Directions sketch of its rows in stream order; sage_fd_finalize
 * freezes every sketch and merges them pairwise (sketch a absorbs sketch a + s for s = 1, 2, 4, ...: the rows a + s
 * kept are appended to a, which is frozen again). Frequent-Directions sketches are mergeable, so the result obeys
 * the same error bound as the sequential sketch, but it is a different sketch. The P chains of Gram / eigen-solve /
 * rebuild run on P streams of the library's own and overlap on the device; device memory grows P-fold. (CUDA maps streams onto
 * a limited number of hardware queues, 8 unless the environment variable CUDA_DEVICE_MAX_CONNECTIONS says otherwise when CUDA
 * is initialised; streams that share a queue do not overlap, so with P > 8 set it to 32 before the process touches CUDA.)
 * Outside a scoring pass: key 8 = 1 for the strict-memory form of Phase II (see sage_score_apply), 0 (default) to keep the
 * N x ell normalised projections.
 * At any time: key 9 = 1 (default) lets a shrink cycle whose ell + 1 new rows all lie in one sage_fd_update call read them
 * where the caller holds them instead of appending them to the buffer first (bfloat16 rows, ell = 32 or 64, tensor-core
 * kernels, the paper's single sketch: the Gram and rebuild kernels take rows 0 .. ell - 2 from the buffer and convert the
 * caller's rows on the way into the operand tiles; same arithmetic and the same results as the appended form); rows that do
 * not fill a cycle are appended as before. 0: always append. Either way `rows` must stay unchanged until the work enqueued by
 * the call has run (stream order on cuda_stream takes care of that for work enqueued there afterwards). */
sage_status_t sage_fd_set_option(sage_fd_t* h, int key, double value);

/* Per-kernel device time of this handle's launches since the previous call, for the classes selected
 * with option 3. Class indices: 0 append, 1 Gram, 2 Gram split reduction, 3 eigen-solve + shrink,
 * 4 rebuild, 5 projection, 6 projection split reduction, 7 normalise + consensus partials, 8 consensus
 * + score. ms[c] is the summed event time in milliseconds and launches[c] the number of timed launches.
 * capacity is the length of both host arrays (>= 9). Synchronises the device. */
sage_status_t sage_fd_profile(sage_fd_t* h, double* ms, int64_t* launches, int32_t capacity);

const char* sage_status_string(sage_status_t s);
const char* sage_last_error(void);
/* Library version string, e.g. for logs. */
const char* sage_version(void);
/* Number of kernels this library has launched in the calling process so far (all handles and
 * sage_select together); a benchmark takes the difference around its timed region. */
int64_t sage_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SAGE_B200_H_ */

// Host orchestration behind the C ABI: state machine, buffer management and the launch sequences of
// pass 1 (append -> Gram -> eigen/shrink -> rebuild), freeze, pass 2 (project -> normalise -> consensus
// -> score) and selection. No device->host synchronisation happens inside sage_fd_update.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "sage_internal.h"

using namespace sage;

namespace {

thread_local char g_err[512] = "";
std::atomic<long long> g_launches{0};

void set_err(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

#define CU_TRY(expr)                                                                       \
    do {                                                                                   \
        cudaError_t e__ = (expr);                                                          \
        if (e__ != cudaSuccess) {                                                          \
            set_err("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e__), __FILE__, __LINE__); \
            return e__ == cudaErrorMemoryAllocation ? SAGE_ERR_ALLOC : SAGE_ERR_CUDA;      \
        }                                                                                  \
    } while (0)

#define ST_TRY(expr)                       \
    do {                                   \
        sage_status_t s__ = (expr);        \
        if (s__ != SAGE_OK) return s__;    \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

enum State { SKETCHING = 0, FROZEN = 1, SCORING = 2 };

// Kernel classes for the optional per-kernel timing (sage_fd_profile).
enum KClass { K_APPEND = 0, K_GRAM, K_GRAM_REDUCE, K_EIG, K_REBUILD, K_PROJECT, K_PROJECT_REDUCE, K_NORMALISE, K_SCORE, K_NCLASS };

struct Prof {
    unsigned mask = 0;
    std::vector<cudaEvent_t> pool;
    struct Pending { int cls; cudaEvent_t a, b; };
    std::vector<Pending> pending;
    double ms[K_NCLASS] = {};
    int64_t n[K_NCLASS] = {};
    // Adds the pairs whose second event has completed to the sums and recycles their events.
    void fold_finished() {
        size_t keep = 0;
        for (size_t i = 0; i < pending.size(); ++i) {
            Pending& p = pending[i];
            float t = 0.f;
            if (cudaEventQuery(p.b) == cudaSuccess && cudaEventElapsedTime(&t, p.a, p.b) == cudaSuccess) {
                ms[p.cls] += t;
                n[p.cls] += 1;
                pool.push_back(p.a);
                pool.push_back(p.b);
            } else {
                pending[keep++] = p;
            }
        }
        pending.resize(keep);
    }
    cudaEvent_t get() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
};

size_t elem_size(sage_dtype_t dt) { return dt == SAGE_F32 ? 4 : 2; }

// Stream-ordered scratch of the selection entry points comes from a pool of the library's own whose memory stays
// cached across synchronisations (the device's default pool gives its memory back at every synchronisation, and
// getting it again costs milliseconds). One pool per device, created on first use, kept until the process exits.
cudaError_t scratch_alloc(void** p, size_t bytes, cudaStream_t st) {
    static cudaMemPool_t pools[64] = {};
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaMallocAsync(p, bytes, st);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!pools[dev]) {
            cudaMemPoolProps props = {};
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            cudaMemPool_t pool = nullptr;
            e = cudaMemPoolCreate(&pool, &props);
            if (e != cudaSuccess) return e;
            unsigned long long keep = ~0ull;
            e = cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
            if (e != cudaSuccess) return e;
            pools[dev] = pool;
        }
    }
    return cudaMallocFromPoolAsync(p, bytes, pools[dev], st);
}

}  // namespace

struct sage_fd {
    int64_t D = 0;
    int ell = 0, m = 0;
    sage_dtype_t dtype = SAGE_F32;
    int device = 0;
    int64_t pitch = 0;             // floats per buffer row (multiple of 32)
    float* B[2] = {nullptr, nullptr};
    int cur = 0;
    int fill = 0;
    int64_t rows_seen = 0;
    State state = SKETCHING;
    int delta_rank = 0, max_sweeps = 30;
    // Gram / eigen workspaces
    float* gram_parts = nullptr;   // split-K partials of the Gram matrix (gram_part_floats floats)
    size_t gram_part_floats = 0;   // at least kGramPartFloats; 16 slices of m x m for buffers of more than 256 rows
    float* Wsplit = nullptr;       // rebuild factors split for the tensor cores: wsplit_ld rows x wsplit_ld floats
    int wsplit_ld = 256;           // 256 (buffers of up to 256 rows) or 512
    float* Kmat = nullptr;         // m x m
    float* Ur = nullptr;           // m x m
    float* eig_work = nullptr;     // m x m
    float* sigma = nullptr;        // ell
    EigInfo* info = nullptr;       // device
    // scoring
    int64_t N_total = 0, next_row = 0, zcap = 0;
    float* zhat = nullptr;
    float* znorm = nullptr;
    float* zwork = nullptr;
    size_t zwork_bytes = 0;
    float* partials = nullptr;
    size_t partials_bytes = 0;
    double* zsum = nullptr;
    float* u = nullptr;
    bool scored = false;           // a scoring pass over N_total rows has finished: zhat holds their normalised projections
    float* bias_t = nullptr;       // structured rows: the bias block of the sketch transposed (C x ell)
    size_t bias_t_bytes = 0;
    float* zred = nullptr;         // projections of a sub-chunk summed over their K slices (when there are many slices)
    size_t zred_bytes = 0;
    bool direct_rows = true;       // option 9: shrink cycles read bfloat16 rows from the caller's memory where the shapes allow it
    bool strict = false;           // option 8: no N x ell store; scores come from a third pass (sage_score_apply)
    bool scored_strict = false;    // the finished pass ran in strict-memory mode: u is known, zhat is not kept
    float* class_U = nullptr;      // class-balanced variant: unit centroids (class_cap x ell) and class sizes
    int* class_counts = nullptr;
    int class_cap = 0, class_num = 0;
    __nv_bfloat16* P16 = nullptr;  // frozen sketch in bf16 (bf16 handles: tensor-core projection operand); with p16_fold
                                   // rows [0, ell) hold bf16(S) and rows [n_pad, n_pad + ell) hold bf16(S - bf16(S))
    int p16_fold = 0, p16_npad = 0;
    float* S32split = nullptr;     // frozen sketch split into tf32 hi / lo rows (fp32 handles with ell <= 64): 128 x pitch
    cudaStream_t side = nullptr;   // appends of the next shrink cycle run here, beside the eigen-solve of the current one
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    int* tc_err = nullptr;         // set by a tensor-core kernel whose bounded wait ran out
    bool use_tc = true;            // option 4: tensor-core kernels where their alignment rules hold
    int eig_variant = 0;           // option 5: 0 cluster eigen-solve in distributed shared memory, 1 the one-CTA / L2 kernels
    int64_t launches = 0;
    int64_t tc_launches = 0;       // how many of them were tensor-core (tcgen05) kernels
    int64_t rows_in_place = 0;     // rows that shrink cycles read where the caller held them (never appended)
    Prof prof;
    // Merged form of pass 1 (option 6): P sketches over interleaved row blocks. This handle is sketch 0; sketches
    // 1..P-1 are handles of their own that only sketch (no scoring state). With P > 1 every sketch runs its
    // Gram / eigen-solve / rebuild chain on a stream of its own, so the chains of different sketches overlap.
    int P = 1;
    int64_t block = 0;             // rows per dealt block
    int64_t dealt = 0;             // rows dealt so far (all sketches)
    std::vector<sage_fd*> kids;
    bool sketch_only = false;      // a sub-sketch: no scoring buffers
    cudaStream_t chain = nullptr;  // P > 1: the stream of this sketch's chain (P == 1: the caller's stream)
    bool app_pending = false;      // appends on `side` that the chain stream has not been made to wait for yet
    int64_t in_epoch = -1;         // the update call whose entry event `side` already waits for
    cudaEvent_t ev_in = nullptr;   // the caller's stream at the entry of an update call (sketch 0 only)
    cudaEvent_t ev_rows = nullptr; // after the last append of the current update call
    cudaEvent_t ev_done = nullptr; // end of the chain stream (joins)
    bool used = false;             // fed during the current update call
};

namespace {

void count(sage_fd* h, int k) {
    if (h) h->launches += k;
    g_launches.fetch_add(k, std::memory_order_relaxed);
}

// Runs one launcher; when the class is selected for timing, brackets it with events on the same stream.
template <typename F>
cudaError_t timed(sage_fd* h, int cls, int nlaunch, cudaStream_t st, F&& f) {
    const bool on = h && (h->prof.mask >> cls) & 1u;
    cudaEvent_t a = nullptr, b = nullptr;
    if (on) {
        a = h->prof.get();
        b = h->prof.get();
        cudaEventRecord(a, st);
    }
    const cudaError_t e = f();
    if (on) {
        cudaEventRecord(b, st);
        h->prof.pending.push_back({cls, a, b});
        if (h->prof.pending.size() >= 65536) h->prof.fold_finished();   // never grows without bound if nobody asks for the profile
    }
    count(h, nlaunch);
    return e;
}

constexpr size_t kGramPartFloats = (size_t)148 * 128 * 128;   // >= 296 tiles of 64 x 64

int gram_tiles(int r) {
    const int t = (r + 63) / 64;
    return t * t;
}

int pick_splits(int tiles, int64_t K, int64_t min_k) {
    int64_t s = 296 / (tiles > 0 ? tiles : 1);
    const int64_t cap = (K + min_k - 1) / min_k;
    if (s > cap) s = cap;
    if (s < 1) s = 1;
    return (int)s;
}

// Split count for a grid of `tiles` CTAs per split on 148 SMs: the count (each slice keeping at least
// min_k of the contraction) that wastes the least of the last wave; ties go to fewer splits.
int pick_splits_waves(int tiles, int64_t K, int64_t min_k, int max_splits) {
    int64_t cap = K / min_k;
    if (cap > max_splits) cap = max_splits;
    if (cap < 1) cap = 1;
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= (int)cap; ++s) {
        const int64_t ctas = (int64_t)tiles * s;
        const double eff = (double)ctas / (double)(((ctas + 147) / 148) * 148);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
    }
    return best;
}

// After the sketch is frozen: the bf16 copy the tensor-core projection reads (bf16 handles only).
sage_status_t enqueue_freeze_aux(sage_fd* h, cudaStream_t st) {
    if (h->dtype == SAGE_F32 && h->S32split)
        CU_TRY(timed(h, K_APPEND, 1, st, [&] { return launch_split_tf32(h->B[h->cur], h->pitch, h->ell, h->pitch, h->S32split, h->pitch, st); }));
    if (h->dtype == SAGE_BF16 && h->P16)
        CU_TRY(timed(h, K_APPEND, 1, st, [&] {
            return launch_to_bf16(h->B[h->cur], h->pitch, h->ell, h->pitch, h->P16,
                                  h->p16_fold ? h->P16 + (size_t)h->p16_npad * h->pitch : nullptr, h->pitch, st);
        }));
    return SAGE_OK;
}

// Gram of the first r buffer rows -> Kmat (r x r, pitch m).
sage_status_t enqueue_gram(sage_fd* h, int r, cudaStream_t st) {
    float* Bc = h->B[h->cur];
    if (h->use_tc) {
        // tensor cores: 128 x 128 output tiles, as many K slices as fill the SMs (each at least 256 columns)
        const int t = (r + 127) / 128;
        const int ldc = ((r + 3) / 4) * 4;
        const int64_t stride = (int64_t)r * ldc;
        const int sym = r <= 128 ? 1 : 0;    // one diagonal tile: one wide MMA per K step, transpose added in the reduction
        int cap = (int)(h->gram_part_floats / (size_t)stride);
        if (cap > 148) cap = 148;
        const int splits = pick_splits_waves(t * (t + 1) / 2, h->D, 256, cap);   // only the tiles on and above the diagonal run
        cudaError_t e = timed(h, K_GRAM, 1, st, [&] {
            return launch_tc_gemm_nt_x3(Bc, h->pitch, Bc, h->pitch, r, r, h->D, splits, h->gram_parts, ldc, stride, sym, h->tc_err, st);
        });
        if (e == cudaSuccess) {
            h->tc_launches += 1;
            if (sym)
                CU_TRY(timed(h, K_GRAM_REDUCE, 1, st, [&] { return launch_gram_sym_reduce(h->gram_parts, splits, stride, r, ldc, h->Kmat, h->m, st); }));
            else   // sums the K slices and fills the tiles below the diagonal from their mirror images
                CU_TRY(timed(h, K_GRAM_REDUCE, 1, st, [&] { return launch_split_reduce(h->gram_parts, splits, stride, r, r, ldc, h->Kmat, h->m, st, 1); }));
            return SAGE_OK;
        }
        if (e != cudaErrorNotSupported) CU_TRY(e);
        count(h, -1);
    }
    // splits * tiles <= 296, and the partials are stored compactly (pitch r_pad), so they always fit in
    // the 296 tiles of 64 x 64 floats allocated at create.
    const int splits = pick_splits(gram_tiles(r), h->D, 256);
    const int r_pad = ((r + 63) / 64) * 64;
    const int64_t stride = (int64_t)r_pad * r_pad;
    if (splits == 1) {
        CU_TRY(timed(h, K_GRAM, 1, st, [&] { return launch_gemm_nt(Bc, SAGE_F32, h->pitch, Bc, h->pitch, r, r, h->D, 1, h->Kmat, h->m, 0, st); }));
    } else {
        CU_TRY(timed(h, K_GRAM, 1, st, [&] {
            return launch_gemm_nt(Bc, SAGE_F32, h->pitch, Bc, h->pitch, r, r, h->D, splits, h->gram_parts, r_pad, stride, st);
        }));
        CU_TRY(timed(h, K_GRAM_REDUCE, 1, st, [&] { return launch_split_reduce(h->gram_parts, splits, stride, r, r, r_pad, h->Kmat, h->m, st); }));
    }
    return SAGE_OK;
}

// Factor the first r rows and rebuild `keep` rows into the other buffer; rows keep..zero_to-1 are zeroed.
sage_status_t enqueue_factor(sage_fd* h, int r, int do_shrink, int keep, int zero_to, cudaStream_t st) {
    ST_TRY(enqueue_gram(h, r, st));
    CU_TRY(cudaEventRecord(h->ev_fork, st));       // from here on HBM is idle until the rebuild: see sage_fd_update
    const int j_pad = ((keep + 15) / 16) * 16;
    const bool tc_rebuild = h->use_tc && h->Wsplit && keep > 0 && j_pad <= h->wsplit_ld / 2 && r <= h->wsplit_ld;
    CU_TRY(timed(h, K_EIG, 1, st, [&] {
        return launch_eig_shrink(h->Kmat, h->m, r, do_shrink, h->delta_rank, keep, h->Ur, h->m, h->sigma, h->ell, h->eig_work,
                                 h->max_sweeps, h->info, tc_rebuild ? h->Wsplit : nullptr, h->wsplit_ld, j_pad, h->eig_variant, st);
    }));
    const int m_total = zero_to > keep ? zero_to : keep;
    bool done = false;
    if (tc_rebuild) {
        const int parts = j_pad > 128 ? 2 : 1;                            // launches: 128 output rows each
        cudaError_t e = timed(h, K_REBUILD, parts, st, [&] {
            return launch_tc_rebuild(h->Wsplit, h->wsplit_ld, j_pad, h->B[h->cur], h->B[1 - h->cur], h->pitch, h->D, r, keep, h->tc_err, st);
        });
        if (e == cudaSuccess) {
            done = true;
            h->tc_launches += parts;
            if (m_total > keep)
                CU_TRY(cudaMemsetAsync(h->B[1 - h->cur] + (size_t)keep * h->pitch, 0, (size_t)(m_total - keep) * h->pitch * sizeof(float), st));
        } else if (e != cudaErrorNotSupported) {
            CU_TRY(e);
        } else {
            count(h, -parts);
        }
    }
    if (!done)
        CU_TRY(timed(h, K_REBUILD, 1, st, [&] {
            return launch_rebuild(h->Ur, h->m, h->B[h->cur], h->B[1 - h->cur], h->pitch, h->D, r, keep, m_total, st);
        }));
    h->cur = 1 - h->cur;
    h->fill = keep;
    return SAGE_OK;
}

sage_status_t ensure(float** p, size_t* have, size_t need) {
    if (*have >= need) return SAGE_OK;
    if (*p) CU_TRY(cudaFree(*p));
    *p = nullptr;
    *have = 0;
    CU_TRY(cudaMalloc(reinterpret_cast<void**>(p), need));
    *have = need;
    return SAGE_OK;
}

sage_status_t check_handle(const sage_fd* h) {
    if (!h) {
        set_err("null handle");
        return SAGE_ERR_INVALID_ARG;
    }
    return SAGE_OK;
}

}  // namespace

namespace sage {
void set_error_message(const char* msg) { set_err("%s", msg); }
void count_launches(int k) { count(nullptr, k); }
}  // namespace sage

extern "C" {

const char* sage_status_string(sage_status_t s) {
    switch (s) {
        case SAGE_OK: return "ok";
        case SAGE_ERR_INVALID_ARG: return "invalid argument";
        case SAGE_ERR_BAD_STATE: return "call not allowed in this state";
        case SAGE_ERR_ALLOC: return "allocation failed";
        case SAGE_ERR_CUDA: return "CUDA error";
        case SAGE_ERR_UNSUPPORTED: return "unsupported size";
        case SAGE_ERR_NOT_CONVERGED: return "eigen-solver did not converge";
        case SAGE_ERR_NONFINITE: return "non-finite input";
    }
    return "unknown status";
}

const char* sage_last_error(void) { return g_err; }
const char* sage_version(void) { return "sage-b200 0.1 (sm_100a)"; }
int64_t sage_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int64_t sage_select_count(int64_t N, double keep_rate) {
    if (N <= 0 || !(keep_rate == keep_rate)) return 0;
    double k = std::floor(keep_rate * (double)N + 0.5);
    if (k < 0.0) k = 0.0;
    if (k > (double)N) k = (double)N;
    return (int64_t)k;
}

static sage_status_t create_handle(sage_fd_t** out, int64_t D, int32_t ell, sage_dtype_t row_dtype, int device, bool sketch_only) {
    if (!out || D < 1 || (row_dtype != SAGE_F32 && row_dtype != SAGE_BF16) || device < 0) {
        set_err("sage_fd_create: bad argument (out=%p D=%lld dtype=%d device=%d)", (void*)out, (long long)D, (int)row_dtype, device);
        return SAGE_ERR_INVALID_ARG;
    }
    if (ell < 2 || ell > 256) {
        set_err("sage_fd_create: ell=%d outside [2, 256]", ell);
        return ell < 2 ? SAGE_ERR_INVALID_ARG : SAGE_ERR_UNSUPPORTED;
    }
    DeviceGuard g(device);
    if (!g.ok) {
        set_err("sage_fd_create: cannot select CUDA device %d: %s", device, cudaGetErrorString(cudaGetLastError()));
        return SAGE_ERR_CUDA;
    }
    sage_fd* h = new (std::nothrow) sage_fd();
    if (!h) return SAGE_ERR_ALLOC;
    h->D = D;
    h->ell = ell;
    h->m = 2 * ell;
    h->dtype = row_dtype;
    h->device = device;
    h->delta_rank = ell;
    h->sketch_only = sketch_only;
    h->block = ell + 1;
    h->pitch = ((D + 31) / 32) * 32;
    const size_t bbytes = (size_t)h->m * h->pitch * sizeof(float);
    const size_t mm = (size_t)h->m * h->m * sizeof(float);
    auto fail = [&](cudaError_t e, const char* what) {
        set_err("sage_fd_create: %s failed: %s", what, cudaGetErrorString(e));
        sage_fd_destroy(h);
        return e == cudaErrorMemoryAllocation ? SAGE_ERR_ALLOC : SAGE_ERR_CUDA;
    };
    cudaError_t e;
    for (int i = 0; i < 2; ++i)
        if ((e = cudaMalloc((void**)&h->B[i], bbytes)) != cudaSuccess) return fail(e, "cudaMalloc(buffer)");
    h->gram_part_floats = kGramPartFloats;
    if ((size_t)16 * h->m * h->m > h->gram_part_floats) h->gram_part_floats = (size_t)16 * h->m * h->m;
    if ((e = cudaMalloc((void**)&h->gram_parts, h->gram_part_floats * sizeof(float))) != cudaSuccess) return fail(e, "cudaMalloc(gram)");
    h->wsplit_ld = h->m <= 256 ? 256 : 512;
    if ((e = cudaMalloc((void**)&h->Wsplit, (size_t)h->wsplit_ld * h->wsplit_ld * sizeof(float))) != cudaSuccess)
        return fail(e, "cudaMalloc(W)");
    // rows of the split factors beyond the ones an eigen-solve writes are read by the rebuild's MMA (and ignored by its
    // epilogue): they must hold finite values
    if ((e = cudaMemset(h->Wsplit, 0, (size_t)h->wsplit_ld * h->wsplit_ld * sizeof(float))) != cudaSuccess) return fail(e, "cudaMemset");
    if ((e = cudaMalloc((void**)&h->Kmat, mm)) != cudaSuccess) return fail(e, "cudaMalloc(K)");
    if ((e = cudaMalloc((void**)&h->Ur, mm)) != cudaSuccess) return fail(e, "cudaMalloc(U)");
    // eigen workspace: the matrix padded to 256 or 512 rows/columns plus a few flag words
    const size_t ew = h->m > 256 ? (size_t)512 * 512 : (size_t)256 * 256;
    if ((e = cudaMalloc((void**)&h->eig_work, (ew + 64) * sizeof(float))) != cudaSuccess)
        return fail(e, "cudaMalloc(eig)");
    if ((e = cudaMalloc((void**)&h->sigma, ell * sizeof(float))) != cudaSuccess) return fail(e, "cudaMalloc(sigma)");
    if ((e = cudaMalloc((void**)&h->info, sizeof(EigInfo))) != cudaSuccess) return fail(e, "cudaMalloc(info)");
    if (!sketch_only) {
        if ((e = cudaMalloc((void**)&h->zsum, 256 * sizeof(double))) != cudaSuccess) return fail(e, "cudaMalloc(zsum)");
        if ((e = cudaMalloc((void**)&h->u, 256 * sizeof(float))) != cudaSuccess) return fail(e, "cudaMalloc(u)");
    }
    if ((e = cudaMalloc((void**)&h->tc_err, sizeof(int))) != cudaSuccess) return fail(e, "cudaMalloc(err)");
    if ((e = cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking)) != cudaSuccess) return fail(e, "cudaStreamCreate");
    for (cudaEvent_t* ev : {&h->ev_fork, &h->ev_join, &h->ev_in, &h->ev_rows, &h->ev_done})
        if ((e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return fail(e, "cudaEventCreate");
    if ((e = cudaMemset(h->tc_err, 0, sizeof(int))) != cudaSuccess) return fail(e, "cudaMemset");
    if (row_dtype == SAGE_BF16 && !sketch_only) {
        // Two-term bf16 sketch (16 significant bits) for short rows, where the rounding errors of a one-term
        // sketch would average over too few terms; long rows take the one-term sketch (half the operand traffic).
        h->p16_npad = ((ell + 15) / 16) * 16;
        h->p16_fold = (2 * h->p16_npad <= 256 && D < 16384) ? 1 : 0;
        const size_t prow = h->p16_fold ? 2 * (size_t)h->p16_npad : (size_t)ell;
        if ((e = cudaMalloc((void**)&h->P16, prow * h->pitch * sizeof(__nv_bfloat16))) != cudaSuccess) return fail(e, "cudaMalloc(P16)");
        if ((e = cudaMemset(h->P16, 0, prow * h->pitch * sizeof(__nv_bfloat16))) != cudaSuccess) return fail(e, "cudaMemset");
    }
    if (row_dtype == SAGE_F32 && ell <= 64 && !sketch_only) {
        // fp32 rows, small sketch: the projection multiplies the rows against the sketch pre-split into tf32 hi / lo rows
        if ((e = cudaMalloc((void**)&h->S32split, (size_t)128 * h->pitch * sizeof(float))) != cudaSuccess) return fail(e, "cudaMalloc(S split)");
        if ((e = cudaMemset(h->S32split, 0, (size_t)128 * h->pitch * sizeof(float))) != cudaSuccess) return fail(e, "cudaMemset");
    }
    if ((e = cudaMemset(h->info, 0, sizeof(EigInfo))) != cudaSuccess) return fail(e, "cudaMemset");
    if ((e = cudaMemset(h->sigma, 0, ell * sizeof(float))) != cudaSuccess) return fail(e, "cudaMemset");
    if ((e = cudaDeviceSynchronize()) != cudaSuccess) return fail(e, "cudaDeviceSynchronize");
    *out = h;
    return SAGE_OK;
}

sage_status_t sage_fd_create(sage_fd_t** out, int64_t D, int32_t ell, sage_dtype_t row_dtype, int device) {
    return create_handle(out, D, ell, row_dtype, device, false);
}

void sage_fd_destroy(sage_fd_t* h) {
    if (!h) return;
    DeviceGuard g(h->device);
    cudaDeviceSynchronize();
    for (sage_fd* k : h->kids) sage_fd_destroy(k);
    h->kids.clear();
    if (h->chain) cudaStreamDestroy(h->chain);
    for (cudaEvent_t ev : {h->ev_in, h->ev_rows, h->ev_done})
        if (ev) cudaEventDestroy(ev);
    cudaFree(h->B[0]);
    cudaFree(h->B[1]);
    cudaFree(h->gram_parts);
    cudaFree(h->Wsplit);
    cudaFree(h->Kmat);
    cudaFree(h->Ur);
    cudaFree(h->eig_work);
    cudaFree(h->sigma);
    cudaFree(h->info);
    cudaFree(h->zhat);
    cudaFree(h->znorm);
    cudaFree(h->zwork);
    cudaFree(h->partials);
    cudaFree(h->zred);
    cudaFree(h->bias_t);
    cudaFree(h->zsum);
    cudaFree(h->u);
    cudaFree(h->class_U);
    cudaFree(h->class_counts);
    cudaFree(h->P16);
    cudaFree(h->S32split);
    cudaFree(h->tc_err);
    if (h->side) cudaStreamDestroy(h->side);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    for (auto& p : h->prof.pending) {
        cudaEventDestroy(p.a);
        cudaEventDestroy(p.b);
    }
    for (cudaEvent_t e : h->prof.pool) cudaEventDestroy(e);
    delete h;
}

sage_status_t sage_fd_reset(sage_fd_t* h) {
    ST_TRY(check_handle(h));
    DeviceGuard g(h->device);
    CU_TRY(cudaDeviceSynchronize());
    CU_TRY(cudaMemset(h->info, 0, sizeof(EigInfo)));
    CU_TRY(cudaMemset(h->sigma, 0, h->ell * sizeof(float)));
    CU_TRY(cudaMemset(h->tc_err, 0, sizeof(int)));
    h->fill = 0;
    h->rows_seen = 0;
    h->dealt = 0;
    h->cur = 0;
    h->scored = false;
    h->scored_strict = false;
    h->state = SKETCHING;
    h->launches = 0;
    h->tc_launches = 0;
    h->rows_in_place = 0;
    h->app_pending = false;
    h->in_epoch = -1;
    for (sage_fd* k : h->kids) ST_TRY(sage_fd_reset(k));
    return SAGE_OK;
}

sage_status_t sage_fd_set_option(sage_fd_t* h, int key, double value) {
    ST_TRY(check_handle(h));
    if (key == 3) {                          // per-kernel event timing mask: allowed at any time
        h->prof.mask = (unsigned)value & ((1u << K_NCLASS) - 1u);
        for (sage_fd* k : h->kids) k->prof.mask = h->prof.mask;
        return SAGE_OK;
    }
    if (key == 4) {                          // 0: CUDA-core kernels only, 1: tensor-core kernels where possible
        h->use_tc = value != 0.0;
        for (sage_fd* k : h->kids) k->use_tc = h->use_tc;
        return SAGE_OK;
    }
    if (key == 9) {                          // 1: whole shrink cycles read their new rows in place (no append), 0: always append
        h->direct_rows = value != 0.0;
        for (sage_fd* k : h->kids) k->direct_rows = h->direct_rows;
        return SAGE_OK;
    }
    if (key == 8) {                          // strict-memory scoring: no N x ell store, scores from a third pass
        if (h->state == SCORING) {
            set_err("sage_fd_set_option: a scoring pass is open");
            return SAGE_ERR_BAD_STATE;
        }
        h->strict = value != 0.0;
        return SAGE_OK;
    }
    if (key == 5) {                          // eigen-solve kernel family (same algorithm, same results up to rounding order)
        h->eig_variant = value != 0.0 ? 1 : 0;
        for (sage_fd* k : h->kids) k->eig_variant = h->eig_variant;
        return SAGE_OK;
    }
    if (h->dealt != 0 || h->state != SKETCHING) {
        set_err("sage_fd_set_option: options must be set before the first update");
        return SAGE_ERR_BAD_STATE;
    }
    const int v = (int)value;
    if (key == 1 && v >= 2 && v <= h->m - 1) {
        h->delta_rank = v;
        for (sage_fd* k : h->kids) k->delta_rank = v;
        return SAGE_OK;
    }
    if (key == 2 && v >= 1 && v <= 1000) {
        h->max_sweeps = v;
        for (sage_fd* k : h->kids) k->max_sweeps = v;
        return SAGE_OK;
    }
    if (key == 6 && v >= 1 && v <= 64 && (double)v == value) {      // number of sketches of the merged form of pass 1
        if (v != h->P) {
            DeviceGuard g(h->device);
            cudaDeviceSynchronize();
            for (sage_fd* k : h->kids) sage_fd_destroy(k);
            h->kids.clear();
            if (v == 1 && h->chain) {
                cudaStreamDestroy(h->chain);
                h->chain = nullptr;
            }
        }
        h->P = v;
        return SAGE_OK;
    }
    if (key == 7 && v >= 1 && v <= (1 << 20) && (double)v == value) { // rows per dealt block of the merged form
        h->block = v;
        return SAGE_OK;
    }
    set_err("sage_fd_set_option: unknown key %d or value %g out of range", key, value);
    return SAGE_ERR_INVALID_ARG;
}

// ---- one sketch: feed rows, factor, freeze ------------------------------------------------------------------
//
// Streams of a sketch: every append runs on its `side` stream, the Gram / eigen-solve / rebuild chain on `chain` (the
// caller's stream for a single sketch, the sketch's own stream in the merged form). An append writes rows
// [fill, fill + take) of the current buffer copy and touches nothing the eigen-solve or the rebuild of the previous
// shrink reads or writes (the rebuild fills rows [0, keep) of the same copy), so appends run beside the eigen-solve,
// which leaves HBM idle. The side stream starts after the Gram kernel of the previous shrink (running beside it only
// takes bandwidth from it; that also puts it after the rebuild before, which read the copy now being filled) and
// the chain waits for the appends before the next Gram kernel.

static sage_status_t sketch_join_appends(sage_fd* s, cudaStream_t chain) {
    if (s->app_pending) {
        CU_TRY(cudaEventRecord(s->ev_join, s->side));
        CU_TRY(cudaStreamWaitEvent(chain, s->ev_join, 0));
        s->app_pending = false;
    }
    return SAGE_OK;
}

static sage_status_t sketch_factor(sage_fd* s, int r, int do_shrink, int keep, int zero_to, cudaStream_t chain) {
    ST_TRY(sketch_join_appends(s, chain));
    ST_TRY(enqueue_factor(s, r, do_shrink, keep, zero_to, chain));
    CU_TRY(cudaStreamWaitEvent(s->side, s->ev_fork, 0));
    return SAGE_OK;
}

// A whole shrink cycle whose new rows (m - fill of them, bfloat16, pitch ld) are read where the caller holds them instead of
// being appended first: the Gram and rebuild kernels take rows 0 .. fill - 1 from the buffer and the rest from `rows`
// (same arithmetic, same results as the appended form). *done = false (and nothing enqueued) when the kernels do not
// support the shape: the caller then appends as usual.
static sage_status_t sketch_factor_direct(sage_fd* s, const void* rows, int64_t ld, cudaStream_t chain, bool* done) {
    *done = false;
    const int r = s->m, old_rows = s->fill, n_new = s->m - s->fill, keep = s->delta_rank - 1;
    const int j_pad = ((keep + 15) / 16) * 16;
    if (!s->use_tc || !s->Wsplit || r > 128 || keep != old_rows || keep <= 0 || (old_rows + 1) % 32 != 0 || r % 32 != 0 ||
        j_pad > s->wsplit_ld / 2 || r > s->wsplit_ld || j_pad > 64 || (reinterpret_cast<uintptr_t>(rows) & 15u) || ((ld * 2) & 15))
        return SAGE_OK;
    ST_TRY(sketch_join_appends(s, chain));
    const int ldc = ((r + 3) / 4) * 4;
    const int64_t stride = (int64_t)r * ldc;
    int cap = (int)(s->gram_part_floats / (size_t)stride);
    if (cap > 148) cap = 148;
    const int splits = pick_splits_waves(1, s->D, 256, cap);
    float* Bc = s->B[s->cur];
    cudaError_t e = timed(s, K_GRAM, 1, chain, [&] {
        return launch_tc_gram_direct(Bc, s->pitch, old_rows, rows, ld, n_new, s->D, splits, s->gram_parts, ldc, stride, s->tc_err, chain);
    });
    if (e == cudaErrorNotSupported) {
        count(s, -1);
        return SAGE_OK;
    }
    CU_TRY(e);
    s->tc_launches += 1;
    CU_TRY(timed(s, K_GRAM_REDUCE, 1, chain, [&] { return launch_gram_sym_reduce(s->gram_parts, splits, stride, r, ldc, s->Kmat, s->m, chain); }));
    CU_TRY(cudaEventRecord(s->ev_fork, chain));
    CU_TRY(timed(s, K_EIG, 1, chain, [&] {
        return launch_eig_shrink(s->Kmat, s->m, r, 1, s->delta_rank, keep, s->Ur, s->m, s->sigma, s->ell, s->eig_work, s->max_sweeps, s->info,
                                 s->Wsplit, s->wsplit_ld, j_pad, s->eig_variant, chain);
    }));
    e = timed(s, K_REBUILD, 1, chain, [&] {
        return launch_tc_rebuild_direct(s->Wsplit, s->wsplit_ld, j_pad, Bc, s->B[1 - s->cur], s->pitch, s->D, r, keep, rows, ld, n_new, s->tc_err,
                                        chain);
    });
    if (e == cudaErrorNotSupported) {
        // the factors exist already: bring the rows into the buffer after all and rebuild from there
        count(s, -1);
        CU_TRY(timed(s, K_APPEND, 1, chain, [&] { return launch_append(rows, SAGE_BF16, n_new, ld, s->D, Bc, s->pitch, old_rows, chain); }));
        CU_TRY(timed(s, K_REBUILD, 1, chain, [&] {
            return launch_tc_rebuild(s->Wsplit, s->wsplit_ld, j_pad, Bc, s->B[1 - s->cur], s->pitch, s->D, r, keep, s->tc_err, chain);
        }));
    } else {
        CU_TRY(e);
    }
    s->tc_launches += 1;
    s->cur = 1 - s->cur;
    s->fill = keep;
    CU_TRY(cudaStreamWaitEvent(s->side, s->ev_fork, 0));
    *done = true;
    return SAGE_OK;
}

// Where the rows of an update come from: a dense matrix (rows, pitch ld), or the two factors of structured last-layer
// rows (q: pitch ldq, C values per row; feat: pitch ldf, F values per row), expanded on the fly.
struct RowSrc {
    const void* rows = nullptr;
    int64_t ld = 0;
    const void* q = nullptr;
    const void* feat = nullptr;
    int64_t ldq = 0, ldf = 0;
    int C = 0, F = 0;
    sage_dtype_t dt = SAGE_F32;
    bool outer() const { return q != nullptr; }
    RowSrc advanced(int64_t k) const {       // the same source, k rows further on
        RowSrc r = *this;
        const size_t es = elem_size(dt);
        if (rows) r.rows = static_cast<const char*>(rows) + (size_t)k * ld * es;
        if (q) r.q = static_cast<const char*>(q) + (size_t)k * ldq * es;
        if (feat) r.feat = static_cast<const char*>(feat) + (size_t)k * ldf * es;
        return r;
    }
    cudaError_t append(int64_t take, int64_t D, float* B, int64_t pitch, int dst_row0, cudaStream_t st) const {
        if (outer()) return launch_append_outer(q, ldq, feat, ldf, dt, take, C, F, B, pitch, dst_row0, st);
        return launch_append(rows, dt, take, ld, D, B, pitch, dst_row0, st);
    }
};

// Appends n rows of type dt and shrinks whenever the buffer fills. e_in (may be null): the event after which `rows`
// are valid; epoch identifies the update call it belongs to. on_chain: appends run on the chain stream itself (used
// where the rows to append are produced by that stream). Leaves s->ev_rows recorded after the last append.
static sage_status_t sketch_feed(sage_fd* s, RowSrc src, int64_t n, cudaStream_t chain, cudaEvent_t e_in, int64_t epoch, bool on_chain) {
    // merged form: the appends run on the chain stream too (the chains of the other sketches fill the device while this
    // one waits, and half as many streams keep every chain on a hardware queue of its own)
    const bool from_caller = !on_chain;
    if (s->chain && chain == s->chain) on_chain = true;
    cudaStream_t as = on_chain ? chain : s->side;
    if (from_caller && e_in && s->in_epoch != epoch) {
        CU_TRY(cudaStreamWaitEvent(as, e_in, 0));
        s->in_epoch = epoch;
    }
    bool appended = false;
    auto body = [&]() -> sage_status_t {
        while (n > 0) {
            const int64_t room = s->m - s->fill;
            const int64_t take = n < room ? n : room;
            // a whole cycle's rows at hand, bfloat16, on the caller's own stream: no append, the kernels read them in place
            if (s->direct_rows && from_caller && !s->chain && !src.outer() && src.dt == SAGE_BF16 && take == room && s->fill > 0 &&
                s->fill == s->delta_rank - 1) {
                bool direct = false;
                ST_TRY(sketch_factor_direct(s, src.rows, src.ld, chain, &direct));
                if (direct) {
                    s->rows_in_place += take;
                    s->rows_seen += take;
                    src = src.advanced(take);
                    n -= take;
                    continue;
                }
            }
            CU_TRY(timed(s, K_APPEND, 1, as, [&] { return src.append(take, s->D, s->B[s->cur], s->pitch, s->fill, as); }));
            appended = true;
            if (!on_chain) s->app_pending = true;
            s->fill += (int)take;
            s->rows_seen += take;
            src = src.advanced(take);
            n -= take;
            if (s->fill == s->m) ST_TRY(sketch_factor(s, s->m, 1, s->delta_rank - 1, 0, chain));
        }
        return SAGE_OK;
    };
    const sage_status_t rc = body();
    if (appended && from_caller) {   // also on the error path: the caller's stream must not run ahead of appends that read `rows`
        const cudaError_t e = cudaEventRecord(s->ev_rows, as);
        if (rc == SAGE_OK) CU_TRY(e);
        s->used = true;
    }
    return rc;
}

// The freeze of one sketch: orthogonalise what the buffer holds, shrink only if more than ell rows are in use.
// Afterwards s->fill is the number of rows kept (at most ell) and rows up to ell are zero.
static sage_status_t sketch_freeze(sage_fd* s, cudaStream_t chain) {
    ST_TRY(sketch_join_appends(s, chain));
    const int r = s->fill;
    if (r == 0) {
        CU_TRY(cudaMemsetAsync(s->B[s->cur], 0, (size_t)s->ell * s->pitch * sizeof(float), chain));
        CU_TRY(cudaMemsetAsync(s->sigma, 0, s->ell * sizeof(float), chain));
    } else {
        const int do_shrink = r > s->ell ? 1 : 0;
        const int keep = do_shrink ? s->delta_rank - 1 : (r < s->ell ? r : s->ell);
        ST_TRY(sketch_factor(s, r, do_shrink, keep < s->ell ? keep : s->ell, s->ell, chain));
    }
    return SAGE_OK;
}

static sage_fd* sketch_at(sage_fd* h, int p) { return p == 0 ? h : h->kids[(size_t)p - 1]; }

// Creates the sketches 1..P-1 and the chain streams of the merged form (first update after option 6).
static sage_status_t ensure_sketches(sage_fd* h) {
    if (h->P <= 1 || (int)h->kids.size() == h->P - 1) return SAGE_OK;
    for (int p = (int)h->kids.size() + 1; p < h->P; ++p) {
        sage_fd* k = nullptr;
        ST_TRY(create_handle(&k, h->D, h->ell, h->dtype, h->device, true));
        k->delta_rank = h->delta_rank;
        k->max_sweeps = h->max_sweeps;
        k->use_tc = h->use_tc;
        k->eig_variant = h->eig_variant;
        k->prof.mask = h->prof.mask;
        h->kids.push_back(k);
    }
    for (int p = 0; p < h->P; ++p) {
        sage_fd* s = sketch_at(h, p);
        if (!s->chain) CU_TRY(cudaStreamCreateWithFlags(&s->chain, cudaStreamNonBlocking));
    }
    return SAGE_OK;
}

// Algorithm 1, Phase I for n rows from `src` (dense rows or the factors of structured rows): shared by sage_fd_update and
// sage_fd_update_outer.
static sage_status_t update_from(sage_fd* h, RowSrc src, int64_t n, cudaStream_t st) {
    DeviceGuard g(h->device);
    ST_TRY(ensure_sketches(h));
    static std::atomic<long long> epochs{0};
    const int64_t epoch = epochs.fetch_add(1) + 1;
    CU_TRY(cudaEventRecord(h->ev_in, st));
    sage_status_t rc = SAGE_OK;
    if (h->P == 1) {
        rc = sketch_feed(h, src, n, st, h->ev_in, epoch, false);
        h->dealt += n;
    } else {
        // block b of the row stream (counted over all calls) goes to sketch b mod P
        while (n > 0 && rc == SAGE_OK) {
            const int64_t b = h->dealt / h->block;
            const int64_t left_in_block = (b + 1) * h->block - h->dealt;
            const int64_t take = n < left_in_block ? n : left_in_block;
            sage_fd* s = sketch_at(h, (int)(b % h->P));
            rc = sketch_feed(s, src, take, s->chain, h->ev_in, epoch, false);
            h->dealt += take;
            src = src.advanced(take);
            n -= take;
        }
    }
    // the caller's stream continues once every row of this call has been copied into a buffer
    for (int p = 0; p < h->P && p <= (int)h->kids.size(); ++p) {
        sage_fd* s = sketch_at(h, p);
        if (s->used) {
            const cudaError_t e = cudaStreamWaitEvent(st, s->ev_rows, 0);
            if (rc == SAGE_OK) CU_TRY(e);
            s->used = false;
        }
    }
    return rc;
}

sage_status_t sage_fd_update(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (n < 0 || (n > 0 && (!rows || ld < h->D))) {
        set_err("sage_fd_update: bad argument (rows=%p n=%lld ld=%lld D=%lld)", rows, (long long)n, (long long)ld, (long long)h->D);
        return SAGE_ERR_INVALID_ARG;
    }
    if (h->state != SKETCHING) {
        set_err("sage_fd_update: the sketch is frozen (call sage_fd_reset to start over)");
        return SAGE_ERR_BAD_STATE;
    }
    if (n == 0) return SAGE_OK;
    RowSrc src;
    src.rows = rows;
    src.ld = ld;
    src.dt = h->dtype;
    return update_from(h, src, n, static_cast<cudaStream_t>(cuda_stream));
}

// Checks the arguments of the entry points that take structured last-layer rows.
static sage_status_t check_outer(const sage_fd* h, const char* who, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n,
                                 int32_t C, int32_t F) {
    if (C < 1 || F < 1 || (int64_t)C * F + C != h->D) {
        set_err("%s: C=%d classes x F=%d features + C biases is not the handle's row dimension D=%lld", who, (int)C, (int)F, (long long)h->D);
        return SAGE_ERR_INVALID_ARG;
    }
    if (n < 0 || (n > 0 && (!q || !feat || ldq < C || ldf < F))) {
        set_err("%s: bad argument (q=%p ldq=%lld feat=%p ldf=%lld n=%lld)", who, q, (long long)ldq, feat, (long long)ldf, (long long)n);
        return SAGE_ERR_INVALID_ARG;
    }
    return SAGE_OK;
}

sage_status_t sage_fd_update_outer(sage_fd_t* h, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n, int32_t C, int32_t F,
                                   void* cuda_stream) {
    ST_TRY(check_handle(h));
    ST_TRY(check_outer(h, "sage_fd_update_outer", q, ldq, feat, ldf, n, C, F));
    if (h->state != SKETCHING) {
        set_err("sage_fd_update_outer: the sketch is frozen (call sage_fd_reset to start over)");
        return SAGE_ERR_BAD_STATE;
    }
    if (n == 0) return SAGE_OK;
    RowSrc src;
    src.q = q;
    src.ldq = ldq;
    src.feat = feat;
    src.ldf = ldf;
    src.C = C;
    src.F = F;
    src.dt = h->dtype;
    return update_from(h, src, n, static_cast<cudaStream_t>(cuda_stream));
}

// Makes `cuda_stream` wait for everything the handle has enqueued on streams of its own.
sage_status_t sage_fd_join(sage_fd_t* h, void* cuda_stream) {
    ST_TRY(check_handle(h));
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    for (int p = 0; p <= (int)h->kids.size(); ++p) {
        sage_fd* s = sketch_at(h, p);
        CU_TRY(cudaEventRecord(s->ev_join, s->side));
        CU_TRY(cudaStreamWaitEvent(st, s->ev_join, 0));
        if (s->chain) {
            CU_TRY(cudaEventRecord(s->ev_done, s->chain));
            CU_TRY(cudaStreamWaitEvent(st, s->ev_done, 0));
        }
    }
    return SAGE_OK;
}

sage_status_t sage_fd_finalize(sage_fd_t* h, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (h->state != SKETCHING) {
        set_err("sage_fd_finalize: already frozen");
        return SAGE_ERR_BAD_STATE;
    }
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int nsk = (int)h->kids.size() + 1;            // sketches that exist (1 unless the merged form has been fed)
    if (nsk == 1) {
        ST_TRY(sketch_freeze(h, (h->P > 1 && h->chain) ? h->chain : st));
    } else {
        // every sketch is frozen on its own, then sketch a absorbs sketch a + s for s = 1, 2, 4, ...: the rows the
        // other one kept are appended to it and it is frozen again (a shrink happens if that fills its buffer)
        for (int p = 0; p < nsk; ++p) ST_TRY(sketch_freeze(sketch_at(h, p), sketch_at(h, p)->chain));
        for (int stride = 1; stride < nsk; stride *= 2)
            for (int a = 0; a + stride < nsk; a += 2 * stride) {
                sage_fd* A = sketch_at(h, a);
                sage_fd* Bs = sketch_at(h, a + stride);
                CU_TRY(cudaEventRecord(Bs->ev_done, Bs->chain));
                CU_TRY(cudaStreamWaitEvent(A->chain, Bs->ev_done, 0));
                if (Bs->fill > 0)
                {
                    RowSrc kept;
                    kept.rows = Bs->B[Bs->cur];
                    kept.ld = Bs->pitch;
                    kept.dt = SAGE_F32;
                    ST_TRY(sketch_feed(A, kept, Bs->fill, A->chain, nullptr, 0, true));
                }
                ST_TRY(sketch_freeze(A, A->chain));
            }
    }
    if (h->P > 1 && h->chain) {                          // merged form: sketch 0 holds the result; back to the caller's stream
        CU_TRY(cudaEventRecord(h->ev_done, h->chain));
        CU_TRY(cudaStreamWaitEvent(st, h->ev_done, 0));
    }
    ST_TRY(enqueue_freeze_aux(h, st));
    h->state = FROZEN;
    EigInfo info;
    int tc_err = 0;
    CU_TRY(cudaMemcpyAsync(&info, h->info, sizeof info, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaMemcpyAsync(&tc_err, h->tc_err, sizeof tc_err, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    for (sage_fd* k : h->kids) {                         // their chains ended before sketch 0's did
        EigInfo ki;
        int kt = 0;
        CU_TRY(cudaMemcpy(&ki, k->info, sizeof ki, cudaMemcpyDeviceToHost));
        CU_TRY(cudaMemcpy(&kt, k->tc_err, sizeof kt, cudaMemcpyDeviceToHost));
        info.flags |= ki.flags;
        tc_err |= kt;
    }
    if (tc_err) {
        set_err("sage_fd_finalize: a tensor-core kernel gave up waiting on its pipeline (results are not valid)");
        return SAGE_ERR_CUDA;
    }
    if (info.flags & kFlagExchangeTimeout) {
        set_err("sage_fd_finalize: an eigen-solve gave up waiting for another thread block of its cluster (results are not valid)");
        return SAGE_ERR_CUDA;
    }
    if (info.flags & kFlagNotConverged) {
        set_err("sage_fd_finalize: an eigen-solve reached the sweep limit (%d)", h->max_sweeps);
        return SAGE_ERR_NOT_CONVERGED;
    }
    if (info.flags & kFlagNonFinite) {
        set_err("sage_fd_finalize: non-finite values were met in the rows of pass 1");
        return SAGE_ERR_NONFINITE;
    }
    return SAGE_OK;
}

sage_status_t sage_fd_sketch(const sage_fd_t* h, const float** S, int64_t* pitch, const float** sigma) {
    ST_TRY(check_handle(h));
    if (h->state == SKETCHING) {
        set_err("sage_fd_sketch: the sketch is not frozen yet");
        return SAGE_ERR_BAD_STATE;
    }
    if (S) *S = h->B[h->cur];
    if (pitch) *pitch = h->pitch;
    if (sigma) *sigma = h->sigma;
    return SAGE_OK;
}

sage_status_t sage_fd_load_sketch(sage_fd_t* h, const float* S, int64_t ld, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (!S || ld < h->D) {
        set_err("sage_fd_load_sketch: bad argument");
        return SAGE_ERR_INVALID_ARG;
    }
    if (h->state == SCORING) {
        set_err("sage_fd_load_sketch: a scoring pass is open");
        return SAGE_ERR_BAD_STATE;
    }
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    CU_TRY(timed(h, K_APPEND, 1, st, [&] { return launch_append(S, SAGE_F32, h->ell, ld, h->D, h->B[h->cur], h->pitch, 0, st); }));
    CU_TRY(cudaMemsetAsync(h->sigma, 0, h->ell * sizeof(float), st));
    ST_TRY(enqueue_freeze_aux(h, st));
    h->fill = h->ell;
    h->scored = false;
    h->scored_strict = false;
    h->state = FROZEN;
    return SAGE_OK;
}

sage_status_t sage_score_begin(sage_fd_t* h, int64_t N_total, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (N_total < 0) {
        set_err("sage_score_begin: negative row count");
        return SAGE_ERR_INVALID_ARG;
    }
    if (h->state != FROZEN) {
        set_err("sage_score_begin: needs a frozen sketch and no open scoring pass");
        return SAGE_ERR_BAD_STATE;
    }
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!h->strict && N_total > h->zcap) {
        CU_TRY(cudaStreamSynchronize(st));
        if (h->zhat) CU_TRY(cudaFree(h->zhat));
        if (h->znorm) CU_TRY(cudaFree(h->znorm));
        h->zhat = h->znorm = nullptr;
        h->zcap = 0;
        CU_TRY(cudaMalloc((void**)&h->zhat, (size_t)N_total * h->ell * sizeof(float)));
        CU_TRY(cudaMalloc((void**)&h->znorm, (size_t)N_total * sizeof(float)));
        h->zcap = N_total;
    }
    CU_TRY(cudaMemsetAsync(h->zsum, 0, 256 * sizeof(double), st));
    h->N_total = N_total;
    h->next_row = 0;
    h->scored = false;
    h->scored_strict = false;
    h->state = SCORING;
    return SAGE_OK;
}

// Projection, normalisation and consensus partials of n rows (sub-chunk by sub-chunk). store_at >= 0: the normalised
// projections go to rows [store_at, store_at + n) of the handle's N x ell store; store_at < 0: to a scratch of one sub-chunk
// (strict-memory mode). accumulate: the rows' sum is added to the consensus sum. scores_out != null (third pass of the
// strict-memory mode): the scores of these rows against the finished consensus are written there.
// Projection, normalisation, consensus partials (and, with scores_out, the scores) of n rows, a sub-chunk at a time.
// Dense rows: `rows` with pitch ld. Structured last-layer rows (outer != nullptr; rows and ld unused): the projection
// factorises over the classes,
//     z_i = S g_i = sum_c q_ic (S_c h_i) + S_b q_i      (S_c: columns [c F, c F + F) of the sketch, S_b: its last C columns),
// so the row g_i is never formed: ONE launch of the projection kernel takes the classes as its K slices (every slice reads
// the same F feature columns, slice c the class block c of the sketch) and leaves the planes T_c = H S_c^T, which a second
// kernel folds with the factors q_ic and the bias block.
static sage_status_t score_rows(sage_fd* h, const void* rows, sage_dtype_t dt, int64_t n, int64_t ld, cudaStream_t st, int64_t store_at,
                                bool accumulate, float* scores_out, const RowSrc* outer = nullptr) {
    const int ell = h->ell;
    const bool structured = outer != nullptr;
    const void* oq = structured ? outer->q : nullptr;
    const int64_t oldq = structured ? outer->ldq : 0;
    const int oC = structured ? outer->C : 0, oF = structured ? outer->F : 0;
    if (structured) {
        rows = outer->feat;
        ld = outer->ldf;
    }
    const int64_t K = structured ? (int64_t)oC * oF : h->D;      // contraction length against the sketch
    const int64_t class_F = structured ? oF : 0;
    int64_t sub_max = 148 * 128;             // one full wave of 128-row tiles
    const char* p = static_cast<const char*>(rows);
    const size_t row_bytes = (size_t)ld * elem_size(dt);
    const float* S = h->B[h->cur];
    // Tensor-core path: bf16 rows against the bf16 copy of the sketch (a one-term bf16 sketch is only used for
    // long rows, where its rounding errors average out).
    const bool tc_ok = h->use_tc && dt == SAGE_BF16 && h->P16 && (h->p16_fold || h->D >= 16384) &&
                       (reinterpret_cast<uintptr_t>(rows) & 15u) == 0 && (row_bytes & 15u) == 0;
    // fp32 rows: the fp32-faithful three-MMA kernel against the fp32 sketch itself (one 128-wide tile of S)
    const bool tc32_ok = h->use_tc && dt == SAGE_F32 && ell <= 128 && (reinterpret_cast<uintptr_t>(rows) & 15u) == 0 &&
                         (row_bytes & 15u) == 0;
    // fp32 rows against a small sketch: the projections of a sub-chunk are small (ell <= 64 floats per row and plane), so
    // up to 8 waves go into one launch (fewer launch-scale overheads per pass)
    if (tc32_ok && h->S32split) sub_max *= 8;
    if (structured) {
        // one plane per class (two with the pre-split sketch): keep the planes of a sub-chunk within 1 GiB
        const int64_t per_row = (int64_t)oC * ((tc32_ok && h->S32split) ? 2 : 1) * ell * (int64_t)sizeof(float);
        int64_t fit = ((int64_t)1 << 30) / per_row / 128 * 128;
        if (fit < 128) fit = 128;
        if (sub_max > fit) sub_max = fit;
    }
    for (int64_t r0 = 0; r0 < n; r0 += sub_max) {
        const int64_t sub = (n - r0 < sub_max) ? n - r0 : sub_max;
        const size_t nb = (size_t)((sub + 63) / 64);
        ST_TRY(ensure(&h->partials, &h->partials_bytes, nb * ell * sizeof(float)));
        if (store_at < 0 && sub > h->zcap) {         // strict-memory mode: normalised projections of one sub-chunk only
            CU_TRY(cudaStreamSynchronize(st));
            if (h->zhat) CU_TRY(cudaFree(h->zhat));
            if (h->znorm) CU_TRY(cudaFree(h->znorm));
            h->zhat = h->znorm = nullptr;
            h->zcap = 0;
            CU_TRY(cudaMalloc((void**)&h->zhat, (size_t)sub * ell * sizeof(float)));
            CU_TRY(cudaMalloc((void**)&h->znorm, (size_t)sub * sizeof(float)));
            h->zcap = sub;
        }
        const size_t zred = (size_t)sub * ell * sizeof(float);
        bool done = false;
        const float* Zparts = nullptr;       // the projections of this sub-chunk as nplanes partial planes of sub x ell floats
        int nplanes = 1;
        if (tc32_ok) {
            const int splits = structured ? oC : pick_splits_waves((int)((sub + 127) / 128), K, 2048, 64);
            // sketches of at most 64 rows: one wide MMA per K step against the pre-split sketch, two partial planes per K slice
            const bool wide = h->S32split != nullptr;
            const int planes = wide ? 2 * splits : splits;
            ST_TRY(ensure(&h->zwork, &h->zwork_bytes, zred * planes));
            float* out = h->zwork;
            cudaError_t e = timed(h, K_PROJECT, 1, st, [&] {
                return launch_tc_gemm_nt_x3(reinterpret_cast<const float*>(p + r0 * row_bytes), ld, wide ? h->S32split : S, h->pitch, (int)sub,
                                            ell, K, splits, out, ell, (int64_t)sub * ell, wide ? 2 : 0, h->tc_err, st, class_F);
            });
            if (e == cudaSuccess) {
                done = true;
                h->tc_launches += 1;
                Zparts = out;
                nplanes = planes;
            } else if (e != cudaErrorNotSupported) {
                CU_TRY(e);
            } else {
                count(h, -1);
            }
        }
        if (tc_ok) {
            // row tiles per CTA: as many as TMEM holds (512 columns), fewer when that would leave SMs without work
            const int n_mma = (h->p16_fold ? 2 : 1) * h->p16_npad;
            const int tiles = (int)((sub + 127) / 128);
            int mt = 512 / n_mma >= 4 ? 4 : (512 / n_mma >= 2 ? 2 : 1);
            if (tiles >= 148 && mt > 2) mt = 2;   // measured: pairs of row tiles with two K slices beat single tiles by 25 %
            // rows a page or more apart: the kernel fetches two K tiles per stage (256 bytes per row visit), two row tiles fit
            if (row_bytes >= ((size_t)2 << 20) && mt > 2) mt = 2;
            const int64_t slices_at_least = structured ? oC : (K / 4096 > 0 ? K / 4096 : 1);
            while (mt > 1 && (int64_t)((tiles + mt - 1) / mt) * slices_at_least < 148) mt >>= 1;
            const int splits = structured ? oC : pick_splits_waves((tiles + mt - 1) / mt, K, 4096, 148);
            ST_TRY(ensure(&h->zwork, &h->zwork_bytes, zred * splits));
            float* out = h->zwork;
            cudaError_t e = timed(h, K_PROJECT, 1, st, [&] {
                return launch_tc_gemm_nt(p + r0 * row_bytes, SAGE_BF16, ld, h->P16, h->pitch, (int)sub, ell, h->p16_fold, mt, K, splits,
                                         out, ell, (int64_t)sub * ell, h->tc_err, st, class_F);
            });
            if (e == cudaSuccess) {
                done = true;
                h->tc_launches += 1;
                Zparts = out;
                nplanes = splits;
            } else if (e != cudaErrorNotSupported) {
                CU_TRY(e);
            } else {
                count(h, -1);
            }
        }
        if (!done) {
            const int tiles = (int)((sub + 63) / 64) * ((ell + 63) / 64);
            const int splits = structured ? oC : pick_splits(tiles, K, 1024);
            ST_TRY(ensure(&h->zwork, &h->zwork_bytes, zred * splits));
            CU_TRY(timed(h, K_PROJECT, 1, st, [&] {
                return launch_gemm_nt(p + r0 * row_bytes, dt, ld, S, h->pitch, (int)sub, ell, K, splits, h->zwork, ell,
                                      (int64_t)sub * ell, st, class_F);
            }));
            Zparts = h->zwork;
            nplanes = splits;
        }
        if (structured) {
            // z = sum_c q_c (T_c + bias column c), classes in ascending order
            ST_TRY(ensure(&h->zred, &h->zred_bytes, zred));
            const float* parts = Zparts;
            const int pp = nplanes / oC;
            const char* qsub = static_cast<const char*>(oq) + (size_t)r0 * oldq * elem_size(dt);
            ST_TRY(ensure(&h->bias_t, &h->bias_t_bytes, (size_t)oC * ell * sizeof(float)));
            CU_TRY(timed(h, K_PROJECT_REDUCE, 2, st, [&] {
                return launch_outer_combine(qsub, oldq, dt, oC, parts, pp, (int64_t)sub * ell, S + K, h->pitch, h->bias_t, sub, ell, h->zred, st);
            }));
            Zparts = h->zred;
            nplanes = 1;
        }
        // Many K slices (few rows per launch, as in the 512-row chunks of very long rows): summed first by a kernel with a
        // thread per element; the normalise kernel has a warp per row and would walk the slices one after the other.
        if (nplanes > 4) {
            ST_TRY(ensure(&h->zred, &h->zred_bytes, zred));
            const float* parts = Zparts;
            const int np = nplanes;
            CU_TRY(timed(h, K_PROJECT_REDUCE, 1, st,
                         [&] { return launch_split_reduce(parts, np, (int64_t)sub * ell, (int)sub, ell, ell, h->zred, ell, st); }));
            Zparts = h->zred;
            nplanes = 1;
        }
        // normalise (summing the K slices of the projection on the way), consensus partials, and in the third pass the scores
        float* zh = store_at >= 0 ? h->zhat + (store_at + r0) * ell : h->zhat;
        float* zn = store_at >= 0 ? h->znorm + (store_at + r0) : h->znorm;
        CU_TRY(timed(h, K_NORMALISE, accumulate ? 2 : 1, st, [&] {
            return launch_normalise(Zparts, nplanes, (int64_t)sub * ell, ell, sub, ell, zh, zn, h->partials, accumulate ? h->zsum : nullptr,
                                    &h->info->flags, st);
        }));
        if (scores_out)
            CU_TRY(timed(h, K_SCORE, 1, st, [&] { return launch_consensus_score(h->zsum, zh, sub, ell, h->u, scores_out + r0, st); }));
    }
    return SAGE_OK;
}


sage_status_t sage_score_chunk(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, int64_t row_offset, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (h->state != SCORING) {
        set_err("sage_score_chunk: no open scoring pass");
        return SAGE_ERR_BAD_STATE;
    }
    if (n < 0 || (n > 0 && (!rows || ld < h->D)) || row_offset != h->next_row || row_offset + n > h->N_total) {
        set_err("sage_score_chunk: bad argument (n=%lld ld=%lld offset=%lld expected offset=%lld N_total=%lld)", (long long)n,
                (long long)ld, (long long)row_offset, (long long)h->next_row, (long long)h->N_total);
        return SAGE_ERR_INVALID_ARG;
    }
    if (n == 0) return SAGE_OK;
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ST_TRY(score_rows(h, rows, h->dtype, n, ld, st, h->strict ? -1 : row_offset, true, nullptr));
    h->next_row += n;
    return SAGE_OK;
}

sage_status_t sage_score_chunk_outer(sage_fd_t* h, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n, int32_t C,
                                     int32_t F, int64_t row_offset, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (h->state != SCORING) {
        set_err("sage_score_chunk_outer: no open scoring pass");
        return SAGE_ERR_BAD_STATE;
    }
    ST_TRY(check_outer(h, "sage_score_chunk_outer", q, ldq, feat, ldf, n, C, F));
    if (row_offset != h->next_row || row_offset + n > h->N_total) {
        set_err("sage_score_chunk_outer: bad argument (n=%lld offset=%lld expected offset=%lld N_total=%lld)", (long long)n,
                (long long)row_offset, (long long)h->next_row, (long long)h->N_total);
        return SAGE_ERR_INVALID_ARG;
    }
    if (n == 0) return SAGE_OK;
    DeviceGuard g(h->device);
    RowSrc src;
    src.q = q;
    src.ldq = ldq;
    src.feat = feat;
    src.ldf = ldf;
    src.C = C;
    src.F = F;
    src.dt = h->dtype;
    ST_TRY(score_rows(h, nullptr, h->dtype, n, 0, static_cast<cudaStream_t>(cuda_stream), h->strict ? -1 : row_offset, true, nullptr, &src));
    h->next_row += n;
    return SAGE_OK;
}

sage_status_t sage_score_end(sage_fd_t* h, float* scores, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (h->state != SCORING) {
        set_err("sage_score_end: no open scoring pass");
        return SAGE_ERR_BAD_STATE;
    }
    if (h->next_row != h->N_total) {
        set_err("sage_score_end: %lld of %lld rows were given", (long long)h->next_row, (long long)h->N_total);
        return SAGE_ERR_BAD_STATE;
    }
    if (!scores && h->N_total > 0 && !h->strict) {
        set_err("sage_score_end: null scores");
        return SAGE_ERR_INVALID_ARG;
    }
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (h->strict) {     // only the consensus direction is formed here; the scores come from sage_score_apply
        CU_TRY(timed(h, K_SCORE, 1, st, [&] { return launch_consensus_score(h->zsum, h->zhat, 0, h->ell, h->u, nullptr, st); }));
        h->scored_strict = true;
    } else {
        CU_TRY(timed(h, K_SCORE, 1, st, [&] { return launch_consensus_score(h->zsum, h->zhat, h->N_total, h->ell, h->u, scores, st); }));
        h->scored = true;
    }
    h->state = FROZEN;
    return SAGE_OK;
}

sage_status_t sage_score_apply(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, float* scores, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (h->state != FROZEN || !(h->scored || h->scored_strict)) {
        set_err("sage_score_apply: needs a finished scoring pass (the consensus direction) on this handle");
        return SAGE_ERR_BAD_STATE;
    }
    if (n < 0 || (n > 0 && (!rows || !scores || ld < h->D))) {
        set_err("sage_score_apply: bad argument (n=%lld ld=%lld)", (long long)n, (long long)ld);
        return SAGE_ERR_INVALID_ARG;
    }
    if (n == 0) return SAGE_OK;
    if (h->scored) {     // the N x ell store of the finished pass must survive: this call works in a scratch of its own size class
        set_err("sage_score_apply: the handle keeps the normalised projections of its last pass (option 8 is off); use sage_score");
        return SAGE_ERR_BAD_STATE;
    }
    DeviceGuard g(h->device);
    return score_rows(h, rows, h->dtype, n, ld, static_cast<cudaStream_t>(cuda_stream), -1, false, scores);
}

sage_status_t sage_score(sage_fd_t* h, const void* rows, int64_t n, int64_t ld, float* scores, void* cuda_stream) {
    ST_TRY(sage_score_begin(h, n, cuda_stream));
    sage_status_t s = sage_score_chunk(h, rows, n, ld, 0, cuda_stream);
    if (s != SAGE_OK) {
        h->state = FROZEN;
        return s;
    }
    s = sage_score_end(h, scores, cuda_stream);
    if (s != SAGE_OK) h->state = FROZEN;
    return s;
}

sage_status_t sage_score_outer(sage_fd_t* h, const void* q, int64_t ldq, const void* feat, int64_t ldf, int64_t n, int32_t C, int32_t F,
                               float* scores, void* cuda_stream) {
    ST_TRY(check_handle(h));
    ST_TRY(check_outer(h, "sage_score_outer", q, ldq, feat, ldf, n, C, F));
    ST_TRY(sage_score_begin(h, n, cuda_stream));
    sage_status_t s = sage_score_chunk_outer(h, q, ldq, feat, ldf, n, C, F, 0, cuda_stream);
    if (s != SAGE_OK) {
        h->state = FROZEN;
        return s;
    }
    s = sage_score_end(h, scores, cuda_stream);
    if (s != SAGE_OK) h->state = FROZEN;
    return s;
}

sage_status_t sage_score_intermediates(const sage_fd_t* h, const float** zhat, const float** znorm, const float** u) {
    ST_TRY(check_handle(h));
    if (h->state != FROZEN || !h->zhat || !h->scored) {
        set_err("sage_score_intermediates: no finished scoring pass that kept its projections");
        return SAGE_ERR_BAD_STATE;
    }
    if (zhat) *zhat = h->zhat;
    if (znorm) *znorm = h->znorm;
    if (u) *u = h->u;
    return SAGE_OK;
}

sage_status_t sage_select(const float* scores, int64_t N, double keep_rate, int64_t* idx, int64_t* k_out, void* cuda_stream) {
    if (N < 0 || N >= (1ll << 31) || !(keep_rate == keep_rate) || (N > 0 && !scores)) {
        set_err("sage_select: bad argument (N=%lld keep_rate=%g)", (long long)N, keep_rate);
        return SAGE_ERR_INVALID_ARG;
    }
    const int64_t k = sage_select_count(N, keep_rate);
    if (k > 0 && !idx) {
        set_err("sage_select: null idx");
        return SAGE_ERR_INVALID_ARG;
    }
    if (k > 0) {
        cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
        size_t bytes = 0;
        select_scratch_bytes(N, &bytes);
        void* scratch = nullptr;
        CU_TRY(scratch_alloc(&scratch, bytes, st));
        cudaError_t e = launch_select(scores, N, k, idx, scratch, st);
        cudaError_t e2 = cudaFreeAsync(scratch, st);
        CU_TRY(e);
        CU_TRY(e2);
        int idx_bits = 1;
        while (idx_bits < 32 && (1ll << idx_bits) < N) ++idx_bits;
        count(nullptr, 2 + 3 * (4 + (idx_bits + 7) / 8));
    }
    if (k_out) *k_out = k;
    return SAGE_OK;
}

sage_status_t sage_score_classes(sage_fd_t* h, const int32_t* labels, int32_t num_classes, float* scores, void* cuda_stream) {
    ST_TRY(check_handle(h));
    if (h->state != FROZEN || !h->scored) {
        set_err("sage_score_classes: needs a finished scoring pass (sage_score or sage_score_end) on this handle");
        return SAGE_ERR_BAD_STATE;
    }
    if (num_classes < 1 || num_classes > 65535 || (h->N_total > 0 && (!labels || !scores))) {
        set_err("sage_score_classes: bad argument (num_classes=%d labels=%p scores=%p)", (int)num_classes, (const void*)labels, (void*)scores);
        return SAGE_ERR_INVALID_ARG;
    }
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (num_classes > h->class_cap) {
        CU_TRY(cudaStreamSynchronize(st));
        if (h->class_U) CU_TRY(cudaFree(h->class_U));
        if (h->class_counts) CU_TRY(cudaFree(h->class_counts));
        h->class_U = nullptr;
        h->class_counts = nullptr;
        h->class_cap = 0;
        CU_TRY(cudaMalloc((void**)&h->class_U, (size_t)num_classes * h->ell * sizeof(float)));
        CU_TRY(cudaMalloc((void**)&h->class_counts, (size_t)num_classes * sizeof(int)));
        h->class_cap = num_classes;
    }
    h->class_num = num_classes;
    CU_TRY(launch_class_scores(h->zhat, labels, h->N_total, h->ell, num_classes, h->class_U, h->class_counts, scores, st));
    count(h, h->N_total > 0 ? 2 : 1);
    return SAGE_OK;
}

sage_status_t sage_score_class_centroids(const sage_fd_t* h, const float** U, const int32_t** counts, int32_t* num_classes) {
    ST_TRY(check_handle(h));
    if (!h->class_U || h->class_num == 0) {
        set_err("sage_score_class_centroids: sage_score_classes has not run on this handle");
        return SAGE_ERR_BAD_STATE;
    }
    if (U) *U = h->class_U;
    if (counts) *counts = h->class_counts;
    if (num_classes) *num_classes = h->class_num;
    return SAGE_OK;
}

sage_status_t sage_select_classes(const float* scores, const int32_t* labels, int64_t N, int32_t num_classes, double keep_rate,
                                  int64_t* idx, int64_t* k_per_class, int64_t* k_out, void* cuda_stream) {
    if (N < 0 || N >= (1ll << 31) || !(keep_rate == keep_rate) || num_classes < 1 || num_classes > 65535 || (N > 0 && (!scores || !labels))) {
        set_err("sage_select_classes: bad argument (N=%lld num_classes=%d keep_rate=%g)", (long long)N, (int)num_classes, keep_rate);
        return SAGE_ERR_INVALID_ARG;
    }
    const int C = num_classes;
    std::vector<long long> kc(C, 0), offs(C, 0);
    long long k = 0;
    if (N > 0) {
        cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
        size_t sel_bytes = 0;
        select_scratch_bytes(N, &sel_bytes);
        const size_t a256 = 255;
        const size_t sorted_off = (sel_bytes + a256) & ~a256;
        const size_t counts_off = (sorted_off + (size_t)N * 8 + a256) & ~a256;
        const size_t kc_off = (counts_off + (size_t)C * 4 + a256) & ~a256;
        const size_t offs_off = (kc_off + (size_t)C * 8 + a256) & ~a256;
        const size_t total = offs_off + (size_t)C * 8;
        char* scratch = nullptr;
        CU_TRY(scratch_alloc((void**)&scratch, total, st));
        auto body = [&]() -> sage_status_t {
            int* d_counts = reinterpret_cast<int*>(scratch + counts_off);
            CU_TRY(launch_class_count(labels, N, C, d_counts, st));
            std::vector<int> counts(C);
            CU_TRY(cudaMemcpyAsync(counts.data(), d_counts, (size_t)C * sizeof(int), cudaMemcpyDeviceToHost, st));
            CU_TRY(cudaStreamSynchronize(st));
            long long n_valid = 0;
            for (int c = 0; c < C; ++c) n_valid += counts[c];
            k = sage_select_count(n_valid, keep_rate);
            // k_c proportional to the class sizes, largest remainder, ties to the smaller class (exact integers)
            std::vector<long long> rem(C, 0);
            long long given = 0;
            if (n_valid > 0)
                for (int c = 0; c < C; ++c) {
                    const long long num = (long long)counts[c] * k;
                    kc[c] = num / n_valid;
                    rem[c] = num - kc[c] * n_valid;
                    given += kc[c];
                }
            std::vector<int> order(C);
            for (int c = 0; c < C; ++c) order[c] = c;
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return rem[a] > rem[b]; });
            for (long long t = 0; t < k - given; ++t) kc[order[(size_t)t]] += 1;
            long long run = 0;
            for (int c = 0; c < C; ++c) { offs[c] = run; run += kc[c]; }
            if (k > 0 && !idx) {
                set_err("sage_select_classes: null idx");
                return SAGE_ERR_INVALID_ARG;
            }
            if (k > 0) {
                CU_TRY(cudaMemcpyAsync(scratch + kc_off, kc.data(), (size_t)C * 8, cudaMemcpyHostToDevice, st));
                CU_TRY(cudaMemcpyAsync(scratch + offs_off, offs.data(), (size_t)C * 8, cudaMemcpyHostToDevice, st));
                int64_t* sorted = reinterpret_cast<int64_t*>(scratch + sorted_off);
                CU_TRY(launch_select(scores, N, N, sorted, scratch, st));
                CU_TRY(launch_class_pick(sorted, labels, N, C, reinterpret_cast<const long long*>(scratch + kc_off),
                                         reinterpret_cast<const long long*>(scratch + offs_off), idx, st));
                CU_TRY(cudaStreamSynchronize(st));        // kc / offs are host vectors of this call
                int idx_bits = 1;
                while (idx_bits < 32 && (1ll << idx_bits) < N) ++idx_bits;
                count(nullptr, 3 + 3 * (4 + (idx_bits + 7) / 8) + 2);
            }
            return SAGE_OK;
        };
        const sage_status_t rc = body();
        cudaFreeAsync(scratch, st);
        if (rc != SAGE_OK) return rc;
    }
    if (k_per_class)
        for (int c = 0; c < C; ++c) k_per_class[c] = kc[c];
    if (k_out) *k_out = k;
    return SAGE_OK;
}

// ---- checkpoint of the sketch state ---------------------------------------------------------------------------
namespace {
struct ExportHeader {
    char magic[8];
    int64_t D;
    int32_t ell, dtype, P, frozen;
    int64_t block, dealt;
    int32_t nsk, delta_rank;
};
struct ExportSketch {
    int32_t rows, pad;
    EigInfo info;
};
const char kExportMagic[8] = {'S', 'A', 'G', 'E', 'F', 'D', '1', 0};

int export_rows(const sage_fd* s, bool frozen) { return frozen ? s->ell : s->fill; }
}  // namespace

sage_status_t sage_fd_export_size(const sage_fd_t* h, size_t* bytes) {
    ST_TRY(check_handle(h));
    if (!bytes) {
        set_err("sage_fd_export_size: null bytes");
        return SAGE_ERR_INVALID_ARG;
    }
    if (h->state == SCORING) {
        set_err("sage_fd_export_size: a scoring pass is open");
        return SAGE_ERR_BAD_STATE;
    }
    const bool frozen = h->state == FROZEN;
    size_t total = sizeof(ExportHeader);
    const int nsk = frozen ? 1 : (int)h->kids.size() + 1;
    for (int p = 0; p < nsk; ++p) {
        const sage_fd* s = p == 0 ? h : h->kids[(size_t)p - 1];
        total += sizeof(ExportSketch) + (size_t)export_rows(s, frozen) * h->D * sizeof(float);
    }
    if (frozen) total += (size_t)h->ell * sizeof(float);
    *bytes = total;
    return SAGE_OK;
}

sage_status_t sage_fd_export(sage_fd_t* h, void* dst_host, size_t capacity, size_t* written) {
    size_t need = 0;
    ST_TRY(sage_fd_export_size(h, &need));
    if (!dst_host || capacity < need) {
        set_err("sage_fd_export: destination of %zu bytes is too small (%zu needed)", capacity, need);
        return SAGE_ERR_INVALID_ARG;
    }
    DeviceGuard g(h->device);
    CU_TRY(cudaDeviceSynchronize());           // everything enqueued so far, on the caller's streams and the handle's own
    const bool frozen = h->state == FROZEN;
    char* out = static_cast<char*>(dst_host);
    ExportHeader hd = {};
    std::memcpy(hd.magic, kExportMagic, 8);
    hd.D = h->D;
    hd.ell = h->ell;
    hd.dtype = (int32_t)h->dtype;
    hd.P = h->P;
    hd.frozen = frozen ? 1 : 0;
    hd.block = h->block;
    hd.dealt = h->dealt;
    hd.nsk = frozen ? 1 : (int)h->kids.size() + 1;
    hd.delta_rank = h->delta_rank;
    std::memcpy(out, &hd, sizeof hd);
    out += sizeof hd;
    for (int p = 0; p < hd.nsk; ++p) {
        sage_fd* s = sketch_at(h, p);
        ExportSketch es = {};
        es.rows = export_rows(s, frozen);
        CU_TRY(cudaMemcpy(&es.info, s->info, sizeof(EigInfo), cudaMemcpyDeviceToHost));
        if (frozen)                             // the counters of all sketches, as sage_fd_stats reports them
            for (sage_fd* k : h->kids) {
                EigInfo ki;
                CU_TRY(cudaMemcpy(&ki, k->info, sizeof ki, cudaMemcpyDeviceToHost));
                es.info.shrinks += ki.shrinks;
                es.info.sum_delta += ki.sum_delta;
                es.info.flags |= ki.flags;
                if (ki.max_sweeps > es.info.max_sweeps) es.info.max_sweeps = ki.max_sweeps;
            }
        std::memcpy(out, &es, sizeof es);
        out += sizeof es;
        if (es.rows > 0)
            CU_TRY(cudaMemcpy2D(out, (size_t)h->D * sizeof(float), s->B[s->cur], (size_t)s->pitch * sizeof(float),
                                (size_t)h->D * sizeof(float), (size_t)es.rows, cudaMemcpyDeviceToHost));
        out += (size_t)es.rows * h->D * sizeof(float);
    }
    if (frozen) {
        CU_TRY(cudaMemcpy(out, h->sigma, (size_t)h->ell * sizeof(float), cudaMemcpyDeviceToHost));
        out += (size_t)h->ell * sizeof(float);
    }
    if (written) *written = (size_t)(out - static_cast<char*>(dst_host));
    return SAGE_OK;
}

sage_status_t sage_fd_import(sage_fd_t* h, const void* src_host, size_t bytes, void* cuda_stream) {
    ST_TRY(check_handle(h));
    ExportHeader hd;
    if (!src_host || bytes < sizeof hd) {
        set_err("sage_fd_import: no data");
        return SAGE_ERR_INVALID_ARG;
    }
    std::memcpy(&hd, src_host, sizeof hd);
    if (std::memcmp(hd.magic, kExportMagic, 8) != 0 || hd.D != h->D || hd.ell != h->ell || hd.dtype != (int32_t)h->dtype || hd.P < 1 ||
        hd.P > 64 || hd.nsk < 1 || hd.nsk > hd.P || hd.block < 1 || hd.dealt < 0 || hd.delta_rank < 2 || hd.delta_rank > h->m - 1) {
        set_err("sage_fd_import: not a checkpoint of a sketch with D=%lld ell=%d and this row type", (long long)h->D, h->ell);
        return SAGE_ERR_INVALID_ARG;
    }
    // sizes first: nothing of the handle changes unless the whole checkpoint is consistent
    {
        const char* q = static_cast<const char*>(src_host) + sizeof hd;
        size_t left = bytes - sizeof hd;
        for (int p = 0; p < hd.nsk; ++p) {
            ExportSketch es;
            if (left < sizeof es) { set_err("sage_fd_import: truncated checkpoint"); return SAGE_ERR_INVALID_ARG; }
            std::memcpy(&es, q, sizeof es);
            const size_t rb = (size_t)(es.rows < 0 ? 0 : es.rows) * h->D * sizeof(float);
            if (es.rows < 0 || es.rows >= h->m + (hd.frozen ? 1 : 0) || left < sizeof es + rb) {
                set_err("sage_fd_import: truncated or inconsistent checkpoint");
                return SAGE_ERR_INVALID_ARG;
            }
            q += sizeof es + rb;
            left -= sizeof es + rb;
        }
        if (hd.frozen && left < (size_t)h->ell * sizeof(float)) { set_err("sage_fd_import: truncated checkpoint"); return SAGE_ERR_INVALID_ARG; }
    }
    DeviceGuard g(h->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ST_TRY(sage_fd_reset(h));
    ST_TRY(sage_fd_set_option(h, 6, (double)hd.P));
    h->block = hd.block;
    h->delta_rank = hd.delta_rank;
    for (sage_fd* k : h->kids) k->delta_rank = hd.delta_rank;
    if (hd.nsk > 1) ST_TRY(ensure_sketches(h));
    const char* q = static_cast<const char*>(src_host) + sizeof hd;
    for (int p = 0; p < hd.nsk; ++p) {
        sage_fd* s = sketch_at(h, p);
        s->delta_rank = hd.delta_rank;
        ExportSketch es;
        std::memcpy(&es, q, sizeof es);
        q += sizeof es;
        CU_TRY(cudaMemcpy(s->info, &es.info, sizeof(EigInfo), cudaMemcpyHostToDevice));
        if (es.rows > 0)
            CU_TRY(cudaMemcpy2D(s->B[0], (size_t)s->pitch * sizeof(float), q, (size_t)h->D * sizeof(float), (size_t)h->D * sizeof(float),
                                (size_t)es.rows, cudaMemcpyHostToDevice));
        if (s->pitch > h->D && es.rows > 0)     // columns between D and the pitch are zero in every buffer row
            CU_TRY(cudaMemset2D(s->B[0] + h->D, (size_t)s->pitch * sizeof(float), 0, (size_t)(s->pitch - h->D) * sizeof(float), (size_t)es.rows));
        q += (size_t)es.rows * h->D * sizeof(float);
        s->cur = 0;
        s->fill = hd.frozen ? h->ell : es.rows;
    }
    h->dealt = hd.dealt;
    h->rows_seen = hd.dealt;
    if (hd.frozen) {
        CU_TRY(cudaMemcpy(h->sigma, q, (size_t)h->ell * sizeof(float), cudaMemcpyHostToDevice));
        CU_TRY(cudaDeviceSynchronize());
        ST_TRY(enqueue_freeze_aux(h, st));
        h->state = FROZEN;
    } else {
        CU_TRY(cudaDeviceSynchronize());
    }
    return SAGE_OK;
}

sage_status_t sage_fd_stats(sage_fd_t* h, sage_stats_t* out) {
    ST_TRY(check_handle(h));
    if (!out) {
        set_err("sage_fd_stats: null out");
        return SAGE_ERR_INVALID_ARG;
    }
    DeviceGuard g(h->device);
    CU_TRY(cudaDeviceSynchronize());
    EigInfo info;
    CU_TRY(cudaMemcpy(&info, h->info, sizeof info, cudaMemcpyDeviceToHost));
    int tc_err = 0;
    CU_TRY(cudaMemcpy(&tc_err, h->tc_err, sizeof tc_err, cudaMemcpyDeviceToHost));
    int64_t launches = h->launches, tc_launches = h->tc_launches, in_place = h->rows_in_place;
    for (sage_fd* k : h->kids) {             // merged form: counters of all sketches together
        EigInfo ki;
        int kt = 0;
        CU_TRY(cudaMemcpy(&ki, k->info, sizeof ki, cudaMemcpyDeviceToHost));
        CU_TRY(cudaMemcpy(&kt, k->tc_err, sizeof kt, cudaMemcpyDeviceToHost));
        info.shrinks += ki.shrinks;
        info.sum_delta += ki.sum_delta;
        info.flags |= ki.flags;
        if (ki.max_sweeps > info.max_sweeps) info.max_sweeps = ki.max_sweeps;
        tc_err |= kt;
        launches += k->launches;
        tc_launches += k->tc_launches;
        in_place += k->rows_in_place;
    }
    out->rows_seen = h->dealt;
    out->shrinks = info.shrinks;
    out->sum_delta = info.sum_delta;
    out->last_sweeps = info.sweeps;
    out->max_sweeps = info.max_sweeps;
    out->last_rank = info.rank;
    out->device_flags = info.flags | (tc_err ? 4u : 0u);
    out->kernel_launches = launches;
    out->tensor_core_launches = tc_launches;
    out->rows_in_place = in_place;
    return SAGE_OK;
}

sage_status_t sage_fd_profile(sage_fd_t* h, double* ms, int64_t* launches, int32_t capacity) {
    ST_TRY(check_handle(h));
    if (!ms || !launches || capacity < K_NCLASS) {
        set_err("sage_fd_profile: need arrays of at least %d entries", (int)K_NCLASS);
        return SAGE_ERR_INVALID_ARG;
    }
    DeviceGuard g(h->device);
    CU_TRY(cudaDeviceSynchronize());
    for (int c = 0; c < K_NCLASS; ++c) {
        ms[c] = 0.0;
        launches[c] = 0;
    }
    for (int q = 0; q <= (int)h->kids.size(); ++q) {     // merged form: all sketches together (their kernels overlap in time)
        Prof& pr = sketch_at(h, q)->prof;
        for (auto& p : pr.pending) {
            float t = 0.f;
            if (cudaEventElapsedTime(&t, p.a, p.b) == cudaSuccess) {
                pr.ms[p.cls] += t;
                pr.n[p.cls] += 1;
            }
            pr.pool.push_back(p.a);
            pr.pool.push_back(p.b);
        }
        pr.pending.clear();
        for (int c = 0; c < K_NCLASS; ++c) {
            ms[c] += pr.ms[c];
            launches[c] += pr.n[c];
            pr.ms[c] = 0.0;
            pr.n[c] = 0;
        }
    }
    return SAGE_OK;
}

sage_status_t sage_select_from_host(const void* rows_host, int64_t N, int64_t D, int64_t ld, int32_t ell,
                                    sage_dtype_t row_dtype, double keep_rate, int64_t chunk_rows, int device,
                                    float* scores_host, int64_t* idx_host, int64_t* k_out) {
    if (!rows_host || N < 1 || D < 1 || ld < D || !(keep_rate == keep_rate)) {
        set_err("sage_select_from_host: bad argument");
        return SAGE_ERR_INVALID_ARG;
    }
    const int64_t k = sage_select_count(N, keep_rate);
    if (k > 0 && !idx_host) {
        set_err("sage_select_from_host: null idx_host");
        return SAGE_ERR_INVALID_ARG;
    }
    sage_fd_t* h = nullptr;
    ST_TRY(sage_fd_create(&h, D, ell, row_dtype, device));
    DeviceGuard g(device);
    const size_t es = elem_size(row_dtype);
    if (chunk_rows <= 0) {
        chunk_rows = (int64_t)((256ull << 20) / ((size_t)ld * es));     // about 256 MB per staging buffer
        if (chunk_rows < 2 * ell) chunk_rows = 2 * ell;
    }
    if (chunk_rows > N) chunk_rows = N;
    const size_t chunk_bytes = (size_t)chunk_rows * ld * es;
    void* stage[2] = {nullptr, nullptr};
    float* d_scores = nullptr;
    int64_t* d_idx = nullptr;
    cudaStream_t s_copy = nullptr, s_comp = nullptr;
    cudaEvent_t copied[2] = {nullptr, nullptr}, consumed[2] = {nullptr, nullptr};
    sage_status_t rc = SAGE_OK;
    auto body = [&]() -> sage_status_t {
        CU_TRY(cudaStreamCreateWithFlags(&s_copy, cudaStreamNonBlocking));
        CU_TRY(cudaStreamCreateWithFlags(&s_comp, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CU_TRY(cudaMalloc(&stage[i], chunk_bytes));
            CU_TRY(cudaEventCreateWithFlags(&copied[i], cudaEventDisableTiming));
            CU_TRY(cudaEventCreateWithFlags(&consumed[i], cudaEventDisableTiming));
        }
        CU_TRY(cudaMalloc((void**)&d_scores, (size_t)N * sizeof(float)));
        if (k > 0) CU_TRY(cudaMalloc((void**)&d_idx, (size_t)k * sizeof(int64_t)));
        const char* src = static_cast<const char*>(rows_host);
        for (int pass = 0; pass < 2; ++pass) {
            if (pass == 1) {
                sage_status_t f = sage_fd_finalize(h, s_comp);
                if (f != SAGE_OK && f != SAGE_ERR_NOT_CONVERGED && f != SAGE_ERR_NONFINITE) return f;
                if (f != SAGE_OK) rc = f;
                ST_TRY(sage_score_begin(h, N, s_comp));
            }
            int64_t c = 0;
            for (int64_t r0 = 0; r0 < N; r0 += chunk_rows, ++c) {
                const int b = (int)(c & 1);
                const int64_t n = (N - r0 < chunk_rows) ? N - r0 : chunk_rows;
                if (c >= 2 || pass == 1) CU_TRY(cudaStreamWaitEvent(s_copy, consumed[b], 0));
                CU_TRY(cudaMemcpyAsync(stage[b], src + (size_t)r0 * ld * es, (size_t)n * ld * es, cudaMemcpyHostToDevice, s_copy));
                CU_TRY(cudaEventRecord(copied[b], s_copy));
                CU_TRY(cudaStreamWaitEvent(s_comp, copied[b], 0));
                if (pass == 0)
                    ST_TRY(sage_fd_update(h, stage[b], n, ld, s_comp));
                else
                    ST_TRY(sage_score_chunk(h, stage[b], n, ld, r0, s_comp));
                CU_TRY(cudaEventRecord(consumed[b], s_comp));
            }
        }
        ST_TRY(sage_score_end(h, d_scores, s_comp));
        int64_t kk = 0;
        ST_TRY(sage_select(d_scores, N, keep_rate, d_idx, &kk, s_comp));
        if (scores_host) CU_TRY(cudaMemcpyAsync(scores_host, d_scores, (size_t)N * sizeof(float), cudaMemcpyDeviceToHost, s_comp));
        if (k > 0) CU_TRY(cudaMemcpyAsync(idx_host, d_idx, (size_t)k * sizeof(int64_t), cudaMemcpyDeviceToHost, s_comp));
        CU_TRY(cudaStreamSynchronize(s_comp));
        CU_TRY(cudaStreamSynchronize(s_copy));
        // what the device recorded during pass 2 (pass 1 was reported by the freeze)
        int tc_err = 0;
        EigInfo info;
        CU_TRY(cudaMemcpy(&tc_err, h->tc_err, sizeof tc_err, cudaMemcpyDeviceToHost));
        CU_TRY(cudaMemcpy(&info, h->info, sizeof info, cudaMemcpyDeviceToHost));
        if (tc_err || (info.flags & kFlagExchangeTimeout)) {
            set_err("sage_select_from_host: a kernel gave up a bounded wait during the scoring pass (results are not valid)");
            return SAGE_ERR_CUDA;
        }
        if ((info.flags & kFlagNonFinite) && rc == SAGE_OK) {
            set_err("sage_select_from_host: non-finite values were met in the rows (such rows score 0)");
            rc = SAGE_ERR_NONFINITE;
        }
        return SAGE_OK;
    };
    sage_status_t s = body();
    cudaDeviceSynchronize();
    for (int i = 0; i < 2; ++i) {
        cudaFree(stage[i]);
        if (copied[i]) cudaEventDestroy(copied[i]);
        if (consumed[i]) cudaEventDestroy(consumed[i]);
    }
    cudaFree(d_scores);
    cudaFree(d_idx);
    if (s_copy) cudaStreamDestroy(s_copy);
    if (s_comp) cudaStreamDestroy(s_comp);
    sage_fd_destroy(h);
    if (s != SAGE_OK) return s;
    if (k_out) *k_out = k;
    return rc;
}

}  // extern "C"

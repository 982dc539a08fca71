// SAGE selection oracle: a plain fp64 CPU statement of what the hot path computes.
//
// THIS IS TEST INFRASTRUCTURE. It exists to check the CUDA library; it shares no code with it and
// is never on the product path. Naive loops, no BLAS/LAPACK. OpenMP is used only over work the
// algorithm leaves independent (disjoint row pairs of one Jacobi round, rows of the scoring pass),
// so results do not depend on the thread count.
//
// What it follows (paper sections / algorithm):
//   * Frequent-Directions sketch, Method section, first paragraph and Algorithm 1, Phase I:
//     insert rows; when the buffer is full take the SVD, delta = sigma_ell^2,
//     Sigma'_jj = sqrt(max(sigma_j^2 - delta, 0)), S <- Sigma' V^T.
//   * Two-pass scoring, Method section, paragraph on two-pass scoring, and Algorithm 1, Phase II:
//     z_i = S g_i, zhat_i = z_i/||z_i|| (0 if z_i = 0), zbar = mean zhat, u = zbar/||zbar|| (0 if zbar = 0),
//     alpha_i = <zhat_i, u>.
//   * Selection, Algorithm 1 last branch: top-k indices by alpha.
//
// Readings taken where the paper is silent or inconsistent (all listed in the design notes):
//   - buffer of m = 2*ell rows, append into free rows, shrink when all m rows are used (the fast
//     Frequent-Directions form of the works the paper cites; a literal ell-row buffer with insertion at
//     r mod ell would overwrite the sketch and cannot satisfy the guarantee the paper quotes);
//   - delta = sigma_ell^2 with sigma sorted descending over the m values, 1-indexed, so ell-1 rows survive;
//   - end of stream: orthogonalise, shrink only if more than ell rows are in use, S = first ell rows;
//   - k = floor(keep_rate*N + 0.5) clamped to [0, N]; order (alpha descending, index ascending).
//
// The SVD is a one-sided (Hestenes) Jacobi on the rows of the buffer: rotating rows until they are
// mutually orthogonal leaves rows sigma_j v_j^T, i.e. Sigma V^T, directly. A second, independent
// route (Gram matrix -> two-sided Jacobi eigen-solve -> rebuild) is provided for cross-checks and for
// inputs whose D makes the first route too slow.
//
// Parity pins: every function here is pinned by tests/test_oracle_*.py (closed forms, brute force
// through numpy's SVD/eigh on tiny inputs, the Frequent-Directions guarantees, invariances).
// "End to end versus values printed in the paper": parity unpinned, the paper prints none.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>

namespace {

using std::int64_t;

inline double bf16_to_double(uint16_t h) {
    uint32_t bits = static_cast<uint32_t>(h) << 16;
    float f;
    std::memcpy(&f, &bits, sizeof f);
    return static_cast<double>(f);
}

// Round-robin tournament: round r of n-1 (n even) pairs up n players so that each pair meets once.
// Pairs of one round are disjoint, which is what makes them independent.
void round_pairs(int n_even, int round, std::vector<std::pair<int, int>>& out) {
    out.clear();
    const int n = n_even;
    for (int i = 0; i < n / 2; ++i) {
        int a = (i == 0) ? n - 1 : (round + i) % (n - 1);
        int b = (round + n - 1 - i) % (n - 1);
        if (i == 0) b = round % (n - 1);
        out.emplace_back(std::min(a, b), std::max(a, b));
    }
}

struct FD {
    int64_t D = 0;
    int ell = 0;
    int m = 0;             // buffer rows = 2*ell
    int delta_rank = 0;    // which sigma (1-indexed, descending) defines delta; default ell
    int route = 0;         // 0: Hestenes on rows, 1: Gram + eigen-solve
    int fill = 0;
    int64_t rows_seen = 0;
    int64_t shrinks = 0;
    double sum_delta = 0.0;
    int last_sweeps = 0;
    bool finalized = false;
    std::vector<double> B;       // m x D row-major
    std::vector<double> sigma;   // after finalize: ell values
    double* row(int i) { return B.data() + static_cast<int64_t>(i) * D; }
};

// Makes rows 0..r-1 of the buffer mutually orthogonal by plane rotations of row pairs (Hestenes).
int hestenes_rows(FD& s, int r) {
    const int64_t D = s.D;
    double F2 = 0.0;
    for (int i = 0; i < r; ++i) {
        const double* b = s.row(i);
        double a = 0.0;
        for (int64_t d = 0; d < D; ++d) a += b[d] * b[d];
        F2 += a;
    }
    if (F2 == 0.0 || r < 2) return 0;
    const int n_even = r + (r & 1);
    std::vector<std::pair<int, int>> pairs;
    int sweep = 0;
    for (; sweep < 60; ++sweep) {
        int rotated = 0;
        for (int round = 0; round < n_even - 1; ++round) {
            round_pairs(n_even, round, pairs);
            const int np = static_cast<int>(pairs.size());
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : rotated)
            for (int t = 0; t < np; ++t) {
                const int i = pairs[t].first, j = pairs[t].second;
                if (j >= r) continue;                       // the bye of an odd row count
                double* bi = s.row(i);
                double* bj = s.row(j);
                double alpha = 0.0, beta = 0.0, gamma = 0.0;
                for (int64_t d = 0; d < D; ++d) {
                    alpha += bi[d] * bi[d];
                    beta += bj[d] * bj[d];
                    gamma += bi[d] * bj[d];
                }
                const double ag = std::fabs(gamma);
                if (ag <= 1e-13 * std::sqrt(alpha * beta) || ag <= 1e-24 * F2) continue;
                const double zeta = (beta - alpha) / (2.0 * gamma);
                const double t_ = (zeta >= 0.0 ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
                const double c = 1.0 / std::sqrt(1.0 + t_ * t_);
                const double sn = c * t_;
                for (int64_t d = 0; d < D; ++d) {
                    const double x = bi[d], y = bj[d];
                    bi[d] = c * x - sn * y;
                    bj[d] = sn * x + c * y;
                }
                ++rotated;
            }
        }
        if (rotated == 0) break;
    }
    return sweep;
}

// Cyclic two-sided Jacobi for a symmetric n x n matrix K (row-major, destroyed): K = U diag(lam) U^T.
int jacobi_eig(std::vector<double>& K, int n, std::vector<double>& U, std::vector<double>& lam) {
    U.assign(static_cast<size_t>(n) * n, 0.0);
    for (int i = 0; i < n; ++i) U[static_cast<size_t>(i) * n + i] = 1.0;
    auto a = [&](int i, int j) -> double& { return K[static_cast<size_t>(i) * n + j]; };
    double F2 = 0.0;
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) F2 += a(i, j) * a(i, j);
    int sweep = 0;
    for (; sweep < 100 && F2 > 0.0; ++sweep) {
        double off = 0.0;
        for (int i = 0; i < n; ++i)
            for (int j = i + 1; j < n; ++j) off += 2.0 * a(i, j) * a(i, j);
        if (off <= 1e-30 * F2) break;
        for (int p = 0; p < n - 1; ++p) {
            for (int q = p + 1; q < n; ++q) {
                const double apq = a(p, q);
                if (apq == 0.0) continue;
                const double zeta = (a(q, q) - a(p, p)) / (2.0 * apq);
                const double t = (zeta >= 0.0 ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
                const double c = 1.0 / std::sqrt(1.0 + t * t);
                const double s = c * t;
                for (int k = 0; k < n; ++k) {           // columns p, q
                    const double x = a(k, p), y = a(k, q);
                    a(k, p) = c * x - s * y;
                    a(k, q) = s * x + c * y;
                }
                for (int k = 0; k < n; ++k) {           // rows p, q
                    const double x = a(p, k), y = a(q, k);
                    a(p, k) = c * x - s * y;
                    a(q, k) = s * x + c * y;
                }
                for (int k = 0; k < n; ++k) {
                    double& up = U[static_cast<size_t>(k) * n + p];
                    double& uq = U[static_cast<size_t>(k) * n + q];
                    const double x = up, y = uq;
                    up = c * x - s * y;
                    uq = s * x + c * y;
                }
            }
        }
    }
    lam.resize(n);
    for (int i = 0; i < n; ++i) lam[i] = a(i, i);
    return sweep;
}

// Leaves rows 0..r-1 as sigma_j v_j^T sorted by sigma descending; returns sigma^2 in sig2 (size r).
void orthogonalise_and_sort(FD& s, int r, std::vector<double>& sig2) {
    const int64_t D = s.D;
    if (s.route == 0) {
        s.last_sweeps = hestenes_rows(s, r);
    } else {
        std::vector<double> K(static_cast<size_t>(r) * r), U, lam;
#pragma omp parallel for schedule(dynamic, 1)
        for (int i = 0; i < r; ++i)
            for (int j = i; j < r; ++j) {
                const double *bi = s.row(i), *bj = s.row(j);
                double acc = 0.0;
                for (int64_t d = 0; d < D; ++d) acc += bi[d] * bj[d];
                K[static_cast<size_t>(i) * r + j] = acc;
            }
        for (int i = 0; i < r; ++i)
            for (int j = 0; j < i; ++j) K[static_cast<size_t>(i) * r + j] = K[static_cast<size_t>(j) * r + i];
        s.last_sweeps = jacobi_eig(K, r, U, lam);
        // rows <- U^T B : row j becomes sum_i U[i][j] B[i], which is sigma_j v_j^T
        std::vector<double> out(static_cast<size_t>(r) * D);
#pragma omp parallel for schedule(static)
        for (int j = 0; j < r; ++j) {
            double* o = out.data() + static_cast<int64_t>(j) * D;
            for (int64_t d = 0; d < D; ++d) o[d] = 0.0;
            for (int i = 0; i < r; ++i) {
                const double u = U[static_cast<size_t>(i) * r + j];
                const double* bi = s.row(i);
                for (int64_t d = 0; d < D; ++d) o[d] += u * bi[d];
            }
        }
        std::memcpy(s.B.data(), out.data(), out.size() * sizeof(double));
    }
    std::vector<double> n2(r);
    for (int i = 0; i < r; ++i) {
        const double* b = s.row(i);
        double a = 0.0;
        for (int64_t d = 0; d < D; ++d) a += b[d] * b[d];
        n2[i] = a;
    }
    std::vector<int> order(r);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return n2[x] > n2[y]; });
    std::vector<double> tmp(static_cast<size_t>(r) * D);
    for (int j = 0; j < r; ++j) std::memcpy(tmp.data() + static_cast<int64_t>(j) * D, s.row(order[j]), D * sizeof(double));
    std::memcpy(s.B.data(), tmp.data(), tmp.size() * sizeof(double));
    sig2.resize(r);
    for (int j = 0; j < r; ++j) sig2[j] = n2[order[j]];
}

// The shrink: rows are sigma_j v_j^T sorted; subtract delta = sigma_rank^2 from every sigma^2.
void apply_shrink(FD& s, int r, const std::vector<double>& sig2) {
    const int64_t D = s.D;
    const int rank = s.delta_rank;                          // 1-indexed
    const double delta = (rank - 1 < r) ? sig2[rank - 1] : 0.0;
    for (int j = 0; j < r; ++j) {
        double* b = s.row(j);
        const double kept = std::max(sig2[j] - delta, 0.0);
        if (j >= rank - 1 || kept == 0.0 || sig2[j] <= 0.0) {
            for (int64_t d = 0; d < D; ++d) b[d] = 0.0;
        } else {
            const double f = std::sqrt(kept) / std::sqrt(sig2[j]);
            for (int64_t d = 0; d < D; ++d) b[d] *= f;
        }
    }
    for (int j = r; j < s.m; ++j) {
        double* b = s.row(j);
        for (int64_t d = 0; d < D; ++d) b[d] = 0.0;
    }
    s.sum_delta += delta;
    s.shrinks += 1;
    s.fill = rank - 1;
}

void shrink_full(FD& s) {
    std::vector<double> sig2;
    orthogonalise_and_sort(s, s.m, sig2);
    apply_shrink(s, s.m, sig2);
}

template <typename Load>
void update_rows(FD& s, int64_t n, Load load) {
    for (int64_t i = 0; i < n; ++i) {
        double* dst = s.row(s.fill);
        for (int64_t d = 0; d < s.D; ++d) dst[d] = load(i, d);
        s.fill += 1;
        s.rows_seen += 1;
        if (s.fill == s.m) shrink_full(s);
    }
}

template <typename Load>
void score_rows(const double* S, int ell, int64_t D, int64_t n, Load load, double* zhat, double* znorm,
                double* zbar, double* u, double* alpha) {
    std::vector<double> zh_local;
    if (!zhat) {
        zh_local.resize(static_cast<size_t>(n) * ell);
        zhat = zh_local.data();
    }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double* z = zhat + i * ell;
        double nn = 0.0;
        for (int j = 0; j < ell; ++j) {
            const double* sj = S + static_cast<int64_t>(j) * D;
            double acc = 0.0;
            for (int64_t d = 0; d < D; ++d) acc += sj[d] * load(i, d);
            z[j] = acc;
            nn += acc * acc;
        }
        nn = std::sqrt(nn);
        if (znorm) znorm[i] = nn;
        if (nn > 0.0) {
            for (int j = 0; j < ell; ++j) z[j] /= nn;
        } else {
            for (int j = 0; j < ell; ++j) z[j] = 0.0;
        }
    }
    std::vector<double> sum(ell, 0.0);
    for (int64_t i = 0; i < n; ++i)
        for (int j = 0; j < ell; ++j) sum[j] += zhat[i * ell + j];
    double un = 0.0;
    std::vector<double> zb(ell), uu(ell, 0.0);
    for (int j = 0; j < ell; ++j) {
        zb[j] = n > 0 ? sum[j] / static_cast<double>(n) : 0.0;
        un += zb[j] * zb[j];
    }
    un = std::sqrt(un);
    if (un > 0.0)
        for (int j = 0; j < ell; ++j) uu[j] = zb[j] / un;
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int j = 0; j < ell; ++j) acc += zhat[i * ell + j] * uu[j];
        alpha[i] = acc;
    }
    if (zbar) std::memcpy(zbar, zb.data(), ell * sizeof(double));
    if (u) std::memcpy(u, uu.data(), ell * sizeof(double));
}

}  // namespace

extern "C" {

void* sage_oracle_fd_create(int64_t D, int ell, int delta_rank, int route) {
    if (D <= 0 || ell < 2) return nullptr;
    FD* s = new FD();
    s->D = D;
    s->ell = ell;
    s->m = 2 * ell;
    s->delta_rank = delta_rank > 0 ? delta_rank : ell;
    s->route = route;
    s->B.assign(static_cast<size_t>(s->m) * D, 0.0);
    return s;
}

void sage_oracle_fd_destroy(void* h) { delete static_cast<FD*>(h); }

void sage_oracle_fd_update_f64(void* h, const double* rows, int64_t n, int64_t ld) {
    update_rows(*static_cast<FD*>(h), n, [=](int64_t i, int64_t d) { return rows[i * ld + d]; });
}
void sage_oracle_fd_update_f32(void* h, const float* rows, int64_t n, int64_t ld) {
    update_rows(*static_cast<FD*>(h), n, [=](int64_t i, int64_t d) { return static_cast<double>(rows[i * ld + d]); });
}
void sage_oracle_fd_update_bf16(void* h, const uint16_t* rows, int64_t n, int64_t ld) {
    update_rows(*static_cast<FD*>(h), n, [=](int64_t i, int64_t d) { return bf16_to_double(rows[i * ld + d]); });
}

// The freeze step of Algorithm 1: orthogonalise what is in the buffer, shrink only when more than ell rows are in use.
void sage_oracle_fd_finalize(void* h) {
    FD& s = *static_cast<FD*>(h);
    std::vector<double> sig2;
    const int r = s.fill;
    orthogonalise_and_sort(s, r, sig2);
    if (r > s.ell) apply_shrink(s, r, sig2);
    s.sigma.assign(s.ell, 0.0);
    for (int j = 0; j < s.ell; ++j) {
        const double* b = s.row(j);
        double a = 0.0;
        for (int64_t d = 0; d < s.D; ++d) a += b[d] * b[d];
        s.sigma[j] = std::sqrt(a);
    }
    s.finalized = true;
}

// Copies the ell x D sketch (row-major, pitch D) and its ell row norms.
void sage_oracle_fd_sketch(void* h, double* S, double* sigma) {
    FD& s = *static_cast<FD*>(h);
    std::memcpy(S, s.B.data(), static_cast<size_t>(s.ell) * s.D * sizeof(double));
    if (sigma) std::memcpy(sigma, s.sigma.data(), s.ell * sizeof(double));
}

// Raw buffer access for tests that inspect the state between updates (m x D, pitch D).
void sage_oracle_fd_buffer(void* h, double* B, int* fill) {
    FD& s = *static_cast<FD*>(h);
    std::memcpy(B, s.B.data(), s.B.size() * sizeof(double));
    *fill = s.fill;
}

void sage_oracle_fd_stats(void* h, int64_t* rows_seen, int64_t* shrinks, double* sum_delta, int* last_sweeps) {
    FD& s = *static_cast<FD*>(h);
    *rows_seen = s.rows_seen;
    *shrinks = s.shrinks;
    *sum_delta = s.sum_delta;
    *last_sweeps = s.last_sweeps;
}

void sage_oracle_score_f64(const double* S, int ell, int64_t D, const double* rows, int64_t n, int64_t ld,
                           double* zhat, double* znorm, double* zbar, double* u, double* alpha) {
    score_rows(S, ell, D, n, [=](int64_t i, int64_t d) { return rows[i * ld + d]; }, zhat, znorm, zbar, u, alpha);
}
void sage_oracle_score_f32(const double* S, int ell, int64_t D, const float* rows, int64_t n, int64_t ld,
                           double* zhat, double* znorm, double* zbar, double* u, double* alpha) {
    score_rows(S, ell, D, n, [=](int64_t i, int64_t d) { return static_cast<double>(rows[i * ld + d]); }, zhat, znorm,
               zbar, u, alpha);
}
void sage_oracle_score_bf16(const double* S, int ell, int64_t D, const uint16_t* rows, int64_t n, int64_t ld,
                            double* zhat, double* znorm, double* zbar, double* u, double* alpha) {
    score_rows(S, ell, D, n, [=](int64_t i, int64_t d) { return bf16_to_double(rows[i * ld + d]); }, zhat, znorm, zbar,
               u, alpha);
}

// Top-k by alpha, ties to the smaller index; idx must hold k entries. Returns k.
int64_t sage_oracle_select_k(int64_t N, double keep_rate) {
    double k = std::floor(keep_rate * static_cast<double>(N) + 0.5);
    if (k < 0.0) k = 0.0;
    if (k > static_cast<double>(N)) k = static_cast<double>(N);
    return static_cast<int64_t>(k);
}
int64_t sage_oracle_select(const double* alpha, int64_t N, double keep_rate, int64_t* idx) {
    const int64_t k = sage_oracle_select_k(N, keep_rate);
    std::vector<int64_t> order(N);
    std::iota(order.begin(), order.end(), int64_t{0});
    std::stable_sort(order.begin(), order.end(), [&](int64_t a, int64_t b) { return alpha[a] > alpha[b]; });
    for (int64_t i = 0; i < k; ++i) idx[i] = order[i];
    return k;
}

// Symmetric eigen-solve exposed for its own pins: K (n x n, row-major) -> U (columns), lam (unsorted).
int sage_oracle_jacobi_eig(const double* K, int n, double* U, double* lam) {
    std::vector<double> k(K, K + static_cast<size_t>(n) * n), u, l;
    const int sweeps = jacobi_eig(k, n, u, l);
    std::memcpy(U, u.data(), u.size() * sizeof(double));
    std::memcpy(lam, l.data(), l.size() * sizeof(double));
    return sweeps;
}

}  // extern "C"

// Host-side builder of the CERAR coefficient matrices (fp64 results; extended
// precision inside where the windows A_l are ill-conditioned by construction).
#include "plan.hpp"
#include <atomic>
#include <thread>
#include <algorithm>

#include <cmath>
#include <limits>

#include "linalg.hpp"

namespace cerar {

using la::MatD;
using la::MatL;
typedef long double ld;

std::vector<double> default_nodes(int c) {
    std::vector<double> v(c, 0.0);
    for (int j = 0; j < c; ++j) v[j] = (c == 1) ? 0.0 : -1.0 + 2.0 * j / (c - 1);
    return v;
}

static inline uint64_t splitmix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

std::vector<double> default_base_matrix(int N, int c, uint64_t seed) {
    std::vector<double> B((size_t)N * c);
    const double two_pi = 6.283185307179586476925286766559;
    for (size_t t = 0; t < B.size(); ++t) {
        uint64_t a = splitmix64(seed * 0x100000001B3ull + 2 * t);
        uint64_t b = splitmix64(seed * 0x100000001B3ull + 2 * t + 1);
        double u1 = ((a >> 11) + 1.0) * (1.0 / 9007199254740993.0);   // (0, 1)
        double u2 = (b >> 11) * (1.0 / 9007199254740992.0);           // [0, 1)
        B[t] = std::sqrt(-2.0 * std::log(u1)) * std::cos(two_pi * u2);
    }
    return B;
}

static void alloc_plan(int N, int c, HostPlan& P) {
    P.N = N; P.c = c; P.L = c + N - 2;
    P.U.assign(N, std::vector<double>((size_t)c * c, 0.0));
    P.R.assign(N, std::vector<double>((size_t)(P.L + 1) * c, 0.0));
}

static bool all_finite(const HostPlan& P) {
    for (const auto& m : P.U) for (double v : m) if (!std::isfinite(v)) return false;
    for (const auto& m : P.R) for (double v : m) if (!std::isfinite(v)) return false;
    return true;
}

static inline void floor_divmod(int l, int N, int& m, int& r) {
    m = l / N; r = l % N;
    if (r < 0) { r += N; m -= 1; }
}

// ---------------------------------------------------------------- Vandermonde
//
// A_l[r, j] = z_j^(l+r) = W[r, j] z_j^l with W the Vandermonde matrix of the
// nodes, so A_l^{-1} = diag(z^-l) W^{-1}, and row j of W^{-1} holds the
// monomial coefficients of the Lagrange basis polynomial
//   L_j(x) = prod_{m != j} (x - z_m) / (z_j - z_m).
// Expanding the product involves no cancellation (all nodes are positive, the
// coefficients alternate in sign) and the node differences come from expm1, so
// every entry keeps full relative accuracy although kappa(A_l) is enormous.
int build_vandermonde(int N, int c, double tau, const double* xi_in, HostPlan& P, std::string& err) {
    if (N < 2 || c < N) { err = "need 2 <= N <= c"; return BUILD_INVALID; }
    if (!(tau > 0) || !std::isfinite(tau)) { err = "tau must be positive"; return BUILD_INVALID; }
    std::vector<double> xi = xi_in ? std::vector<double>(xi_in, xi_in + c) : default_nodes(c);
    for (int a = 0; a < c; ++a)
        for (int b = a + 1; b < c; ++b)
            if (xi[a] == xi[b]) { err = "Vandermonde nodes must be distinct"; return BUILD_INVALID; }
    alloc_plan(N, c, P);
    P.kind = 0; P.param = tau;
    const int L = P.L;
    std::vector<ld> z(c);
    for (int j = 0; j < c; ++j) z[j] = std::exp((ld)tau * (ld)xi[j]);
    // W^{-1}
    MatL Winv(c, c);
    std::vector<ld> poly(c), next(c);
    for (int j = 0; j < c; ++j) {
        std::fill(poly.begin(), poly.end(), (ld)0);
        poly[0] = 1;
        int deg = 0;
        ld denom = 1;
        for (int m = 0; m < c; ++m) {
            if (m == j) continue;
            // poly <- poly * (x - z_m)
            for (int t = 0; t <= deg + 1; ++t) {
                ld lo = (t <= deg) ? -z[m] * poly[t] : (ld)0;
                ld hi = (t >= 1) ? poly[t - 1] : (ld)0;
                next[t] = lo + hi;
            }
            ++deg;
            for (int t = 0; t <= deg; ++t) poly[t] = next[t];
            denom *= z[m] * std::expm1((ld)tau * ((ld)xi[j] - (ld)xi[m]));
        }
        for (int r = 0; r < c; ++r) Winv(j, r) = poly[r] / denom;
    }
    for (int k = 0; k < N; ++k) {
        const int l = N - 1 - k;          // U_k = A_{N-1-k}^{-1}
        for (int j = 0; j < c; ++j) {
            ld zl = std::exp(-(ld)tau * (ld)xi[j] * (ld)l);
            for (int r = 0; r < c; ++r) P.U[k][(size_t)j * c + r] = (double)(zl * Winv(j, r));
        }
    }
    for (int i = 0; i < N; ++i)
        for (int l = 0; l <= L; ++l)
            for (int j = 0; j < c; ++j)
                P.R[i][(size_t)l * c + j] = (double)std::exp((ld)tau * (ld)xi[j] * (ld)(l - i));
    // Prop. 2: Phi = N(N-1)/2 ||D^{-1} - I||_F^2 with D = diag(z_j^N)
    ld ph = 0;
    for (int j = 0; j < c; ++j) { ld e = std::expm1(-(ld)N * (ld)tau * (ld)xi[j]); ph += e * e; }
    P.phi_closed = (double)(ph * (ld)N * (ld)(N - 1) / 2);
    // inverse residual (extended precision, informative only)
    ld worst = 0;
    for (int k = 0; k < N; ++k) {
        const int l = N - 1 - k;
        for (int a = 0; a < c; ++a)
            for (int b = 0; b < c; ++b) {
                ld s = 0;
                for (int r = 0; r < c; ++r)
                    s += (ld)P.U[k][(size_t)a * c + r] * std::exp((ld)tau * (ld)xi[b] * (ld)(l + r));
                worst = std::max(worst, std::fabs(s - (a == b ? (ld)1 : (ld)0)));
            }
    }
    P.inv_residual_max = (double)worst;
    if (!all_finite(P)) { err = "non-finite Vandermonde coefficients"; return BUILD_SINGULAR; }
    return BUILD_OK;
}

// ---------------------------------------------------------------- epsilon
//
// a_{r+mN} = b_r D^m with D = I + eps diag(h).  The window A_l is inverted
// through the finite-difference factorisation of the appendix,
//     F~_l Pi_l A_l = Lambda_l K_l   =>   A_l^{-1} = K_l^{-1} Lambda_l^{-1} F~_l Pi_l,
// where the rows of K_l are b_alpha D^{m_alpha} H^j (formed directly, so the
// eps^j scaling that makes A_l ill-conditioned never enters an elimination),
// Lambda_l = diag(eps^j), F~_l is block diagonal with exact integer binomials.
static ld ipow(ld x, int n) {
    if (n < 0) return (ld)1 / ipow(x, -n);
    ld r = 1;
    for (int t = 0; t < n; ++t) r *= x;
    return r;
}

static ld binom(int n, int k) {
    ld r = 1;
    for (int t = 1; t <= k; ++t) r = r * (ld)(n - k + t) / (ld)t;
    return std::round(r);
}

int build_epsilon(int N, int c, double eps, const double* B, const double* h_in, HostPlan& P,
                  std::string& err) {
    if (N < 2 || c < N) { err = "need 2 <= N <= c"; return BUILD_INVALID; }
    if (!B) { err = "base matrix missing"; return BUILD_INVALID; }
    if (!std::isfinite(eps) || eps < 0) { err = "eps must be >= 0"; return BUILD_INVALID; }
    std::vector<double> h = h_in ? std::vector<double>(h_in, h_in + c) : default_nodes(c);
    double hmax = 0;
    for (double v : h) hmax = std::max(hmax, std::fabs(v));
    if (!(eps * hmax < 1.0)) { err = "need eps * ||H||_2 < 1"; return BUILD_INVALID; }
    if (eps == 0.0 && c > N) { err = "eps = 0 with c > N gives singular windows"; return BUILD_SINGULAR; }
    alloc_plan(N, c, P);
    P.kind = 1; P.param = eps;
    const int L = P.L;
    std::vector<ld> dj(c);
    for (int j = 0; j < c; ++j) dj[j] = (ld)1 + (ld)eps * (ld)h[j];

    ld worst = 0;
    for (int k = 0; k < N; ++k) {
        const int l = N - 1 - k;
        // group the window's rows t = 0..c-1 (sequence index l+t) by remainder
        std::vector<std::vector<int>> rows_of(N);
        std::vector<int> m_first(N, 0);
        for (int t = 0; t < c; ++t) {
            int m, a;
            floor_divmod(l + t, N, m, a);
            if (rows_of[a].empty()) m_first[a] = m;
            rows_of[a].push_back(t);
        }
        MatL K(c, c), Q(c, c);
        int row = 0;
        for (int a = 0; a < N; ++a) {
            const int n_a = (int)rows_of[a].size();
            for (int j = 0; j < n_a; ++j, ++row) {
                for (int col = 0; col < c; ++col)
                    K(row, col) = (ld)B[(size_t)a * c + col] * ipow(dj[col], m_first[a]) * ipow((ld)h[col], j);
                // row (a, j) of Lambda^{-1} F~ Pi: eps^-j * (-1)^(j-kk) C(j,kk) at the kk-th row of the group
                for (int kk = 0; kk <= j; ++kk) {
                    ld f = (((j - kk) & 1) ? (ld)-1 : (ld)1) * binom(j, kk);
                    Q(row, rows_of[a][kk]) = f * ipow((ld)eps, -j);
                }
            }
        }
        MatL Kinv;
        if (!la::inverse(K, Kinv)) { err = "K_l(B, H) is singular: choose another B or H"; return BUILD_SINGULAR; }
        MatL Uk = la::matmul(Kinv, Q);
        for (int a = 0; a < c; ++a)
            for (int b = 0; b < c; ++b) P.U[k][(size_t)a * c + b] = (double)Uk(a, b);
        // residual U_k A_l - I in extended precision
        for (int a = 0; a < c; ++a)
            for (int b = 0; b < c; ++b) {
                ld s = 0;
                for (int t = 0; t < c; ++t) {
                    int m, r;
                    floor_divmod(l + t, N, m, r);
                    s += (ld)P.U[k][(size_t)a * c + t] * (ld)B[(size_t)r * c + b] * ipow(dj[b], m);
                }
                worst = std::max(worst, std::fabs(s - (a == b ? (ld)1 : (ld)0)));
            }
    }
    P.inv_residual_max = (double)worst;
    for (int i = 0; i < N; ++i)
        for (int l = 0; l <= L; ++l) {
            int m, r;
            floor_divmod(l - i, N, m, r);
            for (int j = 0; j < c; ++j)
                P.R[i][(size_t)l * c + j] = (double)((ld)B[(size_t)r * c + j] * ipow(dj[j], m));
        }
    ld ph = 0;
    for (int j = 0; j < c; ++j) { ld e = (ld)1 / dj[j] - (ld)1; ph += e * e; }
    P.phi_closed = (double)(ph * (ld)N * (ld)(N - 1) / 2);
    if (!all_finite(P)) { err = "non-finite epsilon-construction coefficients"; return BUILD_SINGULAR; }
    return BUILD_OK;
}

// ---------------------------------------------------------------- diagnostics

static MatD mat_of(const std::vector<double>& v, int rows, int cols) {
    MatD M(rows, cols);
    M.a = v;
    return M;
}

static MatD m_matrix(const HostPlan& P, int i) {
    const int N = P.N, c = P.c, L = P.L;
    MatD M(N * c, L + 1);
    for (int r = 0; r < N; ++r) {
        const std::vector<double>& U = P.U[(i + r) % N];
        for (int a = 0; a < c; ++a)
            for (int b = 0; b < c; ++b) M(r * c + a, N - 1 - r + b) = U[(size_t)a * c + b];
    }
    return M;
}

template <class Acc>
static double phi_blocks(const HostPlan& P) {
    const int N = P.N, c = P.c;
    Acc tot = 0;
    std::vector<Acc> rowacc(c);
    for (int i = 0; i < N; ++i)
        for (int s = 0; s < N; ++s) {
            const std::vector<double>& U = P.U[((i - 1 - s) % N + N) % N];
            const std::vector<double>& R = P.R[i];
            for (int a = 0; a < c; ++a) {
                // row a of U W_s(R_i) - I, accumulated over the window rows (contiguous in R)
                for (int b = 0; b < c; ++b) rowacc[b] = (a == b) ? (Acc)-1 : (Acc)0;
                for (int t = 0; t < c; ++t) {
                    const Acc u = (Acc)U[(size_t)a * c + t];
                    const double* r = &R[(size_t)(s + t) * c];
                    for (int b = 0; b < c; ++b) rowacc[b] += u * (Acc)r[b];
                }
                for (int b = 0; b < c; ++b) tot += rowacc[b] * rowacc[b];
            }
        }
    return (double)tot;
}

double k_limit_gamma(int N, int c, const double* B, const double* h) {
    const int beta = c / N, s = c % N;
    // rows B H^j for j = 0..beta (the last block only partly used)
    std::vector<double> pw((size_t)(beta + 1) * N * c);
    for (int r = 0; r < N; ++r)
        for (int q = 0; q < c; ++q) {
            double v = B[(size_t)r * c + q];
            for (int j = 0; j <= beta; ++j) {
                pw[((size_t)j * N + r) * c + q] = v;
                v *= h[q];
            }
        }
    double gamma = std::numeric_limits<double>::infinity();
    const int windows = (s == 0) ? 1 : N;          // without the partial block every l gives the same matrix
    for (int l = 0; l < windows; ++l) {
        la::MatD K(c, c);
        int row = 0;
        for (int j = 0; j < beta; ++j)
            for (int r = 0; r < N; ++r, ++row)
                for (int q = 0; q < c; ++q) K(row, q) = pw[((size_t)j * N + r) * c + q];
        for (int t = 0; t < s; ++t, ++row) {
            const int r = (l + t) % N;
            for (int q = 0; q < c; ++q) K(row, q) = pw[((size_t)beta * N + r) * c + q];
        }
        la::MatD Uo, V;
        std::vector<double> sv;
        la::svd_jacobi(K, Uo, sv, V);
        gamma = std::min(gamma, sv.back());
    }
    return gamma;
}

double optimize_h(int N, int c, const double* B, double* h, int sweeps, int grid, int* moves_out) {
    double hmax = 0;
    for (int j = 0; j < c; ++j) hmax = std::max(hmax, std::fabs(h[j]));
    if (hmax > 0) for (int j = 0; j < c; ++j) h[j] /= hmax;
    std::vector<double> cand(grid);
    for (int t = 0; t < grid; ++t) cand[t] = -1.0 + 2.0 * t / (grid - 1);
    double best = k_limit_gamma(N, c, B, h);
    int moves = 0;
    for (int sweep = 0; sweep < sweeps; ++sweep) {
        bool moved = false;
        for (int j = 0; j < c; ++j) {
            const double keep = h[j];
            double val_j = best, best_j = keep;
            bool found = false;
            for (int t = 0; t < grid; ++t) {
                if (cand[t] == keep) continue;
                h[j] = cand[t];
                double m = 0;
                for (int q = 0; q < c; ++q) m = std::max(m, std::fabs(h[q]));
                if (m < 1.0) continue;                         // ||H||_2 = 1 stays: choices remain comparable
                const double v = k_limit_gamma(N, c, B, h);
                if (v > val_j * (1 + 1e-12)) { val_j = v; best_j = cand[t]; found = true; }
            }
            h[j] = best_j;
            if (found) { best = val_j; moved = true; ++moves; }
        }
        if (!moved) break;
    }
    if (moves_out) *moves_out = moves;
    return best;
}

double phi_direct(const HostPlan& P) { return phi_blocks<ld>(P); }

double kappa_U_max(const HostPlan& P) {
    double k = 0;
    for (int i = 0; i < P.N; ++i) k = std::max(k, la::kappa2(mat_of(P.U[i], P.c, P.c)));
    return k;
}

double kappa_M_max(const HostPlan& P) {
    double k = 0;
    for (int i = 0; i < P.N; ++i) k = std::max(k, la::kappa2(m_matrix(P, i)));
    return k;
}

// ---------------------------------------------------------------- kappa-constrained ALS
//
// minimise Phi(U,R) s.t. kappa_2(M_i(U)) <= C (Sec. II-D).  One iteration:
// least squares in U with R fixed, projection of the singular values of every
// U_k into [a0, b0] (sqrt(N) b0 / a0 = C guarantees the constraint), least
// squares in R with U fixed.  Started from an epsilon-construction.

// The N solves of an ALS step are independent (each writes only its own matrix): one thread each,
// up to the host's core count.  The result does not depend on the number of threads.
template <class F>
static void parallel_for(int n, int c, F fn) {
    unsigned hw = std::thread::hardware_concurrency();
    int nt = (int)std::min<unsigned>(hw ? hw : 1u, (unsigned)n);
    if (c < 24) nt = 1;                 // small solves: starting threads costs more than it saves
    if (nt <= 1) { for (int i = 0; i < n; ++i) fn(i); return; }
    std::vector<std::thread> th;
    std::atomic<int> next(0);
    for (int t = 0; t < nt; ++t)
        th.emplace_back([&]() { for (int i = next.fetch_add(1); i < n; i = next.fetch_add(1)) fn(i); });
    for (auto& x : th) x.join();
}

static void ls_R(HostPlan& P) {
    const int N = P.N, c = P.c, L = P.L;
    MatD T(N * c, c);
    for (int r = 0; r < N; ++r)
        for (int a = 0; a < c; ++a) T(r * c + a, a) = 1.0;
    parallel_for(N, c, [&](int i) {
        MatD X;
        la::lstsq(m_matrix(P, i), T, X);
        for (int l = 0; l <= L; ++l)
            for (int j = 0; j < c; ++j) P.R[i][(size_t)l * c + j] = X(l, j);
    });
}

static void ls_U(HostPlan& P) {
    const int N = P.N, c = P.c;
    parallel_for(N, c, [&](int k) {
        // U_k [W_{s_0}(R_0) ... W_{s_{N-1}}(R_{N-1})] ~ [I ... I], s_i = (i-1-k) mod N;
        // transposed: rows of P^T are the columns of the windows.
        MatD Pt(N * c, c), Tt(N * c, c);
        for (int i = 0; i < N; ++i) {
            const int s = ((i - 1 - k) % N + N) % N;
            for (int a = 0; a < c; ++a)          // window row a -> column of P, row block i of P^T
                for (int b = 0; b < c; ++b) Pt(i * c + b, a) = P.R[i][(size_t)(s + a) * c + b];
            for (int a = 0; a < c; ++a) Tt(i * c + a, a) = 1.0;
        }
        MatD X;                                    // X = U_k^T
        la::lstsq(Pt, Tt, X);
        for (int a = 0; a < c; ++a)
            for (int b = 0; b < c; ++b) P.U[k][(size_t)a * c + b] = X(b, a);
    });
}

static void project(HostPlan& P, double a0, double b0) {
    const int c = P.c;
    parallel_for(P.N, c, [&](int k) {
        MatD Uo, V;
        std::vector<double> s;
        la::svd_jacobi(mat_of(P.U[k], c, c), Uo, s, V);
        for (double& v : s) v = std::min(std::max(v, a0), b0);
        for (int a = 0; a < c; ++a)
            for (int b = 0; b < c; ++b) {
                double acc = 0;
                for (int t = 0; t < c; ++t) acc += Uo(a, t) * s[t] * V(b, t);
                P.U[k][(size_t)a * c + b] = acc;
            }
    });
}

int build_kappa(int N, int c, double kappa_max, const double* B, const double* h, double eps_init,
                int iters, double tol, HostPlan& P, std::string& err) {
    if (!(kappa_max > std::sqrt((double)N)) || !std::isfinite(kappa_max)) {
        err = "kappa_max must exceed sqrt(N)"; return BUILD_INVALID;
    }
    if (eps_init <= 0) eps_init = 0.1;
    if (iters <= 0) iters = 200;
    if (tol <= 0) tol = 1e-6;
    int st = build_epsilon(N, c, eps_init, B, h, P, err);
    if (st != BUILD_OK) return st;
    P.kind = 2; P.param = kappa_max; P.phi_closed = -1.0; P.inv_residual_max = -1.0;
    // a0 = min_k sigma_min(U_k) of the initial design.  The initial encoders have condition numbers up
    // to 1e15 (kappa = Theta(eps^-r*), Sec. II-C), where an SVD of U_k itself gets the smallest singular
    // value wrong in the third digit; U_k^{-1} = A_{N-1-k} is at hand without any inversion (its rows are
    // rows N-1-k .. N-1-k+c-1 of R_0, Eq. decoderconstruction) and has that value as the reciprocal of its
    // LARGEST singular value, which the SVD delivers to full accuracy.
    double a0 = std::numeric_limits<double>::infinity();
    const int L = P.L;
    (void)L;
    for (int l = 0; l < N; ++l) {
        MatD A(c, c);
        for (int t = 0; t < c; ++t)
            for (int j = 0; j < c; ++j) A(t, j) = P.R[0][(size_t)(l + t) * c + j];
        MatD Uo, V; std::vector<double> s;
        la::svd_jacobi(A, Uo, s, V);
        if (!(s.front() > 0)) { a0 = 0; break; }
        a0 = std::min(a0, 1.0 / s.front());
    }
    if (!(a0 > 0) || !std::isfinite(a0)) { err = "initial design is singular"; return BUILD_SINGULAR; }
    const double b0 = a0 * kappa_max / std::sqrt((double)N);
    project(P, a0, b0);
    ls_R(P);
    double prev = phi_blocks<double>(P);     // the projected iterates are well conditioned: fp64 is enough here
    int done = 0;
    for (int it = 0; it < iters; ++it) {
        ls_U(P);
        project(P, a0, b0);
        ls_R(P);
        double cur = phi_blocks<double>(P);
        done = it + 1;
        bool stop = std::fabs(prev - cur) <= tol * std::max(cur, 1e-300);
        prev = cur;
        if (stop) break;
    }
    P.als_iters_done = done;
    if (!all_finite(P)) { err = "non-finite coefficients after ALS"; return BUILD_SINGULAR; }
    if (kappa_M_max(P) > kappa_max * (1 + 1e-9)) { err = "condition-number constraint not met"; return BUILD_NOT_CONVERGED; }
    return BUILD_OK;
}

}  // namespace cerar

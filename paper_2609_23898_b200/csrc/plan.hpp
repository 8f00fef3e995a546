// Host-side (fp64) builder of the CERAR coefficient matrices.  No CUDA here.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace cerar {

struct HostPlan {
    int N = 0, c = 0, L = 0;
    int kind = 3;                 // cerar_construction_t, 3 = custom
    double param = 0.0;
    std::vector<std::vector<double>> U;   // N matrices, c*c, row-major
    std::vector<std::vector<double>> R;   // N matrices, (L+1)*c, row-major
    double phi_closed = -1.0;             // Prop. 2 value for explicit constructions, else < 0
    double inv_residual_max = -1.0;
    int als_iters_done = 0;
};

enum BuildStatus { BUILD_OK = 0, BUILD_INVALID = 1, BUILD_SINGULAR = 3, BUILD_NOT_CONVERGED = 4 };

// c equally spaced values in [-1, 1] (default nodes xi_j and default diag(H)).
std::vector<double> default_nodes(int c);
// N x c matrix of N(0,1) draws: splitmix64 counter stream, Box-Muller.
std::vector<double> default_base_matrix(int N, int c, uint64_t seed);

// Vandermonde construction (Sec. II-B.2): z_j = exp(tau xi_j).
int build_vandermonde(int N, int c, double tau, const double* xi, HostPlan& out, std::string& err);
// epsilon-construction (Sec. II-C) with diagonal H = diag(h).
int build_epsilon(int N, int c, double eps, const double* B, const double* h, HostPlan& out,
                  std::string& err);
// Condition-number-constrained alternating least squares (Sec. II-D).
int build_kappa(int N, int c, double kappa_max, const double* B, const double* h, double eps_init,
                int iters, double tol, HostPlan& out, std::string& err);

// gamma(B, H) = min over l = 0..N-1 of sigma_min(K^(l)(B, H)), the quantity the analysis of the
// epsilon-construction assumes positive (Sec. II-C): K^(l) stacks B, BH, .., BH^(beta-1) and, when
// c = beta N + s with s > 0, the rows {l, .., l+s-1} mod N of BH^beta.  H = diag(h).
double k_limit_gamma(int N, int c, const double* B, const double* h);
// Coordinate ascent on gamma over `grid` equally spaced values of [-1, 1] per coordinate; h is the start and the
// result (scaled to max|h| = 1 first); returns gamma of the result.
double optimize_h(int N, int c, const double* B, double* h, int sweeps, int grid, int* moves_out);

// Phi(U,R) from the block form sum_{i,s} ||U_{i-1-s} W_s(R_i) - I||_F^2.
double phi_direct(const HostPlan& P);
double kappa_U_max(const HostPlan& P);
double kappa_M_max(const HostPlan& P);

}  // namespace cerar

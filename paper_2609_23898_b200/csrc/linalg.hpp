// Small dense linear algebra for the host-side plan builder (row-major).
// Sizes are tiny (c <= a few hundred), so clarity beats blocking.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstddef>
#include <limits>
#include <vector>

namespace cerar {
namespace la {

template <class T>
struct Mat {
    int rows = 0, cols = 0;
    std::vector<T> a;
    Mat() {}
    Mat(int r, int c) : rows(r), cols(c), a((size_t)r * c, T(0)) {}
    T& operator()(int i, int j) { return a[(size_t)i * cols + j]; }
    const T& operator()(int i, int j) const { return a[(size_t)i * cols + j]; }
};
using MatD = Mat<double>;
using MatL = Mat<long double>;

template <class T>
Mat<T> matmul(const Mat<T>& A, const Mat<T>& B) {
    Mat<T> C(A.rows, B.cols);
    for (int i = 0; i < A.rows; ++i)
        for (int k = 0; k < A.cols; ++k) {
            T aik = A(i, k);
            if (aik == T(0)) continue;
            for (int j = 0; j < B.cols; ++j) C(i, j) += aik * B(k, j);
        }
    return C;
}

template <class T>
Mat<T> transpose(const Mat<T>& A) {
    Mat<T> B(A.cols, A.rows);
    for (int i = 0; i < A.rows; ++i)
        for (int j = 0; j < A.cols; ++j) B(j, i) = A(i, j);
    return B;
}

// Inverse by LU with partial pivoting (Gauss-Jordan on [A | I]).  Returns false
// if a pivot is zero or non-finite.
template <class T>
bool inverse(const Mat<T>& Ain, Mat<T>& out) {
    const int n = Ain.rows;
    Mat<T> A = Ain;
    out = Mat<T>(n, n);
    for (int i = 0; i < n; ++i) out(i, i) = T(1);
    for (int col = 0; col < n; ++col) {
        int piv = col;
        T best = std::fabs(A(col, col));
        for (int r = col + 1; r < n; ++r)
            if (std::fabs(A(r, col)) > best) { best = std::fabs(A(r, col)); piv = r; }
        if (!(best > T(0)) || !std::isfinite((double)best)) return false;
        if (piv != col)
            for (int j = 0; j < n; ++j) { std::swap(A(piv, j), A(col, j)); std::swap(out(piv, j), out(col, j)); }
        T inv = T(1) / A(col, col);
        for (int j = 0; j < n; ++j) { A(col, j) *= inv; out(col, j) *= inv; }
        for (int r = 0; r < n; ++r) {
            if (r == col) continue;
            T f = A(r, col);
            if (f == T(0)) continue;
            for (int j = 0; j < n; ++j) { A(r, j) -= f * A(col, j); out(r, j) -= f * out(col, j); }
        }
    }
    return true;
}

// Householder QR of an m x n matrix (m >= n), applied to a right-hand side:
// solves min ||A X - Bm||_F.  Also returns the n x n triangular factor if asked.
inline bool lstsq(const MatD& Ain, const MatD& Bin, MatD& X, MatD* Rout = nullptr) {
    const int m = Ain.rows, n = Ain.cols, k = Bin.cols;
    if (m < n || Bin.rows != m) return false;
    MatD A = Ain, B = Bin;
    std::vector<double> v(m);
    for (int j = 0; j < n; ++j) {
        double nrm = 0;
        for (int i = j; i < m; ++i) nrm += A(i, j) * A(i, j);
        nrm = std::sqrt(nrm);
        if (nrm == 0.0) continue;
        double alpha = (A(j, j) > 0) ? -nrm : nrm;
        for (int i = j; i < m; ++i) v[i] = A(i, j);
        v[j] -= alpha;
        double vnorm2 = 0;
        for (int i = j; i < m; ++i) vnorm2 += v[i] * v[i];
        if (vnorm2 == 0.0) continue;
        for (int c2 = j; c2 < n; ++c2) {
            double dot = 0;
            for (int i = j; i < m; ++i) dot += v[i] * A(i, c2);
            double f = 2.0 * dot / vnorm2;
            for (int i = j; i < m; ++i) A(i, c2) -= f * v[i];
        }
        for (int c2 = 0; c2 < k; ++c2) {
            double dot = 0;
            for (int i = j; i < m; ++i) dot += v[i] * B(i, c2);
            double f = 2.0 * dot / vnorm2;
            for (int i = j; i < m; ++i) B(i, c2) -= f * v[i];
        }
    }
    X = MatD(n, k);
    for (int c2 = 0; c2 < k; ++c2)
        for (int i = n - 1; i >= 0; --i) {
            double s = B(i, c2);
            for (int j = i + 1; j < n; ++j) s -= A(i, j) * X(j, c2);
            if (A(i, i) == 0.0 || !std::isfinite(A(i, i))) return false;
            X(i, c2) = s / A(i, i);
        }
    if (Rout) {
        *Rout = MatD(n, n);
        for (int i = 0; i < n; ++i)
            for (int j = i; j < n; ++j) (*Rout)(i, j) = A(i, j);
    }
    return true;
}

// One-sided Jacobi SVD of an m x n matrix (m >= n): A = Uo diag(s) V^T with
// Uo m x n (orthonormal columns where s > 0) and V n x n.  s is returned in
// descending order.
inline void svd_jacobi(const MatD& Ain, MatD& Uo, std::vector<double>& s, MatD& V) {
    const int m = Ain.rows, n = Ain.cols;
    MatD A = Ain;
    V = MatD(n, n);
    for (int i = 0; i < n; ++i) V(i, i) = 1.0;
    const double eps = std::numeric_limits<double>::epsilon();
    for (int sweep = 0; sweep < 60; ++sweep) {
        bool rotated = false;
        for (int p = 0; p < n - 1; ++p)
            for (int q = p + 1; q < n; ++q) {
                double alpha = 0, beta = 0, gamma = 0;
                for (int i = 0; i < m; ++i) {
                    alpha += A(i, p) * A(i, p);
                    beta += A(i, q) * A(i, q);
                    gamma += A(i, p) * A(i, q);
                }
                if (gamma == 0.0 || std::fabs(gamma) <= eps * std::sqrt(alpha * beta)) continue;
                rotated = true;
                double zeta = (beta - alpha) / (2.0 * gamma);
                double t = ((zeta >= 0) ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
                double cs = 1.0 / std::sqrt(1.0 + t * t), sn = cs * t;
                for (int i = 0; i < m; ++i) {
                    double ap = A(i, p), aq = A(i, q);
                    A(i, p) = cs * ap - sn * aq;
                    A(i, q) = sn * ap + cs * aq;
                }
                for (int i = 0; i < n; ++i) {
                    double vp = V(i, p), vq = V(i, q);
                    V(i, p) = cs * vp - sn * vq;
                    V(i, q) = sn * vp + cs * vq;
                }
            }
        if (!rotated) break;
    }
    std::vector<double> nrm(n);
    for (int j = 0; j < n; ++j) {
        double t = 0;
        for (int i = 0; i < m; ++i) t += A(i, j) * A(i, j);
        nrm[j] = std::sqrt(t);
    }
    std::vector<int> order(n);
    for (int j = 0; j < n; ++j) order[j] = j;
    std::sort(order.begin(), order.end(), [&](int a, int b) { return nrm[a] > nrm[b]; });
    Uo = MatD(m, n);
    MatD Vs(n, n);
    s.assign(n, 0.0);
    for (int jj = 0; jj < n; ++jj) {
        int j = order[jj];
        s[jj] = nrm[j];
        for (int i = 0; i < m; ++i) Uo(i, jj) = (nrm[j] > 0) ? A(i, j) / nrm[j] : 0.0;
        for (int i = 0; i < n; ++i) Vs(i, jj) = V(i, j);
    }
    V = Vs;
}

inline double kappa2(const MatD& A) {
    // condition number of a (tall or square) matrix: QR first so that the
    // Jacobi sweeps work on an n x n factor.
    MatD Rf;
    const MatD* src = &A;
    MatD X;
    if (A.rows > A.cols) {
        MatD zero(A.rows, 1);
        if (!lstsq(A, zero, X, &Rf)) return std::numeric_limits<double>::infinity();
        src = &Rf;
    }
    MatD Uo, V;
    std::vector<double> s;
    svd_jacobi(*src, Uo, s, V);
    if (s.empty() || !(s.back() > 0)) return std::numeric_limits<double>::infinity();
    return s.front() / s.back();
}

}  // namespace la
}  // namespace cerar

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
// Works on transposed copies so that every column is contiguous in memory.
inline bool lstsq(const MatD& Ain, const MatD& Bin, MatD& X, MatD* Rout = nullptr) {
    const int m = Ain.rows, n = Ain.cols, k = Bin.cols;
    if (m < n || Bin.rows != m) return false;
    MatD At = transpose(Ain), Bt = transpose(Bin);      // At(j, i) = A(i, j)
    std::vector<double> v(m);
    for (int j = 0; j < n; ++j) {
        double* aj = &At(j, 0);
        double nrm = 0;
        for (int i = j; i < m; ++i) nrm += aj[i] * aj[i];
        nrm = std::sqrt(nrm);
        if (nrm == 0.0) continue;
        const double alpha = (aj[j] > 0) ? -nrm : nrm;
        for (int i = j; i < m; ++i) v[i] = aj[i];
        v[j] -= alpha;
        double vnorm2 = 0;
        for (int i = j; i < m; ++i) vnorm2 += v[i] * v[i];
        if (vnorm2 == 0.0) continue;
        const double inv = 2.0 / vnorm2;
        for (int c2 = j; c2 < n; ++c2) {
            double* ac = &At(c2, 0);
            double dot = 0;
            for (int i = j; i < m; ++i) dot += v[i] * ac[i];
            const double f = dot * inv;
            for (int i = j; i < m; ++i) ac[i] -= f * v[i];
        }
        for (int c2 = 0; c2 < k; ++c2) {
            double* bc = &Bt(c2, 0);
            double dot = 0;
            for (int i = j; i < m; ++i) dot += v[i] * bc[i];
            const double f = dot * inv;
            for (int i = j; i < m; ++i) bc[i] -= f * v[i];
        }
    }
    X = MatD(n, k);
    for (int c2 = 0; c2 < k; ++c2)
        for (int i = n - 1; i >= 0; --i) {
            double s = Bt(c2, i);
            for (int j = i + 1; j < n; ++j) s -= At(j, i) * X(j, c2);
            const double d = At(i, i);
            if (d == 0.0 || !std::isfinite(d)) return false;
            X(i, c2) = s / d;
        }
    if (Rout) {
        *Rout = MatD(n, n);
        for (int i = 0; i < n; ++i)
            for (int j = i; j < n; ++j) (*Rout)(i, j) = At(j, i);
    }
    return true;
}

// One-sided Jacobi SVD of an m x n matrix (m >= n): A = Uo diag(s) V^T with
// Uo m x n (orthonormal columns where s > 0) and V n x n.  s is returned in
// descending order.  Columns are kept contiguous (transposed working copies).
inline void svd_jacobi(const MatD& Ain, MatD& Uo, std::vector<double>& s, MatD& V) {
    const int m = Ain.rows, n = Ain.cols;
    MatD At = transpose(Ain);                           // row j = column j of A
    MatD Vt(n, n);                                      // row j = column j of V
    for (int i = 0; i < n; ++i) Vt(i, i) = 1.0;
    const double eps = std::numeric_limits<double>::epsilon();
    for (int sweep = 0; sweep < 60; ++sweep) {
        bool rotated = false;
        for (int p = 0; p < n - 1; ++p)
            for (int q = p + 1; q < n; ++q) {
                double* ap = &At(p, 0);
                double* aq = &At(q, 0);
                double alpha = 0, beta = 0, gamma = 0;
                for (int i = 0; i < m; ++i) {
                    alpha += ap[i] * ap[i];
                    beta += aq[i] * aq[i];
                    gamma += ap[i] * aq[i];
                }
                if (gamma == 0.0 || std::fabs(gamma) <= eps * std::sqrt(alpha * beta)) continue;
                rotated = true;
                const double zeta = (beta - alpha) / (2.0 * gamma);
                const double t = ((zeta >= 0) ? 1.0 : -1.0) / (std::fabs(zeta) + std::sqrt(1.0 + zeta * zeta));
                const double cs = 1.0 / std::sqrt(1.0 + t * t), sn = cs * t;
                for (int i = 0; i < m; ++i) {
                    const double x = ap[i], y = aq[i];
                    ap[i] = cs * x - sn * y;
                    aq[i] = sn * x + cs * y;
                }
                double* vp = &Vt(p, 0);
                double* vq = &Vt(q, 0);
                for (int i = 0; i < n; ++i) {
                    const double x = vp[i], y = vq[i];
                    vp[i] = cs * x - sn * y;
                    vq[i] = sn * x + cs * y;
                }
            }
        if (!rotated) break;
    }
    std::vector<double> nrm(n);
    for (int j = 0; j < n; ++j) {
        double t = 0;
        for (int i = 0; i < m; ++i) t += At(j, i) * At(j, i);
        nrm[j] = std::sqrt(t);
    }
    std::vector<int> order(n);
    for (int j = 0; j < n; ++j) order[j] = j;
    std::sort(order.begin(), order.end(), [&](int a, int b) { return nrm[a] > nrm[b]; });
    Uo = MatD(m, n);
    V = MatD(n, n);
    s.assign(n, 0.0);
    for (int jj = 0; jj < n; ++jj) {
        const int j = order[jj];
        s[jj] = nrm[j];
        for (int i = 0; i < m; ++i) Uo(i, jj) = (nrm[j] > 0) ? At(j, i) / nrm[j] : 0.0;
        for (int i = 0; i < n; ++i) V(i, jj) = Vt(j, i);
    }
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

// Graph quantities of Sec. 3.1: Laplacian (the Laplacian definition of Sec. 3.1), chi_1 (the definition of chi_1 in Sec. 3.1), chi_2 (the definition of chi_2 in Sec. 3.1).
// Dense symmetric eigen-decomposition by cyclic Jacobi rotations (n is the number of workers,
// at most a few thousand), then the pseudo-inverse through the non-zero eigenpairs.
#include <algorithm>
#include <cmath>
#include <numeric>

#include "a2cid2_internal.h"

namespace a2 {

namespace {

// Eigen-decomposition of the symmetric matrix A (n x n, row-major, destroyed): on return the
// diagonal of A holds the eigenvalues and the columns of V the eigenvectors.
void jacobi_eigen(std::vector<double>& A, std::vector<double>& V, int n) {
    V.assign((size_t)n * n, 0.0);
    for (int i = 0; i < n; ++i) V[(size_t)i * n + i] = 1.0;
    for (int sweep = 0; sweep < 100; ++sweep) {
        double off = 0.0, diag = 0.0;
        for (int p = 0; p < n; ++p) {
            diag += A[(size_t)p * n + p] * A[(size_t)p * n + p];
            for (int q = p + 1; q < n; ++q) off += A[(size_t)p * n + q] * A[(size_t)p * n + q];
        }
        if (off == 0.0 || off <= 1e-30 * (diag + off)) break;
        for (int p = 0; p < n - 1; ++p) {
            for (int q = p + 1; q < n; ++q) {
                const double apq = A[(size_t)p * n + q];
                if (apq == 0.0) continue;
                const double app = A[(size_t)p * n + p], aqq = A[(size_t)q * n + q];
                const double theta = (aqq - app) / (2.0 * apq);
                const double t = (theta >= 0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
                const double c = 1.0 / std::sqrt(t * t + 1.0), sn = t * c;
                for (int k = 0; k < n; ++k) {  // columns p, q
                    const double akp = A[(size_t)k * n + p], akq = A[(size_t)k * n + q];
                    A[(size_t)k * n + p] = c * akp - sn * akq;
                    A[(size_t)k * n + q] = sn * akp + c * akq;
                }
                for (int k = 0; k < n; ++k) {  // rows p, q
                    const double apk = A[(size_t)p * n + k], aqk = A[(size_t)q * n + k];
                    A[(size_t)p * n + k] = c * apk - sn * aqk;
                    A[(size_t)q * n + k] = sn * apk + c * aqk;
                }
                for (int k = 0; k < n; ++k) {
                    const double vkp = V[(size_t)k * n + p], vkq = V[(size_t)k * n + q];
                    V[(size_t)k * n + p] = c * vkp - sn * vkq;
                    V[(size_t)k * n + q] = sn * vkp + c * vkq;
                }
            }
        }
    }
}

}  // namespace

int graph_chi(int32_t n, int64_t n_edges, const int32_t* ei, const int32_t* ej, const double* lambda, double* chi1,
              double* chi2, std::string& err) {
    if (n < 2 || n > 4096) { err = "need 2 <= n <= 4096"; return A2_EINVAL; }
    if (n_edges < 1 || !ei || !ej || !lambda || !chi1 || !chi2) { err = "bad edge list or NULL output"; return A2_EINVAL; }
    std::vector<double> L((size_t)n * n, 0.0), V;
    for (int64_t k = 0; k < n_edges; ++k) {
        const int32_t i = ei[k], j = ej[k];
        if (i < 0 || j < 0 || i >= n || j >= n || i == j) { err = "edge endpoint out of range"; return A2_ERANGE; }
        if (!(lambda[k] > 0.0) || !std::isfinite(lambda[k])) { err = "edge rate must be positive and finite"; return A2_EINVAL; }
        L[(size_t)i * n + i] += lambda[k];
        L[(size_t)j * n + j] += lambda[k];
        L[(size_t)i * n + j] -= lambda[k];
        L[(size_t)j * n + i] -= lambda[k];
    }
    double scale = 0.0;
    for (int i = 0; i < n; ++i) scale = std::max(scale, L[(size_t)i * n + i]);
    jacobi_eigen(L, V, n);
    std::vector<int> order((size_t)n);
    std::iota(order.begin(), order.end(), 0);
    std::sort(order.begin(), order.end(), [&](int a, int b) { return L[(size_t)a * n + a] < L[(size_t)b * n + b]; });
    const double lam2 = L[(size_t)order[1] * n + order[1]];
    if (!(lam2 > 1e-12 * scale)) { err = "graph is not connected (chi_1 is infinite)"; return A2_EINVAL; }
    *chi1 = 1.0 / lam2;
    double best = 0.0;
    for (int64_t k = 0; k < n_edges; ++k) {
        double r = 0.0;  // (e_i - e_j)^T Lambda^+ (e_i - e_j) = sum over non-zero modes (v_i - v_j)^2 / lambda
        for (int m = 1; m < n; ++m) {
            const int c = order[(size_t)m];
            const double dv = V[(size_t)ei[k] * n + c] - V[(size_t)ej[k] * n + c];
            r += dv * dv / L[(size_t)c * n + c];
        }
        best = std::max(best, r);
    }
    *chi2 = 0.5 * best;
    return A2_OK;
}

}  // namespace a2

/*
 * CPU checker for the A2CiD2 event update -- TEST INFRASTRUCTURE, not a product path.
 *
 * Plain, sequential, fp64. Events are applied one by one, strictly in the order given
 * (time order, ties by stream index). Nothing here is blocked, fused or reordered, and
 * nothing is shared with the CUDA library: this file is compared against it.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * What each function follows (paper: "A2CiD2: Accelerating Asynchronous Communication in
 * Decentralized Deep Learning"):
 *   a2o_mix        the drift term eta*(x~ - x) dt of Eq. (dynamic), Sec. 3.2, integrated in
 *                  closed form over the worker's elapsed time: the matrix exponential
 *                  exp(dt * [[-eta, eta],[eta,-eta]]) of Algorithm 1.
 *   gradient event jump -gamma * g on both x^i and x~^i (Eq. (dynamic); Algorithm 1, first loop)
 *   comm event     jump -alpha (x^i - x^j) on x^i, -alpha~ (x^i - x^j) on x~^i, and the same
 *                  with i and j swapped on worker j (Eq. (dynamic); Algorithm 1, second loop;
 *                  symmetric communications, Sec. 3.1)
 *   a2o_consensus  ||pi x||_F^2 = sum_i ||x_i - xbar||^2, App. A (Notations)
 *
 * Closed form used for the mixing step. With A = [[-eta, eta],[eta,-eta]] one has
 * A^2 = -2 eta A, hence exp(dt A) = I + (1 - e)/(2 eta) A with e = exp(-2 eta dt), i.e.
 *     x  <- x  - c (x - x~),   x~ <- x~ + c (x - x~),   c = (1 - e)/2 = -expm1(-2 eta dt)/2.
 *
 * Reading of the order of operations at a communication event: the message x^i - x^j is
 * taken at the event time, after both workers have been mixed forward to that time, as
 * Eq. (dynamic) states (variant 0). Algorithm 1 as printed forms the message before the
 * mixing line; that ordering is available as variant 1.
 *
 * Variant 2 is the asynchronous baseline the paper compares with, Eq. (baselinedynamic) of
 * Sec. 3.2 (restated at the head of the proofs' appendix as what Eq. (dynamic) becomes when
 * the method is not applied): there is no momentum buffer and no drift; a gradient event is
 * x^i -= gamma g, a communication x^i -= alpha (x^i - x^j), x^j += alpha (x^i - x^j). X~ is
 * never read or written; eta and alpha~ are ignored.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { A2O_OK = 0, A2O_EINVAL = -1, A2O_EORDER = -2, A2O_ERANGE = -3 };

/* Mixing coefficient c for an elapsed time dt >= 0. */
double a2o_mix_coeff(double eta, double dt) { return -expm1(-2.0 * eta * dt) / 2.0; }

/* Advance worker w's pair (x, x~) from its last time tl[w] to t, columns [0, d). */
static void a2o_mix(double* x, double* xt, int64_t d, double eta, double dt) {
    const double c = a2o_mix_coeff(eta, dt);
    for (int64_t k = 0; k < d; ++k) {
        const double dlt = x[k] - xt[k];
        x[k] = x[k] - c * dlt;
        xt[k] = xt[k] + c * dlt;
    }
}

/* Eq. (baselinedynamic): the two jumps on x alone. */
static void a2o_plain_grad(double* x, const double* g, int64_t d, double gamma) {
    for (int64_t k = 0; k < d; ++k) x[k] = x[k] - gamma * g[k];
}

static void a2o_plain_comm(double* x, double* y, int64_t d, double alpha) {
    for (int64_t k = 0; k < d; ++k) {
        const double m = x[k] - y[k];
        x[k] = x[k] - alpha * m;
        y[k] = y[k] + alpha * m;
    }
}

/*
 * Apply n_events events in the given order to X, Xt (row-major, row stride ld doubles,
 * d columns used) and the per-worker last-event times tl[n].
 *   wj[e] >= 0 : communication between wi[e] and wj[e]   (slot[e] must be -1)
 *   wj[e] == -1: gradient event on wi[e] with gradient row G[slot[e]] (row stride ldg)
 * variant 0: message after mixing (Eq. (dynamic)); variant 1: message before mixing
 * (Algorithm 1 as printed); variant 2: Eq. (baselinedynamic), x only (Xt is left as it is).
 * Returns 0, or a negative code at the first invalid event (state is then partly updated).
 */
int a2o_run(int32_t n, int64_t d, int64_t ld, double eta, double alpha, double alpha_t, double gamma,
            double* X, double* Xt, double* tl, const double* G, int32_t n_slots, int64_t ldg,
            int64_t n_events, const double* times, const int32_t* wi, const int32_t* wj,
            const int32_t* slot, int32_t variant) {
    if (n < 2 || d < 0 || ld < d || n_events < 0 || variant < 0 || variant > 2) return A2O_EINVAL;
    for (int64_t e = 0; e < n_events; ++e) {
        const double t = times[e];
        const int32_t i = wi[e], j = wj[e], s = slot[e];
        if (!(t == t) || i < 0 || i >= n) return A2O_ERANGE;
        if (e > 0 && t < times[e - 1]) return A2O_EORDER;
        double* xi = X + (size_t)i * ld;
        double* xti = Xt + (size_t)i * ld;
        if (j < 0) {
            /* gradient event */
            if (j != -1 || s < 0 || s >= n_slots) return A2O_ERANGE;
            if (t < tl[i]) return A2O_EORDER;
            const double* g = G + (size_t)s * ldg;
            if (variant == 2) {
                a2o_plain_grad(xi, g, d, gamma);
                tl[i] = t;
                continue;
            }
            a2o_mix(xi, xti, d, eta, t - tl[i]);
            for (int64_t k = 0; k < d; ++k) {
                xi[k] = xi[k] - gamma * g[k];
                xti[k] = xti[k] - gamma * g[k];
            }
            tl[i] = t;
        } else {
            /* communication event */
            if (j >= n || j == i || s != -1) return A2O_ERANGE;
            if (t < tl[i] || t < tl[j]) return A2O_EORDER;
            double* xj = X + (size_t)j * ld;
            double* xtj = Xt + (size_t)j * ld;
            if (variant == 2) {
                a2o_plain_comm(xi, xj, d, alpha);
                tl[i] = t;
                tl[j] = t;
                continue;
            }
            if (variant == 0) {
                a2o_mix(xi, xti, d, eta, t - tl[i]);
                a2o_mix(xj, xtj, d, eta, t - tl[j]);
                for (int64_t k = 0; k < d; ++k) {
                    const double m = xi[k] - xj[k];
                    xi[k] = xi[k] - alpha * m;
                    xti[k] = xti[k] - alpha_t * m;
                    xj[k] = xj[k] + alpha * m;
                    xtj[k] = xtj[k] + alpha_t * m;
                }
            } else {
                const double ci = a2o_mix_coeff(eta, t - tl[i]);
                const double cj = a2o_mix_coeff(eta, t - tl[j]);
                for (int64_t k = 0; k < d; ++k) {
                    const double m = xi[k] - xj[k]; /* from the un-mixed buffers */
                    const double di = xi[k] - xti[k];
                    const double dj = xj[k] - xtj[k];
                    xi[k] = (xi[k] - ci * di) - alpha * m;
                    xti[k] = (xti[k] + ci * di) - alpha_t * m;
                    xj[k] = (xj[k] - cj * dj) + alpha * m;
                    xtj[k] = (xtj[k] + cj * dj) + alpha_t * m;
                }
            }
            tl[i] = t;
            tl[j] = t;
        }
    }
    return A2O_OK;
}

/* sum_i ||x_i - xbar||^2 over columns [0, d) of the stored x. */
double a2o_consensus(int32_t n, int64_t d, int64_t ld, const double* X) {
    double total = 0.0;
    for (int64_t k = 0; k < d; ++k) {
        double mean = 0.0;
        for (int32_t i = 0; i < n; ++i) mean += X[(size_t)i * ld + k];
        mean /= (double)n;
        for (int32_t i = 0; i < n; ++i) {
            const double dev = X[(size_t)i * ld + k] - mean;
            total += dev * dev;
        }
    }
    return total;
}

/*
 * The same quantity at a common time t_eval >= max_i tl[i]: every worker's x is first mixed
 * forward from its own last-event time to t_eval (nothing is written back).
 */
double a2o_consensus_at(int32_t n, int64_t d, int64_t ld, double eta, const double* X, const double* Xt,
                        const double* tl, double t_eval) {
    double total = 0.0;
    for (int64_t k = 0; k < d; ++k) {
        double mean = 0.0;
        for (int32_t i = 0; i < n; ++i) {
            const double c = a2o_mix_coeff(eta, t_eval - tl[i]);
            const double x = X[(size_t)i * ld + k], xt = Xt[(size_t)i * ld + k];
            mean += x - c * (x - xt);
        }
        mean /= (double)n;
        for (int32_t i = 0; i < n; ++i) {
            const double c = a2o_mix_coeff(eta, t_eval - tl[i]);
            const double x = X[(size_t)i * ld + k], xt = Xt[(size_t)i * ld + k];
            const double dev = (x - c * (x - xt)) - mean;
            total += dev * dev;
        }
    }
    return total;
}

/*
 * Model of reduced-precision STORAGE (no passage of the paper: the method is stated in real numbers; this
 * models an implementation that keeps its state in bfloat16 and writes rows back at known points). The
 * value is rounded to IEEE binary32 and then to bfloat16 -- the upper 16 bits of that binary32 -- both to
 * nearest, ties to even. Finite inputs only.
 */
double a2o_to_bf16(double v) {
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    u = (u + 0x7FFFu + ((u >> 16) & 1u)) & 0xFFFF0000u;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* The same for IEEE binary32 storage: one rounding to nearest, ties to even. */
double a2o_to_f32(double v) { return (double)(float)v; }

/* Round columns [0, d) of the rows X[w], Xt[w] (w in rows[0 .. n_rows)) to the storage format
 * (fmt 0: bfloat16, 1: binary32). */
void a2o_round_rows(int64_t d, int64_t ld, double* X, double* Xt, int32_t n_rows, const int32_t* rows, int32_t fmt) {
    for (int32_t r = 0; r < n_rows; ++r) {
        double* x = X + (size_t)rows[r] * ld;
        double* xt = Xt + (size_t)rows[r] * ld;
        for (int64_t k = 0; k < d; ++k) {
            x[k] = fmt == 0 ? a2o_to_bf16(x[k]) : a2o_to_f32(x[k]);
            xt[k] = fmt == 0 ? a2o_to_bf16(xt[k]) : a2o_to_f32(xt[k]);
        }
    }
}

/*
 * a2o_run on consecutive groups of events, with the storage model applied between groups: group k is
 * events [group_end[k-1], group_end[k]) (group_end[-1] = 0), applied in the order given by a2o_run (fp64
 * arithmetic, unchanged); then the rows of workers[worker_ptr[k] .. worker_ptr[k+1]) are rounded to the
 * storage format. The time-order check of a2o_run holds inside a group; groups may overlap in time (they
 * are the items of a schedule, which keeps every worker's own order).
 */
int a2o_run_groups(int32_t n, int64_t d, int64_t ld, double eta, double alpha, double alpha_t, double gamma,
                   double* X, double* Xt, double* tl, const double* G, int32_t n_slots, int64_t ldg,
                   const double* times, const int32_t* wi, const int32_t* wj, const int32_t* slot,
                   int32_t variant, int64_t n_groups, const int64_t* group_end, const int64_t* worker_ptr,
                   const int32_t* workers, int32_t fmt) {
    if (fmt != 0 && fmt != 1) return A2O_EINVAL;
    int64_t e0 = 0;
    for (int64_t k = 0; k < n_groups; ++k) {
        const int64_t e1 = group_end[k];
        if (e1 < e0) return A2O_EINVAL;
        const int rc = a2o_run(n, d, ld, eta, alpha, alpha_t, gamma, X, Xt, tl, G, n_slots, ldg, e1 - e0, times + e0,
                               wi + e0, wj + e0, slot + e0, variant);
        if (rc != A2O_OK) return rc;
        a2o_round_rows(d, ld, X, Xt, (int32_t)(worker_ptr[k + 1] - worker_ptr[k]), workers + worker_ptr[k], fmt);
        e0 = e1;
    }
    return A2O_OK;
}

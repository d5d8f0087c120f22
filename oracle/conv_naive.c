/* Oracle (test infrastructure only): the message-passing convolution, its
 * backward, written as the defining sums in float64.  No blocking, no fusion,
 * no reordering: each function is the paper's equation with the loops spelled
 * out.  Inputs are float32 (the precision the workloads are generated in),
 * promoted to double; all sums and outputs are double.
 *
 * Forward, "Mathematical operations", message-passing-convolution equation:
 *   m[b,i0,q] = sum_{edges e into b} sum_{i1,i2} C[i0,i1,i2]
 *               * x[sender(e),i1,q] * y[e,i2] * s[e,i3(i0),q]
 * (y carries no channel axis: it is shared across channels, as the forward
 * algorithm's data declaration and the backward's sum over q state.)
 *
 * Backward, "Differentiation", message-passing-backward equation, with the
 * edge-scalar cotangent taken per irreducible block k = i3(i0):
 *   dx[a,i1,q] = sum_{edges e out of a} sum C * y[e,i2] * s[e,k,q] * dm[b,i0,q]
 *   dy[e,i2]   = sum_q sum C * x[a,i1,q] * s[e,k,q] * dm[b,i0,q]
 *   ds[e,k,q]  = sum_{i0 in block k} dm[b,i0,q] * sum C * x[a,i1,q] * y[e,i2]
 *
 * The coupling tensor C is passed dense, [D][d][dp]; zero entries are skipped.
 * Edges must be sorted by receiver (non-decreasing); the loops over receivers
 * (forward, dy, ds) and over senders (dx) are split across OpenMP threads,
 * each output element being owned by exactly one thread.
 *
 * Return value: 0, or -1 if receivers are not sorted / an index is out of
 * range.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int e3j_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int check_graph(int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                       const int32_t* receivers) {
    for (int64_t e = 0; e < n_edges; ++e) {
        if (senders[e] < 0 || senders[e] >= n_nodes) return -1;
        if (receivers[e] < 0 || receivers[e] >= n_nodes) return -1;
        if (e > 0 && receivers[e] < receivers[e - 1]) return -1;
    }
    return 0;
}

/* rowptr[b] = first edge whose receiver is >= b */
static int64_t* build_rowptr(int64_t n_nodes, int64_t n_edges, const int32_t* receivers) {
    int64_t* rowptr = (int64_t*)calloc((size_t)n_nodes + 1, sizeof(int64_t));
    for (int64_t e = 0; e < n_edges; ++e) rowptr[receivers[e] + 1] += 1;
    for (int64_t b = 0; b < n_nodes; ++b) rowptr[b + 1] += rowptr[b];
    return rowptr;
}

/* The edge scalars come in as doubles: the float32 entry point promotes them first (exactly), the
 * radial entry points of conv.py pass s = h W formed in float64. */
static int conv_fwd_sums(int64_t n_nodes, int64_t n_edges, int d, int dp, int P, int D, int nq,
                         const double* C, const int32_t* i3, const float* x, const float* y,
                         const double* s, const int32_t* senders, const int32_t* receivers,
                         double* out) {
    if (check_graph(n_nodes, n_edges, senders, receivers)) return -1;
    int64_t* rowptr = build_rowptr(n_nodes, n_edges, receivers);
    memset(out, 0, sizeof(double) * (size_t)n_nodes * D * nq);
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t b = 0; b < n_nodes; ++b) {
        double* mb = out + (size_t)b * D * nq;
        for (int64_t e = rowptr[b]; e < rowptr[b + 1]; ++e) {
            const float* xa = x + (size_t)senders[e] * d * nq;
            const float* ye = y + (size_t)e * dp;
            const double* se = s + (size_t)e * P * nq;
            for (int i0 = 0; i0 < D; ++i0) {
                const int k = i3[i0];
                for (int i1 = 0; i1 < d; ++i1)
                    for (int i2 = 0; i2 < dp; ++i2) {
                        const double c = C[((size_t)i0 * d + i1) * dp + i2];
                        if (c == 0.0) continue;
                        for (int q = 0; q < nq; ++q)
                            mb[(size_t)i0 * nq + q] += c * (double)xa[(size_t)i1 * nq + q] *
                                                       (double)ye[i2] * se[(size_t)k * nq + q];
                    }
            }
        }
    }
    free(rowptr);
    return 0;
}

static double* promote(const float* s, size_t n) {
    double* out = (double*)malloc(sizeof(double) * (n > 0 ? n : 1));
    for (size_t i = 0; i < n; ++i) out[i] = (double)s[i];
    return out;
}

int e3j_oracle_conv_fwd(int64_t n_nodes, int64_t n_edges, int d, int dp, int P, int D, int nq,
                        const double* C, const int32_t* i3, const float* x, const float* y,
                        const float* s, const int32_t* senders, const int32_t* receivers,
                        double* out) {
    double* sd = promote(s, (size_t)n_edges * P * nq);
    const int rc = conv_fwd_sums(n_nodes, n_edges, d, dp, P, D, nq, C, i3, x, y, sd, senders, receivers, out);
    free(sd);
    return rc;
}

/* the same sums with the edge scalars given in float64 */
int e3j_oracle_conv_fwd_sd(int64_t n_nodes, int64_t n_edges, int d, int dp, int P, int D, int nq,
                           const double* C, const int32_t* i3, const float* x, const float* y,
                           const double* s, const int32_t* senders, const int32_t* receivers,
                           double* out) {
    return conv_fwd_sums(n_nodes, n_edges, d, dp, P, D, nq, C, i3, x, y, s, senders, receivers, out);
}

static int conv_bwd_sums(int64_t n_nodes, int64_t n_edges, int d, int dp, int P, int D, int nq,
                         const double* C, const int32_t* i3, const float* x, const float* y,
                         const double* s, const int32_t* senders, const int32_t* receivers,
                         const float* dm, double* dx, double* dy, double* ds) {
    if (check_graph(n_nodes, n_edges, senders, receivers)) return -1;
    memset(dx, 0, sizeof(double) * (size_t)n_nodes * d * nq);
    memset(dy, 0, sizeof(double) * (size_t)n_edges * dp);
    memset(ds, 0, sizeof(double) * (size_t)n_edges * P * nq);

    /* edge-local cotangents dy, ds */
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t e = 0; e < n_edges; ++e) {
        const float* xa = x + (size_t)senders[e] * d * nq;
        const float* ye = y + (size_t)e * dp;
        const double* se = s + (size_t)e * P * nq;
        const float* dmb = dm + (size_t)receivers[e] * D * nq;
        for (int i0 = 0; i0 < D; ++i0) {
            const int k = i3[i0];
            for (int i1 = 0; i1 < d; ++i1)
                for (int i2 = 0; i2 < dp; ++i2) {
                    const double c = C[((size_t)i0 * d + i1) * dp + i2];
                    if (c == 0.0) continue;
                    for (int q = 0; q < nq; ++q) {
                        const double xv = xa[(size_t)i1 * nq + q], yv = ye[i2];
                        const double sv = se[(size_t)k * nq + q], gv = dmb[(size_t)i0 * nq + q];
                        dy[(size_t)e * dp + i2] += c * xv * sv * gv;
                        ds[((size_t)e * P + k) * nq + q] += c * xv * yv * gv;
                    }
                }
        }
    }

    /* sender cotangent dx: list the edges of every sender in edge order */
    int64_t* colptr = (int64_t*)calloc((size_t)n_nodes + 1, sizeof(int64_t));
    int64_t* perm = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n_edges > 0 ? n_edges : 1));
    int64_t* fill = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n_nodes > 0 ? n_nodes : 1));
    for (int64_t e = 0; e < n_edges; ++e) colptr[senders[e] + 1] += 1;
    for (int64_t a = 0; a < n_nodes; ++a) colptr[a + 1] += colptr[a];
    for (int64_t a = 0; a < n_nodes; ++a) fill[a] = colptr[a];
    for (int64_t e = 0; e < n_edges; ++e) perm[fill[senders[e]]++] = e;
#pragma omp parallel for schedule(dynamic, 8)
    for (int64_t a = 0; a < n_nodes; ++a) {
        double* dxa = dx + (size_t)a * d * nq;
        for (int64_t j = colptr[a]; j < colptr[a + 1]; ++j) {
            const int64_t e = perm[j];
            const float* ye = y + (size_t)e * dp;
            const double* se = s + (size_t)e * P * nq;
            const float* dmb = dm + (size_t)receivers[e] * D * nq;
            for (int i0 = 0; i0 < D; ++i0) {
                const int k = i3[i0];
                for (int i1 = 0; i1 < d; ++i1)
                    for (int i2 = 0; i2 < dp; ++i2) {
                        const double c = C[((size_t)i0 * d + i1) * dp + i2];
                        if (c == 0.0) continue;
                        for (int q = 0; q < nq; ++q)
                            dxa[(size_t)i1 * nq + q] += c * (double)ye[i2] *
                                                        se[(size_t)k * nq + q] *
                                                        (double)dmb[(size_t)i0 * nq + q];
                    }
            }
        }
    }
    free(colptr);
    free(perm);
    free(fill);
    return 0;
}

int e3j_oracle_conv_bwd(int64_t n_nodes, int64_t n_edges, int d, int dp, int P, int D, int nq,
                        const double* C, const int32_t* i3, const float* x, const float* y,
                        const float* s, const int32_t* senders, const int32_t* receivers,
                        const float* dm, double* dx, double* dy, double* ds) {
    double* sd = promote(s, (size_t)n_edges * P * nq);
    const int rc = conv_bwd_sums(n_nodes, n_edges, d, dp, P, D, nq, C, i3, x, y, sd, senders, receivers, dm,
                                 dx, dy, ds);
    free(sd);
    return rc;
}

int e3j_oracle_conv_bwd_sd(int64_t n_nodes, int64_t n_edges, int d, int dp, int P, int D, int nq,
                           const double* C, const int32_t* i3, const float* x, const float* y,
                           const double* s, const int32_t* senders, const int32_t* receivers,
                           const float* dm, double* dx, double* dy, double* ds) {
    return conv_bwd_sums(n_nodes, n_edges, d, dp, P, D, nq, C, i3, x, y, s, senders, receivers, dm, dx, dy, ds);
}

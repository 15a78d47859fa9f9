/*
 * EF21 reference oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded CPU statement of what the EF21 hot path
 * computes (Richtarik, Sokolov, Fatkhullin: "EF21", Algorithm 2, with the
 * Top-k compressor of Section 2.1 and the logistic loss with nonconvex
 * regulariser of Section 5, Eq. 19).  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the CUDA library shares no code
 * with it and must never route through it.
 *
 * Precision.  The file is built twice: with `real` = float (the state
 * x, g, g_i and every message are fp32 vectors, each state update is one
 * IEEE-754 fp32 operation in the stated order, so a GPU fed the same fp32
 * gradients can be compared bit for bit), and with -DEF21O_F64 (`real` =
 * double, used to pin the oracle against exact identities).  Loss and gradient
 * arithmetic is always fp64 and is rounded once to `real`.
 * Compile with -ffp-contract=off so no multiply-add is fused unless written
 * as fma().
 *
 * Readings of points the paper leaves open (all listed in the design notes):
 *   - Top-k ties are broken toward the lower index; magnitudes are compared
 *     by the bit pattern of |v| (so +0 and -0 tie and a NaN sorts above Inf).
 *   - Exactly k pairs are always produced, in ascending index order, with the
 *     original signed values.
 *   - Every f_i carries the whole regulariser; f_i averages over its own m_i.
 *   - The master's average is kept incrementally, g += (1/n) * sum_i c_i, the
 *     per-coordinate sum taken over ascending worker index starting from 0.
 *
 * Parity pins: see tests/test_oracle_*.py (finite differences, closed forms,
 * brute-force sort, k = d => gradient descent, n = 1 => Algorithm 1, the
 * contraction bound of Eq. 3, the one-step distortion bound from the proof of
 * Lemma 2, Theorem 1, a hand-worked Algorithm 2 example).  The original error
 * feedback method (Algorithm 4) at the end of the file is pinned by a
 * hand-worked run, the perturbed-iterate identity x - mean e, the contraction
 * of the error, Theorem 3 for the identity compressor and an exact check of
 * every rounding.  The diagnostics (||grad f||^2, G^t) are pinned by closed forms at the origin and a planted
 * distortion; the scaled Rand-k by exact averages over all k-subsets (unbiasedness and second moment of Rand-k,
 * the contraction of Lemma 8 with equality) and by k = d.  The stepsize rule gamma = 1/L is a harness convention:
 * parity unpinned by the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef EF21O_F64
typedef double real;
typedef uint64_t ubits;
#define ABS_MASK 0x7fffffffffffffffULL
#define FMA_REAL(a, b, c) fma((a), (b), (c))
#else
typedef float real;
typedef uint32_t ubits;
#define ABS_MASK 0x7fffffffU
#define FMA_REAL(a, b, c) fmaf((a), (b), (c))
#endif

int ef21o_real_bytes(void) { return (int)sizeof(real); }

/* ------------------------------------------------------------------ */
/* Top-k compressor (Section 2.1, the paragraph after Eq. 3).           */
/* ------------------------------------------------------------------ */

typedef struct { ubits mag; int64_t j; } topk_rec;

static ubits magnitude_bits(real v) {
    ubits b;
    memcpy(&b, &v, sizeof b);
    return b & ABS_MASK;
}

static int cmp_mag_desc_index_asc(const void* pa, const void* pb) {
    const topk_rec* a = (const topk_rec*)pa;
    const topk_rec* b = (const topk_rec*)pb;
    if (a->mag != b->mag) return a->mag > b->mag ? -1 : 1;
    if (a->j != b->j) return a->j < b->j ? -1 : 1;
    return 0;
}

static int cmp_index_asc(const void* pa, const void* pb) {
    const topk_rec* a = (const topk_rec*)pa;
    const topk_rec* b = (const topk_rec*)pb;
    return (a->j > b->j) - (a->j < b->j);
}

/* c = C(v): the k entries of largest |v_j| survive, the rest are zeroed.
 * Output: their indices ascending and their signed values.  Full sort. */
void ef21o_topk(const real* v, int64_t d, int64_t k, int32_t* idx, real* val) {
    topk_rec* r = (topk_rec*)malloc((size_t)d * sizeof(topk_rec));
    for (int64_t j = 0; j < d; ++j) { r[j].mag = magnitude_bits(v[j]); r[j].j = j; }
    qsort(r, (size_t)d, sizeof(topk_rec), cmp_mag_desc_index_asc);
    qsort(r, (size_t)k, sizeof(topk_rec), cmp_index_asc);
    for (int64_t t = 0; t < k; ++t) { idx[t] = (int32_t)r[t].j; val[t] = v[r[t].j]; }
    free(r);
}

/* ------------------------------------------------------------------ */
/* Local objective and gradient (Section 5, Eq. 19; Eq. 1).             */
/* f_i(x) = (1/m_i) sum_r log(1+exp(-y_r a_r.x)) + lam sum_j x_j^2/(1+x_j^2) */
/* ------------------------------------------------------------------ */

/* Objective used by the loss/gradient routines: 0 = logistic loss with regulariser (Section 5, Eq. 19),
 * 1 = least squares (1/m_i) sum_r (a_r.x - y_r)^2 (Appendix A.2), same regulariser term (lam = 0 for none). */
static int g_objective = 0;
void ef21o_set_objective(int objective) { g_objective = objective; }

static double softplus(double t) { /* log(1+exp(t)) without overflow */
    return (t > 0.0 ? t : 0.0) + log1p(exp(-fabs(t)));
}

double ef21o_local_loss(const float* A, const float* y, int64_t m, int64_t d,
                        const real* x, double lam) {
    double loss = 0.0;
    for (int64_t r = 0; r < m; ++r) {
        double z = 0.0;
        for (int64_t j = 0; j < d; ++j) z += (double)A[r * d + j] * (double)x[j];
        if (g_objective == 0) loss += softplus(-(double)y[r] * z);
        else loss += (z - (double)y[r]) * (z - (double)y[r]);
    }
    if (m > 0) loss /= (double)m;
    double reg = 0.0;
    for (int64_t j = 0; j < d; ++j) {
        double xj = (double)x[j];
        reg += xj * xj / (1.0 + xj * xj);
    }
    return loss + lam * reg;
}

/* grad f_i(x)_j = (1/m_i) sum_r rho_r a_rj + 2 lam x_j / (1+x_j^2)^2,
 * rho_r = -y_r / (1 + exp(y_r a_r.x))  (derivative of the logistic term). */
void ef21o_local_grad(const float* A, const float* y, int64_t m, int64_t d,
                      const real* x, double lam, real* grad) {
    double* acc = (double*)calloc((size_t)d, sizeof(double));
    for (int64_t r = 0; r < m; ++r) {
        double z = 0.0;
        for (int64_t j = 0; j < d; ++j) z += (double)A[r * d + j] * (double)x[j];
        double yr = (double)y[r];
        double t = yr * z;
        double rho;
        if (g_objective == 1) { rho = 2.0 * (z - yr); }
        else if (t >= 0.0) { double e = exp(-t); rho = -yr * e / (1.0 + e); }
        else          { rho = -yr / (1.0 + exp(t)); }
        for (int64_t j = 0; j < d; ++j) acc[j] += rho * (double)A[r * d + j];
    }
    for (int64_t j = 0; j < d; ++j) {
        double xj = (double)x[j];
        double q = 1.0 + xj * xj;
        double data = m > 0 ? acc[j] / (double)m : 0.0;
        grad[j] = (real)(data + 2.0 * lam * xj / (q * q));
    }
    free(acc);
}

/* All n local gradients at x, worker i owning rows [row_off[i], row_off[i+1]). */
void ef21o_all_grads(int32_t n, int64_t d, const float* A, const float* y, const int64_t* row_off,
                     const real* x, double lam, real* grads /* [n][d] */) {
    for (int32_t i = 0; i < n; ++i) {
        int64_t r0 = row_off[i], m = row_off[i + 1] - r0;
        ef21o_local_grad(A + r0 * d, y + r0, m, d, x, lam, grads + (int64_t)i * d);
    }
}

/* f(x) = (1/n) sum_i f_i(x)  (Eq. 1). */
double ef21o_loss(int32_t n, int64_t d, const float* A, const float* y, const int64_t* row_off,
                  const real* x, double lam) {
    double f = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        int64_t r0 = row_off[i], m = row_off[i + 1] - r0;
        f += ef21o_local_loss(A + r0 * d, y + r0, m, d, x, lam);
    }
    return f / (double)n;
}

/* ||grad f(x)||^2 and G = (1/n) sum_i ||g_i - grad f_i(x)||^2 (Eq. 12, "G^t"), both fp64
 * from the rounded local gradients. gi may be NULL (then *G_out = 0). */
void ef21o_diagnostics(int32_t n, int64_t d, const float* A, const float* y, const int64_t* row_off,
                       const real* x, double lam, const real* gi, double* grad_norm2, double* G_out) {
    real* grads = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
    double nrm = 0.0, G = 0.0;
    for (int64_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int32_t i = 0; i < n; ++i) s += (double)grads[(int64_t)i * d + j];
        s /= (double)n;
        nrm += s * s;
    }
    if (gi) {
        for (int32_t i = 0; i < n; ++i)
            for (int64_t j = 0; j < d; ++j) {
                double e = (double)gi[(int64_t)i * d + j] - (double)grads[(int64_t)i * d + j];
                G += e * e;
            }
        G /= (double)n;
    }
    *grad_norm2 = nrm;
    *G_out = G;
    free(grads);
}

/* ------------------------------------------------------------------ */
/* Algorithm 2, one communication round given the local gradients.      */
/* ------------------------------------------------------------------ */

/* For every worker (Algorithm 2, the node loop):
 *     c_i = C(grad_i - g_i);  g_i <- g_i + c_i
 * then the master (Algorithm 2, last line of the loop):
 *     g <- g + (1/n) sum_i c_i
 * idx/val receive the n messages, k pairs each. */
void ef21o_round(int32_t n, int64_t d, int64_t k, const real* grads /* [n][d] */,
                 real* gi /* [n][d] */, real* g /* [d] */,
                 int32_t* idx /* [n][k] */, real* val /* [n][k] */) {
    real* v = (real*)malloc((size_t)d * sizeof(real));
    for (int32_t i = 0; i < n; ++i) {
        const real* gr = grads + (int64_t)i * d;
        real* gs = gi + (int64_t)i * d;
        for (int64_t j = 0; j < d; ++j) v[j] = gr[j] - gs[j];
        int32_t* ix = idx + (int64_t)i * k;
        real* vl = val + (int64_t)i * k;
        ef21o_topk(v, d, k, ix, vl);
        for (int64_t t = 0; t < k; ++t) gs[ix[t]] = gs[ix[t]] + vl[t];
    }
    free(v);
    real* s = (real*)calloc((size_t)d, sizeof(real));
    unsigned char* touched = (unsigned char*)calloc((size_t)d, 1);
    for (int32_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < k; ++t) {
            int64_t j = idx[(int64_t)i * k + t];
            s[j] = s[j] + val[(int64_t)i * k + t];
            touched[j] = 1;
        }
    const real inv_n = (real)1 / (real)n;
    for (int64_t j = 0; j < d; ++j)
        if (touched[j]) {
            real p = s[j] * inv_n;
            g[j] = g[j] + p;
        }
    free(s);
    free(touched);
}

/* x^{t+1} = x^t - gamma g^t as one fused multiply-add per coordinate. */
void ef21o_x_update(int64_t d, real gamma, const real* g, real* x) {
    for (int64_t j = 0; j < d; ++j) x[j] = FMA_REAL(-gamma, g[j], x[j]);
}

/* Initial state from the local gradients at x^0 (Algorithm 2, input line; Section 3.3,
 * last paragraph: any g_i^0 is allowed).
 *   mode 0: g_i^0 = C(grad_i),  g^0 = (1/n) sum g_i^0
 *   mode 1: g_i^0 = 0,          g^0 = 0
 *   mode 2: g_i^0 = grad_i,     g^0 = (1/n) sum g_i^0     (the k = d message round) */
void ef21o_init_from_grads(int32_t mode, int32_t n, int64_t d, int64_t k, const real* grads,
                           real* gi, real* g, int32_t* idx, real* val) {
    memset(gi, 0, (size_t)n * (size_t)d * sizeof(real));
    memset(g, 0, (size_t)d * sizeof(real));
    if (mode == 0) {
        ef21o_round(n, d, k, grads, gi, g, idx, val);
    } else if (mode == 2) {
        int32_t* ix = (int32_t*)malloc((size_t)n * (size_t)d * sizeof(int32_t));
        real* vl = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
        ef21o_round(n, d, d, grads, gi, g, ix, vl);
        free(ix);
        free(vl);
    }
}

void ef21o_init(int32_t mode, int32_t n, int64_t d, int64_t k, const float* A, const float* y,
                const int64_t* row_off, double lam, const real* x,
                real* gi, real* g, int32_t* idx, real* val) {
    real* grads = (real*)calloc((size_t)n * (size_t)d, sizeof(real));
    if (mode != 1) ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
    ef21o_init_from_grads(mode, n, d, k, grads, gi, g, idx, val);
    free(grads);
}

/* `steps` iterations of Algorithm 2's loop body:
 *   x <- x - gamma g;  grads at the new x;  message round. */
void ef21o_step(int32_t steps, int32_t n, int64_t d, int64_t k, const float* A, const float* y,
                const int64_t* row_off, double lam, real gamma,
                real* x, real* gi, real* g, int32_t* idx, real* val) {
    real* grads = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    for (int32_t t = 0; t < steps; ++t) {
        ef21o_x_update(d, gamma, g, x);
        ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
        ef21o_round(n, d, k, grads, gi, g, idx, val);
    }
    free(grads);
}

/* The same loop with caller-supplied gradients V[n][d], re-used at every step
 * (the static input sequence of the Markov compressor, Section 3.1). */
void ef21o_step_grads(int32_t steps, int32_t n, int64_t d, int64_t k, const real* V, real gamma,
                      real* x, real* gi, real* g, int32_t* idx, real* val) {
    for (int32_t t = 0; t < steps; ++t) {
        ef21o_x_update(d, gamma, g, x);
        ef21o_round(n, d, k, V, gi, g, idx, val);
    }
}

/* ------------------------------------------------------------------ */
/* Scaled Rand-k (Appendix, Lemma 8 and Example 2)                       */
/* ------------------------------------------------------------------ */

/* Rand-k keeps a uniformly random set S of k coordinates and scales them by d/k, which makes it unbiased
 * with omega = d/k - 1; Lemma 8 turns an unbiased compressor into a contractive one by the factor
 * 1/(1 + omega) = k/d.  The two factors cancel: the scaled Rand-k of Example 2 is C(v)_j = v_j for j in S and
 * 0 elsewhere, in B(k/d).  The set is an input (the caller draws it): S holds k distinct indices in ascending
 * order.  Output: the k pairs (S_t, v[S_t]). */
void ef21o_randk(const real* v, int64_t d, int64_t k, const int32_t* S, int32_t* idx, real* val) {
    (void)d;
    for (int64_t t = 0; t < k; ++t) { idx[t] = S[t]; val[t] = v[S[t]]; }
}

/* The unbiased Rand-k itself, C'(v)_j = (d/k) v_j on S (used only to pin the class U(omega) it belongs to). */
void ef21o_randk_unbiased(const real* v, int64_t d, int64_t k, const int32_t* S, int32_t* idx, real* val) {
    const real scale = (real)d / (real)k;
    for (int64_t t = 0; t < k; ++t) { idx[t] = S[t]; val[t] = scale * v[S[t]]; }
}

/* One message round of Algorithm 2 with the scaled Rand-k in place of Top-k: worker i uses the set
 * sets[i][0..k).  Node loop and master line as in ef21o_round. */
void ef21o_randk_round(int32_t n, int64_t d, int64_t k, const real* grads, const int32_t* sets /* [n][k] */,
                       real* gi, real* g, int32_t* idx, real* val) {
    real* v = (real*)malloc((size_t)d * sizeof(real));
    for (int32_t i = 0; i < n; ++i) {
        const real* gr = grads + (int64_t)i * d;
        real* gs = gi + (int64_t)i * d;
        for (int64_t j = 0; j < d; ++j) v[j] = gr[j] - gs[j];
        int32_t* ix = idx + (int64_t)i * k;
        real* vl = val + (int64_t)i * k;
        ef21o_randk(v, d, k, sets + (int64_t)i * k, ix, vl);
        for (int64_t t = 0; t < k; ++t) gs[ix[t]] = gs[ix[t]] + vl[t];
    }
    free(v);
    /* master: g <- g + (1/n) sum_i c_i, per coordinate in ascending worker order (Algorithm 2, last line) */
    real* s = (real*)calloc((size_t)d, sizeof(real));
    unsigned char* touched = (unsigned char*)calloc((size_t)d, 1);
    for (int32_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < k; ++t) {
            int64_t j = idx[(int64_t)i * k + t];
            s[j] = s[j] + val[(int64_t)i * k + t];
            touched[j] = 1;
        }
    const real inv_n = (real)1 / (real)n;
    for (int64_t j = 0; j < d; ++j)
        if (touched[j]) {
            real p = s[j] * inv_n;
            g[j] = g[j] + p;
        }
    free(s);
    free(touched);
}

/* `steps` iterations of Algorithm 2 with the scaled Rand-k; sets[steps][n][k].  V != NULL: the supplied
 * vectors V[n][d] stand for the local gradients at every step (as in ef21o_step_grads); otherwise the gradients
 * of Eq. 19 on the shards. */
void ef21o_step_randk(int32_t steps, int32_t n, int64_t d, int64_t k, const float* A, const float* y,
                      const int64_t* row_off, double lam, const real* V, real gamma, const int32_t* sets,
                      real* x, real* gi, real* g, int32_t* idx, real* val) {
    real* grads = V ? NULL : (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    for (int32_t t = 0; t < steps; ++t) {
        ef21o_x_update(d, gamma, g, x);
        if (!V) ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
        ef21o_randk_round(n, d, k, V ? V : grads, sets + (int64_t)t * n * k, gi, g, idx, val);
    }
    free(grads);
}

/* ------------------------------------------------------------------ */
/* EF21+ (Algorithm 3): per node the better of C and the Markov compressor */
/* ------------------------------------------------------------------ */

/* One round of Algorithm 3 given the local gradients: for every worker
 *     m_i = g_i + C(grad_i - g_i)        (Markov compressor)
 *     b_i = C(grad_i)                    (plain compressor)
 *     M_i = ||m_i - grad_i||^2,  B_i = ||b_i - grad_i||^2      (fp64 sums over the stored vectors)
 *     g_i <- m_i if M_i <= B_i else b_i
 * and the master's g = (1/n) sum_i g_i (sum over ascending i, then one multiply by 1/n).
 * idx/val receive the compressed vector that was used (C(grad_i - g_i) or C(grad_i)),
 * choice[i] = 0 for the Markov branch, 1 for the plain one. */
void ef21o_plus_round(int32_t n, int64_t d, int64_t k, const real* grads, real* gi, real* g,
                      int32_t* idx, real* val, int32_t* choice) {
    real* v = (real*)malloc((size_t)d * sizeof(real));
    real* m = (real*)malloc((size_t)d * sizeof(real));
    int32_t* ib = (int32_t*)malloc((size_t)k * sizeof(int32_t));
    real* vb = (real*)malloc((size_t)k * sizeof(real));
    unsigned char* inb = (unsigned char*)malloc((size_t)d);
    for (int32_t i = 0; i < n; ++i) {
        const real* gr = grads + (int64_t)i * d;
        real* gs = gi + (int64_t)i * d;
        int32_t* im = idx + (int64_t)i * k;
        real* vm = val + (int64_t)i * k;
        for (int64_t j = 0; j < d; ++j) { v[j] = gr[j] - gs[j]; m[j] = gs[j]; }
        ef21o_topk(v, d, k, im, vm);
        for (int64_t t = 0; t < k; ++t) m[im[t]] = m[im[t]] + vm[t];
        double M = 0.0;
        for (int64_t j = 0; j < d; ++j) { double e = (double)m[j] - (double)gr[j]; M += e * e; }
        ef21o_topk(gr, d, k, ib, vb);
        memset(inb, 0, (size_t)d);
        for (int64_t t = 0; t < k; ++t) inb[ib[t]] = 1;
        double B = 0.0;
        for (int64_t j = 0; j < d; ++j) if (!inb[j]) { double e = (double)gr[j]; B += e * e; }
        if (M <= B) {
            memcpy(gs, m, (size_t)d * sizeof(real));
            choice[i] = 0;
        } else {
            for (int64_t j = 0; j < d; ++j) gs[j] = (real)0;
            for (int64_t t = 0; t < k; ++t) { gs[ib[t]] = vb[t]; im[t] = ib[t]; vm[t] = vb[t]; }
            choice[i] = 1;
        }
    }
    const real inv_n = (real)1 / (real)n;
    for (int64_t j = 0; j < d; ++j) {
        real s = (real)0;
        for (int32_t i = 0; i < n; ++i) s = s + gi[(int64_t)i * d + j];
        g[j] = s * inv_n;
    }
    free(v); free(m); free(ib); free(vb); free(inb);
}

void ef21o_plus_step(int32_t steps, int32_t n, int64_t d, int64_t k, const float* A, const float* y,
                     const int64_t* row_off, double lam, real gamma,
                     real* x, real* gi, real* g, int32_t* idx, real* val, int32_t* choice) {
    real* grads = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    for (int32_t t = 0; t < steps; ++t) {
        ef21o_x_update(d, gamma, g, x);
        ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
        ef21o_plus_round(n, d, k, grads, gi, g, idx, val, choice);
    }
    free(grads);
}

void ef21o_plus_step_grads(int32_t steps, int32_t n, int64_t d, int64_t k, const real* V, real gamma,
                           real* x, real* gi, real* g, int32_t* idx, real* val, int32_t* choice) {
    for (int32_t t = 0; t < steps; ++t) {
        ef21o_x_update(d, gamma, g, x);
        ef21o_plus_round(n, d, k, V, gi, g, idx, val, choice);
    }
}

/* ------------------------------------------------------------------ */
/* Stochastic EF21 (Algorithm 5): minibatch gradient estimates          */
/* ------------------------------------------------------------------ */

/* One iteration of Algorithm 5: x <- x - gamma g; every worker forms the estimate
 *     ghat_i = (1/tau) sum_{r in batch_i} rho_r a_r + regulariser term
 * over the tau rows batch[i][0..tau) of its shard (row numbers inside the shard, drawn by the caller)
 * and uses it in place of grad f_i in the message round of Algorithm 2. */
void ef21o_step_minibatch(int32_t n, int64_t d, int64_t k, const float* A, const float* y,
                          const int64_t* row_off, double lam, real gamma, const int32_t* batch, int32_t tau,
                          real* x, real* gi, real* g, int32_t* idx, real* val) {
    real* grads = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    float* Ab = (float*)malloc((size_t)tau * (size_t)d * sizeof(float));
    float* yb = (float*)malloc((size_t)tau * sizeof(float));
    ef21o_x_update(d, gamma, g, x);
    for (int32_t i = 0; i < n; ++i) {
        for (int32_t r = 0; r < tau; ++r) {
            const int64_t row = row_off[i] + batch[(int64_t)i * tau + r];
            memcpy(Ab + (int64_t)r * d, A + row * d, (size_t)d * sizeof(float));
            yb[r] = y[row];
        }
        ef21o_local_grad(Ab, yb, tau, d, x, lam, grads + (int64_t)i * d);
    }
    ef21o_round(n, d, k, grads, gi, g, idx, val);
    free(grads); free(Ab); free(yb);
}

/* ------------------------------------------------------------------ */
/* EF, the original error feedback method (Algorithm 4)                */
/* ------------------------------------------------------------------ */

/* State of Algorithm 4 between iterations: x, the errors e_i, the messages w_i last sent (idx/val,
 * k pairs per worker) and a_i = gamma * grad f_i(x) at the current x (the vector each worker
 * "would like" to send; it is needed again by the error update of the next iteration).
 * Each of  gamma * grad,  e + a,  (e + a) - w,  s * (1/n),  x - p  is one rounded operation. */

/* Messages of one round: w_i = C(e_i + a_i) for every worker. */
static void ef_messages(int32_t n, int64_t d, int64_t k, const real* e, const real* a, int32_t* idx, real* val) {
    real* p = (real*)malloc((size_t)d * sizeof(real));
    for (int32_t i = 0; i < n; ++i) {
        for (int64_t j = 0; j < d; ++j) p[j] = e[(int64_t)i * d + j] + a[(int64_t)i * d + j];
        ef21o_topk(p, d, k, idx + (int64_t)i * k, val + (int64_t)i * k);
    }
    free(p);
}

static void ef_scale(int32_t n, int64_t d, real gamma, const real* grads, real* a) {
    for (int64_t e = 0; e < (int64_t)n * d; ++e) a[e] = gamma * grads[e];
}

/* Algorithm 4, the two lines before the loop, given the local gradients at x^0:
 *     e_i^0 = 0,   w_i^0 = C(gamma grad f_i(x^0)). */
void ef21o_ef_init_from_grads(int32_t n, int64_t d, int64_t k, real gamma, const real* grads,
                              real* e, real* a, int32_t* idx, real* val) {
    memset(e, 0, (size_t)n * (size_t)d * sizeof(real));
    ef_scale(n, d, gamma, grads, a);
    ef_messages(n, d, k, e, a, idx, val);
}

/* Algorithm 4, the part of one loop iteration that precedes the new gradient:
 *     master:  x^{t+1} = x^t - (1/n) sum_i w_i^t      (per coordinate: sum over ascending i from 0,
 *                                                      one multiply by 1/n, one subtraction)
 *     nodes:   e_i^{t+1} = e_i^t + gamma grad f_i(x^t) - w_i^t */
static void ef_master_and_error(int32_t n, int64_t d, int64_t k, const int32_t* idx, const real* val,
                                const real* a, real* x, real* e) {
    real* s = (real*)calloc((size_t)d, sizeof(real));
    unsigned char* touched = (unsigned char*)calloc((size_t)d, 1);
    for (int32_t i = 0; i < n; ++i)
        for (int64_t t = 0; t < k; ++t) {
            const int64_t j = idx[(int64_t)i * k + t];
            s[j] = s[j] + val[(int64_t)i * k + t];
            touched[j] = 1;
        }
    const real inv_n = (real)1 / (real)n;
    for (int64_t j = 0; j < d; ++j)
        if (touched[j]) {
            const real p = s[j] * inv_n;
            x[j] = x[j] - p;
        }
    free(s); free(touched);
    real* w = (real*)malloc((size_t)d * sizeof(real));
    for (int32_t i = 0; i < n; ++i) {
        for (int64_t j = 0; j < d; ++j) w[j] = 0;
        for (int64_t t = 0; t < k; ++t) w[idx[(int64_t)i * k + t]] = val[(int64_t)i * k + t];
        real* ei = e + (int64_t)i * d;
        const real* ai = a + (int64_t)i * d;
        for (int64_t j = 0; j < d; ++j) {
            const real want = ei[j] + ai[j];
            ei[j] = want - w[j];
        }
    }
    free(w);
}

/* One whole iteration of Algorithm 4's loop given the local gradients at the NEW point
 * (callers that supply gradients pass them in; grads_new is grad f_i(x^{t+1})):
 *     a_i <- gamma grad f_i(x^{t+1}),   w_i^{t+1} = C(e_i^{t+1} + a_i). */
static void ef_new_messages(int32_t n, int64_t d, int64_t k, real gamma, const real* grads_new,
                            const real* e, real* a, int32_t* idx, real* val) {
    ef_scale(n, d, gamma, grads_new, a);
    ef_messages(n, d, k, e, a, idx, val);
}

void ef21o_ef_init(int32_t n, int64_t d, int64_t k, const float* A, const float* y, const int64_t* row_off,
                   double lam, real gamma, const real* x, real* e, real* a, int32_t* idx, real* val) {
    real* grads = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
    ef21o_ef_init_from_grads(n, d, k, gamma, grads, e, a, idx, val);
    free(grads);
}

void ef21o_ef_step(int32_t steps, int32_t n, int64_t d, int64_t k, const float* A, const float* y,
                   const int64_t* row_off, double lam, real gamma,
                   real* x, real* e, real* a, int32_t* idx, real* val) {
    real* grads = (real*)malloc((size_t)n * (size_t)d * sizeof(real));
    for (int32_t t = 0; t < steps; ++t) {
        ef_master_and_error(n, d, k, idx, val, a, x, e);
        ef21o_all_grads(n, d, A, y, row_off, x, lam, grads);
        ef_new_messages(n, d, k, gamma, grads, e, a, idx, val);
    }
    free(grads);
}

/* The same loop with caller-supplied gradients V[n][d] standing in for grad f_i at every point. */
void ef21o_ef_step_grads(int32_t steps, int32_t n, int64_t d, int64_t k, const real* V, real gamma,
                         real* x, real* e, real* a, int32_t* idx, real* val) {
    for (int32_t t = 0; t < steps; ++t) {
        ef_master_and_error(n, d, k, idx, val, a, x, e);
        ef_new_messages(n, d, k, gamma, V, e, a, idx, val);
    }
}

/*
 * E2-TTT oracle: a plain, slow, fp64 CPU statement of what the chunk-parallel fast-weight
 * update computes.  TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; no product code path may.  It shares no code with the CUDA
 * library and is written from the paper's definitions:
 *
 *   - the token-wise recurrence  M_t = beta_t M_{t-1} + eta_t G_t,  W_t = gamma_t W_{t-1} + M_t
 *     (Eq. "tokenwise_ttt_decay_momentum", Section 3.1), run literally, one token at a time;
 *   - G_t = - grad_W L(f_{W_0}(k_t), v_t) taken at the frozen chunk-start weights W_0
 *     (Section 3.1, Eq. "ttt_minibatch_update"), L = 1/2 ||f - v||^2 (Section 2 names the usual choice, a mean
 *     squared error, without a formula; the scale is a reading);
 *   - outputs o_t = f_{W_0}(q_t) from the chunk-start weights (Eq. "chunkwise_output",
 *     Algorithm 1 line 1);
 *   - fast-weight networks of Section 4 "Fast-weight Network":
 *       GELU MLP : f_W(x) = x + LN(W2 GELU(W1 x))
 *       SwiGLU   : f_W(x) = x + LN(W3 (SiLU(W1 x) * (W2 x)))
 *     LN = layer norm over the d outputs, biased variance, eps inside the square root, no
 *     affine parameters; GELU = x Phi(x) with the exact erf (both readings: the paper does
 *     not say).
 *
 *   - optional post-chunk normalisation (Appendix "Implementation details": L2 normalisation of the
 *     fast-weight matrices at each chunk boundary; the paper gives neither axis nor target - a
 *     reading): after the last token of a chunk every row w of every W_i (one output unit's
 *     weights; the momentum is left alone) becomes  n w / (||w||_2 + eps_n), n the row's target norm,
 *     an input.  The next chunk starts from, and the final state is, the normalised W.
 *
 * The closed form of Proposition 1 is NOT used here: this file is the definition the closed
 * form must reproduce.  The reverse pass is the adjoint of exactly this program, swept token
 * by token.
 *
 * Pins (tests/test_oracle_pins.py): inner gradients vs central finite differences; sequential
 * chunk-end states vs Proposition 1 and vs the division-free unrolled Eq. "unroll_recurrence";
 * neutral gates reduce to one plain chunk-wise step; C = 1 reduces to the token-wise update;
 * the hand-expanded C = 2 case; the reverse pass vs finite differences and vs an independent
 * automatic-differentiation run; the normalisation vs an independent chunk-by-chunk restatement and
 * its reverse pass vs finite differences.  The paper prints no output or state VALUES, so absolute
 * values are fixed only by those pins and by the readings above.
 *
 * Layouts (row-major, dense, double): q, k, v, o [N, L, d]; eta, beta, gamma [N, L];
 * matrix i of the fast-weight collection [N, rows_i, cols_i] with
 *   MLP    : W1 [h, d], W2 [d, h]          SwiGLU : W1 [h, d], W2 [h, d], W3 [d, h].
 * N = B*H independent sequences.  A final chunk shorter than C is allowed.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define KIND_MLP 0
#define KIND_SWIGLU 1
#define MAXMAT 3

typedef struct {
    int d, h, kind, nmat;
    double eps;
    size_t n; /* elements per matrix = d*h (every matrix of both networks) */
} net_t;

static net_t make_net(int d, int h, int kind, double eps) {
    net_t n;
    n.d = d; n.h = h; n.kind = kind; n.eps = eps;
    n.nmat = (kind == KIND_MLP) ? 2 : 3;
    n.n = (size_t)d * (size_t)h;
    return n;
}

/* ---------- small dense helpers (plain loops) ---------- */
static void matvec(int rows, int cols, const double* A, const double* x, double* y) { /* y = A x */
    for (int i = 0; i < rows; ++i) {
        double s = 0.0;
        for (int j = 0; j < cols; ++j) s += A[(size_t)i * cols + j] * x[j];
        y[i] = s;
    }
}
static void matvec_t_acc(int rows, int cols, const double* A, const double* x, double* y) { /* y += A^T x */
    for (int i = 0; i < rows; ++i)
        for (int j = 0; j < cols; ++j) y[j] += A[(size_t)i * cols + j] * x[i];
}
static void outer_acc(int rows, int cols, double s, const double* a, const double* b, double* A) { /* A += s a b^T */
    for (int i = 0; i < rows; ++i)
        for (int j = 0; j < cols; ++j) A[(size_t)i * cols + j] += s * a[i] * b[j];
}
static double dot(size_t n, const double* a, const double* b) {
    double s = 0.0;
    for (size_t i = 0; i < n; ++i) s += a[i] * b[i];
    return s;
}

/* ---------- scalar nonlinearities ---------- */
static double Phi(double z) { return 0.5 * (1.0 + erf(z * 0.70710678118654752440)); }
static double phi(double z) { return 0.39894228040143267794 * exp(-0.5 * z * z); }
static double gelu(double z) { return z * Phi(z); }
static double gelu_d1(double z) { return Phi(z) + z * phi(z); }
static double gelu_d2(double z) { return phi(z) * (2.0 - z * z); }
static double sigm(double z) { return 1.0 / (1.0 + exp(-z)); }
static double silu(double z) { return z * sigm(z); }
static double silu_d1(double z) { double s = sigm(z); return s * (1.0 + z * (1.0 - s)); }
static double silu_d2(double z) { double s = sigm(z); return s * (1.0 - s) * (2.0 + z * (1.0 - 2.0 * s)); }

/* ---------- layer norm over d features and the product with its (symmetric) Jacobian ---------- */
static void ln_fwd(int d, double eps, const double* u, double* y, double* r_out) {
    double mu = 0.0, var = 0.0;
    for (int i = 0; i < d; ++i) mu += u[i];
    mu /= d;
    for (int i = 0; i < d; ++i) var += (u[i] - mu) * (u[i] - mu);
    var /= d;
    double r = 1.0 / sqrt(var + eps);
    for (int i = 0; i < d; ++i) y[i] = (u[i] - mu) * r;
    *r_out = r;
}
/* out = (dy/du) e = r ( e - mean(e) - y mean(e*y) ) */
static void ln_jac(int d, const double* y, double r, const double* e, double* out) {
    double me = 0.0, mey = 0.0;
    for (int i = 0; i < d; ++i) { me += e[i]; mey += e[i] * y[i]; }
    me /= d; mey /= d;
    for (int i = 0; i < d; ++i) out[i] = r * (e[i] - me - y[i] * mey);
}

/* ---------- per-token scratch ---------- */
typedef struct {
    double *z1, *z2, *a, *u, *y, *e, *pu, *ph, *pz1, *pz2; /* forward / inner-backward */
    double *t_d0, *t_d1, *t_d2, *t_h0, *t_h1, *t_h2, *t_h3;  /* reverse-pass temporaries */
    double r;
    double* block;
} tok_t;

static int tok_alloc(tok_t* t, int d, int h) {
    size_t nd = 7, nh = 10;
    t->block = (double*)calloc(nd * d + nh * h, sizeof(double));
    if (!t->block) return -1;
    double* p = t->block;
    t->u = p; p += d; t->y = p; p += d; t->e = p; p += d; t->pu = p; p += d;
    t->t_d0 = p; p += d; t->t_d1 = p; p += d; t->t_d2 = p; p += d;
    t->z1 = p; p += h; t->z2 = p; p += h; t->a = p; p += h; t->ph = p; p += h;
    t->pz1 = p; p += h; t->pz2 = p; p += h;
    t->t_h0 = p; p += h; t->t_h1 = p; p += h; t->t_h2 = p; p += h; t->t_h3 = p; p += h;
    return 0;
}
static void tok_free(tok_t* t) { free(t->block); t->block = NULL; }

/* f_W(x): fills t->z1 (,z2), t->a (hidden activation fed to the last matrix), t->u, t->y, t->r.
 * Returns f in out (may be NULL). */
static void net_forward(const net_t* n, const double* const* W, const double* x, tok_t* t, double* out) {
    const int d = n->d, h = n->h;
    if (n->kind == KIND_MLP) {
        matvec(h, d, W[0], x, t->z1);
        for (int j = 0; j < h; ++j) t->a[j] = gelu(t->z1[j]);
        matvec(d, h, W[1], t->a, t->u);
    } else {
        matvec(h, d, W[0], x, t->z1);
        matvec(h, d, W[1], x, t->z2);
        for (int j = 0; j < h; ++j) t->a[j] = silu(t->z1[j]) * t->z2[j];
        matvec(d, h, W[2], t->a, t->u);
    }
    ln_fwd(d, n->eps, t->u, t->y, &t->r);
    if (out)
        for (int i = 0; i < d; ++i) out[i] = x[i] + t->y[i];
}

/* Inner loss L = 1/2 || f_W(k) - v ||^2 and everything its gradient needs (kept in t):
 * e = f - v, pu = dL/du, ph = dL/d(hidden activation), pz* = dL/d(pre-activations). */
static double inner_backward(const net_t* n, const double* const* W, const double* k, const double* v, tok_t* t) {
    const int d = n->d, h = n->h;
    net_forward(n, W, k, t, NULL);
    double loss = 0.0;
    for (int i = 0; i < d; ++i) { t->e[i] = k[i] + t->y[i] - v[i]; loss += 0.5 * t->e[i] * t->e[i]; }
    ln_jac(d, t->y, t->r, t->e, t->pu);
    const double* Wlast = W[n->nmat - 1]; /* [d, h] */
    for (int j = 0; j < h; ++j) t->ph[j] = 0.0;
    matvec_t_acc(d, h, Wlast, t->pu, t->ph);
    if (n->kind == KIND_MLP) {
        for (int j = 0; j < h; ++j) t->pz1[j] = t->ph[j] * gelu_d1(t->z1[j]);
    } else {
        for (int j = 0; j < h; ++j) {
            t->pz1[j] = t->ph[j] * t->z2[j] * silu_d1(t->z1[j]);
            t->pz2[j] = t->ph[j] * silu(t->z1[j]);
        }
    }
    return loss;
}

/* G_i = - dL/dW_i at W (written, not accumulated). */
static void inner_neg_grad(const net_t* n, const double* const* W, const double* k, const double* v, tok_t* t,
                           double* const* G) {
    const int d = n->d, h = n->h;
    inner_backward(n, W, k, v, t);
    for (int i = 0; i < n->nmat; ++i) memset(G[i], 0, n->n * sizeof(double));
    if (n->kind == KIND_MLP) {
        outer_acc(h, d, -1.0, t->pz1, k, G[0]);
        outer_acc(d, h, -1.0, t->pu, t->a, G[1]);
    } else {
        outer_acc(h, d, -1.0, t->pz1, k, G[0]);
        outer_acc(h, d, -1.0, t->pz2, k, G[1]);
        outer_acc(d, h, -1.0, t->pu, t->a, G[2]);
    }
}

/* ---------- reverse-pass pieces ---------- */

/* o = f_W(q); given ob = dLoss/do:  qb = dLoss/dq (written),  Wb_i += dLoss/dW_i. */
static void output_vjp(const net_t* n, const double* const* W, const double* q, const double* ob, tok_t* t,
                       double* qb, double* const* Wb) {
    const int d = n->d, h = n->h;
    net_forward(n, W, q, t, NULL);
    double *ub = t->t_d0, *ab = t->t_h0, *zb1 = t->t_h1, *zb2 = t->t_h2;
    ln_jac(d, t->y, t->r, ob, ub);
    for (int j = 0; j < h; ++j) ab[j] = 0.0;
    matvec_t_acc(d, h, W[n->nmat - 1], ub, ab);
    outer_acc(d, h, 1.0, ub, t->a, Wb[n->nmat - 1]);
    for (int i = 0; i < d; ++i) qb[i] = ob[i];
    if (n->kind == KIND_MLP) {
        for (int j = 0; j < h; ++j) zb1[j] = ab[j] * gelu_d1(t->z1[j]);
        matvec_t_acc(h, d, W[0], zb1, qb);
        outer_acc(h, d, 1.0, zb1, q, Wb[0]);
    } else {
        for (int j = 0; j < h; ++j) {
            zb1[j] = ab[j] * t->z2[j] * silu_d1(t->z1[j]);
            zb2[j] = ab[j] * silu(t->z1[j]);
        }
        matvec_t_acc(h, d, W[0], zb1, qb);
        matvec_t_acc(h, d, W[1], zb2, qb);
        outer_acc(h, d, 1.0, zb1, q, Wb[0]);
        outer_acc(h, d, 1.0, zb2, q, Wb[1]);
    }
}

/* G(W, k, v) = - grad_W L.  Given Gb_i = dLoss/dG_i:  kb, vb written;  Wb_i += dLoss/dW_i.
 * This is the derivative of the scalar  <Gb, G>  with respect to (W, k, v): a second-order
 * (Hessian-vector) quantity of the per-token loss, taken by reversing inner_backward step by step. */
static void neg_grad_vjp(const net_t* n, const double* const* W, const double* k, const double* v,
                         const double* const* Gb, tok_t* t, double* kb, double* vb, double* const* Wb) {
    const int d = n->d, h = n->h;
    const int last = n->nmat - 1;
    inner_backward(n, W, k, v, t);
    double *pub = t->t_d0, *eb = t->t_d1, *ub = t->t_d2;
    double *ab = t->t_h0, *phb = t->t_h1, *zb1 = t->t_h2, *zb2 = t->t_h3;

    /* G_last = - pu a^T :  pub = -Gb_last a ;  ab = -Gb_last^T pu */
    matvec(d, h, Gb[last], t->a, pub);
    for (int i = 0; i < d; ++i) pub[i] = -pub[i];
    for (int j = 0; j < h; ++j) ab[j] = 0.0;
    matvec_t_acc(d, h, Gb[last], t->pu, ab);
    for (int j = 0; j < h; ++j) ab[j] = -ab[j];
    for (int i = 0; i < d; ++i) kb[i] = 0.0;

    if (n->kind == KIND_MLP) {
        /* G_1 = - pz1 k^T :  pzb = -Gb_1 k ;  kb = -Gb_1^T pz1 */
        double* pzb = zb2; /* reuse as temporary */
        matvec(h, d, Gb[0], k, pzb);
        for (int j = 0; j < h; ++j) pzb[j] = -pzb[j];
        matvec_t_acc(h, d, Gb[0], t->pz1, kb);
        for (int i = 0; i < d; ++i) kb[i] = -kb[i];
        /* pz1 = ph * gelu'(z1) */
        for (int j = 0; j < h; ++j) {
            phb[j] = pzb[j] * gelu_d1(t->z1[j]);
            zb1[j] = pzb[j] * t->ph[j] * gelu_d2(t->z1[j]);
        }
    } else {
        double *pzb1 = zb1, *pzb2 = zb2;
        matvec(h, d, Gb[0], k, pzb1);
        matvec(h, d, Gb[1], k, pzb2);
        matvec_t_acc(h, d, Gb[0], t->pz1, kb);
        matvec_t_acc(h, d, Gb[1], t->pz2, kb);
        for (int i = 0; i < d; ++i) kb[i] = -kb[i];
        for (int j = 0; j < h; ++j) {
            double b1 = -pzb1[j], b2 = -pzb2[j];
            double z1 = t->z1[j], z2 = t->z2[j], g1 = silu_d1(z1);
            /* pz1 = ph z2 silu'(z1) ;  pz2 = ph silu(z1) */
            phb[j] = b1 * z2 * g1 + b2 * silu(z1);
            zb2[j] = b1 * t->ph[j] * g1;
            zb1[j] = b1 * t->ph[j] * z2 * silu_d2(z1) + b2 * t->ph[j] * g1;
        }
    }
    /* ph = W_last^T pu */
    {
        double* tmp = eb; /* W_last phb */
        matvec(d, h, W[last], phb, tmp);
        for (int i = 0; i < d; ++i) pub[i] += tmp[i];
        outer_acc(d, h, 1.0, t->pu, phb, Wb[last]);
    }
    /* pu = J(u) e :  eb = J pub ;  ub = d<pub, J(u) e>/du */
    ln_jac(d, t->y, t->r, pub, eb);
    {
        double s_pp = 0.0, m_py = 0.0, m_ey = 0.0;
        for (int i = 0; i < d; ++i) { s_pp += pub[i] * t->pu[i]; m_py += pub[i] * t->y[i]; m_ey += t->e[i] * t->y[i]; }
        m_py /= d; m_ey /= d;
        for (int i = 0; i < d; ++i)
            ub[i] = -(t->r / d) * s_pp * t->y[i] - t->r * (m_py * t->pu[i] + m_ey * eb[i]);
    }
    /* e = k + y - v */
    for (int i = 0; i < d; ++i) { kb[i] += eb[i]; vb[i] = -eb[i]; }
    {
        double* tmp = pub; /* pub is dead: J eb */
        ln_jac(d, t->y, t->r, eb, tmp);
        for (int i = 0; i < d; ++i) ub[i] += tmp[i];
    }
    /* u = W_last a */
    matvec_t_acc(d, h, W[last], ub, ab);
    outer_acc(d, h, 1.0, ub, t->a, Wb[last]);
    if (n->kind == KIND_MLP) {
        for (int j = 0; j < h; ++j) zb1[j] += ab[j] * gelu_d1(t->z1[j]);
        matvec_t_acc(h, d, W[0], zb1, kb);
        outer_acc(h, d, 1.0, zb1, k, Wb[0]);
    } else {
        for (int j = 0; j < h; ++j) {
            zb1[j] += ab[j] * t->z2[j] * silu_d1(t->z1[j]);
            zb2[j] += ab[j] * silu(t->z1[j]);
        }
        matvec_t_acc(h, d, W[0], zb1, kb);
        matvec_t_acc(h, d, W[1], zb2, kb);
        outer_acc(h, d, 1.0, zb1, k, Wb[0]);
        outer_acc(h, d, 1.0, zb2, k, Wb[1]);
    }
}

/* ---------- post-chunk normalisation of one matrix: rows w -> n w / (||w|| + eps_n) ---------- */
static int mat_rows(const net_t* n, int i) { return (i == n->nmat - 1) ? n->d : n->h; }

static void rows_normalise(const net_t* n, int i, double* W, const double* target, double eps_n) {
    const int rows = mat_rows(n, i);
    const size_t cols = n->n / (size_t)rows;
    for (int r = 0; r < rows; ++r) {
        double* w = W + (size_t)r * cols;
        const double s = sqrt(dot(cols, w, w));
        const double f = target[r] / (s + eps_n);
        for (size_t c = 0; c < cols; ++c) w[c] *= f;
    }
}

/* adjoint of rows_normalise: Wt = the rows BEFORE normalisation; Yb (in) = adjoint of the normalised rows, (out) =
 * adjoint of Wt; nb, if not NULL, accumulates the adjoint of the targets.
 *   y = n w / (s + e),  s = ||w||:   wb = n/(s+e) (yb - w <yb, w> / (s (s+e))),   nb = <yb, w> / (s+e)          */
static void rows_normalise_vjp(const net_t* n, int i, const double* Wt, const double* target, double eps_n,
                               double* Yb, double* nb) {
    const int rows = mat_rows(n, i);
    const size_t cols = n->n / (size_t)rows;
    for (int r = 0; r < rows; ++r) {
        const double* w = Wt + (size_t)r * cols;
        double* yb = Yb + (size_t)r * cols;
        const double s = sqrt(dot(cols, w, w));
        const double yw = dot(cols, yb, w);
        if (nb) nb[r] += yw / (s + eps_n);
        const double f = target[r] / (s + eps_n);
        const double g = (s > 0.0) ? yw / (s * (s + eps_n)) : 0.0;
        for (size_t c = 0; c < cols; ++c) yb[c] = f * (yb[c] - w[c] * g);
    }
}

/* ---------- one sequence, forward ---------- */
static int seq_forward(const net_t* n, int L, int C, const double* q, const double* k, const double* v,
                       const double* eta, const double* beta, const double* gamma,
                       double* const* W, double* const* M, /* in: initial state, out: final state */
                       double* o /* may be NULL */, double* chunk_states /* may be NULL: [nchunks][2][nmat][n] */,
                       const double* const* row_norm /* NULL: no post-chunk normalisation */, double eps_n) {
    const int d = n->d;
    tok_t t;
    if (tok_alloc(&t, n->d, n->h)) return -1;
    double* W0[MAXMAT];
    double* G[MAXMAT];
    for (int i = 0; i < n->nmat; ++i) {
        W0[i] = (double*)malloc(n->n * sizeof(double));
        G[i] = (double*)malloc(n->n * sizeof(double));
        if (!W0[i] || !G[i]) return -1;
    }
    int chunk = 0;
    for (int s = 0; s < L; s += C, ++chunk) {
        const int len = (L - s < C) ? (L - s) : C;
        for (int i = 0; i < n->nmat; ++i) memcpy(W0[i], W[i], n->n * sizeof(double)); /* frozen for the chunk */
        if (chunk_states) {
            double* cs = chunk_states + (size_t)chunk * 2 * n->nmat * n->n;
            for (int i = 0; i < n->nmat; ++i) {
                memcpy(cs + (size_t)i * n->n, W[i], n->n * sizeof(double));
                memcpy(cs + (size_t)(n->nmat + i) * n->n, M[i], n->n * sizeof(double));
            }
        }
        if (o)
            for (int tt = s; tt < s + len; ++tt)
                net_forward(n, (const double* const*)W0, q + (size_t)tt * d, &t, o + (size_t)tt * d);
        for (int tt = s; tt < s + len; ++tt) {
            inner_neg_grad(n, (const double* const*)W0, k + (size_t)tt * d, v + (size_t)tt * d, &t, G);
            for (int i = 0; i < n->nmat; ++i) {
                double *Mi = M[i], *Wi = W[i];
                const double* Gi = G[i];
                for (size_t e = 0; e < n->n; ++e) {
                    Mi[e] = beta[tt] * Mi[e] + eta[tt] * Gi[e];
                    Wi[e] = gamma[tt] * Wi[e] + Mi[e];
                }
            }
        }
        if (row_norm)
            for (int i = 0; i < n->nmat; ++i) rows_normalise(n, i, W[i], row_norm[i], eps_n);
    }
    for (int i = 0; i < n->nmat; ++i) { free(W0[i]); free(G[i]); }
    tok_free(&t);
    return 0;
}

/* ---------- one sequence, reverse ---------- */
static int seq_backward(const net_t* n, int L, int C, const double* q, const double* k, const double* v,
                        const double* eta, const double* beta, const double* gamma,
                        const double* const* W_init, const double* const* M_init, /* M_init[i] never NULL here */
                        const double* d_o, double* const* Wb, double* const* Mb, /* in: adjoints of the final state; out: of the initial state */
                        double* dq, double* dk, double* dv, double* deta, double* dbeta, double* dgamma,
                        const double* const* row_norm /* NULL: no post-chunk normalisation */, double eps_n,
                        double* const* row_norm_b /* NULL or out: adjoints of the targets (accumulated) */) {
    const int d = n->d, nm = n->nmat;
    const size_t ne = n->n;
    const int nchunks = (L + C - 1) / C;
    tok_t t;
    if (tok_alloc(&t, n->d, n->h)) return -1;
    /* forward sweep keeping every chunk-start state */
    double* cs = (double*)malloc((size_t)nchunks * 2 * nm * ne * sizeof(double));
    double* W[MAXMAT]; double* M[MAXMAT]; double* G[MAXMAT]; double* Gb[MAXMAT]; double* W0b[MAXMAT];
    /* per-token states of the chunk being reversed: Wprev[t] = W_{t-1}, Mprev[t] = M_{t-1} */
    double* Wprev = (double*)malloc((size_t)C * nm * ne * sizeof(double));
    double* Mprev = (double*)malloc((size_t)C * nm * ne * sizeof(double));
    if (!cs || !Wprev || !Mprev) return -1;
    for (int i = 0; i < nm; ++i) {
        W[i] = (double*)malloc(ne * sizeof(double)); M[i] = (double*)malloc(ne * sizeof(double));
        G[i] = (double*)malloc(ne * sizeof(double)); Gb[i] = (double*)malloc(ne * sizeof(double));
        W0b[i] = (double*)malloc(ne * sizeof(double));
        if (!W[i] || !M[i] || !G[i] || !Gb[i] || !W0b[i]) return -1;
        memcpy(W[i], W_init[i], ne * sizeof(double));
        memcpy(M[i], M_init[i], ne * sizeof(double));
    }
    if (seq_forward(n, L, C, q, k, v, eta, beta, gamma, W, M, NULL, cs, row_norm, eps_n)) return -1;

    for (int c = nchunks - 1; c >= 0; --c) {
        const int s = c * C;
        const int len = (L - s < C) ? (L - s) : C;
        const double* W0[MAXMAT];
        const double* cstate = cs + (size_t)c * 2 * nm * ne;
        for (int i = 0; i < nm; ++i) {
            W0[i] = cstate + (size_t)i * ne;
            memcpy(W[i], cstate + (size_t)i * ne, ne * sizeof(double));
            memcpy(M[i], cstate + (size_t)(nm + i) * ne, ne * sizeof(double));
            memset(W0b[i], 0, ne * sizeof(double));
        }
        /* replay the chunk, remembering the state before every token */
        for (int j = 0; j < len; ++j) {
            const int tt = s + j;
            for (int i = 0; i < nm; ++i) {
                memcpy(Wprev + ((size_t)j * nm + i) * ne, W[i], ne * sizeof(double));
                memcpy(Mprev + ((size_t)j * nm + i) * ne, M[i], ne * sizeof(double));
            }
            inner_neg_grad(n, W0, k + (size_t)tt * d, v + (size_t)tt * d, &t, G);
            for (int i = 0; i < nm; ++i)
                for (size_t e = 0; e < ne; ++e) {
                    M[i][e] = beta[tt] * M[i][e] + eta[tt] * G[i][e];
                    W[i][e] = gamma[tt] * W[i][e] + M[i][e];
                }
        }
        /* W now holds the chunk-end weights before normalisation: pull the adjoint back through it */
        if (row_norm)
            for (int i = 0; i < nm; ++i)
                rows_normalise_vjp(n, i, W[i], row_norm[i], eps_n, Wb[i], row_norm_b ? row_norm_b[i] : NULL);
        /* reverse the token-wise recurrence */
        for (int j = len - 1; j >= 0; --j) {
            const int tt = s + j;
            inner_neg_grad(n, W0, k + (size_t)tt * d, v + (size_t)tt * d, &t, G);
            double gb = 0.0, bb = 0.0, eb = 0.0;
            for (int i = 0; i < nm; ++i) {
                const double* Wp = Wprev + ((size_t)j * nm + i) * ne;
                const double* Mp = Mprev + ((size_t)j * nm + i) * ne;
                /* W_t = gamma_t W_{t-1} + M_t */
                for (size_t e = 0; e < ne; ++e) Mb[i][e] += Wb[i][e];
                gb += dot(ne, Wb[i], Wp);
                for (size_t e = 0; e < ne; ++e) Wb[i][e] *= gamma[tt];
                /* M_t = beta_t M_{t-1} + eta_t G_t */
                bb += dot(ne, Mb[i], Mp);
                eb += dot(ne, Mb[i], G[i]);
                for (size_t e = 0; e < ne; ++e) { Gb[i][e] = eta[tt] * Mb[i][e]; Mb[i][e] *= beta[tt]; }
            }
            dgamma[tt] = gb; dbeta[tt] = bb; deta[tt] = eb;
            neg_grad_vjp(n, W0, k + (size_t)tt * d, v + (size_t)tt * d, (const double* const*)Gb, &t,
                         dk + (size_t)tt * d, dv + (size_t)tt * d, W0b);
        }
        /* outputs of the chunk read the chunk-start weights */
        for (int j = 0; j < len; ++j) {
            const int tt = s + j;
            output_vjp(n, W0, q + (size_t)tt * d, d_o + (size_t)tt * d, &t, dq + (size_t)tt * d, W0b);
        }
        /* W_0 feeds the recurrence (Wb), every G_t and every o_t (W0b) */
        for (int i = 0; i < nm; ++i)
            for (size_t e = 0; e < ne; ++e) Wb[i][e] += W0b[i][e];
    }
    for (int i = 0; i < nm; ++i) { free(W[i]); free(M[i]); free(G[i]); free(Gb[i]); free(W0b[i]); }
    free(cs); free(Wprev); free(Mprev);
    tok_free(&t);
    return 0;
}

/* ---------- exported entry points ---------- */

int e2ttt_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Forward over N sequences.  W_final/M_final receive the final states; M_init may be NULL (zeros).
 * chunk_states, if not NULL, receives [N][nchunks][2][nmat][d*h]: the (W, M) at every chunk start.
 * Returns 0, or -1 on allocation failure / bad arguments.  threads <= 0: all cores. */
int e2ttt_oracle_fwd_norm(int N, int L, int d, int h, int C, int kind, double eps,
                          const double* q, const double* k, const double* v,
                          const double* eta, const double* beta, const double* gamma,
                          const double* const* W_init, const double* const* M_init,
                          double* o, double* const* W_final, double* const* M_final,
                          double* chunk_states, int threads,
                          const double* const* row_norm /* NULL or nmat x [N, rows_i] */, double eps_n) {
    if (N <= 0 || L <= 0 || d <= 0 || h <= 0 || C <= 0 || (kind != KIND_MLP && kind != KIND_SWIGLU)) return -1;
    net_t n = make_net(d, h, kind, eps);
    const int nchunks = (L + C - 1) / C;
    int fail = 0;
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
#endif
    for (int s = 0; s < N; ++s) {
        double* W[MAXMAT]; double* M[MAXMAT];
        for (int i = 0; i < n.nmat; ++i) {
            W[i] = W_final[i] + (size_t)s * n.n;
            M[i] = M_final[i] + (size_t)s * n.n;
            memcpy(W[i], W_init[i] + (size_t)s * n.n, n.n * sizeof(double));
            if (M_init) memcpy(M[i], M_init[i] + (size_t)s * n.n, n.n * sizeof(double));
            else memset(M[i], 0, n.n * sizeof(double));
        }
        const size_t off = (size_t)s * L;
        const double* rn[MAXMAT];
        for (int i = 0; i < n.nmat; ++i) rn[i] = row_norm ? row_norm[i] + (size_t)s * mat_rows(&n, i) : NULL;
        int rc = seq_forward(&n, L, C, q + off * d, k + off * d, v + off * d, eta + off, beta + off, gamma + off,
                             W, M, o ? o + off * d : NULL,
                             chunk_states ? chunk_states + (size_t)s * nchunks * 2 * n.nmat * n.n : NULL,
                             row_norm ? rn : NULL, eps_n);
        if (rc) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        }
    }
    return fail ? -1 : 0;
}

int e2ttt_oracle_fwd(int N, int L, int d, int h, int C, int kind, double eps,
                     const double* q, const double* k, const double* v,
                     const double* eta, const double* beta, const double* gamma,
                     const double* const* W_init, const double* const* M_init,
                     double* o, double* const* W_final, double* const* M_final,
                     double* chunk_states, int threads) {
    return e2ttt_oracle_fwd_norm(N, L, d, h, C, kind, eps, q, k, v, eta, beta, gamma, W_init, M_init, o, W_final,
                                 M_final, chunk_states, threads, NULL, 0.0);
}

/* Reverse pass over N sequences: adjoints of everything the forward reads, given d_o and the
 * adjoints of the final state (dW_final / dM_final, NULL = zeros).  With row_norm (post-chunk normalisation)
 * d_row_norm (NULL or nmat x [N, rows_i]) receives the adjoints of the targets. */
int e2ttt_oracle_bwd_norm(int N, int L, int d, int h, int C, int kind, double eps,
                          const double* q, const double* k, const double* v,
                          const double* eta, const double* beta, const double* gamma,
                          const double* const* W_init, const double* const* M_init,
                          const double* d_o, const double* const* dW_final, const double* const* dM_final,
                          double* dq, double* dk, double* dv, double* deta, double* dbeta, double* dgamma,
                          double* const* dW_init, double* const* dM_init, int threads,
                          const double* const* row_norm, double eps_n, double* const* d_row_norm) {
    if (N <= 0 || L <= 0 || d <= 0 || h <= 0 || C <= 0 || (kind != KIND_MLP && kind != KIND_SWIGLU)) return -1;
    net_t n = make_net(d, h, kind, eps);
    int fail = 0;
#ifdef _OPENMP
    if (threads <= 0) threads = omp_get_max_threads();
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1)
#endif
    for (int s = 0; s < N; ++s) {
        const double* Wi[MAXMAT]; const double* Mi[MAXMAT];
        double* Wb[MAXMAT]; double* Mb[MAXMAT];
        double* zeros = NULL;
        if (!M_init) zeros = (double*)calloc(n.n, sizeof(double));
        for (int i = 0; i < n.nmat; ++i) {
            Wi[i] = W_init[i] + (size_t)s * n.n;
            Mi[i] = M_init ? M_init[i] + (size_t)s * n.n : zeros;
            Wb[i] = dW_init[i] + (size_t)s * n.n;
            Mb[i] = dM_init[i] + (size_t)s * n.n;
            if (dW_final) memcpy(Wb[i], dW_final[i] + (size_t)s * n.n, n.n * sizeof(double));
            else memset(Wb[i], 0, n.n * sizeof(double));
            if (dM_final) memcpy(Mb[i], dM_final[i] + (size_t)s * n.n, n.n * sizeof(double));
            else memset(Mb[i], 0, n.n * sizeof(double));
        }
        const size_t off = (size_t)s * L;
        const double* rn[MAXMAT];
        double* rnb[MAXMAT];
        for (int i = 0; i < n.nmat; ++i) {
            rn[i] = row_norm ? row_norm[i] + (size_t)s * mat_rows(&n, i) : NULL;
            rnb[i] = (row_norm && d_row_norm) ? d_row_norm[i] + (size_t)s * mat_rows(&n, i) : NULL;
            if (rnb[i]) memset(rnb[i], 0, (size_t)mat_rows(&n, i) * sizeof(double));
        }
        int rc = (!M_init && !zeros) ? -1 :
                 seq_backward(&n, L, C, q + off * d, k + off * d, v + off * d, eta + off, beta + off, gamma + off,
                              Wi, Mi, d_o + off * d, Wb, Mb, dq + off * d, dk + off * d, dv + off * d,
                              deta + off, dbeta + off, dgamma + off, row_norm ? rn : NULL, eps_n,
                              (row_norm && d_row_norm) ? rnb : NULL);
        free(zeros);
        if (rc) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            fail = 1;
        }
    }
    return fail ? -1 : 0;
}

int e2ttt_oracle_bwd(int N, int L, int d, int h, int C, int kind, double eps,
                     const double* q, const double* k, const double* v,
                     const double* eta, const double* beta, const double* gamma,
                     const double* const* W_init, const double* const* M_init,
                     const double* d_o, const double* const* dW_final, const double* const* dM_final,
                     double* dq, double* dk, double* dv, double* deta, double* dbeta, double* dgamma,
                     double* const* dW_init, double* const* dM_init, int threads) {
    return e2ttt_oracle_bwd_norm(N, L, d, h, C, kind, eps, q, k, v, eta, beta, gamma, W_init, M_init, d_o, dW_final,
                                 dM_final, dq, dk, dv, deta, dbeta, dgamma, dW_init, dM_init, threads, NULL, 0.0, NULL);
}

/* One token at fixed weights: the inner loss and G_i = -dL/dW_i (for the finite-difference pin and
 * for evaluating the closed form outside this file). G may be NULL (loss only). */
double e2ttt_oracle_inner(int d, int h, int kind, double eps, const double* const* W,
                          const double* k, const double* v, double* const* G) {
    net_t n = make_net(d, h, kind, eps);
    tok_t t;
    if (tok_alloc(&t, d, h)) return NAN;
    double loss;
    if (G) { inner_neg_grad(&n, W, k, v, &t, G); loss = 0.0; for (int i = 0; i < d; ++i) loss += 0.5 * t.e[i] * t.e[i]; }
    else loss = inner_backward(&n, W, k, v, &t);
    tok_free(&t);
    return loss;
}

/* f_W(x) for one token. */
int e2ttt_oracle_net(int d, int h, int kind, double eps, const double* const* W, const double* x, double* out) {
    net_t n = make_net(d, h, kind, eps);
    tok_t t;
    if (tok_alloc(&t, d, h)) return -1;
    net_forward(&n, W, x, &t, out);
    tok_free(&t);
    return 0;
}

/*
 * TEST INFRASTRUCTURE -- not part of the product.
 *
 * Plain, slow, fp64 CPU statement of DSGD-CECA as the paper defines it.  It exists
 * so that tests (and the CPU-baseline leg of the benchmark) have something to compare
 * the CUDA library against.  It shares no code with the CUDA library and the library
 * never calls it.
 *
 * Every function follows the paper's steps in the paper's order and notation:
 *   - auxiliary sequence tau, delta_r, n_r ......... Sec. 3.1, Eq. (bin-n-1), Eq. (iter-nr)
 *   - CECA-2P communication matrix Q^(r) ........... Sec. 3.1, Eq. (2p-gossip-matrix-d1/d0)
 *   - CECA-1P communication matrix Q^(r) ........... Sec. 3.2, Eq. (1p-gossip-matrix)
 *   - weights a^(k), b^(k) and the payload z ....... Algorithm 1
 *   - x and y updates ............................... Sec. 4.1, Eq. (x-iter-dsgd), Eq. (y-iter-dsgd)
 *   - a CECA round = the same update with gamma = 0 . Sec. 3.1 "Main recursions", Algorithm 2
 *   - logistic-regression gradient .................. NOT in the paper (workload chosen by the
 *                                                     benchmark); pinned by calculus only.
 *   - least-squares gradient ........................ Sec. 5 "DSGD: least-squares problem"
 *
 * Indices are 0-based here.  The paper's agents are 1..n with a mod that maps into
 * {1..n}; paper agent p is index p-1, so a paper-odd agent has an even index.
 *
 * Readings taken where the paper is silent (listed again in the design notes):
 *   - n = 1: tau = 0, no peer; the step degenerates to x+ = x - gamma e, y+ = y - gamma e.
 *     parity unpinned (the paper says nothing about n = 1).
 *   - 1-port with odd n is undefined in the paper: returns an error.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_ODD_N_1P 2

#define VARIANT_1P 1
#define VARIANT_2P 2

typedef struct {
  int32_t n, tau, r, delta, n_r;
  int32_t payload;                  /* 0: x is the message base (delta=1); 1: y (delta=0) */
  int32_t a_num, a_den, b_num, b_den;
  double a, b;
} oracle_round_t;

/* tau = ceil(log2 n) computed on integers: the number of binary digits of n-1. */
static int32_t bit_count_of(int32_t v) {
  int32_t t = 0;
  while (v > 0) { t++; v >>= 1; }
  return t;
}

/*
 * Sec. 3.1 "Auxiliary variables" + Algorithm 1 (the branch on delta_r).
 * n-1 = (delta_0 ... delta_{tau-1})_2, delta_0 the most significant digit;
 * n_0 = 0, n_{r+1} = 2 n_r + delta_r; r = k mod tau.
 */
int ceca_oracle_round(int32_t n, int64_t k, oracle_round_t *out) {
  if (n < 1 || k < 0 || !out) return ORACLE_ERR_ARG;
  memset(out, 0, sizeof(*out));
  out->n = n;
  int32_t tau = bit_count_of(n - 1);
  out->tau = tau;
  if (tau == 0) { /* n = 1: reading for the silent case, see header */
    out->r = 0; out->delta = 1; out->n_r = 0; out->payload = 0;
    out->a_num = 1; out->a_den = 1; out->b_num = 1; out->b_den = 1;
    out->a = 1.0; out->b = 1.0;
    return ORACLE_OK;
  }
  int32_t r = (int32_t)(k % (int64_t)tau);
  int32_t n_r = 0, delta = 0;
  for (int32_t q = 0; q <= r; q++) {
    /* digit q of n-1 counted from the most significant one */
    delta = ((n - 1) >> (tau - 1 - q)) & 1;
    if (q < r) n_r = 2 * n_r + delta;
  }
  out->r = r; out->delta = delta; out->n_r = n_r;
  if (delta == 1) {          /* Algorithm 1, branch delta_r = 1 */
    out->payload = 0;
    out->a_num = 1;       out->a_den = 2;
    out->b_num = n_r;     out->b_den = 2 * n_r + 1;
  } else {                   /* Algorithm 1, branch delta_r = 0 */
    out->payload = 1;
    out->a_num = n_r + 1; out->a_den = 2 * n_r + 1;
    out->b_num = 1;       out->b_den = 2;
  }
  out->a = (double)out->a_num / (double)out->a_den;
  out->b = (double)out->b_num / (double)out->b_den;
  return ORACLE_OK;
}

static int32_t wrap(int64_t i, int32_t n) {
  int64_t m = i % n;
  if (m < 0) m += n;
  return (int32_t)m;
}

/*
 * Row i of P^(k) has its single 1 in column recv_from[i] (the agent that sends to i);
 * send_to is the inverse map.
 * 2-port, Eq. (2p-gossip-matrix-d1/d0): Q_{i,j} = 1 iff i - j = n_r + delta_r (mod n).
 * 1-port, Eq. (1p-gossip-matrix): paper-odd i is matched with i + 2 n_r + 1,
 * paper-even i with i - 2 n_r - 1.
 */
int ceca_oracle_peers(int32_t n, int32_t variant, int64_t k, int32_t *recv_from, int32_t *send_to) {
  oracle_round_t rd;
  int rc = ceca_oracle_round(n, k, &rd);
  if (rc) return rc;
  if (variant != VARIANT_1P && variant != VARIANT_2P) return ORACLE_ERR_ARG;
  if (n == 1) {
    if (recv_from) recv_from[0] = 0;
    if (send_to) send_to[0] = 0;
    return ORACLE_OK;
  }
  if (variant == VARIANT_1P && (n % 2) != 0) return ORACLE_ERR_ODD_N_1P;
  for (int32_t i = 0; i < n; i++) {
    int32_t src;
    if (variant == VARIANT_2P) {
      src = wrap((int64_t)i - (rd.n_r + rd.delta), n);
    } else {
      int64_t off = 2 * (int64_t)rd.n_r + 1;
      int paper_index_is_odd = ((i + 1) % 2) == 1;
      src = paper_index_is_odd ? wrap(i + off, n) : wrap(i - off, n);
    }
    if (recv_from) recv_from[i] = src;
    if (send_to) send_to[src] = i;
  }
  return ORACLE_OK;
}

/*
 * One DSGD-CECA iteration, Eq. (x-iter-dsgd) and Eq. (y-iter-dsgd), out of place:
 *   u      = z - gamma e                  (the message every agent sends)
 *   x+_i   = a (x_i - gamma e_i) + (1-a) u_{src(i)}
 *   y+_i   = b (y_i - gamma e_i) + (1-b) u_{src(i)}
 * X, Y, E, X_out, Y_out are dense n x d row-major doubles.  E may be NULL (treated as 0,
 * which with any gamma gives the pure CECA round of Sec. 3.1 / Sec. 3.2).
 */
int ceca_oracle_step(const double *X, const double *Y, const double *E, double gamma,
                     int32_t n, int64_t d, int32_t variant, int64_t k,
                     double *X_out, double *Y_out) {
  if (!X || !Y || !X_out || !Y_out || d < 1) return ORACLE_ERR_ARG;
  oracle_round_t rd;
  int rc = ceca_oracle_round(n, k, &rd);
  if (rc) return rc;
  int32_t *src = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
  double *U = (double *)malloc(sizeof(double) * (size_t)n * (size_t)d);
  if (!src || !U) { free(src); free(U); return ORACLE_ERR_ARG; }
  rc = ceca_oracle_peers(n, variant, k, src, NULL);
  if (rc) { free(src); free(U); return rc; }
  const double *Z = rd.payload == 0 ? X : Y;
  const double a = rd.a, b = rd.b;
#pragma omp parallel for schedule(static)
  for (int32_t i = 0; i < n; i++)
    for (int64_t c = 0; c < d; c++) {
      double e = E ? E[(int64_t)i * d + c] : 0.0;
      U[(int64_t)i * d + c] = Z[(int64_t)i * d + c] - gamma * e;
    }
#pragma omp parallel for schedule(static)
  for (int32_t i = 0; i < n; i++)
    for (int64_t c = 0; c < d; c++) {
      double e = E ? E[(int64_t)i * d + c] : 0.0;
      double recv = U[(int64_t)src[i] * d + c];
      X_out[(int64_t)i * d + c] = a * (X[(int64_t)i * d + c] - gamma * e) + (1.0 - a) * recv;
      Y_out[(int64_t)i * d + c] = b * (Y[(int64_t)i * d + c] - gamma * e) + (1.0 - b) * recv;
    }
  free(src); free(U);
  return ORACLE_OK;
}

/*
 * `rounds` consecutive CECA rounds k0, k0+1, ... applied to (I, J) = (X, Y):
 * Sec. 3.1 "Main recursions" / Algorithm 2 (2-port), Sec. 3.2 (1-port).
 * In place on X and Y.
 */
int ceca_oracle_consensus(double *X, double *Y, int32_t n, int64_t d, int32_t variant,
                          int64_t k0, int32_t rounds) {
  if (rounds < 0) return ORACLE_ERR_ARG;
  size_t bytes = sizeof(double) * (size_t)n * (size_t)d;
  double *Xn = (double *)malloc(bytes), *Yn = (double *)malloc(bytes);
  if (!Xn || !Yn) { free(Xn); free(Yn); return ORACLE_ERR_ARG; }
  int rc = ORACLE_OK;
  for (int32_t t = 0; t < rounds && rc == ORACLE_OK; t++) {
    rc = ceca_oracle_step(X, Y, NULL, 0.0, n, d, variant, k0 + t, Xn, Yn);
    if (rc == ORACLE_OK) { memcpy(X, Xn, bytes); memcpy(Y, Yn, bytes); }
  }
  free(Xn); free(Yn);
  return rc;
}

/*
 * Per-agent logistic-regression gradient (workload definition, not from the paper):
 *   f_i(w)      = (1/m) sum_s log(1 + exp(-l_s <a_s, w>)),   l_s in {-1,+1}
 *   grad f_i(w) = -(1/m) sum_s l_s sigma(-l_s <a_s, w>) a_s,  sigma(t) = 1/(1+exp(-t))
 * evaluated at w = z_i, the model Algorithm 1 selects in iteration k (x if delta_r=1, else y).
 * A is n x m x d, labels n x m, X, Y, G are n x d; all dense row-major doubles.
 */
int ceca_oracle_logreg_grad(const double *A, const double *labels, const double *X, const double *Y,
                            int64_t k, double *G, int32_t n, int32_t m, int64_t d) {
  if (!A || !labels || !X || !Y || !G || m < 1 || d < 1) return ORACLE_ERR_ARG;
  oracle_round_t rd;
  int rc = ceca_oracle_round(n, k, &rd);
  if (rc) return rc;
  const double *Z = rd.payload == 0 ? X : Y;
#pragma omp parallel for schedule(static)
  for (int32_t i = 0; i < n; i++) {
    const double *w = Z + (int64_t)i * d;
    double *g = G + (int64_t)i * d;
    for (int64_t c = 0; c < d; c++) g[c] = 0.0;
    for (int32_t s = 0; s < m; s++) {
      const double *a_s = A + ((int64_t)i * m + s) * d;
      double l = labels[(int64_t)i * m + s];
      double t = 0.0;
      for (int64_t c = 0; c < d; c++) t += a_s[c] * w[c];
      double sig = 1.0 / (1.0 + exp(l * t));      /* sigma(-l t) */
      double coef = -l * sig / (double)m;
      for (int64_t c = 0; c < d; c++) g[c] += coef * a_s[c];
    }
  }
  return ORACLE_OK;
}

/* The loss whose gradient the routine above states; used by the finite-difference pin. */
int ceca_oracle_logreg_loss(const double *A, const double *labels, const double *W,
                            double *loss, int32_t n, int32_t m, int64_t d) {
  if (!A || !labels || !W || !loss || n < 1 || m < 1 || d < 1) return ORACLE_ERR_ARG;
  for (int32_t i = 0; i < n; i++) {
    double acc = 0.0;
    for (int32_t s = 0; s < m; s++) {
      const double *a_s = A + ((int64_t)i * m + s) * d;
      double t = 0.0;
      for (int64_t c = 0; c < d; c++) t += a_s[c] * W[(int64_t)i * d + c];
      double v = -labels[(int64_t)i * m + s] * t;
      /* log(1 + exp(v)) without overflow */
      acc += v > 0 ? v + log1p(exp(-v)) : log1p(exp(v));
    }
    loss[i] = acc / (double)m;
  }
  return ORACLE_OK;
}

/*
 * Per-agent least-squares gradient, Sec. 5 "DSGD: least-squares problem":
 *   f_i(w) = (1/2) ||A_i w - b_i||^2,   stochastic gradient = A_i^T (A_i w - b_i) + eps_i,
 * evaluated at w = z_i, the model Algorithm 1 selects in iteration k.  The noise eps (n x d, may be
 * NULL) is an input: the caller draws it.  A is n x m x d, B is n x m.
 */
int ceca_oracle_lsq_grad(const double *A, const double *B, const double *X, const double *Y,
                         const double *noise, int64_t k, double *G, int32_t n, int32_t m, int64_t d) {
  if (!A || !B || !X || !Y || !G || m < 1 || d < 1) return ORACLE_ERR_ARG;
  oracle_round_t rd;
  int rc = ceca_oracle_round(n, k, &rd);
  if (rc) return rc;
  const double *Z = rd.payload == 0 ? X : Y;
#pragma omp parallel for schedule(static)
  for (int32_t i = 0; i < n; i++) {
    const double *w = Z + (int64_t)i * d;
    double *g = G + (int64_t)i * d;
    for (int64_t c = 0; c < d; c++) g[c] = noise ? noise[(int64_t)i * d + c] : 0.0;
    for (int32_t s = 0; s < m; s++) {
      const double *a_s = A + ((int64_t)i * m + s) * d;
      double resid = -B[(int64_t)i * m + s];
      for (int64_t c = 0; c < d; c++) resid += a_s[c] * w[c];
      for (int64_t c = 0; c < d; c++) g[c] += resid * a_s[c];
    }
  }
  return ORACLE_OK;
}

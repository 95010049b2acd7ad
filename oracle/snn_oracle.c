/*
 * CPU oracle for BPTT training of sparse recurrent / spiking networks.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * training step computes: full-storage back-propagation through time (every
 * membrane state of every step kept, no checkpointing, no event lists, dense
 * loops that skip zero activations).  It shares no code with the CUDA library
 * and must never be linked, imported or called by it.
 *
 * What it follows.  The paper (Methods, "BPTT based SNN training") states that
 * the networks are trained by BPTT with a surrogate gradient for the spike
 * discontinuity, and (Methods, "Standard Checkpointing") that a forward step
 * is two operations: a matrix product driven by the sparse spikes that yields
 * the next state, then spike generation from that state.  The paper prints no
 * neuron equations; the ones below are the reading this repository fixes:
 *
 *   forward, t = 1..T, l = 1..L, every sample b, neuron i (V_0 = 0, S_0 = 0):
 *     I      = sum_{j asc} S^{l-1}_t[b,j] W_ff^l[j,i]   (feed-forward, same step)
 *            + sum_{j asc} S^l_{t-1}[b,j] W_rec^l[j,i]  (recurrent, one-step delay)
 *     V^l_t  = fma(alpha, V^l_{t-1}, I) - theta S^l_{t-1}[b,i]     (LIF cell)
 *     V^l_t  = fma(alpha, V^l_{t-1}, I)                             (graded cell)
 *     S^l_t  = [V^l_t > theta]             (LIF)   |  V^l_t [V^l_t > theta]  (graded)
 *   readout: c = sum_t S^L_t ; logits = scale c W_out ; mean soft-max cross-entropy
 *   backward, t = T..1, l = L..1 (delta_{T+1} = 0):
 *     g_S      = [l=L] g_out + delta^{l+1}_t W_ff^{l+1 T} + delta^l_{t+1} W_rec^{l T}
 *                - theta delta^l_{t+1}                       (last term: LIF only)
 *     delta^l_t = g_S sigma'(V^l_t - theta) + alpha delta^l_{t+1}
 *     dW_ff^l  += S^{l-1 T}_t delta^l_t ;  dW_rec^l += S^{l T}_{t-1} delta^l_t
 *
 * Canonical forward arithmetic.  Spike trains are compared bit for bit, so the
 * forward pass keeps ONE accumulator per (b,i), adds feed-forward terms first,
 * then recurrent terms, each in ascending presynaptic index, every term as one
 * fused multiply-add (for a binary spike that is an exact plain add), followed
 * by one fused multiply-add for the leak and one subtraction for the reset.
 * Compile with -ffp-contract=off so nothing else is fused.
 *
 * Precision.  The file is compiled twice: REAL=float (forward in fp32 in the
 * canonical order; backward reductions in double) and REAL=double (everything
 * in double, used with the optional smooth-spike mode for finite-difference
 * checks of the backward pass).
 *
 * Parity pins (tests/ -m "not gpu"): closed-form leaky integration trace,
 * first-spike time, soft-max regression special case, finite differences in
 * smooth mode and for the graded cell, brute-force dense re-derivation on
 * tiny nets, dW sparsity identities.  The surrogate slope beta, the readout
 * scale and the weight gains are conventions: parity unpinned beyond "both
 * sides are given the same number".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifndef REAL
#define REAL float
#endif
#ifndef PFX
#define PFX f32
#endif
#define CAT_(a, b) a##_##b
#define CAT(a, b) CAT_(a, b)
#define FN(name) CAT(CAT(oracle, PFX), name)

typedef REAL real;

#define CELL_LIF 0
#define CELL_GRADED 1
#define SURR_FAST_SIGMOID 0
#define SURR_SIGMOID 1
#define SURR_TRIANGLE 2   /* compact support; not in the paper (see surrogate_grad) */

typedef struct {
  int32_t L;        /* number of hidden (recurrent) layers                 */
  int32_t cell;     /* CELL_LIF | CELL_GRADED                               */
  int32_t surrogate;/* SURR_FAST_SIGMOID | SURR_SIGMOID | SURR_TRIANGLE     */
  int32_t smooth;   /* 1: S = sigmoid(beta (V - theta)) in the forward too  */
  double alpha;     /* leak per step; cast to REAL before use               */
  double theta;     /* threshold                                            */
  double beta;      /* surrogate slope                                      */
  double scale;     /* readout scale                                        */
} oracle_params;

static inline real fma_real(real a, real b, real c) {
  return sizeof(real) == sizeof(float) ? (real)fmaf((float)a, (float)b, (float)c)
                                       : (real)fma((double)a, (double)b, (double)c);
}

static inline double sigmoid_d(double x) {
  if (x >= 0) { double e = exp(-x); return 1.0 / (1.0 + e); }
  double e = exp(x); return e / (1.0 + e);
}

/* sigma'(x), x = V - theta.  Graded cell: derivative of V [V > theta] away from
 * the jump.  Smooth mode: exact derivative of the sigmoid used in the forward. */
static inline double surrogate_grad(const oracle_params* p, double x) {
  if (p->cell == CELL_GRADED) return x > 0 ? 1.0 : 0.0;
  if (p->smooth || p->surrogate == SURR_SIGMOID) {
    double s = sigmoid_d(p->beta * x);
    return p->beta * s * (1.0 - s);
  }
  if (p->surrogate == SURR_TRIANGLE) {
    /* An extension beyond the paper, which names no surrogate: the triangular pseudo-derivative
     * beta * max(0, 1 - beta |x|), zero outside |x| < 1/beta, unit area.  With it only neurons near
     * the threshold carry gradient, which is what an event-driven backward pass would exploit. */
    double u = 1.0 - p->beta * fabs(x);
    return u > 0.0 ? p->beta * u : 0.0;
  }
  double d = 1.0 + p->beta * fabs(x);
  return 1.0 / (d * d);
}

/* One forward step of one hidden layer (the paper's "MatMul" + "Spike Generation").
 *   S_below [B][N_pre]  activations of layer l-1 at step t   (0/1, or graded values)
 *   S_prev  [B][N]      activations of this layer at step t-1
 *   V_prev  [B][N]      membrane at step t-1
 *   W_ff    [N_pre][N], W_rec [N][N]   row-major by presynaptic neuron
 *   V_out, S_out [B][N] */
void FN(forward_step)(const oracle_params* p, int32_t B, int32_t N_pre, int32_t N,
                      const real* S_below, const real* S_prev, const real* V_prev,
                      const real* W_ff, const real* W_rec, real* V_out, real* S_out) {
  const real alpha = (real)p->alpha, theta = (real)p->theta;
#pragma omp parallel for schedule(static)
  for (int32_t b = 0; b < B; ++b) {
    real* acc = (real*)malloc(sizeof(real) * (size_t)N);
    for (int32_t i = 0; i < N; ++i) acc[i] = 0;
    for (int32_t j = 0; j < N_pre; ++j) {
      const real s = S_below[(size_t)b * N_pre + j];
      if (s == 0) continue;
      const real* w = W_ff + (size_t)j * N;
      for (int32_t i = 0; i < N; ++i) acc[i] = fma_real(s, w[i], acc[i]);
    }
    for (int32_t j = 0; j < N; ++j) {
      const real s = S_prev[(size_t)b * N + j];
      if (s == 0) continue;
      const real* w = W_rec + (size_t)j * N;
      for (int32_t i = 0; i < N; ++i) acc[i] = fma_real(s, w[i], acc[i]);
    }
    for (int32_t i = 0; i < N; ++i) {
      const size_t k = (size_t)b * N + i;
      real v = fma_real(alpha, V_prev[k], acc[i]);
      if (p->cell == CELL_LIF) v = v - theta * S_prev[k];
      V_out[k] = v;
      real s;
      if (p->smooth) s = (real)sigmoid_d(p->beta * ((double)v - p->theta));
      else if (p->cell == CELL_LIF) s = v > theta ? (real)1 : (real)0;
      else s = v > theta ? v : (real)0;
      S_out[k] = s;
    }
    free(acc);
  }
}

/* Readout, loss and the gradient entering the last hidden layer.
 *   c [B][N_L] time-summed activations; targets [B]; W_out [N_L][N_out]
 *   logits [B][N_out], dlogits [B][N_out], g_out [B][N_L], dW_out [N_L][N_out]: double
 *   returns the mean cross-entropy. */
double FN(readout)(const oracle_params* p, int32_t B, int32_t N_L, int32_t N_out,
                   const real* c, const int32_t* targets, const real* W_out,
                   double* logits, double* dlogits, double* g_out, double* dW_out) {
  double loss = 0;
  for (int32_t b = 0; b < B; ++b) {
    double* z = logits + (size_t)b * N_out;
    for (int32_t k = 0; k < N_out; ++k) z[k] = 0;
    for (int32_t i = 0; i < N_L; ++i) {
      const double ci = (double)c[(size_t)b * N_L + i];
      if (ci == 0) continue;
      for (int32_t k = 0; k < N_out; ++k) z[k] += ci * (double)W_out[(size_t)i * N_out + k];
    }
    double m = -INFINITY;
    for (int32_t k = 0; k < N_out; ++k) { z[k] *= p->scale; if (z[k] > m) m = z[k]; }
    double se = 0;
    for (int32_t k = 0; k < N_out; ++k) se += exp(z[k] - m);
    const double lse = m + log(se);
    loss += lse - z[targets[b]];
    for (int32_t k = 0; k < N_out; ++k) {
      double sm = exp(z[k] - lse);
      dlogits[(size_t)b * N_out + k] = (sm - (k == targets[b] ? 1.0 : 0.0)) / (double)B;
    }
  }
  loss /= (double)B;
  for (int32_t b = 0; b < B; ++b)
    for (int32_t i = 0; i < N_L; ++i) {
      double g = 0;
      for (int32_t k = 0; k < N_out; ++k)
        g += (double)W_out[(size_t)i * N_out + k] * dlogits[(size_t)b * N_out + k];
      g_out[(size_t)b * N_L + i] = p->scale * g;
    }
  for (int32_t i = 0; i < N_L; ++i)
    for (int32_t k = 0; k < N_out; ++k) {
      double g = 0;
      for (int32_t b = 0; b < B; ++b)
        g += (double)c[(size_t)b * N_L + i] * dlogits[(size_t)b * N_out + k];
      dW_out[(size_t)i * N_out + k] = p->scale * g;
    }
  return loss;
}

/* One backward step of one hidden layer.
 *   V_t [B][N] membrane of this layer at step t (REAL)
 *   S_below_t [B][N_pre] activations of layer l-1 at step t; S_prev [B][N] own at t-1
 *   delta_next [B][N] delta^l_{t+1}; delta_above [B][N_post] delta^{l+1}_t or NULL
 *   g_out [B][N] or NULL (last hidden layer only)
 *   W_ff_above [N][N_post] or NULL; W_rec [N][N]
 *   delta_out [B][N]; dW_ff [N_pre][N], dW_rec [N][N] accumulated (double) */
void FN(backward_step)(const oracle_params* p, int32_t B, int32_t N_pre, int32_t N, int32_t N_post,
                       const real* V_t, const real* S_below_t, const real* S_prev,
                       const double* delta_next, const double* delta_above, const double* g_out,
                       const real* W_ff_above, const real* W_rec,
                       double* delta_out, double* dW_ff, double* dW_rec) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int32_t b = 0; b < B; ++b)
    for (int32_t i = 0; i < N; ++i) {
      const size_t k = (size_t)b * N + i;
      double g = g_out ? g_out[k] : 0.0;
      if (delta_above) {
        const real* w = W_ff_above + (size_t)i * N_post;
        const double* d = delta_above + (size_t)b * N_post;
        double s = 0;
        for (int32_t q = 0; q < N_post; ++q) s += (double)w[q] * d[q];
        g += s;
      }
      {
        const real* w = W_rec + (size_t)i * N;
        const double* d = delta_next + (size_t)b * N;
        double s = 0;
        for (int32_t q = 0; q < N; ++q) s += (double)w[q] * d[q];
        g += s;
      }
      if (p->cell == CELL_LIF) g -= p->theta * delta_next[k];
      const double sp = surrogate_grad(p, (double)V_t[k] - p->theta);
      delta_out[k] = g * sp + p->alpha * delta_next[k];
    }
  /* weight gradients: rows of presynaptic neurons that were active */
#pragma omp parallel for schedule(dynamic, 8)
  for (int32_t j = 0; j < N_pre; ++j)
    for (int32_t b = 0; b < B; ++b) {
      const double s = (double)S_below_t[(size_t)b * N_pre + j];
      if (s == 0) continue;
      double* g = dW_ff + (size_t)j * N;
      const double* d = delta_out + (size_t)b * N;
      for (int32_t i = 0; i < N; ++i) g[i] += s * d[i];
    }
#pragma omp parallel for schedule(dynamic, 8)
  for (int32_t j = 0; j < N; ++j)
    for (int32_t b = 0; b < B; ++b) {
      const double s = (double)S_prev[(size_t)b * N + j];
      if (s == 0) continue;
      double* g = dW_rec + (size_t)j * N;
      const double* d = delta_out + (size_t)b * N;
      for (int32_t i = 0; i < N; ++i) g[i] += s * d[i];
    }
}

/* Full-storage BPTT of the whole network: the definition every checkpointing
 * strategy must reproduce.
 *   sizes [L+2] = N_0, N_1..N_L, N_out
 *   input   [T][B][N_0]  REAL (0/1 spikes, or graded input values)
 *   targets [B]
 *   W_ff[l] (l=0..L-1) [N_l][N_{l+1}], W_rec[l] [N_{l+1}][N_{l+1}], W_out [N_L][N_out]
 * outputs (any may be NULL):
 *   V_all[l] [T+1][B][N_{l+1}] REAL, S_all[l] [T+1][B][N_{l+1}] REAL (index 0 = initial zeros)
 *   delta_all[l] [T+2][B][N_{l+1}] double (index t; T+1 = zeros; 0 unused)
 *   dW_ff[l], dW_rec[l], dW_out double; logits [B][N_out] double; counts [B][N_L] REAL
 * returns the loss.  When do_backward == 0 only the forward and the loss are computed. */
double FN(bptt_full)(const oracle_params* p, const int32_t* sizes, int32_t T, int32_t B,
                     const real* input, const int32_t* targets,
                     const real* const* W_ff, const real* const* W_rec, const real* W_out,
                     real* const* V_all, real* const* S_all, double* const* delta_all,
                     double* const* dW_ff, double* const* dW_rec, double* dW_out,
                     double* logits_out, real* counts_out, int32_t do_backward) {
  const int32_t L = p->L;
  const int32_t N_L = sizes[L], N_out = sizes[L + 1];
  real** V = (real**)calloc((size_t)L, sizeof(real*));
  real** S = (real**)calloc((size_t)L, sizeof(real*));
  for (int32_t l = 0; l < L; ++l) {
    const size_t n = (size_t)(T + 1) * B * sizes[l + 1];
    V[l] = V_all && V_all[l] ? V_all[l] : (real*)malloc(n * sizeof(real));
    S[l] = S_all && S_all[l] ? S_all[l] : (real*)malloc(n * sizeof(real));
    memset(V[l], 0, (size_t)B * sizes[l + 1] * sizeof(real));
    memset(S[l], 0, (size_t)B * sizes[l + 1] * sizeof(real));
  }
  real* c = (real*)calloc((size_t)B * N_L, sizeof(real));
  for (int32_t t = 1; t <= T; ++t) {
    for (int32_t l = 0; l < L; ++l) {
      const int32_t N_pre = sizes[l], N = sizes[l + 1];
      const size_t st = (size_t)B * N;
      const real* below = l == 0 ? input + (size_t)(t - 1) * B * N_pre
                                 : S[l - 1] + (size_t)t * B * N_pre;
      FN(forward_step)(p, B, N_pre, N, below, S[l] + (size_t)(t - 1) * st, V[l] + (size_t)(t - 1) * st,
                       W_ff[l], W_rec[l], V[l] + (size_t)t * st, S[l] + (size_t)t * st);
    }
    const real* sl = S[L - 1] + (size_t)t * B * N_L;
    for (size_t k = 0; k < (size_t)B * N_L; ++k) c[k] = c[k] + sl[k];
  }
  double* logits = (double*)malloc(sizeof(double) * (size_t)B * N_out);
  double* dlogits = (double*)malloc(sizeof(double) * (size_t)B * N_out);
  double* g_out = (double*)malloc(sizeof(double) * (size_t)B * N_L);
  double* dWo = dW_out ? dW_out : (double*)malloc(sizeof(double) * (size_t)N_L * N_out);
  const double loss = FN(readout)(p, B, N_L, N_out, c, targets, W_out, logits, dlogits, g_out, dWo);
  if (logits_out) memcpy(logits_out, logits, sizeof(double) * (size_t)B * N_out);
  if (counts_out) memcpy(counts_out, c, sizeof(real) * (size_t)B * N_L);
  if (do_backward) {
    /* delta[l]: two rolling buffers unless the caller wants every step */
    double** dcur = (double**)calloc((size_t)L, sizeof(double*));
    double** dnext = (double**)calloc((size_t)L, sizeof(double*));
    for (int32_t l = 0; l < L; ++l) {
      const size_t st = (size_t)B * sizes[l + 1];
      memset(dW_ff[l], 0, sizeof(double) * (size_t)sizes[l] * sizes[l + 1]);
      memset(dW_rec[l], 0, sizeof(double) * (size_t)sizes[l + 1] * sizes[l + 1]);
      if (delta_all && delta_all[l]) {
        memset(delta_all[l], 0, sizeof(double) * (size_t)(T + 2) * st);
      } else {
        dcur[l] = (double*)calloc(st, sizeof(double));
        dnext[l] = (double*)calloc(st, sizeof(double));
      }
    }
    for (int32_t t = T; t >= 1; --t) {
      for (int32_t l = L - 1; l >= 0; --l) {
        const int32_t N_pre = sizes[l], N = sizes[l + 1], N_post = sizes[l + 2];
        const size_t st = (size_t)B * N;
        const int keep = delta_all && delta_all[l];
        double* d_out = keep ? delta_all[l] + (size_t)t * st : dcur[l];
        const double* d_next = keep ? delta_all[l] + (size_t)(t + 1) * st : dnext[l];
        const double* d_above = NULL;
        if (l < L - 1) {
          const int keep_a = delta_all && delta_all[l + 1];
          d_above = keep_a ? delta_all[l + 1] + (size_t)t * B * N_post : dcur[l + 1];
        }
        const real* below = l == 0 ? input + (size_t)(t - 1) * B * N_pre
                                   : S[l - 1] + (size_t)t * B * N_pre;
        FN(backward_step)(p, B, N_pre, N, N_post, V[l] + (size_t)t * st, below,
                          S[l] + (size_t)(t - 1) * st, d_next, d_above,
                          l == L - 1 ? g_out : NULL, l < L - 1 ? W_ff[l + 1] : NULL, W_rec[l],
                          d_out, dW_ff[l], dW_rec[l]);
      }
      for (int32_t l = 0; l < L; ++l)
        if (!(delta_all && delta_all[l])) { double* tmp = dnext[l]; dnext[l] = dcur[l]; dcur[l] = tmp; }
    }
    for (int32_t l = 0; l < L; ++l) { free(dcur[l]); free(dnext[l]); }
    free(dcur); free(dnext);
  }
  for (int32_t l = 0; l < L; ++l) {
    if (!(V_all && V_all[l])) free(V[l]);
    if (!(S_all && S_all[l])) free(S[l]);
  }
  free(V); free(S); free(c); free(logits); free(dlogits); free(g_out);
  if (!dW_out) free(dWo);
  return loss;
}

/* Brute-force spike compaction: the ascending list of indices i with v[i] > theta
 * (the paper's "Spike Generation" output in its sparse representation).
 * Returns the count; idx must have room for n entries. */
int32_t FN(compact)(const real* v, int32_t n, double theta, int32_t* idx) {
  int32_t c = 0;
  const real th = (real)theta;
  for (int32_t i = 0; i < n; ++i)
    if (v[i] > th) idx[c++] = i;
  return c;
}

/*
 * M2RNN scan oracle (fp64, one thread, no blocking, no fusion).
 * TEST INFRASTRUCTURE ONLY -- see m2rnn_ref.h.  Each function cites the passage
 * of the paper it writes out.
 */
#include "m2rnn_ref.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* Forget gate.  VALUE: the tensor is f itself (Algorithm 1 takes F in [0,1]).
 * LOGIT: f = sigmoid(x), i.e. the forget-gate equation with alpha=1, beta=0 and
 * the input reflected.  PSI: the forget-gate equation f = (1+e^{x+beta})^{-alpha},
 * evaluated as exp(-alpha*softplus(x+beta)) so that large |x| neither overflows
 * nor loses f to rounding; df/dx = -alpha * sigmoid(x+beta) * f. */
double m2rnn_ref_gate(int gate_kind, double x, double alpha, double beta, double *dfdx) {
  double f, d;
  if (gate_kind == M2RNN_REF_GATE_VALUE) {
    f = x;
    d = 1.0;
  } else if (gate_kind == M2RNN_REF_GATE_LOGIT) {
    if (x >= 0.0) {
      f = 1.0 / (1.0 + exp(-x));
    } else {
      double e = exp(x);
      f = e / (1.0 + e);
    }
    d = f * (1.0 - f);
  } else {
    double u = x + beta;
    double softplus = (u > 0.0) ? u + log1p(exp(-u)) : log1p(exp(u));
    double sig = (u >= 0.0) ? 1.0 / (1.0 + exp(-u)) : exp(u) / (1.0 + exp(u));
    f = exp(-alpha * softplus);
    d = -alpha * sig * f;
  }
  if (dfdx) *dfdx = d;
  return f;
}

static int bad_params(const m2rnn_ref_params *p) {
  if (!p) return 1;
  if (p->B < 0 || p->T < 0 || p->N <= 0 || p->K <= 0 || p->V <= 0) return 1;
  if (p->Nq <= 0 || p->Nk <= 0 || p->N % p->Nq || p->N % p->Nk) return 1;
  if (p->gate_kind < 0 || p->gate_kind > 2) return 1;
  return 0;
}

/* One application of Eq. 1-3 to one (b,n) state.
 *   H     [K,V] in: H_{t-1}, out: H_t
 *   Zout  [K,V] optional: receives Z_t
 *   y     [V]   optional */
static void step(int K, int V, double *H, const double *W, const double *q, const double *k,
                 const double *v, double f, const double *w_r, double *Zout, double *y,
                 double *Znew /* scratch [K,V] */) {
  /* Eq. 1: Z = tanh(H W + k v^T) */
  for (int i = 0; i < K; ++i)
    for (int j = 0; j < V; ++j) {
      double s = 0.0;
      for (int l = 0; l < V; ++l) s += H[i * V + l] * W[l * V + j];
      Znew[i * V + j] = tanh(s + k[i] * v[j]);
    }
  /* Eq. 2: H = f H + (1-f) Z */
  for (int i = 0; i < K * V; ++i) H[i] = f * H[i] + (1.0 - f) * Znew[i];
  if (Zout) memcpy(Zout, Znew, sizeof(double) * (size_t)K * V);
  /* Eq. 3 / Algorithm 1 readout from the post-update state: y = H^T q (+ w_r (.) v) */
  if (y)
    for (int j = 0; j < V; ++j) {
      double s = 0.0;
      for (int i = 0; i < K; ++i) s += H[i * V + j] * q[i];
      if (w_r) s += w_r[j] * v[j];
      y[j] = s;
    }
}

/* Algorithm 1: for every (b,n), start from H_0 (zero when absent), loop t. */
int m2rnn_ref_fwd(const m2rnn_ref_params *p, const double *q, const double *k, const double *v,
                  const double *gate, const double *W, const double *h0, const double *alpha,
                  const double *beta, const double *w_r, double *y, double *hT, double *H_all) {
  if (bad_params(p)) return -2;
  const int B = p->B, T = p->T, N = p->N, K = p->K, V = p->V;
  const int gq = N / p->Nq, gk = N / p->Nk;
  const size_t KV = (size_t)K * V;
  double *H = (double *)malloc(sizeof(double) * KV);
  double *Zs = (double *)malloc(sizeof(double) * KV);
  if (!H || !Zs) { free(H); free(Zs); return -6; }
  for (int b = 0; b < B; ++b)
    for (int n = 0; n < N; ++n) {
      const size_t bn = (size_t)b * N + n;
      if (h0) memcpy(H, h0 + bn * KV, sizeof(double) * KV);
      else memset(H, 0, sizeof(double) * KV);
      if (H_all) memcpy(H_all + bn * (size_t)(T + 1) * KV, H, sizeof(double) * KV);
      for (int t = 0; t < T; ++t) {
        const size_t bt = (size_t)b * T + t;
        const double *qt = q + (bt * p->Nq + n / gq) * K;
        const double *kt = k + (bt * p->Nk + n / gk) * K;
        const double *vt = v + (bt * N + n) * V;
        double f = m2rnn_ref_gate(p->gate_kind, gate[bt * N + n], alpha ? alpha[n] : 1.0,
                                  beta ? beta[n] : 0.0, NULL);
        step(K, V, H, W + (size_t)n * V * V, qt, kt, vt, f, w_r ? w_r + (size_t)n * V : NULL,
             NULL, y ? y + (bt * N + n) * V : NULL, Zs);
        if (H_all) memcpy(H_all + (bn * (size_t)(T + 1) + t + 1) * KV, H, sizeof(double) * KV);
      }
      if (hT) memcpy(hT + bn * KV, H, sizeof(double) * KV);
    }
  free(H);
  free(Zs);
  return 0;
}

/* One step on a cached state: Eq. 1-3 once (the recurrent / decoding form). */
int m2rnn_ref_decode_step(const m2rnn_ref_params *p, const double *q, const double *k,
                          const double *v, const double *gate, const double *W,
                          const double *alpha, const double *beta, const double *w_r,
                          double *state, double *y) {
  if (bad_params(p)) return -2;
  const int B = p->B, N = p->N, K = p->K, V = p->V;
  const int gq = N / p->Nq, gk = N / p->Nk;
  const size_t KV = (size_t)K * V;
  double *Zs = (double *)malloc(sizeof(double) * KV);
  if (!Zs) return -6;
  for (int b = 0; b < B; ++b)
    for (int n = 0; n < N; ++n) {
      const size_t bn = (size_t)b * N + n;
      double f = m2rnn_ref_gate(p->gate_kind, gate[bn], alpha ? alpha[n] : 1.0,
                                beta ? beta[n] : 0.0, NULL);
      step(K, V, state + bn * KV, W + (size_t)n * V * V, q + ((size_t)b * p->Nq + n / gq) * K,
           k + ((size_t)b * p->Nk + n / gk) * K, v + bn * V, f,
           w_r ? w_r + (size_t)n * V : NULL, NULL, y ? y + bn * V : NULL, Zs);
    }
  free(Zs);
  return 0;
}

/* Algorithm 2 written as exact back-propagation through Eq. 1-3.
 *
 * Pass 1 keeps every H_t (the algorithm's H_full).  Pass 2 runs t = T-1 .. 0
 * with C = dL/dH_t carried from the later steps (C starts as d_hT, or 0):
 *     G   = C + q_t dy_t^T                 total gradient reaching H_t; Algorithm 2's r is
 *                                          q dy^T alone, which is only right at the last
 *                                          step -- every use of r below takes G
 *     dq  = H_t dy_t                                        (Algorithm 2, query-gradient line)
 *     df  = sum( G (.) (H_{t-1} - Z_t) )                    (Algorithm 2, gate-gradient line)
 *     dZ  = (1-f) G ;  dX = dZ (.) (1 - Z (.) Z)            (Algorithm 2, candidate and
 *                                                            pre-activation gradient lines)
 *     C   = f G + dX W^T          both paths into H_{t-1}: the gated residual (Algorithm 2's
 *                                 first state-gradient line) plus the path through the
 *                                 transition (its second one, which as printed multiplies
 *                                 the two where the chain rule adds them)
 *     dW += H_{t-1}^T dX ;  dk = dX v ;  dv = dX^T k (+ w_r (.) dy from Eq. 3)
 * dq/dk add over the heads sharing them, dW over batch (the algorithm's atomic adds).
 * dh0 = C after the last reverse step. */
int m2rnn_ref_bwd(const m2rnn_ref_params *p, const double *q, const double *k, const double *v,
                  const double *gate, const double *W, const double *h0, const double *alpha,
                  const double *beta, const double *w_r, const double *dy, const double *d_hT,
                  double *dq, double *dk, double *dv, double *dgate, double *dW, double *dh0) {
  if (bad_params(p)) return -2;
  const int B = p->B, T = p->T, N = p->N, K = p->K, V = p->V;
  const int gq = N / p->Nq, gk = N / p->Nk;
  const size_t KV = (size_t)K * V;
  double *Hs = (double *)malloc(sizeof(double) * KV * (size_t)(T + 1));
  double *Z = (double *)malloc(sizeof(double) * KV);
  double *G = (double *)malloc(sizeof(double) * KV);
  double *dX = (double *)malloc(sizeof(double) * KV);
  double *C = (double *)malloc(sizeof(double) * KV);
  if (!Hs || !Z || !G || !dX || !C) { free(Hs); free(Z); free(G); free(dX); free(C); return -6; }
  if (dq) memset(dq, 0, sizeof(double) * (size_t)B * T * p->Nq * K);
  if (dk) memset(dk, 0, sizeof(double) * (size_t)B * T * p->Nk * K);
  if (dW) memset(dW, 0, sizeof(double) * (size_t)N * V * V);

  for (int b = 0; b < B; ++b)
    for (int n = 0; n < N; ++n) {
      const size_t bn = (size_t)b * N + n;
      const double *Wn = W + (size_t)n * V * V;
      const double a_n = alpha ? alpha[n] : 1.0, b_n = beta ? beta[n] : 0.0;
      /* pass 1: H_0 .. H_T */
      if (h0) memcpy(Hs, h0 + bn * KV, sizeof(double) * KV);
      else memset(Hs, 0, sizeof(double) * KV);
      for (int t = 0; t < T; ++t) {
        const size_t bt = (size_t)b * T + t;
        double f = m2rnn_ref_gate(p->gate_kind, gate[bt * N + n], a_n, b_n, NULL);
        memcpy(Hs + (size_t)(t + 1) * KV, Hs + (size_t)t * KV, sizeof(double) * KV);
        step(K, V, Hs + (size_t)(t + 1) * KV, Wn, NULL, k + (bt * p->Nk + n / gk) * K,
             v + (bt * N + n) * V, f, NULL, NULL, NULL, Z);
      }
      /* pass 2 */
      if (d_hT) memcpy(C, d_hT + bn * KV, sizeof(double) * KV);
      else memset(C, 0, sizeof(double) * KV);
      for (int t = T - 1; t >= 0; --t) {
        const size_t bt = (size_t)b * T + t;
        const double *qt = q + (bt * p->Nq + n / gq) * K;
        const double *kt = k + (bt * p->Nk + n / gk) * K;
        const double *vt = v + (bt * N + n) * V;
        const double *dyt = dy + (bt * N + n) * V;
        const double *Hprev = Hs + (size_t)t * KV, *Hcur = Hs + (size_t)(t + 1) * KV;
        double dfdx;
        double f = m2rnn_ref_gate(p->gate_kind, gate[bt * N + n], a_n, b_n, &dfdx);
        /* recompute Z_t */
        for (int i = 0; i < K; ++i)
          for (int j = 0; j < V; ++j) {
            double s = 0.0;
            for (int l = 0; l < V; ++l) s += Hprev[i * V + l] * Wn[l * V + j];
            Z[i * V + j] = tanh(s + kt[i] * vt[j]);
          }
        for (int i = 0; i < K; ++i)
          for (int j = 0; j < V; ++j) G[i * V + j] = C[i * V + j] + qt[i] * dyt[j];
        if (dq)
          for (int i = 0; i < K; ++i) {
            double s = 0.0;
            for (int j = 0; j < V; ++j) s += Hcur[i * V + j] * dyt[j];
            dq[(bt * p->Nq + n / gq) * K + i] += s;
          }
        double df = 0.0;
        for (size_t e = 0; e < KV; ++e) df += G[e] * (Hprev[e] - Z[e]);
        if (dgate) dgate[bt * N + n] = df * dfdx;
        for (size_t e = 0; e < KV; ++e) dX[e] = (1.0 - f) * G[e] * (1.0 - Z[e] * Z[e]);
        for (int i = 0; i < K; ++i)
          for (int l = 0; l < V; ++l) {
            double s = 0.0;
            for (int j = 0; j < V; ++j) s += dX[i * V + j] * Wn[l * V + j];
            C[i * V + l] = f * G[i * V + l] + s;
          }
        if (dW)
          for (int l = 0; l < V; ++l)
            for (int j = 0; j < V; ++j) {
              double s = 0.0;
              for (int i = 0; i < K; ++i) s += Hprev[i * V + l] * dX[i * V + j];
              dW[(size_t)n * V * V + l * V + j] += s;
            }
        if (dk)
          for (int i = 0; i < K; ++i) {
            double s = 0.0;
            for (int j = 0; j < V; ++j) s += dX[i * V + j] * vt[j];
            dk[(bt * p->Nk + n / gk) * K + i] += s;
          }
        if (dv)
          for (int j = 0; j < V; ++j) {
            double s = 0.0;
            for (int i = 0; i < K; ++i) s += dX[i * V + j] * kt[i];
            if (w_r) s += w_r[(size_t)n * V + j] * dyt[j];
            dv[(bt * N + n) * V + j] = s;
          }
        /* per-step clipping of the state gradient (section "Gradient Clipping");
         * the paper gives no threshold or form: elementwise clamp, off by default */
        if (p->dh_clip > 0.0)
          for (size_t e = 0; e < KV; ++e) {
            if (C[e] > p->dh_clip) C[e] = p->dh_clip;
            if (C[e] < -p->dh_clip) C[e] = -p->dh_clip;
          }
      }
      if (dh0) memcpy(dh0 + bn * KV, C, sizeof(double) * KV);
    }
  free(Hs); free(Z); free(G); free(dX); free(C);
  return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Output path after the scan: y_gt = RMSNorm(y_t (.) g_t) over the head-concatenated features. */
static double silu_fn(double x, double *dx) {
  const double sg = 1.0 / (1.0 + exp(-x));
  if (dx) *dx = sg * (1.0 + x * (1.0 - sg));
  return x * sg;
}

int m2rnn_ref_gated_norm_fwd(long tokens, int d, const double *y, const double *g_in, const double *w,
                             double eps, int silu, double *out, double *rstd) {
  if (!y || !g_in || !w || !out || d <= 0 || tokens < 0) return -1;
  for (long t = 0; t < tokens; ++t) {
    const double *yt = y + t * d, *gt = g_in + t * d;
    double ss = 0.0;
    for (int j = 0; j < d; ++j) {
      const double g = silu ? silu_fn(gt[j], NULL) : gt[j];
      const double x = yt[j] * g;
      ss += x * x;
    }
    const double s = 1.0 / sqrt(ss / d + eps);
    for (int j = 0; j < d; ++j) {
      const double g = silu ? silu_fn(gt[j], NULL) : gt[j];
      out[t * d + j] = w[j] * (yt[j] * g) * s;
    }
    if (rstd) rstd[t] = s;
  }
  return 0;
}

int m2rnn_ref_gated_norm_bwd(long tokens, int d, const double *y, const double *g_in, const double *w,
                             double eps, int silu, const double *dout, double *dy, double *dg_in,
                             double *dw) {
  if (!y || !g_in || !w || !dout || !dy || !dg_in || !dw || d <= 0 || tokens < 0) return -1;
  for (int j = 0; j < d; ++j) dw[j] = 0.0;
  for (long t = 0; t < tokens; ++t) {
    const double *yt = y + t * d, *gt = g_in + t * d, *dot = dout + t * d;
    double ss = 0.0, r = 0.0;
    for (int j = 0; j < d; ++j) {
      const double g = silu ? silu_fn(gt[j], NULL) : gt[j];
      const double x = yt[j] * g;
      ss += x * x;
      r += w[j] * dot[j] * x;
    }
    const double s = 1.0 / sqrt(ss / d + eps);
    for (int j = 0; j < d; ++j) {
      double dsilu = 1.0;
      const double g = silu ? silu_fn(gt[j], &dsilu) : gt[j];
      const double x = yt[j] * g;
      const double dx = s * w[j] * dot[j] - r * s * s * s * x / d;
      dy[t * d + j] = dx * g;
      dg_in[t * d + j] = dx * yt[j] * dsilu;
      dw[j] += dot[j] * x * s;
    }
  }
  return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Input path before the scan ("M2RNN block" equations): q_t, k_t, v_t = SiLU(conv1d(projection)),
 * a depthwise causal convolution of width 4 along time, one filter per channel:
 *     pre[t][c] = bias[c] + sum_{s=0..3} w[c][s] * x[t-3+s][c],     out = SiLU(pre),
 * so w[c][3] weighs the current token and w[c][0] the one three steps back (the layout of a
 * cross-correlation with three zeros padded on the left).  Inputs before t = 0 are zero, or the
 * three rows of `prev` (the last three inputs of the segment before this one). */
static double conv_in(const double *x, const double *prev, long b, int T, int C, int t, int c) {
  if (t >= 0) return x[((size_t)b * T + t) * C + c];
  return prev ? prev[((size_t)b * 3 + (3 + t)) * C + c] : 0.0;
}

int m2rnn_ref_conv_silu_fwd(int B, int T, int C, const double *x, const double *w, const double *bias,
                            const double *prev, double *out) {
  if (!x || !w || !out || B < 0 || T < 0 || C <= 0) return -1;
  for (long b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t)
      for (int c = 0; c < C; ++c) {
        double pre = bias ? bias[c] : 0.0;
        for (int s = 0; s < 4; ++s) pre += w[c * 4 + s] * conv_in(x, prev, b, T, C, t - 3 + s, c);
        out[((size_t)b * T + t) * C + c] = silu_fn(pre, NULL);
      }
  return 0;
}

/* Its backward: dpre = dout * SiLU'(pre);  dx[t'] = sum_s w[c][s] dpre[t'+3-s] (the steps that
 * read x[t']);  dw[c][s] = sum_{b,t} dpre[t] x[t-3+s];  dbias[c] = sum_{b,t} dpre[t];
 * dprev [B,3,C] likewise for the rows of `prev` (may be NULL). */
int m2rnn_ref_conv_silu_bwd(int B, int T, int C, const double *x, const double *w, const double *bias,
                            const double *prev, const double *dout, double *dx, double *dw,
                            double *dbias, double *dprev) {
  if (!x || !w || !dout || !dx || !dw || B < 0 || T < 0 || C <= 0) return -1;
  for (int i = 0; i < C * 4; ++i) dw[i] = 0.0;
  if (dbias) for (int c = 0; c < C; ++c) dbias[c] = 0.0;
  for (size_t i = 0; i < (size_t)B * T * C; ++i) dx[i] = 0.0;
  if (dprev) for (size_t i = 0; i < (size_t)B * 3 * C; ++i) dprev[i] = 0.0;
  for (long b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t)
      for (int c = 0; c < C; ++c) {
        double pre = bias ? bias[c] : 0.0;
        for (int s = 0; s < 4; ++s) pre += w[c * 4 + s] * conv_in(x, prev, b, T, C, t - 3 + s, c);
        double dsilu;
        (void)silu_fn(pre, &dsilu);
        const double dpre = dout[((size_t)b * T + t) * C + c] * dsilu;
        if (dbias) dbias[c] += dpre;
        for (int s = 0; s < 4; ++s) {
          const int ts = t - 3 + s;
          dw[c * 4 + s] += dpre * conv_in(x, prev, b, T, C, ts, c);
          if (ts >= 0) dx[((size_t)b * T + ts) * C + c] += w[c * 4 + s] * dpre;
          else if (dprev) dprev[((size_t)b * 3 + (3 + ts)) * C + c] += w[c * 4 + s] * dpre;
        }
      }
  return 0;
}

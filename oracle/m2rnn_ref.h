/*
 * M2RNN scan oracle: a plain, slow, fp64 CPU statement of the recurrence.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may include, link or
 * call this; only the test-suite, the smoke check and the bench's CPU-baseline
 * leg do.  It shares no code with the CUDA library.
 *
 * What it follows (paper: "M2RNN: Non-Linear RNNs with Matrix-Valued States"):
 *   Eq. 1-3 (M2RNN layer, recurrence):  Z_t = tanh(H_{t-1} W + k_t v_t^T)
 *                                        H_t = f_t H_{t-1} + (1-f_t) Z_t
 *                                        y_t = H_t^T q_t + w_r (.) v_t
 *   Forget-gate equation (section "Forget Gate"):
 *                                        f = (1 + exp(x + beta_n))^(-alpha_n)
 *   Algorithm 1 (loop order, y read from the post-update state, tensor layouts)
 *   Algorithm 2 (reverse sweep), with the carried state-gradient restored
 *   (the printed "dH" lines drop it; see m2rnn_ref_bwd).
 *
 * Layouts (Algorithm 1/2 I/O lists, token-major, heads interleaved), all fp64,
 * host memory, contiguous:
 *   q [B,T,Nq,K]  k [B,T,Nk,K]  v [B,T,N,V]  gate [B,T,N]  W [N,V,V]
 *   h0/hT [B,N,K,V]  y/dy [B,T,N,V]  alpha,beta [N]  w_r [N,V]
 * Head n reads q-head n / (N/Nq) and k-head n / (N/Nk) (contiguous groups;
 * Nq = Nk = 1 is the paper's multi-value layout).
 */
#ifndef M2RNN_REF_H
#define M2RNN_REF_H

#ifdef __cplusplus
extern "C" {
#endif

enum { M2RNN_REF_GATE_VALUE = 0, /* gate tensor already holds f in [0,1] (Algorithm 1 input F) */
       M2RNN_REF_GATE_LOGIT = 1, /* f = 1/(1+exp(-gate))  (psi with alpha=1, beta=0, x=-gate)   */
       M2RNN_REF_GATE_PSI   = 2  /* f = (1+exp(gate+beta_n))^(-alpha_n)   (forget-gate equation) */
};

typedef struct {
  int B, T, N, Nq, Nk, K, V;
  int gate_kind;
  double dh_clip; /* <= 0: off; else clamp the carried state gradient to [-c, c] after each reverse step */
} m2rnn_ref_params;

/* f and df/dgate for one gate entry of head n. */
double m2rnn_ref_gate(int gate_kind, double x, double alpha, double beta, double *dfdx);

/* Forward scan.  h0, alpha, beta, w_r, hT, H_all may be NULL.
 * H_all, when given, receives every state: [B,N,T+1,K,V] with H_all[..,0,..] = H_0. */
int m2rnn_ref_fwd(const m2rnn_ref_params *p, const double *q, const double *k, const double *v,
                  const double *gate, const double *W, const double *h0, const double *alpha,
                  const double *beta, const double *w_r, double *y, double *hT, double *H_all);

/* Backward through time.  d_hT (seed of the carried gradient) and dh0 may be NULL.
 * dq [B,T,Nq,K] and dk [B,T,Nk,K] hold the sum over the heads that share them,
 * dW [N,V,V] the sum over batch, dgate the gradient w.r.t. the gate tensor as passed. */
int m2rnn_ref_bwd(const m2rnn_ref_params *p, const double *q, const double *k, const double *v,
                  const double *gate, const double *W, const double *h0, const double *alpha,
                  const double *beta, const double *w_r, const double *dy, const double *d_hT,
                  double *dq, double *dk, double *dv, double *dgate, double *dW, double *dh0);

/* One step of the recurrence on a cached state [B,N,K,V] (updated in place).
 * q [B,Nq,K], k [B,Nk,K], v [B,N,V], gate [B,N], y [B,N,V]. */
int m2rnn_ref_decode_step(const m2rnn_ref_params *p, const double *q, const double *k,
                          const double *v, const double *gate, const double *W,
                          const double *alpha, const double *beta, const double *w_r,
                          double *state, double *y);

/* Output path of the layer after the scan ("M2RNN block" equations, y_gt = RMSNorm(y_t (.) g_t), and
 * the RMSNorm appendix): per token, over the d features of all heads concatenated,
 *     x = y (.) g,   s = 1 / sqrt(mean_j x_j^2 + eps),   out_i = w_i x_i s,
 * with g = g_in (silu = 0) or g = SiLU(g_in) = g_in / (1 + exp(-g_in)) (silu != 0).
 * y, g_in, out [tokens, d]; w [d]; rstd [tokens] receives s (may be NULL). */
int m2rnn_ref_gated_norm_fwd(long tokens, int d, const double *y, const double *g_in, const double *w,
                             double eps, int silu, double *out, double *rstd);

/* Its backward (RMSNorm appendix: p = w (.) dout, r = sum_j p_j x_j, dx = s p - r s^3 x / d,
 * dw_i = sum over tokens of dout_i x_i s), then through the product: dy = dx (.) g,
 * dg = dx (.) y, and through SiLU when silu != 0.  dw [d] is the sum over tokens. */
int m2rnn_ref_gated_norm_bwd(long tokens, int d, const double *y, const double *g_in, const double *w,
                             double eps, int silu, const double *dout, double *dy, double *dg_in,
                             double *dw);

/* Input path before the scan ("M2RNN block" equations: q_t, k_t, v_t = SiLU(conv1d(projection))):
 * depthwise causal convolution of width 4 along time, then SiLU.
 *     pre[b][t][c] = bias[c] + sum_{s=0..3} w[c][s] x[b][t-3+s][c],   out = pre / (1 + exp(-pre))
 * x, out [B,T,C]; w [C,4] (w[c][3] weighs the current token); bias [C] or NULL; prev [B,3,C] or NULL:
 * the inputs at t = -3, -2, -1 (NULL: zeros). */
int m2rnn_ref_conv_silu_fwd(int B, int T, int C, const double *x, const double *w, const double *bias,
                            const double *prev, double *out);

/* Its backward: dx [B,T,C], dw [C,4] and dbias [C] (may be NULL) summed over batch and time,
 * dprev [B,3,C] (may be NULL). */
int m2rnn_ref_conv_silu_bwd(int B, int T, int C, const double *x, const double *w, const double *bias,
                            const double *prev, const double *dout, double *dx, double *dw,
                            double *dbias, double *dprev);

#ifdef __cplusplus
}
#endif
#endif

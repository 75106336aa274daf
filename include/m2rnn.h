/*
 * m2rnn.h -- C ABI of the B200 (sm_100a) M2RNN recurrent-scan library.
 *
 * The library computes the sequential part of one M2RNN layer, per (batch b, head n)
 * on a K x V matrix state H (paper, Eq. 1-3 of the M2RNN layer):
 *
 *     Z_t = tanh(H_{t-1} W_n + k_t v_t^T)
 *     H_t = f_t H_{t-1} + (1 - f_t) Z_t
 *     y_t = H_t^T q_t  (+ w_r (.) v_t)
 *
 * forward (Algorithm 1), backward through time (Algorithm 2) and one decoding step.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, contiguous in the
 *     stated layout and 16-byte aligned.  `params` is a HOST pointer.
 *   - Layouts are the paper's (Algorithm 1/2 I/O lists): token-major, heads interleaved
 *     (variable-length batches and strided q/k/v: see m2rnn_params).
 *       q [B,T,Nq,K]  k [B,T,Nk,K]  v [B,T,N,V]  gate [B,T,N]  W [N,V,V]
 *       h0,hT [B,N,K,V]  y,dy [B,T,N,V]  alpha,beta [N]  w_r [N,V]
 *     Head n reads q-head n/(N/Nq) and k-head n/(N/Nk) (contiguous groups);
 *     Nq = Nk = 1 is the paper's multi-value layout, Nq = Nk = N plain multi-head.
 *   - q,k,v,W,w_r,y,dy,dq,dk,dv have the element type `io_dtype`; gate, alpha, beta,
 *     every state (h0,hT,ckpt,d_hT,dh0,decode state), dgate and dW are fp32.
 *     With M2RNN_BF16 the state x W product runs on tensor cores (bf16 operands, fp32
 *     accumulate) and the state itself stays fp32; with M2RNN_F32 everything is fp32 FMA.
 *   - The library allocates nothing and keeps nothing between calls.  Outputs are
 *     overwritten, never accumulated into.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the
 *     default stream) and never synchronise.  The return value is an m2rnn_status.
 *     Argument errors (every code but M2RNN_ERR_CUDA) are found on the host first: nothing
 *     has been launched when one is returned.  M2RNN_ERR_CUDA means the runtime refused a
 *     launch or a copy; a call is several launches, earlier ones may already be on the
 *     stream, and the outputs are then undefined.
 *   - `dev_status` (device int32, may be NULL): every wait inside a kernel is bounded;
 *     if one runs out the kernel stores M2RNN_ERR_TIMEOUT there and returns early.
 *     The caller zeroes it and reads it back after synchronising.
 *   - Supported sizes: K a multiple of 16 in 16..128, V in {16,32,64,128}, B,T,N >= 1
 *     (T = 0 or B = 0 is a valid empty call: nothing is launched, hT = h0 is NOT written).
 */
#ifndef M2RNN_H
#define M2RNN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  M2RNN_OK = 0,
  M2RNN_ERR_NULL = -1,        /* a required pointer is NULL                         */
  M2RNN_ERR_SHAPE = -2,       /* a size is non-positive or a head count does not divide N */
  M2RNN_ERR_UNSUPPORTED = -3, /* K, V, dtype, gate kind or ckpt_interval outside the supported set */
  M2RNN_ERR_ALIGN = -4,       /* a pointer is not 16-byte aligned                   */
  M2RNN_ERR_WORKSPACE = -5,   /* workspace missing or smaller than m2rnn_bwd_workspace_bytes */
  M2RNN_ERR_CUDA = -6,        /* the CUDA runtime refused a launch or attribute     */
  M2RNN_ERR_TIMEOUT = -7      /* device-side only: a bounded wait ran out           */
} m2rnn_status;

typedef enum { M2RNN_F32 = 0, M2RNN_BF16 = 1 } m2rnn_dtype;

typedef enum {
  M2RNN_GATE_VALUE = 0, /* gate tensor IS f_t in [0,1]                 (Algorithm 1, input F)    */
  M2RNN_GATE_LOGIT = 1, /* f_t = 1/(1+exp(-gate))                      (forget-gate eq., alpha=1, beta=0, x=-gate) */
  M2RNN_GATE_PSI = 2    /* f_t = (1+exp(gate+beta_n))^(-alpha_n)       (forget-gate equation)    */
} m2rnn_gate_kind;

typedef struct {
  int32_t B, T, N;       /* batch, steps, value heads (N = N_v = N_f = N_w)                   */
  int32_t Nq, Nk;        /* query / key heads: 1..N, each divides N                           */
  int32_t K, V;          /* state is K x V per (b,n); the transition matrix is V x V          */
  int32_t io_dtype;      /* m2rnn_dtype                                                       */
  int32_t gate_kind;     /* m2rnn_gate_kind                                                   */
  int32_t ckpt_interval; /* steps between saved states; 0 = library default for (K,V,dtype);
                            at most m2rnn_ckpt_interval's bound, and even for M2RNN_BF16        */
  float dh_clip;         /* <= 0: off.  Else the state gradient carried to the previous step is
                            clamped elementwise to [-dh_clip, dh_clip] after every reverse step
                            (section "Gradient Clipping"; the paper gives no threshold or form) */
  /* Token addressing of the scan calls (m2rnn_fwd, m2rnn_bwd; ignored by the decoding step).
   * All zero / NULL = the dense layouts above. */
  int64_t q_stride, k_stride, v_stride; /* elements between consecutive tokens of q, k, v; 0 = dense
                            (Nq K, Nk K, N V).  A larger stride lets q, k and v be views into one fused
                            projection output [tokens, Nq K + Nk K + N V + ...]; a token's heads stay
                            contiguous.  Multiples of 16 bytes.  Outputs and gradients are always dense. */
  int64_t total_tokens;  /* packed batches (cu_seqlens != NULL): tokens in the batch; else 0 */
  const int32_t *cu_seqlens; /* DEVICE pointer to B + 1 token offsets, or NULL.  With it the B sequences
                            are packed one after the other along the token axis: q [total_tokens,Nq,K],
                            k, v, gate [total_tokens,N], y, dy and the gradients likewise; sequence b is
                            tokens cu_seqlens[b] .. cu_seqlens[b+1]-1; T is the LONGEST sequence (it
                            sizes checkpoints and workspaces; a longer sequence is cut to T).  Offsets
                            are non-decreasing from 0 to total_tokens; a sequence may be empty (its
                            hT = h0, its dh0 = d_hT).  States stay [B,N,K,V]. */
} m2rnn_params;

/* Library version: major*10000 + minor*100 + patch. */
int m2rnn_version(void);

/* Static text for a status code. */
const char *m2rnn_status_string(int status);

/* The checkpoint interval C the library will use for `params` (params->ckpt_interval if it is
 * non-zero and supported, else the default); <= 0 is an m2rnn_status.  The backward kernel
 * recomputes C states at a time from a checkpoint, so C is bounded by on-chip memory. */
int m2rnn_ckpt_interval(const m2rnn_params *params);

/* Rows of a state that one CTA of the backward kernel takes for `params` (a divisor of K); <= 0
 * is an m2rnn_status.  The K rows of a state are independent recurrences (Eq. 1-2 act row by row),
 * so the backward pass may split them over K/rows CTAs; when it does, dv and dgate (sums over all
 * rows) are finished by two extra reduction launches. */
int m2rnn_bwd_row_slab(const m2rnn_params *params);

/* Bytes of the checkpoint tensor [B,N,ceil(T/C),K,V] (fp32). */
size_t m2rnn_ckpt_bytes(const m2rnn_params *params);

/* Scratch the forward call needs for `params`: 0 unless the library splits the rows of a state
 * over several CTAs (it does when there are few (b,n) units, to fill the GPU), in which case the
 * per-slab shares of y pass through this scratch before a second launch adds them. */
size_t m2rnn_fwd_workspace_bytes(const m2rnn_params *params);

/* Forward scan (Algorithm 1; Eq. 1-3).
 *   in : q,k,v,gate,W; h0 or NULL (= zero state); alpha,beta (GATE_PSI only, else ignored,
 *        may be NULL); w_r or NULL (residual term of Eq. 3 omitted, as in Algorithm 1)
 *   out: y [B,T,N,V]; hT or NULL: final state H_T (fp32);
 *        ckpt or NULL: ckpt[b,n,c] = H_{c*C}, the state BEFORE step c*C (so ckpt[..,0] = h0),
 *        for m2rnn_bwd.
 *   workspace: device scratch of at least m2rnn_fwd_workspace_bytes(params), 256-byte aligned
 *        (NULL and 0 when that is 0); contents undefined afterwards. */
int m2rnn_fwd(const m2rnn_params *params, const void *q, const void *k, const void *v,
              const float *gate, const void *W, const float *h0, const float *alpha,
              const float *beta, const void *w_r, void *y, float *hT, float *ckpt,
              void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

/* Scratch the backward call needs for `params`; `have_ckpt` != 0 if the caller will pass the
 * checkpoints written by m2rnn_fwd (otherwise the workspace also holds them). */
size_t m2rnn_bwd_workspace_bytes(const m2rnn_params *params, int have_ckpt);

/* Backward through time (Algorithm 2, with the state gradient carried across steps:
 * G_t = C_t + q_t dy_t^T, C_{t-1} = f_t G_t + dX_t W^T, dX_t = (1-f_t) G_t (.) (1 - Z_t (.) Z_t)).
 *   in : the forward inputs; ckpt from m2rnn_fwd with the same params, or NULL (recomputed here);
 *        dy [B,T,N,V]; d_hT or NULL: gradient w.r.t. the final state (seed of C_T)
 *   out: dq [B,T,Nq,K], dk [B,T,Nk,K] (summed over the heads sharing them), dv [B,T,N,V],
 *        dgate [B,T,N] (w.r.t. the gate tensor as passed, i.e. through the gate function),
 *        dW [N,V,V] fp32 (summed over batch, fixed order: results repeat bit for bit),
 *        dh0 or NULL [B,N,K,V] fp32.
 *   workspace: device scratch of at least m2rnn_bwd_workspace_bytes(params, ckpt != NULL),
 *        256-byte aligned; contents undefined afterwards.
 * w_r's own gradient (sum over b,t of v (.) dy) is an elementwise reduction outside the scan. */
int m2rnn_bwd(const m2rnn_params *params, const void *q, const void *k, const void *v,
              const float *gate, const void *W, const float *h0, const float *alpha,
              const float *beta, const void *w_r, const float *ckpt, const void *dy,
              const float *d_hT, void *dq, void *dk, void *dv, float *dgate, float *dW,
              float *dh0, void *workspace, size_t workspace_bytes, int32_t *dev_status,
              void *stream);

/* m2rnn_bwd without a workspace argument, for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a convenience of the library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside a host
 * application that owns the allocator and hands out only input/output buffers, a real-time or
 * safety-reviewed service that forbids allocation after start-up, or a caller whose memory pool
 * is exhausted or fragmented by the time the backward pass runs.  Such callers still pass every
 * input and output tensor; only the scratch comes from the library.
 *
 * The scratch is a fixed array of M2RNN_STATIC_SCRATCH_BYTES inside the library's device image:
 * every GPU that loads the library's device code holds that much memory until the process exits,
 * whether or not this function is ever called.  The function itself calls no allocating routine.
 * The CUDA runtime, however, may load a library's device code lazily (its default), and the
 * array's memory is claimed at that moment: on a device that is already full the first call can
 * therefore fail with M2RNN_ERR_CUDA.  So make the first call on each device at start-up, while
 * memory is still to be had (any small problem will do), or run with CUDA_MODULE_LOADING=EAGER.
 *   - A problem whose m2rnn_bwd_workspace_bytes(params, ckpt != NULL) exceeds
 *     M2RNN_STATIC_SCRATCH_BYTES is refused with M2RNN_ERR_WORKSPACE before anything runs;
 *     passing the checkpoints written by m2rnn_fwd lowers the need.
 *   - The first call on each device looks up the array's device address (the device that is
 *     current at the call); that same start-up call must come before any stream capture.
 *   - All calls share the one array, which keeps whatever the last call left in it.  Nothing in
 *     it has to start at zero (each call writes what it later reads), but two calls that overlap
 *     on the GPU -- different streams, or different host threads -- race on it: run them one
 *     after the other.
 * Arguments, outputs and status codes are otherwise exactly those of m2rnn_bwd. */
#define M2RNN_STATIC_SCRATCH_BYTES (8u << 20)
int m2rnn_bwd_static_scratch(const m2rnn_params *params, const void *q, const void *k,
                             const void *v, const float *gate, const void *W, const float *h0,
                             const float *alpha, const float *beta, const void *w_r,
                             const float *ckpt, const void *dy, const float *d_hT, void *dq,
                             void *dk, void *dv, float *dgate, float *dW, float *dh0,
                             int32_t *dev_status, void *stream);

/* One decoding step on a cached state (Eq. 1-3 once; params->T is ignored).
 *   in : q [B,Nq,K], k [B,Nk,K], v [B,N,V], gate [B,N], W, alpha/beta/w_r as in m2rnn_fwd
 *   io : state [B,N,K,V] fp32, updated in place
 *   out: y [B,N,V] */
int m2rnn_decode_step(const m2rnn_params *params, const void *q, const void *k, const void *v,
                      const float *gate, const void *W, const float *alpha, const float *beta,
                      const void *w_r, float *state, void *y, int32_t *dev_status, void *stream);

/* Self-test of the bounded waits (`dev_status` above).  Launches one warp that waits, with the
 * library's own wait routine and a limit of `limit_cycles` SM clocks (0 .. 1e8), on a barrier that
 * nothing ever completes.  The wait gives up, the kernel stores M2RNN_ERR_TIMEOUT in *dev_status
 * and returns normally; the context stays usable.  `waited_cycles` (device int64, may be NULL)
 * receives the SM clocks the wait took.  The paper has no counterpart: this exercises the
 * library's failure reporting without making anything fail. */
int m2rnn_wait_selftest(int64_t limit_cycles, int32_t *dev_status, int64_t *waited_cycles, void *stream);

/* ---- Output path after the scan ("M2RNN block" equations: y_gt = RMSNorm(y_t (.) g_t) with
 * g_t = SiLU of the gate projection; "RMSNormTP Module" appendix for RMSNorm and its backward).
 * Fuses the product with the gate and the normalisation over the d = N V features of all heads of
 * a token, so that y (.) g never goes to memory:
 *     x = y (.) g,   s = 1 / sqrt((1/d) sum_j x_j^2 + eps),   out_i = w_i x_i s
 * where g = g_in (silu = 0) or g = SiLU(g_in) = g_in / (1 + exp(-g_in)) (silu != 0).  The paper
 * prints RMSNorm without an epsilon: eps = 0 reproduces it, a positive eps guards all-zero rows.
 *   in : y, g_in [tokens, d] (the scan's y [B,T,N,V] has tokens = B T, d = N V), w [d], io_dtype
 *   out: out [tokens, d] io_dtype; rstd [tokens] fp32 = s (NULL: not stored; the backward needs it)
 * d is a multiple of 8, at most 8192.  tokens = 0 is a valid empty call.  Pointers: device, 16-byte
 * aligned, caller-owned; asynchronous on `stream`; errors as for the scan calls. */
int m2rnn_gated_norm_fwd(int64_t tokens, int32_t d, int32_t io_dtype, const void *y, const void *g_in,
                         const void *w, float eps, int32_t silu, void *out, float *rstd, void *stream);

/* Bytes of workspace m2rnn_gated_norm_bwd needs (per-CTA partial sums of dw). */
size_t m2rnn_gated_norm_bwd_workspace_bytes(int64_t tokens, int32_t d);

/* Backward of m2rnn_gated_norm_fwd (appendix formulas: p = w (.) dout, r = sum_j p_j x_j,
 * dx = s p - r s^3 x / d, dw_i = sum over tokens of dout_i x_i s), continued through the product
 * (dy = dx (.) g, dg = dx (.) y) and through SiLU when silu != 0.
 *   in : y, g_in, w as in the forward call; rstd [tokens] as the forward call stored it;
 *        dout [tokens, d]
 *   out: dy, dg_in [tokens, d] io_dtype; dw [d] fp32 (sum over tokens, fixed order: bitwise
 *        repeatable); all overwritten
 *   workspace: 256-byte aligned device memory of at least the queried size. */
int m2rnn_gated_norm_bwd(int64_t tokens, int32_t d, int32_t io_dtype, const void *y, const void *g_in,
                         const void *w, const float *rstd, int32_t silu, const void *dout, void *dy,
                         void *dg_in, float *dw, void *workspace, size_t workspace_bytes, void *stream);

/* ---- Input path before the scan ("M2RNN block" equations: q_t, k_t, v_t = SiLU(conv1d(projection)):
 * a depthwise causal convolution of width 4 along time, one filter per channel, then SiLU).
 *     pre[b][t][c] = bias[c] + sum_{s=0..3} w[c][s] x[b][t-3+s][c],     out = pre / (1 + exp(-pre))
 * (w[c][3] weighs the current token, w[c][0] the one three steps back; the paper gives the
 * convolution no bias of its own: bias = NULL.)
 *   in : x [B,T,C] with `x_stride` elements between tokens (0 = C); w [C,4]; bias [C] or NULL;
 *        prev [B,3,C] or NULL: the inputs at t = -3, -2, -1 (the last three of the segment before;
 *        NULL = zeros), io_dtype all
 *   out: out [B,T,C] with `out_stride` elements between tokens (0 = C); may be x itself only if
 *        nothing else reads x afterwards AND the call is the only one on those rows (in place is
 *        not supported: a tile reads three rows that its neighbour writes).
 * The strides let the three projections be handled as ONE tensor: x = the fused projection output
 * [B,T,Nq K + Nk K + N V], out of the same shape, whose column slices are then the q, k, v of
 * m2rnn_fwd (see m2rnn_params.q_stride).  C is a multiple of 16 bytes of channels.  B = 0 or T = 0
 * is a valid empty call.  Device pointers, 16-byte aligned, asynchronous on `stream`. */
int m2rnn_conv_silu_fwd(int32_t B, int32_t T, int32_t C, int32_t io_dtype, const void *x, int64_t x_stride,
                        const void *w, const void *bias, const void *prev, void *out, int64_t out_stride,
                        void *stream);

/* Bytes of workspace m2rnn_conv_silu_bwd needs (per-tile partial sums of dw and dbias). */
size_t m2rnn_conv_silu_bwd_workspace_bytes(int32_t B, int32_t T, int32_t C);

/* Backward of m2rnn_conv_silu_fwd: with dpre = dout (.) SiLU'(pre) (pre recomputed from x),
 *     dx[t] = sum_s w[c][s] dpre[t+3-s],   dw[c][s] = sum_{b,t} dpre[t] x[t-3+s],   dbias[c] = sum_{b,t} dpre[t].
 *   in : x, w, bias, prev as in the forward call; dout [B,T,C] (token stride dout_stride)
 *   out: dx [B,T,C] (token stride dx_stride); dw [C,4] fp32; dbias [C] fp32 or NULL; dprev [B,3,C]
 *        io_dtype or NULL; all overwritten; sums in a fixed order (bitwise repeatable)
 *   workspace: 256-byte aligned device memory of at least the queried size. */
int m2rnn_conv_silu_bwd(int32_t B, int32_t T, int32_t C, int32_t io_dtype, const void *x, int64_t x_stride,
                        const void *w, const void *bias, const void *prev, const void *dout,
                        int64_t dout_stride, void *dx, int64_t dx_stride, float *dw, float *dbias,
                        void *dprev, void *workspace, size_t workspace_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* M2RNN_H */

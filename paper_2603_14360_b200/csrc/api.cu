// C ABI of the M2RNN scan library: argument checks, workspace layout, dispatch.
// No allocation, no synchronisation, no state kept between calls.
#include <cuda_runtime.h>

#include <cstdlib>
#include <cstring>

#include "internal.h"
#include "m2rnn.h"

namespace m2rnn {

// SMs of the current device (the plans size their grids by it); 148, a B200's count, when no device
// can be asked -- the size queries of the ABI also run on hosts without a GPU.
int sm_count() {
  int dev = -1, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
    (void)cudaGetLastError();
    return 148;
  }
  return sms;
}

bool bwd_use_tc(int B, int N, int K, int V, int io_dtype) {
  if (io_dtype != M2RNN_BF16 || V != 128 || K % bwd_tc_rows_per_cta()) return false;   // 32-row CTAs
  const char *variant = getenv("M2RNN_BWD_VARIANT");
  if (variant && !strcmp(variant, "mma")) return false;
  (void)B; (void)N;
  return true;
}

BwdPlan plan_bwd(int B, int N, int K, int V, int io_dtype) {
  BwdPlan pl{};
  if (io_dtype == M2RNN_F32) {  // recomputed states live in global scratch
    pl.KC = K; pl.C = 16; pl.C_max = 64;
    return pl;
  }
  if (bwd_use_tc(B, N, K, V, io_dtype)) {   // 32-row CTAs, chunks of four steps
    pl.KC = bwd_tc_rows_per_cta(); pl.C = pl.C_max = bwd_tc_chunk();
    return pl;
  }
  // Rows per CTA: the largest slab that still spreads the problem over the SMs (rows are independent
  // recurrences; a smaller slab only shortens the work per step).  V = 128 keeps the slab at 32 rows
  // for the sake of registers.
  const int kSMs = sm_count();
  const long units = (long)(B > 0 ? B : 1) * N;
  const int cap = V > 64 ? 32 : 64;
  int KC = 16;
  for (int cand = 32; cand <= cap; cand *= 2)
    if (K % cand == 0) KC = cand;
  while (KC > 16 && units * (K / KC) < kSMs && units * (K / (KC / 2)) <= kSMs) KC /= 2;
  // V = 16, whole 64-row states, more units than two CTAs per SM hold (the paper's layer shape: 336
  // units): 32-row CTAs at three per SM where that needs fewer waves, a 32-row CTA's wave counted
  // as 0.9 of a 64-row one (measured: the step is latency, not rows; 3.50 -> 3.16 ms at that shape)
  bool v16_split = false;
  if (V == 16 && KC == 64 && units > 2L * kSMs) {
    const long waves64 = (units + 2L * kSMs - 1) / (2L * kSMs), waves32 = (2 * units + 3L * kSMs - 1) / (3L * kSMs);
    v16_split = 9 * waves32 < 10 * waves64;
  }
  if (v16_split) KC = 32;
  pl.KC = KC;
  // Checkpoint interval: as many steps as two chunk buffers fit in shared memory (even, <= 16)
  constexpr size_t kSmemLimit = 227 * 1024;
  int c = 16;
  while (c > 2 && bwd_bf16_smem_bytes(KC, V, c) > kSmemLimit) c -= 2;
  pl.C_max = c;
  // V = 16 with more CTAs than SMs (the paper's layer shape: 84 heads): a shorter chunk lets two
  // (32-row CTAs: three) CTAs share an SM, which saves a wave
  if (V == 16 && units * (K / KC) > kSMs)
    while (c > 2 && bwd_bf16_smem_bytes(KC, V, c) > (v16_split ? 72 : 110) * 1024) c -= 2;
  pl.C = c;
  return pl;
}

bool fwd_use_tc(int B, int N, int K, int V, int io_dtype) {
  if (io_dtype != M2RNN_BF16) return false;
  const char *variant = getenv("M2RNN_FWD_VARIANT");
  if (variant && !strcmp(variant, "tc")) return true;
  if (variant && (!strcmp(variant, "mma") || !strcmp(variant, "wide"))) return false;
  // Measured (B200): the round trip of a tcgen05 step (operand store, proxy fence, barrier, eight
  // MMAs at ~30 cycles of issue each, commit, mbarrier, tcgen05.ld) is ~400 cycles before any
  // arithmetic, against ~30 for mma.sync on registers.  It pays only where the register kernels
  // are bound by the legacy tensor path and there are rows to amortise it over: V = 128 with 64-row
  // CTAs on at least three quarters of the SMs (the K = V = 128 point of the state-size sweep: 6.8
  // against 7.8 ms).
  return V == 128 && K % 64 == 0 && 4L * (B > 0 ? B : 1) * N * (K / 64) >= 3L * sm_count();
}

int plan_fwd_rows(int B, int N, int K, int V, int io_dtype) {
  if (io_dtype == M2RNN_F32) return K;
  if (fwd_use_tc(B, N, K, V, io_dtype)) return fwd_tc_rows_per_cta(B, N, K, V);
  // The smallest slab (a multiple of 16 rows that divides K) that still gives every CTA an SM of
  // its own; with more units than SMs the whole state stays in one CTA.  V = 128 keeps the slab
  // at 64 rows or fewer for the sake of registers.
  const int kSMs = sm_count();
  const long units = (long)(B > 0 ? B : 1) * N;
  const int cap = V > 64 ? 32 : 128;
  int best = 0;
  for (int kc = 16; kc <= K && kc <= cap; kc += 16) {
    if (K % kc) continue;
    best = kc;                                   // largest admissible slab so far
    if (units * (K / kc) <= kSMs) break;         // first (smallest) slab that fits one wave
  }
  return best;
}

namespace {

// A refused launch, attribute or copy: the runtime's last-error slot is cleared here, so that the
// caller's own next cudaGetLastError() does not report this library's failure a second time.
int cuda_failed() {
  (void)cudaGetLastError();
  return M2RNN_ERR_CUDA;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_params(const m2rnn_params *p, bool need_T) {
  if (!p) return M2RNN_ERR_NULL;
  if (p->B < 0 || p->N <= 0 || p->K <= 0 || p->V <= 0 || (need_T && p->T < 0)) return M2RNN_ERR_SHAPE;
  if (p->Nq <= 0 || p->Nk <= 0 || p->Nq > p->N || p->Nk > p->N || p->N % p->Nq || p->N % p->Nk)
    return M2RNN_ERR_SHAPE;
  if (p->io_dtype != M2RNN_F32 && p->io_dtype != M2RNN_BF16) return M2RNN_ERR_UNSUPPORTED;
  if (p->gate_kind < M2RNN_GATE_VALUE || p->gate_kind > M2RNN_GATE_PSI) return M2RNN_ERR_UNSUPPORTED;
  if (p->K % 16 || p->K < 16 || p->K > 128) return M2RNN_ERR_UNSUPPORTED;
  if (p->V != 16 && p->V != 32 && p->V != 64 && p->V != 128) return M2RNN_ERR_UNSUPPORTED;
  if (p->ckpt_interval < 0 || p->ckpt_interval > plan_bwd(p->B, p->N, p->K, p->V, p->io_dtype).C_max)
    return M2RNN_ERR_UNSUPPORTED;
  // the bf16 kernels take steps in pairs and checkpoint between pairs
  if (p->io_dtype == M2RNN_BF16 && (p->ckpt_interval & 1)) return M2RNN_ERR_UNSUPPORTED;
  // token strides: at least a token's heads, in 16-byte units
  const int64_t unit16 = p->io_dtype == M2RNN_BF16 ? 8 : 4;
  const int64_t dense[3] = {(int64_t)p->Nq * p->K, (int64_t)p->Nk * p->K, (int64_t)p->N * p->V};
  const int64_t given[3] = {p->q_stride, p->k_stride, p->v_stride};
  for (int x = 0; x < 3; ++x)
    if (given[x] != 0 && (given[x] < dense[x] || given[x] % unit16)) return M2RNN_ERR_SHAPE;
  if (p->total_tokens < 0 || (!p->cu_seqlens && p->total_tokens != 0)) return M2RNN_ERR_SHAPE;
  if (p->cu_seqlens && (need_T && p->total_tokens > (int64_t)p->B * p->T)) return M2RNN_ERR_SHAPE;
  return M2RNN_OK;
}

// tokens in the batch
size_t tokens_of(const m2rnn_params *p) { return p->cu_seqlens ? (size_t)p->total_tokens : (size_t)p->B * p->T; }

int interval_of(const m2rnn_params *p) {
  return p->ckpt_interval ? p->ckpt_interval : plan_bwd(p->B, p->N, p->K, p->V, p->io_dtype).C;
}

struct Workspace {
  size_t ckpt, dW_part, dq_part, dk_part, chunk_states, dv_part, dgate_part, total;
};

Workspace layout(const m2rnn_params *p, bool have_ckpt) {
  Workspace w{};
  const int C = interval_of(p);
  const size_t nch = p->T > 0 ? (size_t)(p->T + C - 1) / C : 0;
  const size_t BN = (size_t)p->B * p->N, KV = (size_t)p->K * p->V;
  size_t off = 0;
  w.ckpt = off;
  if (!have_ckpt) off += align_up(BN * nch * KV * sizeof(float));
  const int RS = p->K / plan_bwd(p->B, p->N, p->K, p->V, p->io_dtype).KC;   // row slabs per state (1 on the fp32 path)
  w.dW_part = off;
  off += align_up(BN * RS * p->V * p->V * sizeof(float));
  const size_t TT = tokens_of(p);
  w.dq_part = off;
  if (p->Nq < p->N) off += align_up(TT * p->N * p->K * sizeof(float));
  w.dk_part = off;
  if (p->Nk < p->N) off += align_up(TT * p->N * p->K * sizeof(float));
  w.chunk_states = off;
  if (p->io_dtype == M2RNN_F32) off += align_up(BN * C * KV * sizeof(float));
  w.dv_part = off;
  if (RS > 1) off += align_up((size_t)RS * TT * p->N * p->V * sizeof(float));
  w.dgate_part = off;
  if (RS > 1) off += align_up((size_t)RS * TT * p->N * sizeof(float));
  w.total = off;
  return w;
}

ScanArgs base_args(const m2rnn_params *p) {
  ScanArgs a{};
  a.B = p->B; a.T = p->T; a.N = p->N; a.Nq = p->Nq; a.Nk = p->Nk; a.K = p->K; a.V = p->V;
  a.gate_kind = p->gate_kind;
  a.KC = plan_bwd(p->B, p->N, p->K, p->V, p->io_dtype).KC;
  a.KCf = plan_fwd_rows(p->B, p->N, p->K, p->V, p->io_dtype);
  a.C = interval_of(p);
  a.nchunks = p->T > 0 ? (p->T + a.C - 1) / a.C : 0;
  a.dh_clip = p->dh_clip;
  a.qs = p->q_stride ? p->q_stride : (long long)p->Nq * p->K;
  a.ks = p->k_stride ? p->k_stride : (long long)p->Nk * p->K;
  a.vs = p->v_stride ? p->v_stride : (long long)p->N * p->V;
  a.TT = (long long)tokens_of(p);
  a.cu = p->cu_seqlens;
  return a;
}

}  // namespace
}  // namespace m2rnn

using namespace m2rnn;

extern "C" {

int m2rnn_version(void) { return 100; }

const char *m2rnn_status_string(int status) {
  switch (status) {
    case M2RNN_OK: return "ok";
    case M2RNN_ERR_NULL: return "a required pointer is NULL";
    case M2RNN_ERR_SHAPE: return "bad size: non-positive, or a head count that does not divide N";
    case M2RNN_ERR_UNSUPPORTED: return "unsupported K, V, dtype, gate kind or checkpoint interval";
    case M2RNN_ERR_ALIGN: return "a pointer is not 16-byte aligned (workspace: 256-byte)";
    case M2RNN_ERR_WORKSPACE: return "workspace missing or too small";
    case M2RNN_ERR_CUDA: return "the CUDA runtime refused the launch";
    case M2RNN_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

int m2rnn_ckpt_interval(const m2rnn_params *params) {
  int rc = check_params(params, false);
  if (rc != M2RNN_OK) return rc;
  return interval_of(params);
}

int m2rnn_bwd_row_slab(const m2rnn_params *params) {
  int rc = check_params(params, false);
  if (rc != M2RNN_OK) return rc;
  return plan_bwd(params->B, params->N, params->K, params->V, params->io_dtype).KC;
}

size_t m2rnn_ckpt_bytes(const m2rnn_params *params) {
  if (check_params(params, true) != M2RNN_OK || params->T == 0) return 0;
  const int C = interval_of(params);
  return (size_t)params->B * params->N * ((params->T + C - 1) / C) * params->K * params->V * sizeof(float);
}

size_t m2rnn_fwd_workspace_bytes(const m2rnn_params *params) {
  if (check_params(params, true) != M2RNN_OK) return 0;
  const int kcf = plan_fwd_rows(params->B, params->N, params->K, params->V, params->io_dtype);
  const int RS = (params->K + kcf - 1) / kcf;
  if (RS <= 1) return 0;
  return align_up((size_t)RS * tokens_of(params) * params->N * params->V * sizeof(float));
}

int m2rnn_fwd(const m2rnn_params *params, const void *q, const void *k, const void *v,
              const float *gate, const void *W, const float *h0, const float *alpha,
              const float *beta, const void *w_r, void *y, float *hT, float *ckpt,
              void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream) {
  int rc = check_params(params, true);
  if (rc != M2RNN_OK) return rc;
  if (params->B == 0 || params->T == 0 || tokens_of(params) == 0) return M2RNN_OK;
  if (!q || !k || !v || !gate || !W || !y) return M2RNN_ERR_NULL;
  if (params->gate_kind == M2RNN_GATE_PSI && (!alpha || !beta)) return M2RNN_ERR_NULL;
  const void *ptrs[] = {q, k, v, gate, W, h0, w_r, y, hT, ckpt};
  for (const void *p : ptrs)
    if (!aligned16(p)) return M2RNN_ERR_ALIGN;
  ScanArgs a = base_args(params);
  a.q = q; a.k = k; a.v = v; a.gate = gate; a.W = W; a.h0 = h0; a.w_r = w_r;
  a.alpha = params->gate_kind == M2RNN_GATE_PSI ? alpha : nullptr;
  a.beta = params->gate_kind == M2RNN_GATE_PSI ? beta : nullptr;
  a.y = y; a.hT = hT; a.ckpt = ckpt; a.dev_status = dev_status;
  const size_t need = m2rnn_fwd_workspace_bytes(params);
  if (need > 0) {
    if (!workspace || workspace_bytes < need) return M2RNN_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return M2RNN_ERR_ALIGN;
    a.y_part = static_cast<float *>(workspace);
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = params->io_dtype == M2RNN_F32 ? launch_fwd_f32(a, s) : launch_fwd_bf16(a, s);
  if (e == cudaSuccess && a.y_part)
    e = launch_reduce_slabs(a.y_part, y, params->io_dtype, (params->K + a.KCf - 1) / a.KCf,
                            tokens_of(params) * params->N * params->V, s);
  return e == cudaSuccess ? M2RNN_OK : cuda_failed();
}

size_t m2rnn_bwd_workspace_bytes(const m2rnn_params *params, int have_ckpt) {
  if (check_params(params, true) != M2RNN_OK) return 0;
  return layout(params, have_ckpt != 0).total;
}

int m2rnn_bwd(const m2rnn_params *params, const void *q, const void *k, const void *v,
              const float *gate, const void *W, const float *h0, const float *alpha,
              const float *beta, const void *w_r, const float *ckpt, const void *dy,
              const float *d_hT, void *dq, void *dk, void *dv, float *dgate, float *dW,
              float *dh0, void *workspace, size_t workspace_bytes, int32_t *dev_status,
              void *stream) {
  int rc = check_params(params, true);
  if (rc != M2RNN_OK) return rc;
  if (!dW) return M2RNN_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (params->B == 0 || params->T == 0 || tokens_of(params) == 0) {
    // empty scan: the only defined outputs are dW = 0 and dh0 = d_hT (or 0)
    if (!aligned16(dW) || !aligned16(dh0) || !aligned16(d_hT)) return M2RNN_ERR_ALIGN;
    cudaError_t e = cudaMemsetAsync(dW, 0, sizeof(float) * params->N * params->V * params->V, s);
    if (e == cudaSuccess && dh0 && params->B > 0) {
      const size_t bytes = sizeof(float) * (size_t)params->B * params->N * params->K * params->V;
      e = d_hT ? cudaMemcpyAsync(dh0, d_hT, bytes, cudaMemcpyDeviceToDevice, s) : cudaMemsetAsync(dh0, 0, bytes, s);
    }
    return e == cudaSuccess ? M2RNN_OK : cuda_failed();
  }
  if (!q || !k || !v || !gate || !W || !dy || !dq || !dk || !dv || !dgate) return M2RNN_ERR_NULL;
  if (params->gate_kind == M2RNN_GATE_PSI && (!alpha || !beta)) return M2RNN_ERR_NULL;
  const void *ptrs[] = {q, k, v, gate, W, h0, w_r, ckpt, dy, d_hT, dq, dk, dv, dgate, dW, dh0};
  for (const void *p : ptrs)
    if (!aligned16(p)) return M2RNN_ERR_ALIGN;
  const Workspace w = layout(params, ckpt != nullptr);
  if (w.total > 0 && (!workspace || workspace_bytes < w.total)) return M2RNN_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return M2RNN_ERR_ALIGN;
  char *ws = static_cast<char *>(workspace);

  ScanArgs a = base_args(params);
  a.q = q; a.k = k; a.v = v; a.gate = gate; a.W = W; a.h0 = h0; a.w_r = w_r;
  a.alpha = params->gate_kind == M2RNN_GATE_PSI ? alpha : nullptr;
  a.beta = params->gate_kind == M2RNN_GATE_PSI ? beta : nullptr;
  a.dev_status = dev_status;
  const bool f32 = params->io_dtype == M2RNN_F32;
  cudaError_t e = cudaSuccess;
  if (!ckpt) {
    // pass 1 of Algorithm 2, thinned: save the state every C steps only
    ScanArgs f = a;
    f.y = nullptr; f.hT = nullptr;
    f.ckpt = reinterpret_cast<float *>(ws + w.ckpt);
    e = f32 ? launch_fwd_f32(f, s) : launch_fwd_bf16(f, s);
    if (e != cudaSuccess) return cuda_failed();
    a.ckpt = f.ckpt;
  } else {
    a.ckpt = const_cast<float *>(ckpt);
  }
  a.dy = dy; a.d_hT = d_hT; a.dq = dq; a.dk = dk; a.dv = dv; a.dgate = dgate; a.dh0 = dh0;
  a.dW_part = reinterpret_cast<float *>(ws + w.dW_part);
  a.dq_part = params->Nq < params->N ? reinterpret_cast<float *>(ws + w.dq_part) : nullptr;
  a.dk_part = params->Nk < params->N ? reinterpret_cast<float *>(ws + w.dk_part) : nullptr;
  a.chunk_states = f32 ? reinterpret_cast<float *>(ws + w.chunk_states) : nullptr;
  const int RS = params->K / a.KC;
  a.dv_part = RS > 1 ? reinterpret_cast<float *>(ws + w.dv_part) : nullptr;
  a.dgate_part = RS > 1 ? reinterpret_cast<float *>(ws + w.dgate_part) : nullptr;
  e = f32 ? launch_bwd_f32(a, s)
          : (bwd_use_tc(params->B, params->N, params->K, params->V, params->io_dtype) ? launch_bwd_bf16_tc(a, s) : launch_bwd_bf16(a, s));
  if (e != cudaSuccess) return cuda_failed();
  e = launch_reduce_dW(a.dW_part, dW, params->B * RS, params->N, params->V, s);
  if (e != cudaSuccess) return cuda_failed();
  const size_t BT = tokens_of(params);
  if (RS > 1) {
    e = launch_reduce_slabs(a.dv_part, dv, params->io_dtype, RS, BT * params->N * params->V, s);
    if (e != cudaSuccess) return cuda_failed();
    e = launch_reduce_slabs(a.dgate_part, dgate, M2RNN_F32, RS, BT * params->N, s);
    if (e != cudaSuccess) return cuda_failed();
  }
  if (a.dq_part) {
    e = launch_reduce_heads(a.dq_part, dq, params->io_dtype, BT, params->N, params->Nq, params->K, s);
    if (e != cudaSuccess) return cuda_failed();
  }
  if (a.dk_part) {
    e = launch_reduce_heads(a.dk_part, dk, params->io_dtype, BT, params->N, params->Nk, params->K, s);
    if (e != cudaSuccess) return cuda_failed();
  }
  return M2RNN_OK;
}

int m2rnn_decode_step(const m2rnn_params *params, const void *q, const void *k, const void *v,
                      const float *gate, const void *W, const float *alpha, const float *beta,
                      const void *w_r, float *state, void *y, int32_t *dev_status, void *stream) {
  int rc = check_params(params, false);
  if (rc != M2RNN_OK) return rc;
  if (params->B == 0) return M2RNN_OK;
  if (!q || !k || !v || !gate || !W || !state || !y) return M2RNN_ERR_NULL;
  if (params->gate_kind == M2RNN_GATE_PSI && (!alpha || !beta)) return M2RNN_ERR_NULL;
  const void *ptrs[] = {q, k, v, gate, W, w_r, state, y};
  for (const void *p : ptrs)
    if (!aligned16(p)) return M2RNN_ERR_ALIGN;
  ScanArgs a = base_args(params);
  a.T = 1; a.nchunks = 1;
  a.q = q; a.k = k; a.v = v; a.gate = gate; a.W = W; a.w_r = w_r;
  a.alpha = params->gate_kind == M2RNN_GATE_PSI ? alpha : nullptr;
  a.beta = params->gate_kind == M2RNN_GATE_PSI ? beta : nullptr;
  a.h0 = state; a.hT = state; a.y = y; a.ckpt = nullptr; a.dev_status = dev_status;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // one step of Eq. 1-3: a T=1 scan whose initial and final state share storage (each CTA reads
  // its own slice of the state completely before it writes it back)
  cudaError_t e = params->io_dtype == M2RNN_F32 ? launch_fwd_f32(a, s) : launch_decode_bf16(a, s);
  return e == cudaSuccess ? M2RNN_OK : cuda_failed();
}

}  // extern "C"

// Internal declarations shared by the host API and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "m2rnn.h"

namespace m2rnn {

// Everything a kernel needs, by value.  Pointers are device pointers.
struct ScanArgs {
  int B, T, N, Nq, Nk, K, V;
  int gate_kind;
  int KC;         // bf16 backward: state rows per CTA (a divisor of K)
  int KCf;        // bf16 forward: state rows per CTA (a divisor of K)
  int C;          // checkpoint interval (steps)
  int nchunks;    // ceil(T / C)
  float dh_clip;
  const void *q, *k, *v, *W, *w_r;
  const float *gate, *h0, *alpha, *beta;
  void *y;
  float *y_part;  // bf16 forward, K/KCf > 1: [K/KCf][B,T,N,V] fp32 per-row-slab y, else null
  float *hT;
  float *ckpt;    // fwd: written (may be null); bwd: read
  // backward only
  const void *dy;
  const float *d_hT;
  void *dq, *dk, *dv;  // dq/dk: final tensors when the head is not shared, else see dq_part
  float *dgate, *dh0;
  float *dW_part;      // [B*K/KC,N,V,V] per-CTA partial sums of dW
  float *dv_part;      // [K/KC][B,T,N,V] fp32 per-row-slab dv when K/KC > 1, else null
  float *dgate_part;   // [K/KC][B,T,N] fp32 per-row-slab dgate when K/KC > 1, else null
  float *dq_part;      // [B,T,N,K] fp32 per-head dq when Nq < N, else null
  float *dk_part;      // [B,T,N,K] fp32 per-head dk when Nk < N, else null
  float *chunk_states; // fp32 path: [B*N, C, K, V] scratch for the recomputed states
  int32_t *dev_status;
  // token addressing: elements between consecutive tokens of q, k, v (dense: Nq K, Nk K, N V; larger
  // when they alias one fused projection output), the tokens in the batch (B T, or the packed total)
  // and, for packed variable-length batches, the device array of B + 1 token offsets
  long long qs, ks, vs;
  long long TT;
  const int32_t *cu;
};

// First token and length of batch entry b: a slice [cu[b], cu[b+1]) of a packed batch, else b T .. b T + T
struct UnitSpan { size_t tok0; int T; };
#ifdef __CUDACC__
__device__ __forceinline__ UnitSpan unit_span(const ScanArgs &a, int b) {
  if (a.cu) {   // lengths outside 0 .. T are cut to that range: nothing is addressed beyond what T sized
    const int s = a.cu[b], len = a.cu[b + 1] - s;
    return UnitSpan{(size_t)s, len < 0 ? 0 : (len > a.T ? a.T : len)};
  }
  return UnitSpan{(size_t)b * a.T, a.T};
}
#endif

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// How the backward pass splits a problem: state rows per CTA and the checkpoint interval (bounded
// by shared memory in the bf16 backward kernel, which keeps two chunks of recomputed states on chip).
struct BwdPlan {
  int KC;     // rows per CTA (== K on the fp32 path)
  int C;      // default checkpoint interval
  int C_max;  // largest supported checkpoint interval
};
int sm_count();   // SMs of the current device (148 when there is none to ask)
BwdPlan plan_bwd(int B, int N, int K, int V, int io_dtype);
int plan_fwd_rows(int B, int N, int K, int V, int io_dtype);   // state rows per CTA of the forward kernel
// Which bf16 forward kernel takes a problem: the tcgen05 kernel (scan_fwd_tc.cu) or the mma.sync
// kernels (scan_fwd_bf16*.cu).  The environment variable M2RNN_FWD_VARIANT = tc | mma | wide
// overrides the choice (benchmarking only).
bool fwd_use_tc(int B, int N, int K, int V, int io_dtype);
int fwd_tc_rows_per_cta(int B, int N, int K, int V);                 // scan_fwd_tc.cu: 32 or 64
cudaError_t launch_fwd_bf16_tc(const ScanArgs &a, cudaStream_t s);  // scan_fwd_tc.cu
size_t bwd_bf16_smem_bytes(int KC, int V, int C);  // scan_bwd_bf16.cu

// fp32 FMA path (scan_f32.cu)
cudaError_t launch_fwd_f32(const ScanArgs &a, cudaStream_t s);
cudaError_t launch_bwd_f32(const ScanArgs &a, cudaStream_t s);

// bf16 tensor-core path
cudaError_t launch_fwd_bf16(const ScanArgs &a, cudaStream_t s);     // scan_fwd_bf16.cu: picks a variant
bool fwd_cs_supported(const ScanArgs &a);                            // scan_fwd_bf16_cs.cu
cudaError_t launch_fwd_bf16_cs(const ScanArgs &a, cudaStream_t s);  // scan_fwd_bf16_cs.cu: two or four warps per 16-row slab
cudaError_t launch_bwd_bf16(const ScanArgs &a, cudaStream_t s);     // scan_bwd_bf16.cu
// The tcgen05 backward kernel (scan_bwd_tc.cu) takes V = 128; M2RNN_BWD_VARIANT = tc | mma overrides
// the choice (benchmarking only).
bool bwd_use_tc(int B, int N, int K, int V, int io_dtype);
int bwd_tc_rows_per_cta();
int bwd_tc_chunk();
cudaError_t launch_bwd_bf16_tc(const ScanArgs &a, cudaStream_t s);  // scan_bwd_tc.cu
cudaError_t launch_decode_bf16(const ScanArgs &a, cudaStream_t s);  // decode_bf16.cu: picks a kernel
bool decode_tc_supported(const ScanArgs &a);                         // decode_tc_bf16.cu
cudaError_t launch_decode_tc_bf16(const ScanArgs &a, cudaStream_t s);  // decode_tc_bf16.cu: tcgen05 path

// reductions shared by both paths (reduce.cu)
cudaError_t launch_reduce_dW(const float *dW_part, float *dW, int B, int N, int V, cudaStream_t s);
cudaError_t launch_reduce_slabs(const float *part, void *out, int io_dtype, int R, size_t n, cudaStream_t s);
cudaError_t launch_reduce_heads(const float *part, void *out, int io_dtype, size_t BT, int N,
                                int Ng, int K, cudaStream_t s);

}  // namespace m2rnn

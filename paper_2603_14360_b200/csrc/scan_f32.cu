// fp32 FMA path of the M2RNN scan (forward, decode step, backward through time).
//
// One CTA per (b,n).  The K x V state is spread over K*TPR threads: thread (i,c) owns row i
// and the columns {(jj*TPR + c)*4 + e}; a row's TPR threads sit in one warp, so the
// row-by-W product (Eq. 1) only needs warp-level synchronisation through shared memory.
// Everything is plain fp32 FMA with tanhf/expf: this is the accuracy path (<= 1e-4).
#include "device_common.cuh"
#include "internal.h"

namespace m2rnn {
namespace {

constexpr int kPad = 4;  // row pitch V+4 floats: rows land on different banks

__device__ __forceinline__ int col_of(int jj, int c, int TPR) { return (jj * TPR + c) * 4; }

// Z row-segment = tanh( sum_l H[i][l] W[l][cols] + k_i v[cols] )   (Eq. 1)
template <int NJ4>
__device__ __forceinline__ void transition(const float *__restrict__ Hrow, const float *__restrict__ Ws,
                                           int V, int HP, int c, int TPR, float k_i,
                                           const float4 (&v4)[NJ4], float (&z)[NJ4 * 4]) {
  float acc[NJ4 * 4];
#pragma unroll
  for (int jj = 0; jj < NJ4; ++jj) {
    acc[jj * 4 + 0] = k_i * v4[jj].x;
    acc[jj * 4 + 1] = k_i * v4[jj].y;
    acc[jj * 4 + 2] = k_i * v4[jj].z;
    acc[jj * 4 + 3] = k_i * v4[jj].w;
  }
  for (int l = 0; l < V; l += 4) {
    const float4 h4 = *reinterpret_cast<const float4 *>(Hrow + l);
    const float hv[4] = {h4.x, h4.y, h4.z, h4.w};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
#pragma unroll
      for (int jj = 0; jj < NJ4; ++jj) {
        const float4 w4 = *reinterpret_cast<const float4 *>(Ws + (l + u) * HP + col_of(jj, c, TPR));
        acc[jj * 4 + 0] = fmaf(hv[u], w4.x, acc[jj * 4 + 0]);
        acc[jj * 4 + 1] = fmaf(hv[u], w4.y, acc[jj * 4 + 1]);
        acc[jj * 4 + 2] = fmaf(hv[u], w4.z, acc[jj * 4 + 2]);
        acc[jj * 4 + 3] = fmaf(hv[u], w4.w, acc[jj * 4 + 3]);
      }
    }
  }
#pragma unroll
  for (int x = 0; x < NJ4 * 4; ++x) z[x] = tanhf(acc[x]);
}

template <int NJ4>
__device__ __forceinline__ void load_cols(const float *__restrict__ base, int c, int TPR, float4 (&out)[NJ4]) {
#pragma unroll
  for (int jj = 0; jj < NJ4; ++jj) out[jj] = *reinterpret_cast<const float4 *>(base + col_of(jj, c, TPR));
}

template <int NJ4>
__device__ __forceinline__ void store_cols(float *__restrict__ base, int c, int TPR, const float (&h)[NJ4 * 4]) {
#pragma unroll
  for (int jj = 0; jj < NJ4; ++jj)
    *reinterpret_cast<float4 *>(base + col_of(jj, c, TPR)) =
        make_float4(h[jj * 4], h[jj * 4 + 1], h[jj * 4 + 2], h[jj * 4 + 3]);
}

// ------------------------------------------------------------------ forward (Algorithm 1)
template <int NJ4>
__global__ void __launch_bounds__(1024) fwd_f32_kernel(ScanArgs a, int TPR) {
  extern __shared__ __align__(16) float smem[];
  const int K = a.K, V = a.V, N = a.N, HP = V + kPad;
  const int tid = threadIdx.x, nthreads = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const int nwarps = nthreads >> 5;
  const int i = tid / TPR, c = tid % TPR;
  const int bn = blockIdx.x, b = bn / N, n = bn % N;
  const UnitSpan span = unit_span(a, b);   // this batch entry's tokens (a slice of a packed batch, or b T ..)
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int hq = n / (N / a.Nq), hk = n / (N / a.Nk);

  float *Ws = smem;                    // [V][HP]
  float *Hs = Ws + V * HP;             // [K][HP]
  float *ypart = Hs + K * HP;          // [2][nwarps][V]

  const float *Wg = static_cast<const float *>(a.W) + (size_t)n * V * V;
  for (int x = tid; x < V * V; x += nthreads) Ws[(x / V) * HP + (x % V)] = Wg[x];

  const size_t KV = (size_t)K * V;
  float h[NJ4 * 4];
  if (a.h0) {
    float4 t4[NJ4];
    load_cols<NJ4>(a.h0 + bn * KV + (size_t)i * V, c, TPR, t4);
#pragma unroll
    for (int jj = 0; jj < NJ4; ++jj) { h[jj * 4] = t4[jj].x; h[jj * 4 + 1] = t4[jj].y; h[jj * 4 + 2] = t4[jj].z; h[jj * 4 + 3] = t4[jj].w; }
  } else {
#pragma unroll
    for (int x = 0; x < NJ4 * 4; ++x) h[x] = 0.f;
  }
  const float al = a.alpha ? a.alpha[n] : 1.f, be = a.beta ? a.beta[n] : 0.f;
  const float *qg = static_cast<const float *>(a.q), *kg = static_cast<const float *>(a.k);
  const float *vg = static_cast<const float *>(a.v), *wr = static_cast<const float *>(a.w_r);
  float *yg = static_cast<float *>(a.y);
  __syncthreads();

  for (int t = 0; t < T; ++t) {
    const size_t bt = tok0 + t;
    if (a.ckpt && (t % a.C) == 0)
      store_cols<NJ4>(a.ckpt + ((size_t)bn * a.nchunks + t / a.C) * KV + (size_t)i * V, c, TPR, h);
    const float k_i = kg[bt * a.ks + hk * K + i];
    const float q_i = qg[bt * a.qs + hq * K + i];
    const float f = gate_value(a.gate_kind, a.gate[bt * N + n], al, be, nullptr);
    float4 v4[NJ4];
    load_cols<NJ4>(vg + bt * a.vs + n * V, c, TPR, v4);

    store_cols<NJ4>(Hs + i * HP, c, TPR, h);
    __syncwarp();
    float z[NJ4 * 4];
    transition<NJ4>(Hs + i * HP, Ws, V, HP, c, TPR, k_i, v4, z);
    __syncwarp();
#pragma unroll
    for (int x = 0; x < NJ4 * 4; ++x) h[x] = f * h[x] + (1.f - f) * z[x];  // Eq. 2
    if (!yg) continue;  // checkpoint-only pass (first pass of the backward call)
    // readout partial q_i * H_t[i][cols] summed over the warp's rows (Eq. 3)
    float *yp = ypart + ((t & 1) * nwarps + warp) * V;
#pragma unroll
    for (int x = 0; x < NJ4 * 4; ++x) {
      float yv = q_i * h[x];
      for (int off = TPR; off < 32; off <<= 1) yv += __shfl_xor_sync(0xffffffffu, yv, off);
      if (lane < TPR) yp[col_of(x >> 2, c, TPR) + (x & 3)] = yv;
    }
    __syncthreads();
    if (tid < V) {
      float s = 0.f;
      for (int w = 0; w < nwarps; ++w) s += ypart[((t & 1) * nwarps + w) * V + tid];
      if (wr) s += wr[(size_t)n * V + tid] * vg[bt * a.vs + n * V + tid];
      yg[(bt * N + n) * V + tid] = s;
    }
  }
  if (a.hT) store_cols<NJ4>(a.hT + bn * KV + (size_t)i * V, c, TPR, h);
}

// ------------------------------------------------------------------ backward (Algorithm 2)
template <int NJ4>
__global__ void __launch_bounds__(1024) bwd_f32_kernel(ScanArgs a, int TPR) {
  extern __shared__ __align__(16) float smem[];
  const int K = a.K, V = a.V, N = a.N, HP = V + kPad;
  const int tid = threadIdx.x, nthreads = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const int nwarps = nthreads >> 5;
  const int i = tid / TPR, c = tid % TPR;
  const int bn = blockIdx.x, b = bn / N, n = bn % N;
  const UnitSpan span = unit_span(a, b);   // this batch entry's tokens (a slice of a packed batch, or b T ..)
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int hq = n / (N / a.Nq), hk = n / (N / a.Nk);

  float *Ws = smem;                 // [V][HP]
  float *Hs = Ws + V * HP;          // [K][HP]  H_{t-1}
  float *Xs = Hs + K * HP;          // [K][HP]  dX_t
  float *dvpart = Xs + K * HP;      // [nwarps][V]
  float *red = dvpart + nwarps * V; // [nwarps]

  const float *Wg = static_cast<const float *>(a.W) + (size_t)n * V * V;
  for (int x = tid; x < V * V; x += nthreads) Ws[(x / V) * HP + (x % V)] = Wg[x];

  const size_t KV = (size_t)K * V;
  const float al = a.alpha ? a.alpha[n] : 1.f, be = a.beta ? a.beta[n] : 0.f;
  const float *qg = static_cast<const float *>(a.q), *kg = static_cast<const float *>(a.k);
  const float *vg = static_cast<const float *>(a.v), *wr = static_cast<const float *>(a.w_r);
  const float *dyg = static_cast<const float *>(a.dy);
  float *scratch = a.chunk_states + (size_t)bn * a.C * KV;

  float Cg[NJ4 * 4];  // carried dL/dH_t, this thread's segment
  if (a.d_hT) {
    float4 t4[NJ4];
    load_cols<NJ4>(a.d_hT + bn * KV + (size_t)i * V, c, TPR, t4);
#pragma unroll
    for (int jj = 0; jj < NJ4; ++jj) { Cg[jj * 4] = t4[jj].x; Cg[jj * 4 + 1] = t4[jj].y; Cg[jj * 4 + 2] = t4[jj].z; Cg[jj * 4 + 3] = t4[jj].w; }
  } else {
#pragma unroll
    for (int x = 0; x < NJ4 * 4; ++x) Cg[x] = 0.f;
  }
  // dW[l][j4..j4+3] accumulators: float4 slot d = l*(V/4) + j4/4, strided over the CTA
  constexpr int kMaxDW = 8;
  float4 dWacc[kMaxDW];
#pragma unroll
  for (int x = 0; x < kMaxDW; ++x) dWacc[x] = make_float4(0.f, 0.f, 0.f, 0.f);
  const int ndw = V * V / 4;
  __syncthreads();

  for (int ch = (T + a.C - 1) / a.C - 1; ch >= 0; --ch) {   // this unit's chunks; a.nchunks is the checkpoint tensor's extent
    const int t0 = ch * a.C, len = min(a.C, T - t0);
    // pass 1 for this chunk: states H_{t0} .. H_{t0+len-1}, each the H_{t-1} of one step
    float h[NJ4 * 4];
    {
      float4 t4[NJ4];
      load_cols<NJ4>(a.ckpt + ((size_t)bn * a.nchunks + ch) * KV + (size_t)i * V, c, TPR, t4);
#pragma unroll
      for (int jj = 0; jj < NJ4; ++jj) { h[jj * 4] = t4[jj].x; h[jj * 4 + 1] = t4[jj].y; h[jj * 4 + 2] = t4[jj].z; h[jj * 4 + 3] = t4[jj].w; }
    }
    for (int s = 0; s < len; ++s) {
      store_cols<NJ4>(scratch + (size_t)s * KV + (size_t)i * V, c, TPR, h);
      if (s == len - 1) break;
      const size_t bt = tok0 + t0 + s;
      const float k_i = kg[bt * a.ks + hk * K + i];
      const float f = gate_value(a.gate_kind, a.gate[bt * N + n], al, be, nullptr);
      float4 v4[NJ4];
      load_cols<NJ4>(vg + bt * a.vs + n * V, c, TPR, v4);
      store_cols<NJ4>(Hs + i * HP, c, TPR, h);
      __syncwarp();
      float z[NJ4 * 4];
      transition<NJ4>(Hs + i * HP, Ws, V, HP, c, TPR, k_i, v4, z);
      __syncwarp();
#pragma unroll
      for (int x = 0; x < NJ4 * 4; ++x) h[x] = f * h[x] + (1.f - f) * z[x];
    }
    __syncthreads();
    // pass 2: reverse sweep over the chunk
    for (int s = len - 1; s >= 0; --s) {
      const size_t bt = tok0 + t0 + s;
      const float k_i = kg[bt * a.ks + hk * K + i];
      const float q_i = qg[bt * a.qs + hq * K + i];
      float dfdx;
      const float f = gate_value(a.gate_kind, a.gate[bt * N + n], al, be, &dfdx);
      float4 v4[NJ4], dy4[NJ4], hp4[NJ4];
      load_cols<NJ4>(vg + bt * a.vs + n * V, c, TPR, v4);
      load_cols<NJ4>(dyg + (bt * N + n) * V, c, TPR, dy4);
      load_cols<NJ4>(scratch + (size_t)s * KV + (size_t)i * V, c, TPR, hp4);
      float hp[NJ4 * 4], vv[NJ4 * 4], dyv[NJ4 * 4];
#pragma unroll
      for (int jj = 0; jj < NJ4; ++jj) {
        hp[jj * 4] = hp4[jj].x; hp[jj * 4 + 1] = hp4[jj].y; hp[jj * 4 + 2] = hp4[jj].z; hp[jj * 4 + 3] = hp4[jj].w;
        vv[jj * 4] = v4[jj].x; vv[jj * 4 + 1] = v4[jj].y; vv[jj * 4 + 2] = v4[jj].z; vv[jj * 4 + 3] = v4[jj].w;
        dyv[jj * 4] = dy4[jj].x; dyv[jj * 4 + 1] = dy4[jj].y; dyv[jj * 4 + 2] = dy4[jj].z; dyv[jj * 4 + 3] = dy4[jj].w;
      }
      store_cols<NJ4>(Hs + i * HP, c, TPR, hp);
      __syncwarp();
      float z[NJ4 * 4];
      transition<NJ4>(Hs + i * HP, Ws, V, HP, c, TPR, k_i, v4, z);

      float G[NJ4 * 4], dX[NJ4 * 4];
      float dq_i = 0.f, dk_i = 0.f, df = 0.f;
#pragma unroll
      for (int x = 0; x < NJ4 * 4; ++x) {
        const float ht = f * hp[x] + (1.f - f) * z[x];   // H_t
        G[x] = Cg[x] + q_i * dyv[x];                     // G = C + q dy^T
        dq_i = fmaf(ht, dyv[x], dq_i);                   // dq = H_t dy
        df = fmaf(G[x], hp[x] - z[x], df);               // df = sum G (.) (H_{t-1} - Z)
        dX[x] = (1.f - f) * G[x] * (1.f - z[x] * z[x]);  // through the gate and tanh
        dk_i = fmaf(dX[x], vv[x], dk_i);                 // dk = dX v
      }
      store_cols<NJ4>(Xs + i * HP, c, TPR, dX);
      for (int off = 1; off < TPR; off <<= 1) {
        dq_i += __shfl_xor_sync(0xffffffffu, dq_i, off);
        dk_i += __shfl_xor_sync(0xffffffffu, dk_i, off);
      }
      for (int off = 1; off < 32; off <<= 1) df += __shfl_xor_sync(0xffffffffu, df, off);
      if (c == 0) {
        if (a.dq_part) a.dq_part[(bt * N + n) * K + i] = dq_i;
        else static_cast<float *>(a.dq)[(bt * a.Nq + hq) * K + i] = dq_i;
        if (a.dk_part) a.dk_part[(bt * N + n) * K + i] = dk_i;
        else static_cast<float *>(a.dk)[(bt * a.Nk + hk) * K + i] = dk_i;
      }
      if (lane == 0) red[warp] = df;
      // dv partial: sum over the warp's rows of dX[i][col] * k_i
#pragma unroll
      for (int x = 0; x < NJ4 * 4; ++x) {
        float dvv = dX[x] * k_i;
        for (int off = TPR; off < 32; off <<= 1) dvv += __shfl_xor_sync(0xffffffffu, dvv, off);
        if (lane < TPR) dvpart[warp * V + col_of(x >> 2, c, TPR) + (x & 3)] = dvv;
      }
      __syncthreads();  // Hs, Xs, dvpart, red complete for every row

      // C_{t-1}[i][l] = f G[i][l] + sum_j dX[i][j] W[l][j]
      float Cn[NJ4 * 4];
#pragma unroll
      for (int x = 0; x < NJ4 * 4; ++x) Cn[x] = f * G[x];
      for (int j = 0; j < V; j += 4) {
        const float4 x4 = *reinterpret_cast<const float4 *>(Xs + i * HP + j);
#pragma unroll
        for (int x = 0; x < NJ4 * 4; ++x) {
          const int l = col_of(x >> 2, c, TPR) + (x & 3);
          const float4 w4 = *reinterpret_cast<const float4 *>(Ws + l * HP + j);
          Cn[x] = fmaf(x4.x, w4.x, Cn[x]);
          Cn[x] = fmaf(x4.y, w4.y, Cn[x]);
          Cn[x] = fmaf(x4.z, w4.z, Cn[x]);
          Cn[x] = fmaf(x4.w, w4.w, Cn[x]);
        }
      }
#pragma unroll
      for (int x = 0; x < NJ4 * 4; ++x) {
        float cv = Cn[x];
        if (a.dh_clip > 0.f) cv = fminf(fmaxf(cv, -a.dh_clip), a.dh_clip);
        Cg[x] = cv;
      }
      // dW += H_{t-1}^T dX
#pragma unroll
      for (int x = 0; x < kMaxDW; ++x) {
        const int d = tid + x * nthreads;
        if (d < ndw) {
          const int l = d / (V / 4), j = (d % (V / 4)) * 4;
          float4 acc = dWacc[x];
          for (int r = 0; r < K; ++r) {
            const float hv = Hs[r * HP + l];
            const float4 x4 = *reinterpret_cast<const float4 *>(Xs + r * HP + j);
            acc.x = fmaf(hv, x4.x, acc.x);
            acc.y = fmaf(hv, x4.y, acc.y);
            acc.z = fmaf(hv, x4.z, acc.z);
            acc.w = fmaf(hv, x4.w, acc.w);
          }
          dWacc[x] = acc;
        }
      }
      if (tid < V) {
        float sdv = 0.f;
        for (int w = 0; w < nwarps; ++w) sdv += dvpart[w * V + tid];
        if (wr) sdv += wr[(size_t)n * V + tid] * dyg[(bt * N + n) * V + tid];
        static_cast<float *>(a.dv)[(bt * N + n) * V + tid] = sdv;
      }
      if (tid == 0) {
        float sdf = 0.f;
        for (int w = 0; w < nwarps; ++w) sdf += red[w];
        a.dgate[bt * N + n] = sdf * dfdx;
      }
      __syncthreads();  // before Hs / Xs / dvpart / red are overwritten
    }
  }
  if (a.dh0) store_cols<NJ4>(a.dh0 + bn * KV + (size_t)i * V, c, TPR, Cg);
  float *dWp = a.dW_part + (size_t)bn * V * V;
#pragma unroll
  for (int x = 0; x < kMaxDW; ++x) {
    const int d = tid + x * nthreads;
    if (d < ndw) *reinterpret_cast<float4 *>(dWp + (size_t)d * 4) = dWacc[x];
  }
}

int pick_tpr(int K, int V) {
  int tpr = 32;
  while (tpr > V / 4 || tpr * K > 1024) tpr >>= 1;
  return tpr;
}

}  // namespace

cudaError_t launch_fwd_f32(const ScanArgs &a, cudaStream_t s) {
  const int TPR = pick_tpr(a.K, a.V), nthreads = a.K * TPR, nj4 = a.V / TPR / 4, HP = a.V + kPad;
  const size_t smem = sizeof(float) * ((size_t)a.V * HP + (size_t)a.K * HP + 2 * (nthreads / 32) * a.V);
  auto kern = nj4 == 1 ? fwd_f32_kernel<1> : nj4 == 2 ? fwd_f32_kernel<2> : fwd_f32_kernel<4>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<a.B * a.N, nthreads, smem, s>>>(a, TPR);
  return cudaGetLastError();
}

cudaError_t launch_bwd_f32(const ScanArgs &a, cudaStream_t s) {
  const int TPR = pick_tpr(a.K, a.V), nthreads = a.K * TPR, nj4 = a.V / TPR / 4, HP = a.V + kPad;
  const int nwarps = nthreads / 32;
  const size_t smem = sizeof(float) * ((size_t)a.V * HP + 2 * (size_t)a.K * HP + (size_t)nwarps * a.V + nwarps);
  auto kern = nj4 == 1 ? bwd_f32_kernel<1> : nj4 == 2 ? bwd_f32_kernel<2> : bwd_f32_kernel<4>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<a.B * a.N, nthreads, smem, s>>>(a, TPR);
  return cudaGetLastError();
}

}  // namespace m2rnn

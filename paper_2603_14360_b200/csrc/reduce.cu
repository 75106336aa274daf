// Second-stage reductions of the backward pass, in a fixed order so results repeat bit for bit
// (the paper's Algorithm 2 uses atomic adds for these sums).
#include "device_common.cuh"
#include "internal.h"

namespace m2rnn {
namespace {

// dW[n] = sum_b dW_part[b][n]   (Algorithm 2 sums dW over the batch with an atomic add)
__global__ void reduce_dW_kernel(const float *__restrict__ part, float *__restrict__ dW, int B, size_t NVV) {
  const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= NVV) return;
  float s = 0.f;
  for (int b = 0; b < B; ++b) s += part[(size_t)b * NVV + x];
  dW[x] = s;
}

// out[bt][g][:] = sum over the heads n of group g of part[bt][n][:]
// (Algorithm 2 sums dq and dk over the heads that share them with atomic adds)
template <typename TIO>
__global__ void reduce_heads_kernel(const float *__restrict__ part, TIO *__restrict__ out, size_t BT,
                                    int N, int Ng, int K) {
  const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t total = BT * Ng * K;
  if (x >= total) return;
  const int i = (int)(x % K);
  const int g = (int)((x / K) % Ng);
  const size_t bt = x / ((size_t)K * Ng);
  const int per = N / Ng;
  float s = 0.f;
  for (int h = 0; h < per; ++h) s += part[(bt * N + (size_t)g * per + h) * K + i];
  out[x] = from_f32<TIO>(s);
}

// out[x] = sum_r part[r][x]: sums over the row slabs of a state that were handled by different CTAs
// (dv and dgate are sums over all K rows)
template <typename TIO>
__global__ void reduce_slabs_kernel(const float *__restrict__ part, TIO *__restrict__ out, int R, size_t n) {
  const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (x >= n) return;
  float s = 0.f;
  for (int r = 0; r < R; ++r) s += part[(size_t)r * n + x];
  out[x] = from_f32<TIO>(s);
}

}  // namespace

cudaError_t launch_reduce_slabs(const float *part, void *out, int io_dtype, int R, size_t n, cudaStream_t s) {
  const unsigned grid = (unsigned)((n + 255) / 256);
  if (io_dtype == M2RNN_F32)
    reduce_slabs_kernel<float><<<grid, 256, 0, s>>>(part, static_cast<float *>(out), R, n);
  else
    reduce_slabs_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(part, static_cast<__nv_bfloat16 *>(out), R, n);
  return cudaGetLastError();
}

cudaError_t launch_reduce_dW(const float *dW_part, float *dW, int B, int N, int V, cudaStream_t s) {
  const size_t NVV = (size_t)N * V * V;
  reduce_dW_kernel<<<(unsigned)((NVV + 255) / 256), 256, 0, s>>>(dW_part, dW, B, NVV);
  return cudaGetLastError();
}

cudaError_t launch_reduce_heads(const float *part, void *out, int io_dtype, size_t BT, int N, int Ng,
                                int K, cudaStream_t s) {
  const size_t total = BT * Ng * K;
  const unsigned grid = (unsigned)((total + 255) / 256);
  if (io_dtype == M2RNN_F32)
    reduce_heads_kernel<float><<<grid, 256, 0, s>>>(part, static_cast<float *>(out), BT, N, Ng, K);
  else
    reduce_heads_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(part, static_cast<__nv_bfloat16 *>(out), BT, N, Ng, K);
  return cudaGetLastError();
}

}  // namespace m2rnn

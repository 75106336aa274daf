// Output path of the layer after the scan ("M2RNN block" equations: y_gt = RMSNorm(y_t (.) g_t),
// g_t = SiLU of the gate projection; RMSNorm appendix for the formulas and their backward), fused
// into one pass each way: y and g are read once, the normalised product is written once, the
// product y (.) g never goes to memory.  Per token over the d = N V features of all heads:
//     x = y (.) g,   s = 1 / sqrt(mean x^2 + eps),   out = w (.) x s            (s is cached)
//     p = w (.) dout, r = sum p x, dx = s p - r s^3 x / d, dy = dx (.) g, dg = dx (.) y (SiLU'),
//     dw = sum over tokens of dout (.) x s.
// HBM-bound.  One warp per token (tokens are plentiful and a row is 2-16 KB), 16-byte loads and
// stores.  Forward: for the common row lengths (d = 256 x 1, 2, 4, 8) a lane keeps its share of the
// product in registers between the reduction and the scaling; other lengths walk the row twice
// and the second walk is served by the L1.  No shared memory limits the resident warps there.
// (A variant that streamed blocks of rows through a shared-memory ring with bulk copies and eight
// compute warps per SM was slower: the sigmoid makes the row work latency-bound and needs the
// warps.)  dw: per-warp accumulators in shared memory, one partial per CTA, then a fixed-order
// second stage.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "internal.h"
#include "m2rnn.h"

namespace m2rnn {
namespace {

constexpr int kFwdWarps = 8;
constexpr int kMaxCtas = 592;   // 4 per SM on 148 SMs: also the number of dw partials at most
constexpr int kMaxD = 8192;
constexpr int kBwdSmemBudget = 48 * 1024;   // per-warp dw accumulators of a CTA

// 8 consecutive elements as floats
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&f)[8]) {
  const uint4 r = *reinterpret_cast<const uint4 *>(p);
  const uint32_t u[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(u[i] << 16); f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
}
__device__ __forceinline__ void load8(const float *p, float (&f)[8]) {
  const float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ void store8(__nv_bfloat16 *p, const float (&f)[8]) {
  *reinterpret_cast<uint4 *>(p) = make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
}
__device__ __forceinline__ void store8(float *p, const float (&f)[8]) {
  *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]);
  *reinterpret_cast<float4 *>(p + 4) = make_float4(f[4], f[5], f[6], f[7]);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// SiLU and its derivative.  fp32 I/O: sigmoid through ex2.approx + rcp.approx (~1e-6 relative);
// bf16 I/O: through one tanh.approx (~2^-11, below the rounding of the bf16 result) -- the kernels
// are bound by the special-function unit as much as by HBM, and this halves its work
template <typename T>
__device__ __forceinline__ float silu_t(float x, float *dx) {
  float sg;
  if constexpr (sizeof(T) == 2) {
    float th;
    asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * x));
    sg = fmaf(0.5f, th, 0.5f);
  } else {
    sg = __fdividef(1.f, 1.f + __expf(-x));
  }
  if (dx) *dx = sg * (1.f + x * (1.f - sg));
  return x * sg;
}

// CPL > 0: d = 256 CPL, every lane owns CPL chunks and keeps their products in registers.
// CPL = 0: any d, the row is read twice.
template <typename T, int CPL>
__global__ void __launch_bounds__(kFwdWarps * 32) gated_norm_fwd_kernel(long tokens, int d, const T *__restrict__ y,
                                                                          const T *__restrict__ g_in, const T *__restrict__ w,
                                                                          float eps, int use_silu, T *__restrict__ out,
                                                                          float *__restrict__ rstd) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = d >> 3;
  for (long t = (long)blockIdx.x * kFwdWarps + warp; t < tokens; t += (long)gridDim.x * kFwdWarps) {
    const T *yt = y + t * d, *gt = g_in + t * d;
    float ss = 0.f;
    if constexpr (CPL > 0) {
      float x[CPL][8];
      {
        float a[CPL][8], b[CPL][8];
#pragma unroll
        for (int j = 0; j < CPL; ++j) { load8(yt + 8 * (lane + 32 * j), a[j]); load8(gt + 8 * (lane + 32 * j), b[j]); }
#pragma unroll
        for (int j = 0; j < CPL; ++j)
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            x[j][e] = a[j][e] * (use_silu ? silu_t<T>(b[j][e], nullptr) : b[j][e]);
            ss = fmaf(x[j][e], x[j][e], ss);
          }
      }
      ss = warp_sum(ss);
      const float s = 1.f / sqrtf(ss / (float)d + eps);
#pragma unroll
      for (int j = 0; j < CPL; ++j) {
        float wv[8], o[8];
        load8(w + 8 * (lane + 32 * j), wv);
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = wv[e] * x[j][e] * s;
        store8(out + t * d + 8 * (lane + 32 * j), o);
      }
      if (rstd && lane == 0) rstd[t] = s;
    } else {
#pragma unroll 4
      for (int c = lane; c < chunks; c += 32) {
        float a[8], b[8];
        load8(yt + 8 * c, a);
        load8(gt + 8 * c, b);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x = a[e] * (use_silu ? silu_t<T>(b[e], nullptr) : b[e]);
          ss = fmaf(x, x, ss);
        }
      }
      ss = warp_sum(ss);
      const float s = 1.f / sqrtf(ss / (float)d + eps);
#pragma unroll 4
      for (int c = lane; c < chunks; c += 32) {   // the same lane reads the same bytes again: L1 hits
        float a[8], b[8], wv[8], o[8];
        load8(yt + 8 * c, a);
        load8(gt + 8 * c, b);
        load8(w + 8 * c, wv);
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] = wv[e] * (a[e] * (use_silu ? silu_t<T>(b[e], nullptr) : b[e])) * s;
        store8(out + t * d + 8 * c, o);
      }
      if (rstd && lane == 0) rstd[t] = s;
    }
  }
}

template <typename T, int kWarps>
__global__ void __launch_bounds__(kWarps * 32) gated_norm_bwd_kernel(long tokens, int d, const T *__restrict__ y,
                                                                       const T *__restrict__ g_in, const T *__restrict__ w,
                                                                       const float *__restrict__ rstd, int use_silu,
                                                                       const T *__restrict__ dout, T *__restrict__ dy,
                                                                       T *__restrict__ dg_in, float *__restrict__ dw_part) {
  extern __shared__ __align__(16) float acc_all[];   // [kWarps][d] partial sums of dw
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float *acc = acc_all + (size_t)warp * d;
  const int chunks = d >> 3;
  for (int c = lane; c < chunks; c += 32) {
    *reinterpret_cast<float4 *>(acc + 8 * c) = make_float4(0.f, 0.f, 0.f, 0.f);
    *reinterpret_cast<float4 *>(acc + 8 * c + 4) = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (long t = (long)blockIdx.x * kWarps + warp; t < tokens; t += (long)gridDim.x * kWarps) {
    const T *yt = y + t * d, *gt = g_in + t * d, *dot = dout + t * d;
    const float s = rstd[t];
    // r = sum_j w_j dout_j x_j
    float r = 0.f;
#pragma unroll 2
    for (int c = lane; c < chunks; c += 32) {
      float a[8], b[8], wv[8], dv[8];
      load8(yt + 8 * c, a);
      load8(gt + 8 * c, b);
      load8(w + 8 * c, wv);
      load8(dot + 8 * c, dv);
#pragma unroll
      for (int e = 0; e < 8; ++e) r = fmaf(wv[e] * dv[e], a[e] * (use_silu ? silu_t<T>(b[e], nullptr) : b[e]), r);
    }
    r = warp_sum(r);
    const float k3 = r * s * s * s / (float)d;
    // second pass over the same row (served by the L1): the gradients
#pragma unroll 2
    for (int c = lane; c < chunks; c += 32) {
      float a[8], b[8], wv[8], dv[8], o1[8], o2[8];
      load8(yt + 8 * c, a);
      load8(gt + 8 * c, b);
      load8(w + 8 * c, wv);
      load8(dot + 8 * c, dv);
      float4 w0 = *reinterpret_cast<const float4 *>(acc + 8 * c), w1 = *reinterpret_cast<const float4 *>(acc + 8 * c + 4);
      float aw[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float dsl = 1.f;
        const float g = use_silu ? silu_t<T>(b[e], &dsl) : b[e];
        const float x = a[e] * g;
        const float dx = s * wv[e] * dv[e] - k3 * x;
        o1[e] = dx * g;
        o2[e] = dx * a[e] * dsl;
        aw[e] = fmaf(dv[e] * x, s, aw[e]);
      }
      store8(dy + t * d + 8 * c, o1);
      store8(dg_in + t * d + 8 * c, o2);
      *reinterpret_cast<float4 *>(acc + 8 * c) = make_float4(aw[0], aw[1], aw[2], aw[3]);
      *reinterpret_cast<float4 *>(acc + 8 * c + 4) = make_float4(aw[4], aw[5], aw[6], aw[7]);
    }
  }
  __syncthreads();
  // this CTA's partial of dw: the warps' sums in a fixed order
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float v = 0.f;
#pragma unroll
    for (int wi = 0; wi < kWarps; ++wi) v += acc_all[(size_t)wi * d + j];
    dw_part[(size_t)blockIdx.x * d + j] = v;
  }
}

// The same for d = 256 CPL (CPL = 1, 2, 4): a lane owns CPL fixed chunks of every row, keeps the
// row's inputs in registers as loaded (16 bytes per chunk and tensor for bf16) between the
// reduction and the gradients, and sums its columns of dw in registers over all its tokens.
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 v;
  __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = *reinterpret_cast<const uint4 *>(p); }
  __device__ __forceinline__ void get(float (&f)[8]) const {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(u[i] << 16); f[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u); }
  }
};
template <> struct Raw8<float> {
  float4 lo, hi;
  __device__ __forceinline__ void load(const float *p) { lo = *reinterpret_cast<const float4 *>(p); hi = *reinterpret_cast<const float4 *>(p + 4); }
  __device__ __forceinline__ void get(float (&f)[8]) const {
    f[0] = lo.x; f[1] = lo.y; f[2] = lo.z; f[3] = lo.w; f[4] = hi.x; f[5] = hi.y; f[6] = hi.z; f[7] = hi.w;
  }
};

constexpr int kRegWarps = 8;

template <typename T, int CPL>
__global__ void __launch_bounds__(kRegWarps * 32) gated_norm_bwd_reg_kernel(long tokens, const T *__restrict__ y,
                                                                              const T *__restrict__ g_in, const T *__restrict__ w,
                                                                              const float *__restrict__ rstd, int use_silu,
                                                                              const T *__restrict__ dout, T *__restrict__ dy,
                                                                              T *__restrict__ dg_in, float *__restrict__ dw_part) {
  constexpr int d = 256 * CPL;
  extern __shared__ __align__(16) float acc_all[];   // [kRegWarps][d]: the warps' sums at the end
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  Raw8<T> wr[CPL];
  float acc[CPL][8];
#pragma unroll
  for (int j = 0; j < CPL; ++j) {
    wr[j].load(w + 8 * (lane + 32 * j));
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;
  }
  // bf16: the next token's three rows are on their way (cp.async into a two-slot ring of the warp, a
  // lane copies and later reads its own chunks only) while this token is worked on; without that a
  // warp's loads and its arithmetic took turns and the kernel ran at half of the HBM bandwidth
  constexpr bool kRing = sizeof(T) == 2;
  const long t_first = (long)blockIdx.x * kRegWarps + warp, t_step = (long)gridDim.x * kRegWarps;
  uint4 *ring = reinterpret_cast<uint4 *>(acc_all + (size_t)kRegWarps * d) + (size_t)warp * (2 * 3 * CPL * 32);
  auto fetch = [&](long t, int slot) {   // always one group, possibly empty
    if (t < tokens) {
      const T *src[3] = {y + t * d, g_in + t * d, dout + t * d};
#pragma unroll
      for (int x = 0; x < 3; ++x)
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
          const uint32_t dst = (uint32_t)__cvta_generic_to_shared(ring + ((slot * 3 + x) * CPL + j) * 32 + lane);
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src[x] + 8 * (lane + 32 * j)) : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  if constexpr (kRing) fetch(t_first, 0);
  int slot = 0;
  for (long t = t_first; t < tokens; t += t_step) {
    const T *yt = y + t * d, *gt = g_in + t * d, *dot = dout + t * d;
    Raw8<T> ar[CPL], br[CPL], dr[CPL];
    if constexpr (kRing) {
      fetch(t + t_step, slot ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
#pragma unroll
      for (int j = 0; j < CPL; ++j) {
        ar[j].v = ring[((slot * 3 + 0) * CPL + j) * 32 + lane];
        br[j].v = ring[((slot * 3 + 1) * CPL + j) * 32 + lane];
        dr[j].v = ring[((slot * 3 + 2) * CPL + j) * 32 + lane];
      }
      slot ^= 1;
    } else {
#pragma unroll
      for (int j = 0; j < CPL; ++j) {
        ar[j].load(yt + 8 * (lane + 32 * j));
        br[j].load(gt + 8 * (lane + 32 * j));
        dr[j].load(dot + 8 * (lane + 32 * j));
      }
    }
    const float s = rstd[t];
    float r = 0.f;   // r = sum_j w_j dout_j x_j
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
      float a[8], b[8], dv[8], wv[8];
      ar[j].get(a); br[j].get(b); dr[j].get(dv); wr[j].get(wv);
#pragma unroll
      for (int e = 0; e < 8; ++e) r = fmaf(wv[e] * dv[e], a[e] * (use_silu ? silu_t<T>(b[e], nullptr) : b[e]), r);
    }
    r = warp_sum(r);
    const float k3 = r * s * s * s / (float)d;
#pragma unroll
    for (int j = 0; j < CPL; ++j) {
      float a[8], b[8], dv[8], wv[8], o1[8], o2[8];
      ar[j].get(a); br[j].get(b); dr[j].get(dv); wr[j].get(wv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float dsl = 1.f;
        const float g = use_silu ? silu_t<T>(b[e], &dsl) : b[e];
        const float x = a[e] * g;
        const float dx = s * wv[e] * dv[e] - k3 * x;
        o1[e] = dx * g;
        o2[e] = dx * a[e] * dsl;
        acc[j][e] = fmaf(dv[e] * x, s, acc[j][e]);
      }
      store8(dy + t * d + 8 * (lane + 32 * j), o1);
      store8(dg_in + t * d + 8 * (lane + 32 * j), o2);
    }
  }
  if constexpr (kRing) asm volatile("cp.async.wait_group 0;" ::: "memory");
#pragma unroll
  for (int j = 0; j < CPL; ++j) {
    float *p = acc_all + (size_t)warp * d + 8 * (lane + 32 * j);
    *reinterpret_cast<float4 *>(p) = make_float4(acc[j][0], acc[j][1], acc[j][2], acc[j][3]);
    *reinterpret_cast<float4 *>(p + 4) = make_float4(acc[j][4], acc[j][5], acc[j][6], acc[j][7]);
  }
  __syncthreads();
  // this CTA's partial of dw: the warps' sums in a fixed order
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float v = 0.f;
#pragma unroll
    for (int wi = 0; wi < kRegWarps; ++wi) v += acc_all[(size_t)wi * d + j];
    dw_part[(size_t)blockIdx.x * d + j] = v;
  }
}

// dw[j] = sum over the R per-CTA partials, in a fixed order: eight interleaved running sums per
// column (one per warp of the CTA), then their sum in warp order
__global__ void __launch_bounds__(256) reduce_partials_kernel(const float *__restrict__ part, float *__restrict__ out, int R, int n) {
  __shared__ float sm[8][32];
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + lane;
  float v = 0.f;
  if (j < n)
    for (int r = grp; r < R; r += 8) v += part[(size_t)r * n + j];
  sm[grp][lane] = v;
  __syncthreads();
  if (grp == 0 && j < n) {
    float t = 0.f;
#pragma unroll
    for (int g = 0; g < 8; ++g) t += sm[g][lane];
    out[j] = t;
  }
}

// warps per CTA of the backward kernel: as many as the budget for their dw accumulators allows
int bwd_warps(int d) {
  if (d == 256 || d == 512 || d == 1024) return kRegWarps;   // the register variant
  return d * 4 * 8 <= kBwdSmemBudget ? 8 : (d * 4 * 4 <= kBwdSmemBudget ? 4 : (d * 4 * 2 <= kBwdSmemBudget ? 2 : 1));
}

int grid_for(long tokens, int warps) {
  const long need = (tokens + warps - 1) / warps;
  return (int)(need < kMaxCtas ? need : kMaxCtas);
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check(long tokens, int d, int io_dtype) {
  if (tokens < 0 || d <= 0) return M2RNN_ERR_SHAPE;
  if (io_dtype != M2RNN_F32 && io_dtype != M2RNN_BF16) return M2RNN_ERR_UNSUPPORTED;
  if (d % 8 || d > kMaxD) return M2RNN_ERR_UNSUPPORTED;
  return M2RNN_OK;
}

template <typename T>
cudaError_t launch_fwd(long tokens, int d, const void *y, const void *g, const void *w, float eps, int silu_on, void *out,
                       float *rstd, cudaStream_t s) {
  const long need = (tokens + kFwdWarps - 1) / kFwdWarps;
  const int grid = (int)(need < 148 * 8 ? need : 148 * 8);
  const T *yp = static_cast<const T *>(y), *gp = static_cast<const T *>(g), *wp = static_cast<const T *>(w);
  T *op = static_cast<T *>(out);
  switch (d) {
    case 256: gated_norm_fwd_kernel<T, 1><<<grid, kFwdWarps * 32, 0, s>>>(tokens, d, yp, gp, wp, eps, silu_on, op, rstd); break;
    case 512: gated_norm_fwd_kernel<T, 2><<<grid, kFwdWarps * 32, 0, s>>>(tokens, d, yp, gp, wp, eps, silu_on, op, rstd); break;
    case 1024: gated_norm_fwd_kernel<T, 4><<<grid, kFwdWarps * 32, 0, s>>>(tokens, d, yp, gp, wp, eps, silu_on, op, rstd); break;
    case 2048: gated_norm_fwd_kernel<T, 8><<<grid, kFwdWarps * 32, 0, s>>>(tokens, d, yp, gp, wp, eps, silu_on, op, rstd); break;
    default: gated_norm_fwd_kernel<T, 0><<<grid, kFwdWarps * 32, 0, s>>>(tokens, d, yp, gp, wp, eps, silu_on, op, rstd); break;
  }
  return cudaGetLastError();
}

template <typename T, int kWarps>
cudaError_t launch_bwd_w(long tokens, int d, const void *y, const void *g, const void *w, const float *rstd, int silu_on,
                         const void *dout, void *dy, void *dg, float *dw_part, cudaStream_t s) {
  const size_t smem = (size_t)kWarps * d * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(gated_norm_bwd_kernel<T, kWarps>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  gated_norm_bwd_kernel<T, kWarps><<<grid_for(tokens, kWarps), kWarps * 32, smem, s>>>(
      tokens, d, static_cast<const T *>(y), static_cast<const T *>(g), static_cast<const T *>(w), rstd, silu_on,
      static_cast<const T *>(dout), static_cast<T *>(dy), static_cast<T *>(dg), dw_part);
  return cudaGetLastError();
}

// persistent CTAs for the register variant: as many as are resident at once (its register need
// grows with CPL), so that the per-CTA prologue and partial of dw are paid once per SM slot
int reg_grid(long tokens, int cpl) {
  const long need = (tokens + kRegWarps - 1) / kRegWarps;
  const long slots = (long)sm_count() * (cpl >= 4 ? 1 : (cpl == 2 ? 2 : 4));
  return (int)(need < slots ? need : slots);
}

template <typename T, int CPL>
cudaError_t launch_bwd_reg(long tokens, const void *y, const void *g, const void *w, const float *rstd, int silu_on,
                           const void *dout, void *dy, void *dg, float *dw_part, cudaStream_t s) {
  // the warps' dw sums, then (bf16) the warps' two-slot rings of three rows each
  const size_t smem = (size_t)kRegWarps * 256 * CPL * sizeof(float) + (sizeof(T) == 2 ? (size_t)kRegWarps * 2 * 3 * 256 * CPL * sizeof(T) : 0);
  cudaError_t e = cudaFuncSetAttribute(gated_norm_bwd_reg_kernel<T, CPL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  gated_norm_bwd_reg_kernel<T, CPL><<<reg_grid(tokens, CPL), kRegWarps * 32, smem, s>>>(
      tokens, static_cast<const T *>(y), static_cast<const T *>(g), static_cast<const T *>(w), rstd, silu_on,
      static_cast<const T *>(dout), static_cast<T *>(dy), static_cast<T *>(dg), dw_part);
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bwd(long tokens, int d, const void *y, const void *g, const void *w, const float *rstd, int silu_on,
                       const void *dout, void *dy, void *dg, float *dw_part, cudaStream_t s) {
  if (d == 256) return launch_bwd_reg<T, 1>(tokens, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
  if (d == 512) return launch_bwd_reg<T, 2>(tokens, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
  if (d == 1024) return launch_bwd_reg<T, 4>(tokens, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
  switch (bwd_warps(d)) {
    case 8: return launch_bwd_w<T, 8>(tokens, d, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
    case 4: return launch_bwd_w<T, 4>(tokens, d, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
    case 2: return launch_bwd_w<T, 2>(tokens, d, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
    default: return launch_bwd_w<T, 1>(tokens, d, y, g, w, rstd, silu_on, dout, dy, dg, dw_part, s);
  }
}

}  // namespace
}  // namespace m2rnn

using namespace m2rnn;

extern "C" {

int m2rnn_gated_norm_fwd(int64_t tokens, int32_t d, int32_t io_dtype, const void *y, const void *g_in, const void *w,
                         float eps, int32_t silu_on, void *out, float *rstd, void *stream) {
  const int rc = check((long)tokens, d, io_dtype);
  if (rc != M2RNN_OK) return rc;
  if (tokens == 0) return M2RNN_OK;   // nothing to read or write
  if (!y || !g_in || !w || !out) return M2RNN_ERR_NULL;
  if (!aligned16(y) || !aligned16(g_in) || !aligned16(w) || !aligned16(out)) return M2RNN_ERR_ALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const cudaError_t e = io_dtype == M2RNN_BF16 ? launch_fwd<__nv_bfloat16>((long)tokens, d, y, g_in, w, eps, silu_on, out, rstd, s)
                                               : launch_fwd<float>((long)tokens, d, y, g_in, w, eps, silu_on, out, rstd, s);
  if (e != cudaSuccess) (void)cudaGetLastError();   // leave the runtime's last-error slot clear
  return e == cudaSuccess ? M2RNN_OK : M2RNN_ERR_CUDA;
}

size_t m2rnn_gated_norm_bwd_workspace_bytes(int64_t tokens, int32_t d) {
  if (tokens <= 0 || d <= 0) return 0;
  return (size_t)kMaxCtas * (size_t)d * sizeof(float);   // an upper bound that does not depend on the dtype
}

int m2rnn_gated_norm_bwd(int64_t tokens, int32_t d, int32_t io_dtype, const void *y, const void *g_in, const void *w,
                         const float *rstd, int32_t silu_on, const void *dout, void *dy, void *dg_in, float *dw,
                         void *workspace, size_t workspace_bytes, void *stream) {
  const int rc = check((long)tokens, d, io_dtype);
  if (rc != M2RNN_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (tokens == 0) {   // an empty sum
    if (!dw) return M2RNN_ERR_NULL;
    return cudaMemsetAsync(dw, 0, (size_t)d * sizeof(float), s) == cudaSuccess ? M2RNN_OK : M2RNN_ERR_CUDA;
  }
  if (!y || !g_in || !w || !rstd || !dout || !dy || !dg_in || !dw) return M2RNN_ERR_NULL;
  if (!aligned16(y) || !aligned16(g_in) || !aligned16(w) || !aligned16(dout) || !aligned16(dy) || !aligned16(dg_in) || !aligned16(dw))
    return M2RNN_ERR_ALIGN;
  if (!workspace || workspace_bytes < m2rnn_gated_norm_bwd_workspace_bytes(tokens, d)) return M2RNN_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return M2RNN_ERR_ALIGN;
  float *part = static_cast<float *>(workspace);
  cudaError_t e = io_dtype == M2RNN_BF16 ? launch_bwd<__nv_bfloat16>((long)tokens, d, y, g_in, w, rstd, silu_on, dout, dy, dg_in, part, s)
                                         : launch_bwd<float>((long)tokens, d, y, g_in, w, rstd, silu_on, dout, dy, dg_in, part, s);
  if (e != cudaSuccess) { (void)cudaGetLastError(); return M2RNN_ERR_CUDA; }
  const int partials = (d == 256 || d == 512 || d == 1024) ? reg_grid((long)tokens, d / 256) : grid_for((long)tokens, bwd_warps(d));
  reduce_partials_kernel<<<(d + 31) / 32, 256, 0, s>>>(part, dw, partials, d);
  return cudaGetLastError() == cudaSuccess ? M2RNN_OK : M2RNN_ERR_CUDA;
}

}  // extern "C"

// Input path before the scan ("M2RNN block" equations): q, k, v = SiLU(conv1d(projection)), a
// depthwise causal convolution of width 4 along time, forward and backward.
//
// HBM-bound streaming kernels.  A thread owns four channels and walks a
// run of consecutive time steps with the last three inputs in registers, so every input row is
// read from HBM once (a run's three-row halo comes from L2) and every output row written once.  The
// rows travel through a per-thread ring in shared memory filled by cp.async two or three batches
// ahead (no registers held while they are in flight); batches that lie wholly inside the run take
// a form without range checks.  Input, output and
// gradient tensors take a token stride, so that the three projections can be processed in place as
// one [tokens, Nq K + Nk K + N V] tensor whose column slices feed the scan.
// Backward: the thread recomputes the pre-activation, forms dpre = dout SiLU'(pre), emits
// dx[t] = sum_s w[s] dpre[t+3-s] three steps behind, and keeps its channels' dw and dbias sums in
// registers; per-tile partial sums are added by a second launch in a fixed order (bitwise
// repeatable).
#include <cuda_bf16.h>

#include <type_traits>

#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"

namespace m2rnn {
namespace {

// A CTA is 32 channel chunks (one warp = 256 or 512 contiguous bytes of a token) x 4 time sub-tiles.
constexpr int kLanes = 32, kSub = 4;
constexpr int kConvThreads = kLanes * kSub;
constexpr int kStepsFwd = 64;                    // time steps per thread of the forward kernel
constexpr int kUFwd = 8, kGFwd = 3;              // ... fetched in batches of kUFwd steps, kGFwd batches ahead
constexpr int kOccFwd = 6;
constexpr int kTileFwd = kSub * kStepsFwd;       // ... per CTA
constexpr int kStepsBwd = 64;                    // backward: longer runs, fewer halo steps
constexpr int kUBwd = 4, kGBwd = 2;              // fetched in batches of kUBwd steps, kGBwd batches ahead
constexpr int kOccBwd = 4;                       // CTAs per SM the backward kernel is compiled for
constexpr int kTileBwd = kSub * kStepsBwd;       // one partial sum of dw and dbias per CTA

template <typename T> struct Chunk;             // the channels of one thread
template <> struct Chunk<float> {
  static constexpr int CH = 4;
  using Raw = float4;
  __device__ static void unpack(const Raw &t, float (&v)[4]) { v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
  __device__ static void load(const float *p, float (&v)[4]) { unpack(*reinterpret_cast<const Raw *>(p), v); }
  __device__ static void store(float *p, const float (&v)[4]) { *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};
template <> struct Chunk<__nv_bfloat16> {   // 8 bytes: four channels keep a thread's filter taps, window and sums
  static constexpr int CH = 4;               // within ~64 (forward) / ~100 (backward) registers, i.e. enough warps
  using Raw = uint2;                          // in flight to cover the memory latency
  __device__ static void unpack(const Raw &r, float (&v)[4]) {
    v[0] = __uint_as_float(r.x << 16); v[1] = __uint_as_float(r.x & 0xffff0000u);
    v[2] = __uint_as_float(r.y << 16); v[3] = __uint_as_float(r.y & 0xffff0000u);
  }
  __device__ static void load(const __nv_bfloat16 *p, float (&v)[4]) { unpack(*reinterpret_cast<const Raw *>(p), v); }
  __device__ static void store(__nv_bfloat16 *p, const float (&v)[4]) {
    *reinterpret_cast<uint2 *>(p) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
  }
};

// sigmoid: through tanh.approx (one special-function instruction, error ~2^-11: below the bf16
// rounding of the result) on the bf16 path, through expf on the fp32 path
template <typename T> __device__ __forceinline__ float sigmoid_of(float x);
template <> __device__ __forceinline__ float sigmoid_of<float>(float x) {
  return x >= 0.f ? 1.f / (1.f + expf(-x)) : expf(x) / (1.f + expf(x));
}
template <> __device__ __forceinline__ float sigmoid_of<__nv_bfloat16>(float x) { return fmaf(0.5f, tanh_approx(0.5f * x), 0.5f); }

// both halves of a pair (the arithmetic below is in packed fp32 pairs: one instruction per two channels)
template <typename T> __device__ __forceinline__ float2 sigmoid2(float2 x) {
  if constexpr (sizeof(T) == 2) {
    const float2 h = __fmul2_rn(x, make_float2(0.5f, 0.5f));
    return __ffma2_rn(make_float2(tanh_approx(h.x), tanh_approx(h.y)), make_float2(0.5f, 0.5f), make_float2(0.5f, 0.5f));
  } else {
    return make_float2(sigmoid_of<T>(x.x), sigmoid_of<T>(x.y));
  }
}
template <int CH>
__device__ __forceinline__ void to_pairs(const float (&v)[CH], float2 (&p)[CH / 2]) {
#pragma unroll
  for (int e = 0; e < CH / 2; ++e) p[e] = make_float2(v[2 * e], v[2 * e + 1]);
}

// asynchronous copy of one chunk (8 or 16 bytes) from global to shared memory; groups of copies are
// committed and waited for per thread, and a thread reads back only what it copied itself
template <int BYTES>
__device__ __forceinline__ void cp_async_chunk(void *dst, const void *src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src), "n"(BYTES) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// row t of batch entry b: x for t >= 0, the carried rows `prev` [B,3,C] for t = -3..-1 (zeros without)
template <typename T, int CH>
__device__ __forceinline__ void load_row(const T *x, long long xs, const T *prev, int b, int Tn, int C, int t, int c0, float (&v)[CH]) {
  if (t >= 0) { Chunk<T>::load(x + ((size_t)b * Tn + t) * xs + c0, v); return; }
  if (prev) { Chunk<T>::load(prev + ((size_t)b * 3 + (3 + t)) * C + c0, v); return; }
#pragma unroll
  for (int e = 0; e < CH; ++e) v[e] = 0.f;
}

template <typename T>
__global__ void __launch_bounds__(kConvThreads, kOccFwd) conv_silu_fwd_kernel(int B, int Tn, int C, const T *__restrict__ x, long long xs,
                                                                     const T *__restrict__ w, const T *__restrict__ bias,
                                                                     const T *__restrict__ prev, T *__restrict__ out, long long os) {
  constexpr int CH = Chunk<T>::CH;
  const int cc = blockIdx.x * kLanes + (threadIdx.x % kLanes), sub = threadIdx.x / kLanes;
  if (cc * CH >= C) return;
  const int c0 = cc * CH, ntile = (Tn + kTileFwd - 1) / kTileFwd;
  const int b = blockIdx.y / ntile, t0 = (blockIdx.y % ntile) * kTileFwd + sub * kStepsFwd, t1 = min(Tn, t0 + kStepsFwd);
  if (t0 >= Tn) return;
  constexpr int CP = CH / 2;            // channel pairs
  float2 w2[4][CP], b2[CP];             // w2[s][p] = tap s of channels 2p, 2p+1
#pragma unroll
  for (int e = 0; e < CP; ++e) {
#pragma unroll
    for (int s = 0; s < 4; ++s) w2[s][e] = make_float2(to_f32<T>(w[(size_t)(c0 + 2 * e) * 4 + s]), to_f32<T>(w[(size_t)(c0 + 2 * e + 1) * 4 + s]));
    b2[e] = bias ? make_float2(to_f32<T>(bias[c0 + 2 * e]), to_f32<T>(bias[c0 + 2 * e + 1])) : make_float2(0.f, 0.f);
  }
  float2 xm3[CP], xm2[CP], xm1[CP];
  {
    float r3[CH], r2[CH], r1[CH];
    load_row<T, CH>(x, xs, prev, b, Tn, C, t0 - 3, c0, r3);
    load_row<T, CH>(x, xs, prev, b, Tn, C, t0 - 2, c0, r2);
    load_row<T, CH>(x, xs, prev, b, Tn, C, t0 - 1, c0, r1);
    to_pairs<CH>(r3, xm3); to_pairs<CH>(r2, xm2); to_pairs<CH>(r1, xm1);
  }
  // The rows of a run travel through a per-thread ring in shared memory: G batches of U rows are
  // requested ahead with cp.async (no registers held while they are in flight), so that a thread
  // has up to G U rows outstanding: the kernel is bound by the latency of HBM, not by arithmetic.
  constexpr int U = kUFwd;
  using Raw = typename Chunk<T>::Raw;
  constexpr int G = sizeof(Raw) == 16 ? 2 : kGFwd;
  __shared__ Raw ring[G][U][kConvThreads];
  const int tid = threadIdx.x;
  const T *xp = x + ((size_t)b * Tn + t0) * xs + c0;
  T *op = out + ((size_t)b * Tn + t0) * os + c0;
  auto fetch = [&](int slot, const T *src, int tbase) {   // always one group, possibly empty
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (tbase + u < t1) cp_async_chunk<sizeof(Raw)>(&ring[slot][u][tid], src + u * xs);
    cp_async_commit();
  };
#pragma unroll
  for (int g = 0; g < G; ++g) fetch(g, xp + (size_t)g * U * xs, t0 + g * U);
  int slot = 0;
  for (int tb = t0; tb < t1; tb += U, xp += U * xs, op += U * os) {
    cp_async_wait<G - 1>();
    auto batch = [&](auto interior) {   // interior: the whole batch lies inside the run, no range checks
      constexpr bool IN = decltype(interior)::value;
      Raw cur[U];
#pragma unroll
      for (int u = 0; u < U; ++u) cur[u] = IN || tb + u < t1 ? ring[slot][u][tid] : Raw{};
#pragma unroll
      for (int u = 0; u < U; ++u) {
        float xr[CH], o[CH];
        float2 x0[CP];
        Chunk<T>::unpack(cur[u], xr);
        to_pairs<CH>(xr, x0);
#pragma unroll
        for (int e = 0; e < CP; ++e) {
          const float2 pre = __ffma2_rn(w2[3][e], x0[e], __ffma2_rn(w2[2][e], xm1[e], __ffma2_rn(w2[1][e], xm2[e], __ffma2_rn(w2[0][e], xm3[e], b2[e]))));
          const float2 r = __fmul2_rn(pre, sigmoid2<T>(pre));
          o[2 * e] = r.x; o[2 * e + 1] = r.y;
          xm3[e] = xm2[e]; xm2[e] = xm1[e]; xm1[e] = x0[e];
        }
        if (IN || tb + u < t1) Chunk<T>::store(op + u * os, o);   // (past the end: arithmetic on stale registers, nothing stored)
      }
    };
    if (tb + U <= t1) batch(std::true_type{});
    else batch(std::false_type{});
    fetch(slot, xp + (size_t)G * U * xs, tb + G * U);       // refill the batch just used
    slot = slot + 1 == G ? 0 : slot + 1;
  }
  cp_async_wait<0>();
}

// partial sums of a tile: part[tile][5][C] = dw taps 0..3 and dbias
template <typename T>
__global__ void __launch_bounds__(kConvThreads, kOccBwd) conv_silu_bwd_kernel(int B, int Tn, int C, const T *__restrict__ x, long long xs,
                                                                     const T *__restrict__ w, const T *__restrict__ bias,
                                                                     const T *__restrict__ prev, const T *__restrict__ dout, long long ds,
                                                                     T *__restrict__ dx, long long dxs, T *__restrict__ dprev,
                                                                     float *__restrict__ part) {
  constexpr int CH = Chunk<T>::CH;
  __shared__ float red[kSub - 1][5 * CH][kLanes];    // the sub-tiles' sums, added by sub-tile 0
  const int lane = threadIdx.x % kLanes, sub = threadIdx.x / kLanes;
  const int cc = blockIdx.x * kLanes + lane;
  const bool live = cc * CH < C;
  const int c0 = live ? cc * CH : 0, ntile = (Tn + kTileBwd - 1) / kTileBwd;
  const int b = blockIdx.y / ntile, t0 = (blockIdx.y % ntile) * kTileBwd + sub * kStepsBwd;
  const int t1 = max(t0, min(Tn, t0 + kStepsBwd));   // an empty run when the sequence ends before it
  constexpr int CP = CH / 2;            // channel pairs
  float2 w2[4][CP], b2[CP];
#pragma unroll
  for (int e = 0; e < CP; ++e) {
#pragma unroll
    for (int s = 0; s < 4; ++s) w2[s][e] = make_float2(to_f32<T>(w[(size_t)(c0 + 2 * e) * 4 + s]), to_f32<T>(w[(size_t)(c0 + 2 * e + 1) * 4 + s]));
    b2[e] = bias ? make_float2(to_f32<T>(bias[c0 + 2 * e]), to_f32<T>(bias[c0 + 2 * e + 1])) : make_float2(0.f, 0.f);
  }
  float2 dw2[4][CP], db2[CP];
#pragma unroll
  for (int e = 0; e < CP; ++e) { dw2[0][e] = dw2[1][e] = dw2[2][e] = dw2[3][e] = db2[e] = make_float2(0.f, 0.f); }
  // The run that starts a sequence also emits the gradient of the carried rows (t' = -3..-1): its
  // sweep starts three steps early with dpre = 0 there.
  const int ts = t0 == 0 ? -3 : t0;         // first t' whose dx this thread emits
  float2 xm3[CP], xm2[CP], xm1[CP];
  const bool work = live && t1 > t0;        // (an empty run loads nothing: its halo rows may lie past the end)
  if (work) {
    float r3[CH], r2[CH], r1[CH];
    load_row<T, CH>(x, xs, prev, b, Tn, C, t0 - 3, c0, r3);
    load_row<T, CH>(x, xs, prev, b, Tn, C, t0 - 2, c0, r2);
    load_row<T, CH>(x, xs, prev, b, Tn, C, t0 - 1, c0, r1);
    to_pairs<CH>(r3, xm3); to_pairs<CH>(r2, xm2); to_pairs<CH>(r1, xm1);
  }
  float2 d3[CP], d2[CP], d1[CP];            // dpre at t-3, t-2, t-1
#pragma unroll
  for (int e = 0; e < CP; ++e) d3[e] = d2[e] = d1[e] = make_float2(0.f, 0.f);
  // t runs three steps past the run: dx[t'] needs dpre[t' .. t'+3].  The loads of four steps are
  // issued before the first is used.
  constexpr int U = kUBwd;
  using Raw = typename Chunk<T>::Raw;
  const T *xp = x + ((size_t)b * Tn + t0) * xs + c0, *gp = dout + ((size_t)b * Tn + t0) * ds + c0;
  T *dxp = dx + ((size_t)b * Tn + t0 - 3) * dxs + c0;       // three steps behind
  const int tend = min(Tn, t1 + 3);                          // steps with inputs to read
  const float2 one = make_float2(1.f, 1.f), mone = make_float2(-1.f, -1.f);
  // x and dout travel through per-thread rings in shared memory, G batches of U rows ahead (cp.async)
  constexpr int G = sizeof(Raw) == 16 ? 2 : kGBwd;
  __shared__ Raw ringx[G][U][kConvThreads], ringg[G][U][kConvThreads];
  const int tid = threadIdx.x;
  auto fetch = [&](int slot, const T *sx, const T *sg, int tbase) {   // always one group, possibly empty
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (work && tbase + u < tend) {
        cp_async_chunk<sizeof(Raw)>(&ringx[slot][u][tid], sx + u * xs);
        cp_async_chunk<sizeof(Raw)>(&ringg[slot][u][tid], sg + u * ds);
      }
    cp_async_commit();
  };
#pragma unroll
  for (int g = 0; g < G; ++g) fetch(g, xp + (size_t)g * U * xs, gp + (size_t)g * U * ds, t0 + g * U);
  int slot = 0;
  for (int tb = t0; tb < t1 + 3 && work; tb += U, xp += U * xs, gp += U * ds, dxp += U * dxs) {
    cp_async_wait<G - 1>();
    // interior batches (every step inside the run, every dx row inside it too) take the form
    // without the per-step range checks, which were a third of the kernel's instructions
    auto batch = [&](auto interior) {
      constexpr bool IN = decltype(interior)::value;
      Raw rx[U], rg[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        rx[u] = IN || tb + u < tend ? ringx[slot][u][tid] : Raw{};
        rg[u] = IN || tb + u < tend ? ringg[slot][u][tid] : Raw{};
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int t = tb + u;
        float2 d0[CP];
        if (IN || t < tend) {
          float xr[CH], gr[CH];
          float2 x0[CP], g[CP];
          Chunk<T>::unpack(rx[u], xr);
          Chunk<T>::unpack(rg[u], gr);
          to_pairs<CH>(xr, x0); to_pairs<CH>(gr, g);
#pragma unroll
          for (int e = 0; e < CP; ++e) {
            const float2 pre = __ffma2_rn(w2[3][e], x0[e], __ffma2_rn(w2[2][e], xm1[e], __ffma2_rn(w2[1][e], xm2[e], __ffma2_rn(w2[0][e], xm3[e], b2[e]))));
            const float2 sg = sigmoid2<T>(pre);
            // dout * SiLU'(pre),  SiLU'(x) = sg (1 + x (1 - sg))
            d0[e] = __fmul2_rn(__fmul2_rn(g[e], sg), __ffma2_rn(pre, __ffma2_rn(sg, mone, one), one));
            if (IN || t < t1) {                                // sums over this run's own steps only
              dw2[0][e] = __ffma2_rn(d0[e], xm3[e], dw2[0][e]); dw2[1][e] = __ffma2_rn(d0[e], xm2[e], dw2[1][e]);
              dw2[2][e] = __ffma2_rn(d0[e], xm1[e], dw2[2][e]); dw2[3][e] = __ffma2_rn(d0[e], x0[e], dw2[3][e]);
              db2[e] = __fadd2_rn(db2[e], d0[e]);
            }
            xm3[e] = xm2[e]; xm2[e] = xm1[e]; xm1[e] = x0[e];
          }
        } else {
#pragma unroll
          for (int e = 0; e < CP; ++e) d0[e] = make_float2(0.f, 0.f);
        }
        const int tp = t - 3;                                  // dx[tp] = w3 dpre[tp] + w2 dpre[tp+1] + w1 dpre[tp+2] + w0 dpre[tp+3]
        if (IN || (tp >= ts && tp < t1)) {
          float o[CH];
#pragma unroll
          for (int e = 0; e < CP; ++e) {
            const float2 r = __ffma2_rn(w2[3][e], d3[e], __ffma2_rn(w2[2][e], d2[e], __ffma2_rn(w2[1][e], d1[e], __fmul2_rn(w2[0][e], d0[e]))));
            o[2 * e] = r.x; o[2 * e + 1] = r.y;
          }
          if (IN || tp >= 0) Chunk<T>::store(dxp + u * dxs, o);
          else if (dprev) Chunk<T>::store(dprev + ((size_t)b * 3 + (3 + tp)) * C + c0, o);
        }
#pragma unroll
        for (int e = 0; e < CP; ++e) { d3[e] = d2[e]; d2[e] = d1[e]; d1[e] = d0[e]; }
      }
    };
    if (tb >= t0 + 3 && tb + U <= t1) batch(std::true_type{});
    else batch(std::false_type{});
    fetch(slot, xp + (size_t)G * U * xs, gp + (size_t)G * U * ds, tb + G * U);   // refill the batch just used
    slot = slot + 1 == G ? 0 : slot + 1;
  }
  cp_async_wait<0>();
  // the sums, channel by channel, for the hand-over below
  float dwv[CH][4], dbv[CH];
#pragma unroll
  for (int e = 0; e < CP; ++e) {
#pragma unroll
    for (int s = 0; s < 4; ++s) { dwv[2 * e][s] = dw2[s][e].x; dwv[2 * e + 1][s] = dw2[s][e].y; }
    dbv[2 * e] = db2[e].x; dbv[2 * e + 1] = db2[e].y;
  }
  // (dprev of the first tile: the three steps before t = 0 were emitted while t = 0, 1, 2 -- with
  // d3/d2/d1 still zero where they stand for dpre at negative times)
  // one partial sum per CTA: sub-tiles 1.. hand theirs to sub-tile 0 in a fixed order
  if (sub > 0) {
#pragma unroll
    for (int e = 0; e < CH; ++e) {
#pragma unroll
      for (int s = 0; s < 4; ++s) red[sub - 1][s * CH + e][lane] = dwv[e][s];
      red[sub - 1][4 * CH + e][lane] = dbv[e];
    }
  }
  __syncthreads();
  if (sub == 0 && live) {
    float *pp = part + (size_t)blockIdx.y * 5 * C + c0;
#pragma unroll
    for (int e = 0; e < CH; ++e) {
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        float acc = dwv[e][s];
        for (int r = 0; r < kSub - 1; ++r) acc += red[r][s * CH + e][lane];
        pp[(size_t)s * C + e] = acc;
      }
      float acc = dbv[e];
      for (int r = 0; r < kSub - 1; ++r) acc += red[r][4 * CH + e][lane];
      pp[(size_t)4 * C + e] = acc;
    }
  }
}

// dw[c][s] = sum over tiles of part[tile][s][c]; dbias[c] likewise from row 4.  Eight lanes share an
// output: each sums every eighth tile, then a shuffle tree adds the eight (a fixed order).
__global__ void conv_silu_reduce_kernel(const float *__restrict__ part, int ntiles, int C, float *__restrict__ dw, float *__restrict__ dbias) {
  const int x = (blockIdx.x * blockDim.x + threadIdx.x) >> 3, r = threadIdx.x & 7;
  const bool live = x < 5 * C;
  const int s = live ? x / C : 0, c = live ? x % C : 0;
  float acc = 0.f;
  if (live)
    for (int tl = r; tl < ntiles; tl += 8) acc += part[((size_t)tl * 5 + s) * C + c];
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  acc += __shfl_xor_sync(0xffffffffu, acc, 2);
  acc += __shfl_xor_sync(0xffffffffu, acc, 4);
  if (!live || r) return;
  if (s < 4) dw[(size_t)c * 4 + s] = acc;
  else if (dbias) dbias[c] = acc;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check(int B, int T, int C, int io_dtype, long long strides[], int nstrides) {
  if (B < 0 || T < 0 || C <= 0) return M2RNN_ERR_SHAPE;
  if (io_dtype != M2RNN_F32 && io_dtype != M2RNN_BF16) return M2RNN_ERR_UNSUPPORTED;
  const int ch = io_dtype == M2RNN_BF16 ? 8 : 4;   // rows and row starts stay 16-byte aligned
  if (C % ch) return M2RNN_ERR_UNSUPPORTED;
  for (int i = 0; i < nstrides; ++i) {
    if (strides[i] == 0) strides[i] = C;
    if (strides[i] < C || strides[i] % ch) return M2RNN_ERR_SHAPE;
  }
  return M2RNN_OK;
}

}  // namespace
}  // namespace m2rnn

using namespace m2rnn;

extern "C" int m2rnn_conv_silu_fwd(int32_t B, int32_t T, int32_t C, int32_t io_dtype, const void *x, int64_t x_stride,
                                   const void *w, const void *bias, const void *prev, void *out, int64_t out_stride,
                                   void *stream) {
  long long st[2] = {x_stride, out_stride};
  const int rc = check(B, T, C, io_dtype, st, 2);
  if (rc != M2RNN_OK) return rc;
  if (B == 0 || T == 0) return M2RNN_OK;
  if (!x || !w || !out) return M2RNN_ERR_NULL;
  if (!aligned16(x) || !aligned16(w) || !aligned16(bias) || !aligned16(prev) || !aligned16(out)) return M2RNN_ERR_ALIGN;
  const int ch = 4, ntile = (T + kTileFwd - 1) / kTileFwd;   // channels per thread
  const dim3 grid((C / ch + kLanes - 1) / kLanes, (unsigned)(B * ntile));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (io_dtype == M2RNN_BF16)
    conv_silu_fwd_kernel<__nv_bfloat16><<<grid, kConvThreads, 0, s>>>(
        B, T, C, static_cast<const __nv_bfloat16 *>(x), st[0], static_cast<const __nv_bfloat16 *>(w),
        static_cast<const __nv_bfloat16 *>(bias), static_cast<const __nv_bfloat16 *>(prev), static_cast<__nv_bfloat16 *>(out), st[1]);
  else
    conv_silu_fwd_kernel<float><<<grid, kConvThreads, 0, s>>>(B, T, C, static_cast<const float *>(x), st[0], static_cast<const float *>(w),
                                                              static_cast<const float *>(bias), static_cast<const float *>(prev),
                                                              static_cast<float *>(out), st[1]);
  return cudaGetLastError() == cudaSuccess ? M2RNN_OK : M2RNN_ERR_CUDA;
}

extern "C" size_t m2rnn_conv_silu_bwd_workspace_bytes(int32_t B, int32_t T, int32_t C) {
  if (B <= 0 || T <= 0 || C <= 0) return 0;
  return align_up((size_t)B * ((T + kTileBwd - 1) / kTileBwd) * 5 * C * sizeof(float));
}

extern "C" int m2rnn_conv_silu_bwd(int32_t B, int32_t T, int32_t C, int32_t io_dtype, const void *x, int64_t x_stride,
                                   const void *w, const void *bias, const void *prev, const void *dout,
                                   int64_t dout_stride, void *dx, int64_t dx_stride, float *dw, float *dbias,
                                   void *dprev, void *workspace, size_t workspace_bytes, void *stream) {
  long long st[3] = {x_stride, dout_stride, dx_stride};
  const int rc = check(B, T, C, io_dtype, st, 3);
  if (rc != M2RNN_OK) return rc;
  if (!dw) return M2RNN_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (B == 0 || T == 0) {   // no step: the sums are empty, nothing flows to the carried rows
    cudaError_t e = cudaMemsetAsync(dw, 0, sizeof(float) * 4 * C, s);
    if (e == cudaSuccess && dbias) e = cudaMemsetAsync(dbias, 0, sizeof(float) * C, s);
    if (e == cudaSuccess && dprev && B > 0) e = cudaMemsetAsync(dprev, 0, (size_t)B * 3 * C * (io_dtype == M2RNN_BF16 ? 2 : 4), s);
    if (e != cudaSuccess) (void)cudaGetLastError();
    return e == cudaSuccess ? M2RNN_OK : M2RNN_ERR_CUDA;
  }
  if (!x || !w || !dout || !dx) return M2RNN_ERR_NULL;
  const void *ptrs[] = {x, w, bias, prev, dout, dx, dw, dbias, dprev};
  for (const void *p : ptrs)
    if (!aligned16(p)) return M2RNN_ERR_ALIGN;
  const size_t need = m2rnn_conv_silu_bwd_workspace_bytes(B, T, C);
  if (!workspace || workspace_bytes < need) return M2RNN_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return M2RNN_ERR_ALIGN;
  const int ch = 4, ntile = (T + kTileBwd - 1) / kTileBwd;   // channels per thread
  const dim3 grid((C / ch + kLanes - 1) / kLanes, (unsigned)(B * ntile));
  float *part = static_cast<float *>(workspace);
  if (io_dtype == M2RNN_BF16)
    conv_silu_bwd_kernel<__nv_bfloat16><<<grid, kConvThreads, 0, s>>>(
        B, T, C, static_cast<const __nv_bfloat16 *>(x), st[0], static_cast<const __nv_bfloat16 *>(w),
        static_cast<const __nv_bfloat16 *>(bias), static_cast<const __nv_bfloat16 *>(prev), static_cast<const __nv_bfloat16 *>(dout),
        st[1], static_cast<__nv_bfloat16 *>(dx), st[2], static_cast<__nv_bfloat16 *>(dprev), part);
  else
    conv_silu_bwd_kernel<float><<<grid, kConvThreads, 0, s>>>(B, T, C, static_cast<const float *>(x), st[0], static_cast<const float *>(w),
                                                              static_cast<const float *>(bias), static_cast<const float *>(prev),
                                                              static_cast<const float *>(dout), st[1], static_cast<float *>(dx), st[2],
                                                              static_cast<float *>(dprev), part);
  if (cudaGetLastError() != cudaSuccess) return M2RNN_ERR_CUDA;
  conv_silu_reduce_kernel<<<(8 * 5 * C + 255) / 256, 256, 0, s>>>(part, B * ntile, C, dw, dbias);
  return cudaGetLastError() == cudaSuccess ? M2RNN_OK : M2RNN_ERR_CUDA;
}

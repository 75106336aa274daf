// bf16 tensor-core forward scan (Algorithm 1) for sm_100a.
//
// One CTA per (b,n): K/16 compute warps, each holding a 16 x V slab of the state in registers
// for all T steps (see mma_tile.cuh), plus one service warp.  Per step a compute warp
//   1. seeds its accumulators with the outer product k_t v_t^T (fp32 FMA),
//   2. adds H_{t-1} W with V/16 x V/8 mma.sync.m16n8k16 (bf16 operands, fp32 accumulate),
//   3. applies tanh.approx and the gate, keeping H_t in fp32 and re-packing it to the bf16
//      A fragments of the next step,
//   4. forms its partial readout q_t-weighted column sums with shuffles and leaves them in
//      shared memory.
// The service warp runs ahead of and behind the compute warps: it fetches q/k/v/gate for a
// stage of steps from global memory, converts them to fp32, evaluates the forget gate, and,
// once a stage is done, adds the warps' readout partials and writes y with 16-byte stores.
// Stages are handed over with mbarriers; every wait is bounded and reports through dev_status.
#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"

namespace m2rnn {
namespace {

constexpr int kStages = 3;
constexpr int kBarrierBytes = 64;  // 2 * kStages mbarriers, padded so the stages stay 16-byte aligned

template <int V>
struct FwdSmem {
  // Per stage (floats): q [TC][K], k [TC][K], v [TC][V], f [TC], ypart [TC][NW][V]
  __host__ __device__ static int stage_floats(int K, int TC) { return TC * (2 * K + V + 1 + (K / 16) * V); }
  __host__ __device__ static int tc(int K) { return (V >= 128 || K > 64) ? 8 : 16; }
  __host__ static size_t bytes(int K) {
    const int TC = tc(K);
    size_t b = sizeof(float) * (size_t)kStages * stage_floats(K, TC);
    if (V > 64) b += (size_t)V * V * 2;  // W fragments
    return b + kBarrierBytes;
  }
};

template <int V>
__global__ void __launch_bounds__(288, 1) fwd_bf16_kernel(ScanArgs a) {
  using G = TileGeom<V>;
  constexpr int NT = G::NT, KT = G::KT, SEG = G::SEG;
  constexpr bool kWInRegs = V <= 64;
  extern __shared__ __align__(16) unsigned char smem_raw[];

  const int K = a.K, N = a.N, T = a.T;
  const int NW = K >> 4;
  const int TC = FwdSmem<V>::tc(K);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bn = blockIdx.x, b = bn / N, n = bn % N;
  const int stage_floats = FwdSmem<V>::stage_floats(K, TC);

  uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw);  // [kStages]
  uint64_t *done = full + kStages;                          // [kStages]
  float *stages = reinterpret_cast<float *>(smem_raw + kBarrierBytes);
  uint2 *Wf = reinterpret_cast<uint2 *>(stages + (size_t)kStages * stage_floats);  // [KT][NT][32], V > 64 only

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&done[s], NW);
    }
    fence_mbar_init();
  }
  const __nv_bfloat16 *Wn = static_cast<const __nv_bfloat16 *>(a.W) + (size_t)n * V * V;
  if constexpr (!kWInRegs) {
    for (int x = tid; x < KT * NT * 32; x += blockDim.x) {
      uint32_t b0, b1;
      load_w_fragment<V>(Wn, x / (NT * 32), (x / 32) % NT, x & 31, b0, b1);
      Wf[x] = make_uint2(b0, b1);
    }
  }
  __syncthreads();

  const int nchunks = (T + TC - 1) / TC;
  const bool want_y = a.y != nullptr;

  if (warp == NW) {
    // ------------------------------------------------------------------ service warp
    const int hq = n / (N / a.Nq), hk = n / (N / a.Nk);
    const float al = a.alpha ? a.alpha[n] : 1.f, be = a.beta ? a.beta[n] : 0.f;
    const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(a.q);
    const __nv_bfloat16 *kg = static_cast<const __nv_bfloat16 *>(a.k);
    const __nv_bfloat16 *vg = static_cast<const __nv_bfloat16 *>(a.v);
    const __nv_bfloat16 *wr = static_cast<const __nv_bfloat16 *>(a.w_r);
    __nv_bfloat16 *yg = static_cast<__nv_bfloat16 *>(a.y);

    // A stage holds at most 16 x 128 / 8 = 128 (TC = 8, K or V = 128) or 16 x 64 / 8 = 128 rows of
    // 16 bytes per tensor: 4 per lane.  All loads of a stage are issued before the first use so
    // that one global round trip covers the whole stage.
    constexpr int kPerLane = 4;
    auto fill = [&](int ch) {
      const int s = ch % kStages, t0 = ch * TC, len = min(TC, T - t0);
      float *qS = stages + (size_t)s * stage_floats, *kS = qS + TC * K, *vS = kS + TC * K, *fS = vS + TC * V;
      const size_t bt0 = (size_t)b * T + t0;
      const int kq8 = K / 8, v8 = V / 8;
      uint4 rk[kPerLane], rq[kPerLane], rv[kPerLane];
      float gt = 0.f;
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const int x = lane + 32 * i;
        if (x < len * kq8) {
          const int t = x / kq8, j = (x % kq8) * 8;
          rk[i] = *reinterpret_cast<const uint4 *>(kg + ((bt0 + t) * a.Nk + hk) * K + j);
          if (want_y) rq[i] = *reinterpret_cast<const uint4 *>(qg + ((bt0 + t) * a.Nq + hq) * K + j);
        }
        if (x < len * v8) {
          const int t = x / v8, j = (x % v8) * 8;
          rv[i] = *reinterpret_cast<const uint4 *>(vg + ((bt0 + t) * N + n) * V + j);
        }
      }
      if (lane < len) gt = a.gate[(bt0 + lane) * N + n];
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const int x = lane + 32 * i;
        if (x < len * kq8) {
          const int t = x / kq8, j = (x % kq8) * 8;
          store8_bf16_as_f32(kS + t * K + j, rk[i]);
          if (want_y) store8_bf16_as_f32(qS + t * K + j, rq[i]);
        }
        if (x < len * v8) {
          const int t = x / v8, j = (x % v8) * 8;
          store8_bf16_as_f32(vS + t * V + j, rv[i]);
        }
      }
      if (lane < len) fS[lane] = gate_value(a.gate_kind, gt, al, be, nullptr);
      __syncwarp();
      if (lane == 0) mbar_arrive(&full[s]);
    };

    const int pre = min(kStages, nchunks);
    for (int ch = 0; ch < pre; ++ch) fill(ch);
    for (int ch = 0; ch < nchunks; ++ch) {
      const int s = ch % kStages, t0 = ch * TC, len = min(TC, T - t0);
      if (!mbar_wait(&done[s], (ch / kStages) & 1)) { report_timeout(a.dev_status); return; }
      if (want_y) {
        // y[t][col] = sum over compute warps of their partials (+ w_r (.) v), 8 columns per lane
        const float *vS = stages + (size_t)s * stage_floats + 2 * TC * K;
        const float *yp = vS + TC * V + TC;
        const int v8 = V / 8;
        for (int x = lane; x < len * v8; x += 32) {
          const int t = x / v8, j = (x % v8) * 8;
          float acc[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] = 0.f;
          for (int w = 0; w < NW; ++w) {
            const float4 p0 = *reinterpret_cast<const float4 *>(yp + ((size_t)t * NW + w) * V + j);
            const float4 p1 = *reinterpret_cast<const float4 *>(yp + ((size_t)t * NW + w) * V + j + 4);
            acc[0] += p0.x; acc[1] += p0.y; acc[2] += p0.z; acc[3] += p0.w;
            acc[4] += p1.x; acc[5] += p1.y; acc[6] += p1.z; acc[7] += p1.w;
          }
          if (wr) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(__bfloat162float(wr[(size_t)n * V + j + e]), vS[t * V + j + e], acc[e]);
          }
          uint4 o;
          o.x = pack_bf16(acc[0], acc[1]); o.y = pack_bf16(acc[2], acc[3]);
          o.z = pack_bf16(acc[4], acc[5]); o.w = pack_bf16(acc[6], acc[7]);
          *reinterpret_cast<uint4 *>(yg + (((size_t)b * T + t0 + t) * N + n) * V + j) = o;
        }
        __syncwarp();
      }
      if (ch + kStages < nchunks) fill(ch + kStages);
    }
    return;
  }

  // -------------------------------------------------------------------- compute warps
  const int g = lane >> 2, c = lane & 3;
  const int row0 = 16 * warp + 2 * g;   // memory rows row0, row0+1  <->  MMA rows g, g+8
  const size_t KV = (size_t)K * V;

  uint32_t Wr[kWInRegs ? KT : 1][kWInRegs ? NT : 1][2];
  if constexpr (kWInRegs) {
#pragma unroll
    for (int kt = 0; kt < KT; ++kt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) load_w_fragment<V>(Wn, kt, nt, lane, Wr[kt][nt][0], Wr[kt][nt][1]);
  }

  // H[nt] = {row g: cols 2nt,2nt+1 of the segment | row g+8: same}
  float H[NT][4];
  if (a.h0) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float *src = a.h0 + bn * KV + (size_t)(row0 + h) * V + SEG * c;
#pragma unroll
      for (int x = 0; x < SEG / 4; ++x) {
        const float4 t4 = *reinterpret_cast<const float4 *>(src + 4 * x);
        H[2 * x][2 * h] = t4.x; H[2 * x][2 * h + 1] = t4.y; H[2 * x + 1][2 * h] = t4.z; H[2 * x + 1][2 * h + 1] = t4.w;
      }
    }
  } else {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) H[nt][0] = H[nt][1] = H[nt][2] = H[nt][3] = 0.f;
  }
  uint32_t A[KT][4];
#pragma unroll
  for (int kt = 0; kt < KT; ++kt) {
    A[kt][0] = pack_bf16(H[2 * kt][0], H[2 * kt][1]);
    A[kt][1] = pack_bf16(H[2 * kt][2], H[2 * kt][3]);
    A[kt][2] = pack_bf16(H[2 * kt + 1][0], H[2 * kt + 1][1]);
    A[kt][3] = pack_bf16(H[2 * kt + 1][2], H[2 * kt + 1][3]);
  }

  auto store_state = [&](float *dst) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float *p = dst + (size_t)(row0 + h) * V + SEG * c;
#pragma unroll
      for (int x = 0; x < SEG / 4; ++x)
        *reinterpret_cast<float4 *>(p + 4 * x) =
            make_float4(H[2 * x][2 * h], H[2 * x][2 * h + 1], H[2 * x + 1][2 * h], H[2 * x + 1][2 * h + 1]);
    }
  };

  int ck_left = 0, ck_idx = 0;  // steps until the next checkpoint, index of the next checkpoint
  for (int ch = 0; ch < nchunks; ++ch) {
    const int s = ch % kStages, len = min(TC, T - ch * TC);
    if (!mbar_wait(&full[s], (ch / kStages) & 1)) { report_timeout(a.dev_status); return; }
    const float *qS = stages + (size_t)s * stage_floats, *kS = qS + TC * K, *vS = kS + TC * K, *fS = vS + TC * V;
    float *yp = const_cast<float *>(fS) + TC;

    for (int t = 0; t < len; ++t) {
      if (a.ckpt) {
        if (ck_left == 0) {
          store_state(a.ckpt + ((size_t)bn * a.nchunks + ck_idx) * KV);
          ++ck_idx;
          ck_left = a.C;
        }
        --ck_left;
      }
      const float2 kk = *reinterpret_cast<const float2 *>(kS + t * K + row0);
      const float f = fS[t];
      float vv[SEG];
#pragma unroll
      for (int x = 0; x < SEG / 4; ++x) {
        const float4 t4 = *reinterpret_cast<const float4 *>(vS + t * V + SEG * c + 4 * x);
        vv[4 * x] = t4.x; vv[4 * x + 1] = t4.y; vv[4 * x + 2] = t4.z; vv[4 * x + 3] = t4.w;
      }
      // Eq. 1: P = k v^T + H W
      float P[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        P[nt][0] = kk.x * vv[2 * nt]; P[nt][1] = kk.x * vv[2 * nt + 1];
        P[nt][2] = kk.y * vv[2 * nt]; P[nt][3] = kk.y * vv[2 * nt + 1];
      }
#pragma unroll
      for (int kt = 0; kt < KT; ++kt) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if constexpr (kWInRegs) {
            mma_bf16_16816(P[nt], A[kt], Wr[kt][nt][0], Wr[kt][nt][1]);
          } else {
            const uint2 w = Wf[(kt * NT + nt) * 32 + lane];
            mma_bf16_16816(P[nt], A[kt], w.x, w.y);
          }
        }
      }
      // Eq. 2: H = Z + f (H - Z), Z = tanh(P); then the bf16 operand of the next step
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const float z = tanh_approx(P[nt][r]);
          H[nt][r] = fmaf(f, H[nt][r] - z, z);
        }
      }
#pragma unroll
      for (int kt = 0; kt < KT; ++kt) {
        A[kt][0] = pack_bf16(H[2 * kt][0], H[2 * kt][1]);
        A[kt][1] = pack_bf16(H[2 * kt][2], H[2 * kt][3]);
        A[kt][2] = pack_bf16(H[2 * kt + 1][0], H[2 * kt + 1][1]);
        A[kt][3] = pack_bf16(H[2 * kt + 1][2], H[2 * kt + 1][3]);
      }
      // Eq. 3: this warp's share of H_t^T q_t
      if (want_y) {
        const float2 qq = *reinterpret_cast<const float2 *>(qS + t * K + row0);
        float part[SEG];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          part[2 * nt] = fmaf(qq.y, H[nt][2], qq.x * H[nt][0]);
          part[2 * nt + 1] = fmaf(qq.y, H[nt][3], qq.x * H[nt][1]);
        }
        reduce_over_rows<SEG>(part, lane);
        using RO = RowReduceOut<V>;
        if (RO::owner(lane)) {
          float *dst = yp + ((size_t)t * NW + warp) * V + RO::first_col(lane);
          if constexpr (RO::CNT == 4) *reinterpret_cast<float4 *>(dst) = make_float4(part[0], part[1], part[2], part[3]);
          else if constexpr (RO::CNT == 2) *reinterpret_cast<float2 *>(dst) = make_float2(part[0], part[1]);
          else dst[0] = part[0];
        }
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&done[s]);
  }
  if (a.hT) store_state(a.hT + bn * KV);
}

template <int V>
cudaError_t launch_v(const ScanArgs &a, cudaStream_t s) {
  const size_t smem = FwdSmem<V>::bytes(a.K);
  cudaError_t e = cudaFuncSetAttribute(fwd_bf16_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  fwd_bf16_kernel<V><<<a.B * a.N, (a.K / 16 + 1) * 32, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_bf16(const ScanArgs &a, cudaStream_t s) {
  switch (a.V) {
    case 16: return launch_v<16>(a, s);
    case 32: return launch_v<32>(a, s);
    case 64: return launch_v<64>(a, s);
    case 128: return launch_v<128>(a, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace m2rnn

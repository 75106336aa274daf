// bf16 decoding step (Eq. 1-3 once on a cached fp32 state) for sm_100a.
//
// The step streams the whole state through the chip once (read + write, fp32), so the kernel is
// laid out around HBM: persistent CTAs walk a contiguous range of (head, batch) units in
// head-major order, keep the head's transition matrix as MMA fragments in shared memory (re-read
// only when the head changes), and prefetch the states of the next units with the bulk async-copy
// engine (cp.async.bulk into a two-stage shared-memory buffer, completion on an mbarrier) while
// the current ones are computed.  Every warp takes 16 state rows from the staged copy into
// accumulator-layout registers, runs the state x W product
// on tensor cores (mma.sync, bf16 operands, fp32 accumulate), applies the outer product, tanh
// and the gate in registers, writes the rows back in place and leaves its share of the readout
// in shared memory, where the unit's warps are summed.
#include <cstdlib>
#include <cstring>

#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"

namespace m2rnn {
namespace {

// Memory column of MMA column m = 8nt + 2c + e: a thread's registers of the tile pair
// (2x, 2x+1) are the four adjacent columns 16x + 4c .. 16x + 4c + 3, so the four lanes of a row
// group read 64 contiguous bytes of a row per load.
template <int V>
__host__ __device__ constexpr int dec_col(int m) {
  return V == 16 ? 4 * ((m & 7) >> 1) + 2 * (m >> 3) + (m & 1)
                 : 16 * (m >> 4) + 4 * ((m & 7) >> 1) + 2 * ((m >> 3) & 1) + (m & 1);
}

template <int V>
__device__ __forceinline__ uint2 dec_w_fragment(const uint16_t *__restrict__ w, int kt, int nt, int lane) {
  const int g = lane >> 2, c = lane & 3;
  const int col = dec_col<V>(8 * nt + g);
  const int r0 = dec_col<V>(16 * kt + 2 * c), r1 = dec_col<V>(16 * kt + 2 * c + 1);
  const int r2 = dec_col<V>(16 * kt + 8 + 2 * c), r3 = dec_col<V>(16 * kt + 8 + 2 * c + 1);
  return make_uint2((uint32_t)w[r0 * V + col] | ((uint32_t)w[r1 * V + col] << 16),
                    (uint32_t)w[r2 * V + col] | ((uint32_t)w[r3 * V + col] << 16));
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// global -> shared bulk copy (no multicast); both addresses 16-byte aligned, size a multiple of 16
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

template <int V>
__global__ void __launch_bounds__(256, 1) decode_bf16_kernel(ScanArgs a, int WPU, int GPI, int tasks_per_head) {
  constexpr int NT = V / 8, KT = V / 16, SEG = V / 4, NX = V == 16 ? 1 : V / 16;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw);                // [2] stage landed
  uint2 *Wf = reinterpret_cast<uint2 *>(smem_raw + 16);                   // [KT][NT][32]
  float *ypart = reinterpret_cast<float *>(smem_raw + 16 + KT * NT * 32 * 8);  // [2][GPI][WPU][V]

  const int K = a.K, N = a.N, B = a.B;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, c = lane & 3;
  const int grp = warp / WPU, wu = warp % WPU;      // unit slot of this warp, its 16-row slab
  const bool active_warp = grp < GPI;
  const size_t KV = (size_t)K * V;
  const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(a.q), *kg = static_cast<const __nv_bfloat16 *>(a.k);
  const __nv_bfloat16 *vg = static_cast<const __nv_bfloat16 *>(a.v), *wr = static_cast<const __nv_bfloat16 *>(a.w_r);
  __nv_bfloat16 *yg = static_cast<__nv_bfloat16 *>(a.y);
  float *state = a.hT;   // == a.h0: updated in place

  const size_t unit_floats = KV;                                          // one unit's state
  float *stage = ypart + 2 * GPI * WPU * V;                               // [2][GPI][K][V] fp32
  if (tid == 0) {
    mbar_init(&full[0], 1);
    mbar_init(&full[1], 1);
    fence_mbar_init();
  }
  __syncthreads();

  const long ntasks = (long)N * tasks_per_head;
  const long t_begin = ntasks * blockIdx.x / gridDim.x, t_end = ntasks * (blockIdx.x + 1) / gridDim.x;
  // one thread streams the states of a task's units into a stage, 16 KB per copy
  auto prefetch = [&](long task, int st) {
    const int n = (int)(task / tasks_per_head), b0 = (int)(task % tasks_per_head) * GPI;
    const int units = min(GPI, B - b0);
    const uint32_t bytes = (uint32_t)(unit_floats * 4);
    mbar_expect_tx(&full[st], bytes * units);
    for (int u = 0; u < units; ++u) {
      const char *src = reinterpret_cast<const char *>(state + ((size_t)(b0 + u) * N + n) * unit_floats);
      char *dst = reinterpret_cast<char *>(stage + ((size_t)st * GPI + u) * unit_floats);
      for (uint32_t off = 0; off < bytes; off += 16384u) bulk_g2s(dst + off, src + off, min(16384u, bytes - off), &full[st]);
    }
  };
  if (tid == 0 && t_begin < t_end) prefetch(t_begin, 0);
  int cur_head = -1;
  int it = 0;
  for (long task = t_begin; task < t_end; ++task, ++it) {
    const int n = (int)(task / tasks_per_head);
    const int b = (int)(task % tasks_per_head) * GPI + grp;
    // the other stage was last read before the barrier that closed the previous iteration
    if (tid == 0 && task + 1 < t_end) prefetch(task + 1, (it + 1) & 1);
    if (n != cur_head) {
      __syncthreads();   // everyone is done with the previous head's fragments
      const uint16_t *w = reinterpret_cast<const uint16_t *>(a.W) + (size_t)n * V * V;
      for (int x = tid; x < KT * NT * 32; x += blockDim.x) Wf[x] = dec_w_fragment<V>(w, x / (NT * 32), (x / 32) % NT, x & 31);
      cur_head = n;
      __syncthreads();
    }
    const bool live = active_warp && b < B;
    if (!mbar_wait(&full[it & 1], (it >> 1) & 1)) { report_timeout(a.dev_status); return; }
    float *yp = ypart + (size_t)(((it & 1) * GPI + (active_warp ? grp : 0)) * WPU + wu) * V;
    if (live) {
      const size_t bn = (size_t)b * N + n;
      const int hq = n / (N / a.Nq), hk = n / (N / a.Nk);
      const int r0 = 16 * wu + g;
      // state rows r0 and r0+8 in accumulator layout
      float H[NT][4];
      float *hrow0 = state + bn * KV + (size_t)r0 * V, *hrow1 = hrow0 + 8 * V;
      const float *srow0 = stage + ((size_t)(it & 1) * GPI + grp) * unit_floats + (size_t)r0 * V, *srow1 = srow0 + 8 * V;
#pragma unroll
      for (int x = 0; x < NX; ++x) {
        const float4 t0 = *reinterpret_cast<const float4 *>(srow0 + 16 * x + 4 * c);
        const float4 t1 = *reinterpret_cast<const float4 *>(srow1 + 16 * x + 4 * c);
        H[2 * x][0] = t0.x; H[2 * x][1] = t0.y; H[2 * x + 1][0] = t0.z; H[2 * x + 1][1] = t0.w;
        H[2 * x][2] = t1.x; H[2 * x][3] = t1.y; H[2 * x + 1][2] = t1.z; H[2 * x + 1][3] = t1.w;
      }
      const float k0 = __bfloat162float(kg[((size_t)b * a.Nk + hk) * K + r0]), k1 = __bfloat162float(kg[((size_t)b * a.Nk + hk) * K + r0 + 8]);
      const float q0 = __bfloat162float(qg[((size_t)b * a.Nq + hq) * K + r0]), q1 = __bfloat162float(qg[((size_t)b * a.Nq + hq) * K + r0 + 8]);
      const float f = gate_value(a.gate_kind, a.gate[bn], a.alpha ? a.alpha[n] : 1.f, a.beta ? a.beta[n] : 0.f, nullptr);
      // P = k v^T + H W
      float P[NT][4];
#pragma unroll
      for (int x = 0; x < NX; ++x) {
        const uint2 vr = *reinterpret_cast<const uint2 *>(vg + bn * V + 16 * x + 4 * c);
        const float v0 = __uint_as_float(vr.x << 16), v1 = __uint_as_float(vr.x & 0xffff0000u);
        const float v2 = __uint_as_float(vr.y << 16), v3 = __uint_as_float(vr.y & 0xffff0000u);
        P[2 * x][0] = k0 * v0; P[2 * x][1] = k0 * v1; P[2 * x][2] = k1 * v0; P[2 * x][3] = k1 * v1;
        P[2 * x + 1][0] = k0 * v2; P[2 * x + 1][1] = k0 * v3; P[2 * x + 1][2] = k1 * v2; P[2 * x + 1][3] = k1 * v3;
      }
#pragma unroll
      for (int kt = 0; kt < KT; ++kt) {
        const uint32_t Ak[4] = {pack_bf16(H[2 * kt][0], H[2 * kt][1]), pack_bf16(H[2 * kt][2], H[2 * kt][3]),
                                pack_bf16(H[2 * kt + 1][0], H[2 * kt + 1][1]), pack_bf16(H[2 * kt + 1][2], H[2 * kt + 1][3])};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const uint2 wv = Wf[(kt * NT + nt) * 32 + lane];
          mma_bf16_16816(P[nt], Ak, wv.x, wv.y);
        }
      }
      float part[SEG];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const float z = tanh_approx(P[nt][r]);        // Eq. 1
          H[nt][r] = fmaf(f, H[nt][r] - z, z);          // Eq. 2
        }
        part[2 * nt] = fmaf(q1, H[nt][2], q0 * H[nt][0]);       // Eq. 3, this thread's two rows
        part[2 * nt + 1] = fmaf(q1, H[nt][3], q0 * H[nt][1]);
      }
#pragma unroll
      for (int x = 0; x < NX; ++x) {
        *reinterpret_cast<float4 *>(hrow0 + 16 * x + 4 * c) = make_float4(H[2 * x][0], H[2 * x][1], H[2 * x + 1][0], H[2 * x + 1][1]);
        *reinterpret_cast<float4 *>(hrow1 + 16 * x + 4 * c) = make_float4(H[2 * x][2], H[2 * x][3], H[2 * x + 1][2], H[2 * x + 1][3]);
      }
      // column sums over the warp's 16 rows; idx = 2nt+e of a thread <-> memory column 16(idx>>2)+4c+(idx&3)
      reduce_over_rows<SEG>(part, lane);
      using RO = RowReduceOut<V>;
      if (RO::owner(lane)) {
        const int idx0 = (g >> (3 - RO::R)) * RO::CNT;
#pragma unroll
        for (int j = 0; j < RO::CNT; ++j) {
          const int idx = idx0 + j;
          const int col = V == 16 ? 4 * c + idx : 16 * (idx >> 2) + 4 * c + (idx & 3);
          yp[col] = part[j];
        }
      }
    }
    __syncthreads();
    // y = sum over the unit's warps (+ w_r (.) v)
    for (int x = tid; x < GPI * V; x += blockDim.x) {
      const int gi = x / V, j = x % V;
      const int bb = (int)(task % tasks_per_head) * GPI + gi;
      if (bb < B) {
        const float *p = ypart + (size_t)(((it & 1) * GPI + gi) * WPU) * V + j;
        float s = 0.f;
        for (int w = 0; w < WPU; ++w) s += p[(size_t)w * V];
        const size_t bn = (size_t)bb * N + n;
        if (wr) s = fmaf(__bfloat162float(wr[(size_t)n * V + j]), __bfloat162float(vg[bn * V + j]), s);
        yg[bn * V + j] = __float2bfloat16_rn(s);
      }
    }
  }
}

template <int V>
cudaError_t launch_decode_v(const ScanArgs &a, cudaStream_t s) {
  const int WPU = a.K / 16;
  const int GPI = WPU >= 8 ? 1 : 8 / WPU;   // units taken by a CTA at a time
  const int tasks_per_head = (a.B + GPI - 1) / GPI;
  const long ntasks = (long)a.N * tasks_per_head;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = (int)(ntasks < sms ? ntasks : sms);
  const size_t smem = 16 + (size_t)(V / 16) * (V / 8) * 32 * 8 + sizeof(float) * 2 * GPI * WPU * V   // barriers, W, y partials
                      + sizeof(float) * 2 * (size_t)GPI * a.K * V;                                   // two stages of states
  cudaError_t e = cudaFuncSetAttribute(decode_bf16_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  decode_bf16_kernel<V><<<grid, 256, smem, s>>>(a, WPU, GPI, tasks_per_head);
  return cudaGetLastError();
}

}  // namespace

// The tcgen05 kernel takes the shapes whose states stack into a 128-row tile; the mma.sync kernel
// above covers the rest.  M2RNN_DECODE_VARIANT=legacy forces the latter (benchmarking only).
cudaError_t launch_decode_bf16(const ScanArgs &a, cudaStream_t s) {
  const char *variant = getenv("M2RNN_DECODE_VARIANT");
  if (decode_tc_supported(a) && !(variant && !strcmp(variant, "legacy"))) return launch_decode_tc_bf16(a, s);
  switch (a.V) {
    case 16: return launch_decode_v<16>(a, s);
    case 32: return launch_decode_v<32>(a, s);
    case 64: return launch_decode_v<64>(a, s);
    case 128: return launch_decode_v<128>(a, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace m2rnn

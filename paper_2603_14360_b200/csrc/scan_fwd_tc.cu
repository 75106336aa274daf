// bf16 forward scan (Algorithm 1) on the 5th-generation tensor cores: tcgen05.mma with operand A
// and the accumulator in tensor memory, transposed so that the transition matrix is stationary.
//
// Per step the state x W product of Eq. 1 is computed as its transpose,
//     P^T [V x rows] = W^T [V x V]  .  H^T [V x rows],
// with M = 128 lanes of tensor memory = state columns, N = 16 state rows per chain group and
// K = 128.  W^T sits in tensor memory for the whole scan (the MMA's A operand: read from there, the
// tensor core does not stream the 32 KB of W through shared memory every step, which cost ~90 cycles
// per MMA when A was a shared-memory tile); the B operand is the bf16 copy of the 16 x 128 state
// slab in shared memory, row-major (which is K-major for B), rewritten by the epilogue threads every
// step.  For V < 128 the tile takes 128 / V heads at once: A is block diagonal (W_n^T per head), a
// tensor-memory lane is (head slot, column).  The wasted MMA work is free: the step is bound by the
// tanh unit and by the latency of the round trip, not by the tensor pipe.
//
// What this layout buys along the step's dependency chain:
//   - a thread owns one state column and 8 of the slab's 16 rows (tcgen05.ld 32x32b: lane = column,
//     registers = rows; two warps share a lane quarter), so v_t[j] and f_t are per-thread scalars
//     and k_t[i], q_t[i] are warp-uniform broadcasts;
//   - the readout y_t[j] = sum_i q_t[i] H_t[i][j] is a sum over a thread's own registers: no shuffles;
//   - the state stays in fp32 registers; one thread per group issues the 8 MMAs of the next step.
// A CTA runs two independent chain groups of 8 warps (two 16-row slabs of the same unit group):
// while one waits for its MMAs the other one's epilogue keeps the tanh unit busy.  Service warps
// stage q, k, v and the gate (as in the other forward kernels) and write y.  Every wait is bounded.
#include <cstdlib>

#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"

namespace m2rnn {
namespace {

constexpr int kStagesTc = 3;
constexpr int kGroups = 2;            // chain groups per CTA
constexpr int kWarpsG = 8;            // warps per group: lane quarter (warp % 4) x row half (warp / 4)
constexpr int kSvcWarps = 4;
constexpr int kChainThreads = kGroups * kWarpsG * 32;
constexpr int kThreadsTc = kChainThreads + kSvcWarps * 32;
constexpr int kTmemCols = 128;        // 64 columns of W^T (128 K indices, two bf16 per column) + NR (<= 32) per group
constexpr int kTmemD = 64;            // first accumulator column

template <int V, int NR>
struct TcFwdSmem {
  static constexpr int kRowsG = NR, kRowsCta = kGroups * NR;
  static constexpr int HS = 128 / V;                         // heads per tile
  static constexpr int TC = HS * NR >= 64 ? 8 : 16;          // steps per stage
  static constexpr uint32_t b_bytes = kRowsG * 128 * 2;      // B of one group: 2 blocks of [NR rows][128 bytes]
  static constexpr uint32_t oB = 0, oBar = oB + kGroups * b_bytes, oStage = oBar + 128;
  // per stage (floats): k [TC][HS][rows of the CTA], q likewise, v [TC][128], f [TC][8],
  // y [TC][groups][row halves][128]
  static constexpr int kOff = 0, qOff = TC * HS * kRowsCta, vOff = 2 * qOff, fOff = vOff + TC * 128, yOff = fOff + TC * 8;
  static constexpr int stage_floats = yOff + TC * kGroups * 2 * 128;
  static constexpr uint32_t total = oStage + kStagesTc * stage_floats * 4 + 1024;   // + slack to align the base
};

template <int V, int NR, bool CKPT>
__global__ void __launch_bounds__(kThreadsTc, 1) fwd_tc_kernel(ScanArgs a) {
  using S = TcFwdSmem<V, NR>;
  constexpr int HS = S::HS, TC = S::TC;
  constexpr int kRowsG = NR;            // state rows per group = N of the MMA
  constexpr int kRowsT = NR / 2;        // state rows per thread
  constexpr int kRowsCta = kGroups * NR;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base_sa = (smem_u32(smem_dyn) + 1023u) & ~1023u;   // the swizzled tiles want 1024-byte alignment
  unsigned char *base = smem_dyn + (base_sa - smem_u32(smem_dyn));
  uint64_t *full = reinterpret_cast<uint64_t *>(base + S::oBar);    // [kStagesTc] a stage's inputs are staged
  uint64_t *done = full + kStagesTc;                                // [kStagesTc] the chain warps are through with it
  uint64_t *mma_done = done + kStagesTc;                            // [kGroups] the group's product has landed in tensor memory
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(mma_done + kGroups);
  float *stages = reinterpret_cast<float *>(base + S::oStage);

  const int K = a.K, N = a.N;
  // the warp index by way of a shuffle: the compiler then knows it is the same in all lanes, and
  // what is derived from it (the group's tiles and barriers, the MMA descriptors) stays in uniform
  // registers; an MMA issued from values it takes for per-thread ones cost ~65 cycles each
  const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
  const int NG = (N + HS - 1) / HS;               // head groups
  const int RS = (K + kRowsCta - 1) / kRowsCta;   // CTAs per (b, head group)
  const int rs = blockIdx.x % RS, hg = (blockIdx.x / RS) % NG, b = blockIdx.x / (RS * NG);
  const int rbase = rs * kRowsCta;
  const UnitSpan span = unit_span(a, b);   // this batch entry's tokens (a slice of a packed batch, or b T ..)
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int groups_live = min(kGroups, (K - rbase) / kRowsG);
  const int nchunks = (T + TC - 1) / TC;
  const bool want_y = a.y != nullptr || a.y_part != nullptr;

  if (tid == 0) {
    for (int s = 0; s < kStagesTc; ++s) {
      mbar_init(&full[s], kSvcWarps);
      mbar_init(&done[s], kWarpsG * groups_live);
    }
    for (int g = 0; g < kGroups; ++g) mbar_init(&mma_done[g], 1);
    fence_mbar_init();
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // inputs of absent heads (N not a multiple of the heads per tile) read as zero in every stage
  for (int x = tid; x < kStagesTc * S::stage_floats; x += kThreadsTc) stages[x] = 0.f;
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  bool failed = false;

  if (warp < 4) {
    // A = block-diagonal W_n^T of the group's heads, into tensor memory: lane jj = (head slot, column
    // j) holds W_n[l][j] at K index ll = (same head slot, l), zero elsewhere; column c holds the K
    // indices 2c (low half) and 2c + 1
    const int jj = 32 * warp + lane, hs = jj / V, j = jj % V, n = hg * HS + hs;
    const uint16_t *w = reinterpret_cast<const uint16_t *>(a.W) + (size_t)(n < N ? n : 0) * V * V + j;
#pragma unroll 1
    for (int c0 = 0; c0 < 64; c0 += 8) {
      uint32_t r[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int ll = 2 * (c0 + e);
        r[e] = (ll / V == hs && n < N) ? ((uint32_t)w[(size_t)(ll % V) * V] | ((uint32_t)w[(size_t)(ll % V + 1) * V] << 16)) : 0u;
      }
      tmem_st8(tmem_base + ((uint32_t)(32 * warp) << 16) + (uint32_t)c0, r);
    }
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  if (warp >= kGroups * kWarpsG) {
    // ------------------------------------------------------------------ service warps
    const int sl = tid - kChainThreads;          // 0 .. 127
    constexpr int kSvc = kSvcWarps * 32;
    const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(a.q), *kg = static_cast<const __nv_bfloat16 *>(a.k);
    const __nv_bfloat16 *vg = static_cast<const __nv_bfloat16 *>(a.v), *wr = static_cast<const __nv_bfloat16 *>(a.w_r);
    const int rows_cta = groups_live * kRowsG;        // live rows of this CTA's slab pair
    const int heads_live = min(HS, N - hg * HS);
    const int dq = N / a.Nq, dk = N / a.Nk;

    auto fill = [&](int ch) {
      const int s = ch % kStagesTc, t0 = ch * TC, len = min(TC, T - t0);
      float *st = stages + (size_t)s * S::stage_floats;
      const size_t bt0 = tok0 + t0;
      // k and q: per (step, head slot) rows_cta bf16 = rows_cta / 8 chunks of 16 bytes
      const int cpr = rows_cta / 8, nkq = len * heads_live * cpr;
      for (int x = sl; x < nkq; x += kSvc) {
        const int c = x % cpr, hs = (x / cpr) % heads_live, t = x / (cpr * heads_live), n = hg * HS + hs;
        const uint4 rk = *reinterpret_cast<const uint4 *>(kg + (bt0 + t) * a.ks + (n / dk) * K + rbase + 8 * c);
        store8_bf16_as_f32(st + S::kOff + (t * HS + hs) * kRowsCta + 8 * c, rk);
        if (want_y) {
          const uint4 rq = *reinterpret_cast<const uint4 *>(qg + (bt0 + t) * a.qs + (n / dq) * K + rbase + 8 * c);
          store8_bf16_as_f32(st + S::qOff + (t * HS + hs) * kRowsCta + 8 * c, rq);
        }
      }
      // v: the group's heads are adjacent in memory: heads_live * V contiguous bf16 per step
      const int vpr = heads_live * V / 8, nv = len * vpr;
      for (int x = sl; x < nv; x += kSvc) {
        const int c = x % vpr, t = x / vpr;
        const uint4 rv = *reinterpret_cast<const uint4 *>(vg + (bt0 + t) * a.vs + hg * HS * V + 8 * c);
        store8_bf16_as_f32(st + S::vOff + t * 128 + 8 * c, rv);
      }
      for (int x = sl; x < len * heads_live; x += kSvc) {
        const int hs = x % heads_live, t = x / heads_live, n = hg * HS + hs;
        st[S::fOff + t * 8 + hs] = gate_value(a.gate_kind, a.gate[(bt0 + t) * N + n], a.alpha ? a.alpha[n] : 1.f,
                                              a.beta ? a.beta[n] : 0.f, nullptr);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&full[s]);
    };

    const int pre = min(kStagesTc, nchunks);
    for (int ch = 0; ch < pre; ++ch) fill(ch);
    for (int ch = 0; ch < nchunks; ++ch) {
      const int s = ch % kStagesTc, t0 = ch * TC, len = min(TC, T - t0);
      if (!mbar_wait<1000>(&done[s], (ch / kStagesTc) & 1)) { failed = true; break; }
      if (want_y) {
        // y[t][8 columns] = the groups' and row halves' shares (+ w_r (.) v); a step's 128 lanes are
        // contiguous in y
        const float *st = stages + (size_t)s * S::stage_floats;
        const int cpt = heads_live * V / 8;
        for (int x = sl; x < len * cpt; x += kSvc) {
          const int c = x % cpt, t = x / cpt;
          float acc[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] = 0.f;
          for (int p = 0; p < 2 * groups_live; ++p) {
            const float4 p0 = *reinterpret_cast<const float4 *>(st + S::yOff + (t * 2 * kGroups + p) * 128 + 8 * c);
            const float4 p1 = *reinterpret_cast<const float4 *>(st + S::yOff + (t * 2 * kGroups + p) * 128 + 8 * c + 4);
            acc[0] += p0.x; acc[1] += p0.y; acc[2] += p0.z; acc[3] += p0.w;
            acc[4] += p1.x; acc[5] += p1.y; acc[6] += p1.z; acc[7] += p1.w;
          }
          if (wr && rs == 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              acc[e] = fmaf(__bfloat162float(wr[(size_t)hg * 128 + 8 * c + e]), st[S::vOff + t * 128 + 8 * c + e], acc[e]);
          }
          const size_t yo = ((tok0 + t0 + t) * N + hg * HS) * V + 8 * c;
          if (a.y_part) {   // this CTA's share of y, fp32; the shares are added by a second kernel
            float *yp = a.y_part + (size_t)rs * a.TT * N * V + yo;
            *reinterpret_cast<float4 *>(yp) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            *reinterpret_cast<float4 *>(yp + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
          } else {
            uint4 o;
            o.x = pack_bf16(acc[0], acc[1]); o.y = pack_bf16(acc[2], acc[3]);
            o.z = pack_bf16(acc[4], acc[5]); o.w = pack_bf16(acc[6], acc[7]);
            *reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(a.y) + yo) = o;
          }
        }
        __syncwarp();
      }
      if (ch + kStagesTc < nchunks) fill(ch + kStagesTc);
    }
  } else if (warp / kWarpsG < groups_live) {
    // -------------------------------------------------------------------- chain warps
    const int g = warp / kWarpsG, wg = warp % kWarpsG;
    const int quarter = wg & 3, half = wg >> 2;      // tensor-memory lane quarter, row half of the slab
    const int L = 32 * quarter + lane;               // tensor-memory lane = (head slot, state column)
    const int hs = L / V, j = L % V, n = hg * HS + hs;
    const bool head_live = n < N;
    const int r0 = rbase + kRowsG * g + kRowsT * half;   // first of this thread's 8 state rows
    const size_t KV = (size_t)K * V;
    const size_t bn = (size_t)b * N + (head_live ? n : 0);
    const uint32_t d_tmem = tmem_base + (uint32_t)(kTmemD + kRowsG * g);
    const uint32_t taddr = d_tmem + ((uint32_t)(32 * quarter) << 16) + (uint32_t)(kRowsT * half);
    const uint32_t b_sa = base_sa + S::oB + (uint32_t)g * S::b_bytes;
    // this thread's 2-byte slots in the B tile: row i = 8 half + x, K index L: block L / 64, 16-byte
    // chunk ((L % 64) / 8) ^ (i % 8) of the row
    uint32_t b_addr[kRowsT];
#pragma unroll
    for (int x = 0; x < kRowsT; ++x) {
      const int i = kRowsT * half + x;
      b_addr[x] = b_sa + (uint32_t)(L >> 6) * (kRowsG * 128) + (uint32_t)i * 128u + ((((uint32_t)(L & 63) >> 3) ^ (uint32_t)(i & 7)) << 4) +
                  (uint32_t)(L & 7) * 2u;
    }
    constexpr uint32_t idesc = idesc_bf16(128, kRowsG);

    float H[kRowsT];
    if (a.h0 && head_live) {
#pragma unroll
      for (int i = 0; i < kRowsT; ++i) H[i] = a.h0[bn * KV + (size_t)(r0 + i) * V + j];
    } else {
#pragma unroll
      for (int i = 0; i < kRowsT; ++i) H[i] = 0.f;
    }
    // bf16 copy of the slab -> B tile, then the 8 MMAs of the next step's product (one thread)
    auto publish_and_issue = [&](bool issue) {
#pragma unroll
      for (int i = 0; i < kRowsT; i += 2) {
        const uint32_t pk = pack_bf16(H[i], H[i + 1]);
        asm volatile("st.shared.b16 [%0], %1;" ::"r"(b_addr[i]), "h"((uint16_t)(pk & 0xffffu)) : "memory");
        asm volatile("st.shared.b16 [%0], %1;" ::"r"(b_addr[i + 1]), "h"((uint16_t)(pk >> 16)) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> visible to the tensor core
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "n"(kWarpsG * 32) : "memory");
      if (issue && wg == 0 && elect_one()) {   // warp-uniform condition, then one elected lane
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          // 16 K indices per MMA: 8 columns of A, 32 bytes inside a 128-byte row of B (then the next
          // 64-index block)
          const uint32_t bo = (uint32_t)(kk >> 2) * (kRowsG * 128) + (uint32_t)(kk & 3) * 32u;
          umma_bf16_ts(d_tmem, tmem_base + 8u * kk, smem_desc_sw128(b_sa + bo), idesc, kk > 0);
        }
        umma_commit_tc(&mma_done[g]);
      }
    };
    publish_and_issue(T > 0);

    uint32_t it = 0;           // products waited for so far
    int ck_left = 0, ck_idx = 0;
    for (int ch = 0; ch < nchunks && !failed; ++ch) {
      const int s = ch % kStagesTc, len = min(TC, T - ch * TC);
      if (!mbar_wait(&full[s], (ch / kStagesTc) & 1)) { failed = true; break; }
      float *st = stages + (size_t)s * S::stage_floats;
      const float *kp = st + S::kOff + hs * kRowsCta + kRowsG * g + kRowsT * half;
      const float *qp = st + S::qOff + hs * kRowsCta + kRowsG * g + kRowsT * half;
      const float *vp = st + S::vOff + L, *fp = st + S::fOff + hs;
      float *yp = st + S::yOff + (2 * g + half) * 128 + L;
#pragma unroll 1
      for (int tl = 0; tl < len; ++tl) {
        if constexpr (CKPT) {
          if (ck_left == 0) {
            if (head_live) {
              float *dst = a.ckpt + (bn * a.nchunks + ck_idx) * KV + (size_t)r0 * V + j;
#pragma unroll
              for (int i = 0; i < kRowsT; ++i) dst[(size_t)i * V] = H[i];
            }
            ++ck_idx;
            ck_left = a.C;
          }
          --ck_left;
        }
        // this step's vectors (they do not depend on the product in flight)
        float kk[kRowsT], qq[kRowsT];
#pragma unroll
        for (int x = 0; x < kRowsT / 4; ++x) {
          const float4 k4 = *reinterpret_cast<const float4 *>(kp + 4 * x), q4 = *reinterpret_cast<const float4 *>(qp + 4 * x);
          kk[4 * x] = k4.x; kk[4 * x + 1] = k4.y; kk[4 * x + 2] = k4.z; kk[4 * x + 3] = k4.w;
          qq[4 * x] = q4.x; qq[4 * x + 1] = q4.y; qq[4 * x + 2] = q4.z; qq[4 * x + 3] = q4.w;
        }
        const float vj = *vp, f = *fp;
        // P = H_{t-1} W, this thread's column and rows
        if (!mbar_wait(&mma_done[g], it & 1u)) { failed = true; break; }
        ++it;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float P[kRowsT];
        tmem_ld(taddr, P);
        const float2 v2 = make_float2(vj, vj), f2 = make_float2(f, f), m1 = make_float2(-1.f, -1.f);
        float2 yacc = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kRowsT; i += 2) {
          const float2 pre = __ffma2_rn(make_float2(kk[i], kk[i + 1]), v2, make_float2(P[i], P[i + 1]));
          const float2 z = make_float2(tanh_approx(pre.x), tanh_approx(pre.y));           // Eq. 1
          const float2 d = __ffma2_rn(z, m1, make_float2(H[i], H[i + 1]));                 // H - Z
          const float2 h = __ffma2_rn(f2, d, z);                                          // Eq. 2
          H[i] = h.x; H[i + 1] = h.y;
          yacc = __ffma2_rn(make_float2(qq[i], qq[i + 1]), h, yacc);                      // Eq. 3, this thread's rows
        }
        if (want_y) *yp = yacc.x + yacc.y;
        const bool last = ch == nchunks - 1 && tl == len - 1;
        publish_and_issue(!last);
        kp += HS * kRowsCta; qp += HS * kRowsCta; vp += 128; fp += 8; yp += 2 * kGroups * 128;
      }
      __syncwarp();
      if (lane == 0 && !failed) mbar_arrive(&done[s]);
    }
    if (a.hT && head_live && !failed) {
#pragma unroll
      for (int i = 0; i < kRowsT; ++i) a.hT[bn * KV + (size_t)(r0 + i) * V + j] = H[i];
    }
  }
  if (failed) report_timeout(a.dev_status);
  // common exit: every loop above ends after a bounded time
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

template <int V, int NR, bool CKPT>
cudaError_t launch_tc_fwd(const ScanArgs &a, cudaStream_t s) {
  constexpr int HS = 128 / V, kRowsCta = kGroups * NR;
  const size_t smem = TcFwdSmem<V, NR>::total;
  cudaError_t e = cudaFuncSetAttribute(fwd_tc_kernel<V, NR, CKPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int NG = (a.N + HS - 1) / HS, RS = (a.K + kRowsCta - 1) / kRowsCta;
  fwd_tc_kernel<V, NR, CKPT><<<a.B * NG * RS, kThreadsTc, smem, s>>>(a);
  return cudaGetLastError();
}

template <int V>
cudaError_t launch_tc_v(const ScanArgs &a, cudaStream_t s) {
  // a.KCf = rows per CTA chosen by the plan: two groups of 16 or of 32 rows
  if (a.KCf == 64) return a.ckpt ? launch_tc_fwd<V, 32, true>(a, s) : launch_tc_fwd<V, 32, false>(a, s);
  return a.ckpt ? launch_tc_fwd<V, 16, true>(a, s) : launch_tc_fwd<V, 16, false>(a, s);
}

}  // namespace

// Rows per CTA of this kernel for a problem: two groups of 32 rows where that still spreads the
// problem over the SMs (or fills them twice), else two groups of 16; K itself when it is smaller.
int fwd_tc_rows_per_cta(int B, int N, int K, int V) {
  const char *rows = getenv("M2RNN_TC_ROWS");      // benchmarking only: 32 or 64
  int r;
  if (rows) {
    r = atoi(rows) == 64 ? 64 : 32;
  } else {
    const int HS = 128 / V;
    const long tiles = (long)(B > 0 ? B : 1) * ((N + HS - 1) / HS);
    r = (K % 64 == 0 && 4 * tiles * (K / 64) >= 3L * sm_count()) ? 64 : 32;
  }
  if (r == 64 && K % 32) r = 32;
  return r;
}

cudaError_t launch_fwd_bf16_tc(const ScanArgs &a, cudaStream_t s) {
  switch (a.V) {
    case 16: return launch_tc_v<16>(a, s);
    case 32: return launch_tc_v<32>(a, s);
    case 64: return launch_tc_v<64>(a, s);
    case 128: return launch_tc_v<128>(a, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace m2rnn

// bf16 tensor-core forward scan (Algorithm 1) for sm_100a.
//
// One CTA per (b, n, row slab) -- the K rows of a state are independent recurrences (Eq. 1-2 act
// row by row), so a state may be split over several CTAs, whose partial readouts a second-stage
// kernel adds.  Below, K is the slab's row count.  Per CTA: K/16 compute warps, each holding a 16 x V slab of the state in registers
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
#include <cstdlib>
#include <cstring>

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
  __host__ __device__ static constexpr int tc(int K) { return (V >= 128 || K > 64) ? 8 : 16; }
  __host__ static size_t bytes(int K) {
    const int TC = tc(K);
    size_t b = sizeof(float) * (size_t)kStages * stage_floats(K, TC);
    if (V > 64) b += (size_t)V * V * 2;  // W fragments
    return b + kBarrierBytes;
  }
};

// MAXW: most compute warps the instantiation is launched with (K <= 16*MAXW).  Registers are
// granted per 4 warps: up to 4+1 warps leave 255 per thread, 8+1 warps only 168.
// CKPT: whether checkpoints are written (a compile-time switch keeps the branch out of the hot loop).
// OCC: CTAs per SM the kernel is compiled for.  With more (b,n) units than SMs, two co-resident
// CTAs (two chain warps per scheduler) hide each other's latencies; the price is a smaller
// register budget.
// NWT: the slab count when it is known at compile time (0: read from the arguments); with it every
// shared-memory offset of a step is an immediate.
template <int V, int MAXW, bool CKPT, int OCC, int NWT = 0>
__global__ void __launch_bounds__((MAXW + 1) * 32, OCC) fwd_bf16_kernel(ScanArgs a) {
  using G = TileGeom<V>;
  constexpr int NT = G::NT, KT = G::KT, SEG = G::SEG;
  constexpr bool kWInRegs = V <= 64;
  // The product of a step is split over NSET accumulator sets (k-tile kt adds into set kt % NSET,
  // the sets are summed where they are used): an mma.sync that accumulates onto the previous
  // one's result waits for its whole latency (well over 100 cycles), so KT of them in a row
  // would be most of the step.
  constexpr int NSET = V == 128 ? 1 : (KT >= 2 ? 2 : 1);
  extern __shared__ __align__(16) unsigned char smem_raw[];

  const int Kf = a.K, N = a.N;                       // rows of the whole state
  const int K = NWT ? 16 * NWT : a.KCf;              // rows of this CTA's slab
  const int RS = Kf / K;
  const int NW = NWT ? NWT : (K >> 4);
  constexpr bool kPacked = V <= 64;                  // packed fp32x2 arithmetic (spills at V = 128)
  constexpr int TC = FwdSmem<V>::tc(MAXW * 16);   // K > 64 <=> MAXW == 8
  const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;   // (through a shuffle: known to be warp-uniform)
  const int bn = blockIdx.x / RS, rs = blockIdx.x % RS, b = bn / N, n = bn % N;
  const UnitSpan span = unit_span(a, b);   // this batch entry's tokens (a slice of a packed batch, or b T ..)
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int rbase = rs * K;   // first state row of this CTA
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
      const size_t bt0 = tok0 + t0;
      const int kq8 = K / 8, v8 = V / 8;
      uint4 rk[kPerLane], rq[kPerLane], rv[kPerLane];
      float gt = 0.f;
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        const int x = lane + 32 * i;
        if (x < len * kq8) {
          const int t = x / kq8, j = (x % kq8) * 8;
          rk[i] = *reinterpret_cast<const uint4 *>(kg + (bt0 + t) * a.ks + hk * Kf + rbase + j);
          if (want_y) rq[i] = *reinterpret_cast<const uint4 *>(qg + (bt0 + t) * a.qs + hq * Kf + rbase + j);
        }
        if (x < len * v8) {
          const int t = x / v8, j = (x % v8) * 8;
          rv[i] = *reinterpret_cast<const uint4 *>(vg + (bt0 + t) * a.vs + n * V + j);
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
      if (!mbar_wait<1000>(&done[s], (ch / kStages) & 1)) { report_timeout(a.dev_status); return; }
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
          if (wr && rs == 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(__bfloat162float(wr[(size_t)n * V + j + e]), vS[t * V + j + e], acc[e]);
          }
          const size_t yo = ((tok0 + t0 + t) * N + n) * V + j;
          if (a.y_part) {   // this slab's share of y, fp32; the slabs are added by a second kernel
            float *yp = a.y_part + (size_t)rs * a.TT * N * V + yo;
            *reinterpret_cast<float4 *>(yp) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            *reinterpret_cast<float4 *>(yp + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
          } else {
            uint4 o;
            o.x = pack_bf16(acc[0], acc[1]); o.y = pack_bf16(acc[2], acc[3]);
            o.z = pack_bf16(acc[4], acc[5]); o.w = pack_bf16(acc[6], acc[7]);
            *reinterpret_cast<uint4 *>(yg + yo) = o;
          }
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
  const size_t KV = (size_t)Kf * V;

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
      const float *src = a.h0 + bn * KV + (size_t)(rbase + row0 + h) * V + SEG * c;
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
  auto store_state = [&](float *dst) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float *p = dst + (size_t)(rbase + row0 + h) * V + SEG * c;
#pragma unroll
      for (int x = 0; x < SEG / 4; ++x)
        *reinterpret_cast<float4 *>(p + 4 * x) =
            make_float4(H[2 * x][2 * h], H[2 * x][2 * h + 1], H[2 * x + 1][2 * h], H[2 * x + 1][2 * h + 1]);
    }
  };

  // P <- k v^T  (the outer-product term of Eq. 1 seeds the accumulators)
  // (shared-memory operands of the hot loop are 32-bit shared addresses, in bytes)
  auto seed = [&](float (&P)[NSET][NT][4], uint32_t krow, uint32_t vrow) {
    const float2 kk = lds64(krow + 4 * row0);
#pragma unroll
    for (int x = 0; x < SEG / 4; ++x) {
      const float4 v4 = lds128(vrow + 4 * (SEG * c + 4 * x));
      if constexpr (kPacked) {   // one instruction per two products
        const float2 k02 = make_float2(kk.x, kk.x), k12 = make_float2(kk.y, kk.y);
        const float2 a0 = __fmul2_rn(k02, make_float2(v4.x, v4.y)), a1 = __fmul2_rn(k12, make_float2(v4.x, v4.y));
        const float2 b0 = __fmul2_rn(k02, make_float2(v4.z, v4.w)), b1 = __fmul2_rn(k12, make_float2(v4.z, v4.w));
        P[0][2 * x][0] = a0.x; P[0][2 * x][1] = a0.y; P[0][2 * x][2] = a1.x; P[0][2 * x][3] = a1.y;
        P[0][2 * x + 1][0] = b0.x; P[0][2 * x + 1][1] = b0.y; P[0][2 * x + 1][2] = b1.x; P[0][2 * x + 1][3] = b1.y;
      } else {
        P[0][2 * x][0] = kk.x * v4.x; P[0][2 * x][1] = kk.x * v4.y; P[0][2 * x][2] = kk.y * v4.x; P[0][2 * x][3] = kk.y * v4.y;
        P[0][2 * x + 1][0] = kk.x * v4.z; P[0][2 * x + 1][1] = kk.x * v4.w; P[0][2 * x + 1][2] = kk.y * v4.z; P[0][2 * x + 1][3] = kk.y * v4.w;
      }
    }
  };
  // P += A[kt] * W[kt][:]  : one k tile of H W
  auto mma_ktile = [&](float (&P)[NSET][NT][4], const uint32_t (&Ak)[4], int kt) {
    const int set = kt % NSET;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      if constexpr (kWInRegs) {
        if (kt >= 1 && kt < NSET) mma_bf16_16816_zero(P[set][nt], Ak, Wr[kt][nt][0], Wr[kt][nt][1]);
        else mma_bf16_16816(P[set][nt], Ak, Wr[kt][nt][0], Wr[kt][nt][1]);
      } else {
        const uint2 w = Wf[(kt * NT + nt) * 32 + lane];
        if (kt >= 1 && kt < NSET) mma_bf16_16816_zero(P[set][nt], Ak, w.x, w.y);
        else mma_bf16_16816(P[set][nt], Ak, w.x, w.y);
      }
    }
  };

  // transpose of an 8 x 8 tile of 16-bit elements held by a warp: half of an A fragment -> half of a B fragment
  auto movmatrix_trans = [](uint32_t x) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(x));
    return d;
  };
  // One step, software-pipelined by hand: while the MUFU works through tanh of step t, column
  // tile pair by column tile pair, the tensor pipe already runs the k tiles of step t+1 that
  // depend only on the pairs finished so far.  The body is branch-free (one basic block) so the
  // instruction scheduler can interleave the MUFU, tensor and FMA streams.
  //   Pc: H_{t-1} W + k_t v_t^T, complete (or in flight) on entry
  //   Pn: receives H_t W + k_{t+1} v_{t+1}^T; after the last step it is fed a valid but
  //       meaningless row and its result is never read
  auto step = [&](float (&Pc)[NSET][NT][4], float (&Pn)[NSET][NT][4], float f, uint32_t qrow, uint32_t ydst,
                  uint32_t krow_n, uint32_t vrow_n) {
    seed(Pn, krow_n, vrow_n);
    const float2 qq = lds64(qrow + 4 * row0);
    float part[SEG];
    // packed path: the readout (Eq. 3) on the tensor cores, y^T = q^T H over the slab's 16 rows as
    // one more product per accumulator tile: q is row 0 of an otherwise empty A operand (MMA row m
    // <-> memory row 2m, m + 8 <-> 2m + 1), the packed bf16 fragments of H_t, transposed in
    // registers, are B.  It replaces the products and the shuffle tree over the rows, which were
    // half of a V = 16 step's instructions.
    uint32_t Aq[4] = {0u, 0u, 0u, 0u};
    float Y[NT][4];
    if constexpr (kPacked) {
      const float4 q4 = lds128(qrow + 4 * (16 * warp + 4 * c));
      if (g == 0) { Aq[0] = pack_bf16(q4.x, q4.z); Aq[2] = pack_bf16(q4.y, q4.w); }
    }
#pragma unroll
    for (int kt = 0; kt < KT; ++kt) {
#pragma unroll
      for (int nt = 2 * kt; nt < 2 * kt + 2; ++nt) {
        if constexpr (kPacked) {
          float2 hh[2];
#pragma unroll
          for (int h = 0; h < 2; ++h) {   // the two rows' column pairs, as packed fp32 pairs
            float2 x = make_float2(Pc[0][nt][2 * h], Pc[0][nt][2 * h + 1]);
            if constexpr (NSET == 2) x = __fadd2_rn(x, make_float2(Pc[1][nt][2 * h], Pc[1][nt][2 * h + 1]));
            const float2 z = make_float2(tanh_approx(x.x), tanh_approx(x.y));                                      // Eq. 1
            const float2 dd = __ffma2_rn(z, make_float2(-1.f, -1.f), make_float2(H[nt][2 * h], H[nt][2 * h + 1]));  // H - Z
            hh[h] = __ffma2_rn(make_float2(f, f), dd, z);                                                          // Eq. 2
            H[nt][2 * h] = hh[h].x; H[nt][2 * h + 1] = hh[h].y;
          }
        } else {
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            float x = Pc[0][nt][r];
            if constexpr (NSET == 2) x += Pc[1][nt][r];
            const float z = tanh_approx(x);                  // Eq. 1
            H[nt][r] = fmaf(f, H[nt][r] - z, z);             // Eq. 2: f H + (1-f) Z
          }
          part[2 * nt] = fmaf(qq.y, H[nt][2], qq.x * H[nt][0]);      // Eq. 3, this thread's two rows
          part[2 * nt + 1] = fmaf(qq.y, H[nt][3], qq.x * H[nt][1]);
        }
      }
      uint32_t Ak[4];
      Ak[0] = pack_bf16(H[2 * kt][0], H[2 * kt][1]);
      Ak[1] = pack_bf16(H[2 * kt][2], H[2 * kt][3]);
      Ak[2] = pack_bf16(H[2 * kt + 1][0], H[2 * kt + 1][1]);
      Ak[3] = pack_bf16(H[2 * kt + 1][2], H[2 * kt + 1][3]);
      mma_ktile(Pn, Ak, kt);
      if constexpr (kPacked) {   // Eq. 3 for accumulator tiles 2 kt and 2 kt + 1
        mma_bf16_16816_zero(Y[2 * kt], Aq, movmatrix_trans(Ak[0]), movmatrix_trans(Ak[1]));
        mma_bf16_16816_zero(Y[2 * kt + 1], Aq, movmatrix_trans(Ak[2]), movmatrix_trans(Ak[3]));
      }
    }
    if constexpr (kPacked) {
      // row 0 of the products: lanes 0-3 hold the sums over the slab's rows for their SEG columns
      if (g == 0) {
#pragma unroll
        for (int x = 0; x < SEG / 4; ++x)
          sts128(ydst + 4 * (SEG * c + 4 * x), make_float4(Y[2 * x][0], Y[2 * x][1], Y[2 * x + 1][0], Y[2 * x + 1][1]));
      }
    } else {
      reduce_over_rows<SEG>(part, lane);
      using RO = RowReduceOut<V>;
      if (RO::owner(lane)) {
        const uint32_t dst = ydst + 4 * RO::first_col(lane);
        if constexpr (RO::CNT == 4) sts128(dst, make_float4(part[0], part[1], part[2], part[3]));
        else if constexpr (RO::CNT == 2) sts64(dst, make_float2(part[0], part[1]));
        else sts32(dst, part[0]);
      }
    }
  };

  float P0[NSET][NT][4], P1[NSET][NT][4];
  int ck_left = 0, ck_idx = 0;  // steps until the next checkpoint, index of the next checkpoint
  auto maybe_checkpoint = [&](int steps) {   // called before an even-numbered step
    if constexpr (CKPT) {
      if (ck_left == 0) {
        store_state(a.ckpt + ((size_t)bn * a.nchunks + ck_idx) * KV);
        ++ck_idx;
        ck_left = a.C;
      }
      ck_left -= steps;
    }
  };
  const uint32_t stages_sa = smem_u32(stages);
  auto stage_sa = [&](int s) { return stages_sa + 4u * (uint32_t)(s * stage_floats); };
  // byte offsets of the arrays inside a stage
  const uint32_t oK = 4u * TC * K, oV = 2 * oK, oF = oV + 4u * TC * V, oY = oF + 4u * TC;

  if (T > 0) {
    if (!mbar_wait(&full[0], 0)) { report_timeout(a.dev_status); return; }
    // prologue: the first step's product from the initial state
    seed(P0, stages_sa + oK, stages_sa + oV);
#pragma unroll
    for (int kt = 0; kt < KT; ++kt) {
      uint32_t Ak[4];
      Ak[0] = pack_bf16(H[2 * kt][0], H[2 * kt][1]);
      Ak[1] = pack_bf16(H[2 * kt][2], H[2 * kt][3]);
      Ak[2] = pack_bf16(H[2 * kt + 1][0], H[2 * kt + 1][1]);
      Ak[3] = pack_bf16(H[2 * kt + 1][2], H[2 * kt + 1][3]);
      mma_ktile(P0, Ak, kt);
    }
  }
  // Steps are taken in pairs (P0 -> P1 -> P0); the two steps of a pair form one basic block, so
  // the tail of the first (row reduction, last MMAs in flight) overlaps the head of the second.
  // TC and the checkpoint interval are even: stage hand-over and checkpoints fall between pairs.
  // All hand-over logic sits outside the loop over the pairs of a stage, whose body is
  // straight-line code: a warp issues in order, and every branch in that loop used to cost the
  // chain tens of cycles per step.
  auto pair = [&](uint32_t st, int tl, uint32_t k2, uint32_t v2) {
    const uint32_t yp = st + oY + 4u * ((tl * NW + warp) * V);
    step(P0, P1, lds32(st + oF + 4u * tl), st + 4u * (tl * K), yp, st + oK + 4u * ((tl + 1) * K), st + oV + 4u * ((tl + 1) * V));
    step(P1, P0, lds32(st + oF + 4u * (tl + 1)), st + 4u * ((tl + 1) * K), yp + 4u * (NW * V), k2, v2);
  };
  for (int ch = 0, s = 0; ch < nchunks; ++ch) {
    const int sn = s + 1 == kStages ? 0 : s + 1;
    const uint32_t st = stage_sa(s);
    const int len = min(TC, T - ch * TC);
    // the last step of a stage seeds the first step of the next one (after the last step of the
    // scan: any valid row, the product is never read)
    uint32_t kN = st + oK, vN = st + oV;
    if (ch + 1 < nchunks) {
      if (!mbar_wait(&full[sn], ((ch + 1) / kStages) & 1)) { report_timeout(a.dev_status); return; }
      kN = stage_sa(sn) + oK;
      vN = stage_sa(sn) + oV;
    }
    if (len == TC) {
      constexpr int kUnroll = 4;   // steps per loop iteration (TC is a multiple of 4)
#pragma unroll 1
      for (int t0 = 0; t0 < TC - kUnroll; t0 += kUnroll) {
#pragma unroll
        for (int u = 0; u < kUnroll; u += 2) {
          const int tl = t0 + u;
          maybe_checkpoint(2);
          pair(st, tl, st + oK + 4u * ((tl + 2) * K), st + oV + 4u * ((tl + 2) * V));
        }
      }
#pragma unroll
      for (int u = 0; u < kUnroll; u += 2) {
        const int tl = TC - kUnroll + u;
        maybe_checkpoint(2);
        if (u + 2 < kUnroll) pair(st, tl, st + oK + 4u * ((tl + 2) * K), st + oV + 4u * ((tl + 2) * V));
        else pair(st, tl, kN, vN);
      }
    } else {   // ragged last stage
      int tl = 0;
      for (; tl + 1 < len; tl += 2) {
        maybe_checkpoint(2);
        const int nx = tl + 2 < len ? tl + 2 : tl + 1;
        pair(st, tl, st + oK + 4u * (nx * K), st + oV + 4u * (nx * V));
      }
      if (len & 1) {
        maybe_checkpoint(1);
        step(P0, P1, lds32(st + oF + 4u * tl), st + 4u * (tl * K), st + oY + 4u * ((tl * NW + warp) * V),
             st + oK + 4u * (tl * K), st + oV + 4u * (tl * V));
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&done[s]);
    s = sn;
  }
  if (a.hT) store_state(a.hT + bn * KV);
}

template <int V, int MAXW, bool CKPT, int OCC>
cudaError_t launch_vwco(const ScanArgs &a, cudaStream_t s) {
  const size_t smem = FwdSmem<V>::bytes(a.KCf);
  const unsigned grid = a.B * a.N * (a.K / a.KCf), threads = (a.KCf / 16 + 1) * 32;
  if constexpr (V == 16 && MAXW == 4) {
    if (a.KCf == 64) {   // the paper's layer shape (K = 64, V = 16): slab count known at compile time
      cudaError_t e = cudaFuncSetAttribute(fwd_bf16_kernel<V, MAXW, CKPT, OCC, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      fwd_bf16_kernel<V, MAXW, CKPT, OCC, 4><<<grid, threads, smem, s>>>(a);
      return cudaGetLastError();
    }
  }
  cudaError_t e = cudaFuncSetAttribute(fwd_bf16_kernel<V, MAXW, CKPT, OCC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  fwd_bf16_kernel<V, MAXW, CKPT, OCC><<<grid, threads, smem, s>>>(a);
  return cudaGetLastError();
}

template <int V, int MAXW, bool CKPT>
cudaError_t launch_vwc(const ScanArgs &a, cudaStream_t s) {
  // two CTAs per SM where there are units to fill them and the slab count leaves the registers
  if constexpr (MAXW == 4 && V <= 64) {
    const long ctas = (long)a.B * a.N * (a.K / a.KCf);
    // V = 16: the state is small enough for three CTAs per SM, which takes e.g. the 336 units of
    // the paper's layer shape (84 heads x batch 4) in one wave instead of two
    if constexpr (V == 16) {
      if (ctas > 2 * sm_count()) return launch_vwco<V, MAXW, CKPT, 3>(a, s);
    }
    if (ctas > sm_count()) return launch_vwco<V, MAXW, CKPT, 2>(a, s);
  }
  return launch_vwco<V, MAXW, CKPT, 1>(a, s);
}

template <int V, int MAXW>
cudaError_t launch_vw(const ScanArgs &a, cudaStream_t s) {
  return a.ckpt ? launch_vwc<V, MAXW, true>(a, s) : launch_vwc<V, MAXW, false>(a, s);
}

template <int V>
cudaError_t launch_v(const ScanArgs &a, cudaStream_t s) {
  return a.KCf <= 64 ? launch_vw<V, 4>(a, s) : launch_vw<V, 8>(a, s);
}

}  // namespace

// The column-split variant (two chain warps per 16-row slab) takes the shapes it supports; the
// environment variable M2RNN_FWD_VARIANT=wide forces the one-warp-per-slab kernel of this file
// (benchmarking only).
cudaError_t launch_fwd_bf16(const ScanArgs &a, cudaStream_t s) {
  if (fwd_use_tc(a.B, a.N, a.K, a.V, M2RNN_BF16)) return launch_fwd_bf16_tc(a, s);
  const char *variant = getenv("M2RNN_FWD_VARIANT");
  if (fwd_cs_supported(a) && !(variant && !strcmp(variant, "wide"))) return launch_fwd_bf16_cs(a, s);
  switch (a.V) {
    case 16: return launch_v<16>(a, s);
    case 32: return launch_v<32>(a, s);
    case 64: return launch_v<64>(a, s);
    case 128: return launch_v<128>(a, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace m2rnn

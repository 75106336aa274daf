// bf16 tensor-core forward scan (Algorithm 1), column-split variant, for sm_100a.
//
// Same CTA layout and staging as scan_fwd_bf16.cu, but every 16-row slab of the state is shared by
// SP = 2 or 4 chain warps, each owning V/SP of the columns.  A warp's step needs the whole slab as
// the A operand of H W, so the warps of a slab exchange their freshly packed bf16 fragments
// through shared memory once per step (one named barrier per slab).  The exchange hides behind
// the MMAs a warp can already issue from its own fragments.  Each warp holds only its part of W
// (V x V/SP) in registers, which keeps W out of shared memory up to V = 128 (SP = 4 there).  The
// slab count NW is a template parameter and four steps form one loop iteration, so that every
// shared-memory offset of a step is an immediate: the chain warps are bound by the number of
// instructions they issue per step.  Up to four service warps stage q, k, v and the gate and write
// y, one per scheduler, so that no scheduler's chain warps fall behind the others.
//
// Accumulator element map of warp (slab s, part hf), lane (g = lane/4, c = lane%4):
//   rows 16s+g and 16s+g+8; MMA column m of the part  <->  memory column hf*V/SP + SEG*c' + 2*(m>>3) + (m&1)
//   with SEG = V/(4 SP) and c' = (m&7)>>1, i.e. a thread holds SEG adjacent columns of two rows.
#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"

namespace m2rnn {
namespace {

constexpr int kStages = 3;
constexpr int kBarrierBytes = 64;

template <int V>
struct CsSmem {
  // Per stage (floats): q [TC][K], k [TC][K], v [TC][V], f [TC], ypart [TC][K/16][V]
  __host__ __device__ static constexpr int stage_floats(int K, int TC) { return TC * (2 * K + V + 1 + (K / 16) * V); }
  __host__ __device__ static constexpr int tc() { return V >= 128 ? 8 : 16; }
  // fragment exchange: [2 parities][K/16 slabs][V/16 k-tiles (part-major)][32 lanes] x 16 bytes
  __host__ __device__ static int xchg_bytes(int K) { return 2 * (K / 16) * (V / 16) * 32 * 16; }
  __host__ static size_t bytes(int K) {
    return sizeof(float) * (size_t)kStages * stage_floats(K, tc()) + xchg_bytes(K) + kBarrierBytes;
  }
};

// transpose of an 8 x 8 tile of 16-bit elements held by a warp (lane holds row lane/4, elements
// 2 (lane%4), +1 before and after): turns half of an A fragment into half of a B fragment
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// memory column (inside a part of VP columns) of MMA column m of that part
template <int VP>
__host__ __device__ constexpr int part_col(int m) { return (VP / 4) * ((m & 7) >> 1) + 2 * (m >> 3) + (m & 1); }

// service warps of a CTA: one per scheduler that also hosts chain warps, so that staging does not
// weigh on a single scheduler (the chain warps of a slab advance in lockstep with the slowest)
__host__ __device__ constexpr int cs_service_warps(int chain_warps) { return chain_warps < 4 ? chain_warps : 4; }

template <int V, int SP, int NW, bool CKPT, int OCC>
__global__ void __launch_bounds__((SP * NW + cs_service_warps(SP * NW)) * 32, OCC) fwd_bf16_cs_kernel(ScanArgs a) {
  constexpr int kSvc = cs_service_warps(SP * NW);
  constexpr int VH = V / SP;         // columns of a part
  constexpr int NTH = VH / 8;        // accumulator tiles of a warp
  constexpr int KT = V / 16;         // k-tiles of the product
  constexpr int KTH = KT / SP;       // k-tiles a warp produces itself
  constexpr int KTP = KT - KTH;      // k-tiles it receives
  constexpr int SEGH = VH / 4;       // adjacent memory columns per thread
  constexpr int TC = CsSmem<V>::tc();
  constexpr int kUnroll = 4;         // steps per iteration of the stage loop
  extern __shared__ __align__(16) unsigned char smem_raw[];

  constexpr int K = 16 * NW;              // rows of this CTA's slab group (NW slabs of 16 rows): a.KCf
  const int Kf = a.K, N = a.N;            // rows of the whole state
  const int RS = Kf / K;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bn = blockIdx.x / RS, rs = blockIdx.x % RS, b = bn / N, n = bn % N;
  const UnitSpan span = unit_span(a, b);   // this batch entry's tokens (a slice of a packed batch, or b T ..)
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int rbase = rs * K;
  constexpr int stage_floats = CsSmem<V>::stage_floats(K, TC);

  uint64_t *full = reinterpret_cast<uint64_t *>(smem_raw);  // [kStages]
  uint64_t *done = full + kStages;                          // [kStages]
  float *stages = reinterpret_cast<float *>(smem_raw + kBarrierBytes);
  const uint32_t xchg_sa = smem_u32(stages + (size_t)kStages * stage_floats);

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full[s], kSvc);
      mbar_init(&done[s], SP * NW);
    }
    fence_mbar_init();
  }
  const __nv_bfloat16 *Wn = static_cast<const __nv_bfloat16 *>(a.W) + (size_t)n * V * V;
  __syncthreads();

  const int nchunks = (T + TC - 1) / TC;
  const bool want_y = a.y != nullptr;

  if (warp >= SP * NW) {
    // ------------------------------------------------------------------ service warps
    const int sw = warp - SP * NW;   // each takes every kSvc-th group of 32 rows of a stage
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
        if (i % kSvc != sw) continue;
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
      if (sw == kSvc - 1 && lane < len) gt = a.gate[(bt0 + lane) * N + n];
#pragma unroll
      for (int i = 0; i < kPerLane; ++i) {
        if (i % kSvc != sw) continue;
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
      if (sw == kSvc - 1 && lane < len) fS[lane] = gate_value(a.gate_kind, gt, al, be, nullptr);
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
        for (int x = lane + 32 * sw; x < len * v8; x += 32 * kSvc) {
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
      // (a service warp reads, for the residual term, only the rows of v that it refills itself:
      // the two loops split a stage's rows among the service warps in the same way)
      if (ch + kStages < nchunks) fill(ch + kStages);
    }
    return;
  }

  // -------------------------------------------------------------------- chain warps
  const int g = lane >> 2, c = lane & 3;
  const int slab = warp / SP, hf = warp % SP;
  const int r0 = 16 * slab + g;          // slab rows r0 and r0+8  <->  MMA rows g, g+8
  const int col0 = hf * VH + SEGH * c;   // first of this thread's SEGH adjacent memory columns
  const size_t KV = (size_t)Kf * V;

  // B fragments of this warp's half of W: all KT k-tiles x NTH column tiles, kept in the order the
  // warp uses them (its own k-tiles first, then the partner's) so that every index is static
  uint32_t Wr[KT][NTH][2];
  {
    const uint16_t *w = reinterpret_cast<const uint16_t *>(Wn);
#pragma unroll
    for (int kt = 0; kt < KT; ++kt) {
      const int hk = (hf + kt / KTH) % SP, kth = kt % KTH;   // the k-tile's part (own part first, then round the ring) and its index inside it
      const int l0 = hk * VH + part_col<VH>(16 * kth + 2 * c), l1 = hk * VH + part_col<VH>(16 * kth + 2 * c + 1);
      const int l2 = hk * VH + part_col<VH>(16 * kth + 8 + 2 * c), l3 = hk * VH + part_col<VH>(16 * kth + 8 + 2 * c + 1);
#pragma unroll
      for (int nt = 0; nt < NTH; ++nt) {
        const int j = hf * VH + part_col<VH>(8 * nt + g);
        Wr[kt][nt][0] = (uint32_t)w[l0 * V + j] | ((uint32_t)w[l1 * V + j] << 16);
        Wr[kt][nt][1] = (uint32_t)w[l2 * V + j] | ((uint32_t)w[l3 * V + j] << 16);
      }
    }
  }

  // H[nt] = {row r0: cols 2nt, 2nt+1 of the thread's segment | row r0+8: same}
  float H[NTH][4];
  if (a.h0) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float *src = a.h0 + bn * KV + (size_t)(rbase + r0 + 8 * h) * V + col0;
#pragma unroll
      for (int x = 0; x < SEGH / 4; ++x) {
        const float4 t4 = *reinterpret_cast<const float4 *>(src + 4 * x);
        H[2 * x][2 * h] = t4.x; H[2 * x][2 * h + 1] = t4.y; H[2 * x + 1][2 * h] = t4.z; H[2 * x + 1][2 * h + 1] = t4.w;
      }
    }
  } else {
#pragma unroll
    for (int nt = 0; nt < NTH; ++nt) H[nt][0] = H[nt][1] = H[nt][2] = H[nt][3] = 0.f;
  }
  auto store_state = [&](float *dst) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float *p = dst + (size_t)(rbase + r0 + 8 * h) * V + col0;
#pragma unroll
      for (int x = 0; x < SEGH / 4; ++x)
        *reinterpret_cast<float4 *>(p + 4 * x) =
            make_float4(H[2 * x][2 * h], H[2 * x][2 * h + 1], H[2 * x + 1][2 * h], H[2 * x + 1][2 * h + 1]);
    }
  };

  // A fragments of the thread's own columns: k-tile kth of the half = accumulator tiles 2kth, 2kth+1
  auto pack_own = [&](uint32_t (&A)[KTH][4]) {
#pragma unroll
    for (int kth = 0; kth < KTH; ++kth) {
      A[kth][0] = pack_bf16(H[2 * kth][0], H[2 * kth][1]);
      A[kth][1] = pack_bf16(H[2 * kth][2], H[2 * kth][3]);
      A[kth][2] = pack_bf16(H[2 * kth + 1][0], H[2 * kth + 1][1]);
      A[kth][3] = pack_bf16(H[2 * kth + 1][2], H[2 * kth + 1][3]);
    }
  };
  // exchange slot of (parity, slab, half): KTH rows of 32 lanes x 16 bytes
  auto xslot = [&](int par, int h) { return xchg_sa + (uint32_t)((((par * NW + slab) * SP + h) * KTH) * 32 + lane) * 16u; };
  auto xstore = [&](int par, const uint32_t (&A)[KTH][4]) {
#pragma unroll
    for (int kth = 0; kth < KTH; ++kth)
      asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(xslot(par, hf) + 512u * kth), "r"(A[kth][0]), "r"(A[kth][1]),
                   "r"(A[kth][2]), "r"(A[kth][3]) : "memory");
  };
  auto xload = [&](int par, uint32_t (&A)[KTP][4]) {
#pragma unroll
    for (int i = 0; i < KTP; ++i) {
      const int h = (hf + 1 + i / KTH) % SP, kth = i % KTH;   // same ring order as Wr
      asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(A[i][0]), "=r"(A[i][1]), "=r"(A[i][2]), "=r"(A[i][3])
                   : "r"(xslot(par, h) + 512u * kth) : "memory");
    }
  };
  auto pair_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(1 + slab), "n"(32 * SP) : "memory"); };

  // P <- k v^T, then the own k-tiles, then the received ones
  auto seed = [&](float (&P)[NTH][4], uint32_t krow, uint32_t vrow) {
    const float k0 = lds32(krow + 4u * r0), k1 = lds32(krow + 4u * (r0 + 8));
#pragma unroll
    for (int x = 0; x < SEGH / 4; ++x) {
      const float4 v4 = lds128(vrow + 4u * (col0 + 4 * x));
      // packed fp32 pairs (one instruction per two products on sm_100)
      const float2 a0 = __fmul2_rn(make_float2(k0, k0), make_float2(v4.x, v4.y)), a1 = __fmul2_rn(make_float2(k1, k1), make_float2(v4.x, v4.y));
      const float2 b0 = __fmul2_rn(make_float2(k0, k0), make_float2(v4.z, v4.w)), b1 = __fmul2_rn(make_float2(k1, k1), make_float2(v4.z, v4.w));
      P[2 * x][0] = a0.x; P[2 * x][1] = a0.y; P[2 * x][2] = a1.x; P[2 * x][3] = a1.y;
      P[2 * x + 1][0] = b0.x; P[2 * x + 1][1] = b0.y; P[2 * x + 1][2] = b1.x; P[2 * x + 1][3] = b1.y;
    }
  };
  auto mma_own = [&](float (&P)[NTH][4], const uint32_t (&A)[KTH][4]) {
#pragma unroll
    for (int kth = 0; kth < KTH; ++kth)
#pragma unroll
      for (int nt = 0; nt < NTH; ++nt) mma_bf16_16816(P[nt], A[kth], Wr[kth][nt][0], Wr[kth][nt][1]);
  };
  auto mma_partner = [&](float (&P)[NTH][4], const uint32_t (&A)[KTP][4]) {
#pragma unroll
    for (int i = 0; i < KTP; ++i)
#pragma unroll
      for (int nt = 0; nt < NTH; ++nt) mma_bf16_16816(P[nt], A[i], Wr[KTH + i][nt][0], Wr[KTH + i][nt][1]);
  };

  // One step.  Pc: H_{t-1} W + k_t v_t^T, complete or in flight on entry.
  // Pn receives the same for step t+1 (after the last step: fed a valid but meaningless row).
  auto step = [&](float (&Pc)[NTH][4], float (&Pn)[NTH][4], float f, uint32_t qrow, uint32_t ydst,
                  uint32_t krow_n, uint32_t vrow_n, int par) {
    seed(Pn, krow_n, vrow_n);
    // Readout (Eq. 3) on the tensor cores: y^T = q^T H over the slab's 16 rows is one more product
    // per accumulator tile, with q as row 0 of an otherwise empty A operand and the freshly packed
    // bf16 fragments of H_t, transposed in registers, as B.  It replaces the products and the
    // shuffle tree over the rows (39 instructions per warp and step by 8 movmatrix + 4 MMAs + a
    // dozen others); the chain is bound by its instruction count, the tensor pipe has room.
    uint32_t Aq[4] = {0u, 0u, 0u, 0u};
    {
      const float2 qa = lds64(qrow + 4u * (16 * slab + 2 * c)), qb = lds64(qrow + 4u * (16 * slab + 2 * c + 8));
      if (g == 0) { Aq[0] = pack_bf16(qa.x, qa.y); Aq[2] = pack_bf16(qb.x, qb.y); }
    }
    float Y[NTH][4];
    const float2 f2 = make_float2(f, f), m1 = make_float2(-1.f, -1.f);
    // Unit u = (accumulator tile u/2, row half u%2): Eq. 1 and 2 for two elements, and after the
    // tile's second unit its share of Eq. 3.
    auto unit = [&](int u) {
      const int nt = u >> 1, h = u & 1;
      const float2 z = make_float2(tanh_approx(Pc[nt][2 * h]), tanh_approx(Pc[nt][2 * h + 1]));   // Eq. 1
      const float2 d = __ffma2_rn(z, m1, make_float2(H[nt][2 * h], H[nt][2 * h + 1]));            // H - Z
      const float2 hh = __ffma2_rn(f2, d, z);                                                     // Eq. 2
      H[nt][2 * h] = hh.x; H[nt][2 * h + 1] = hh.y;
    };
    uint32_t Aown[KTH][4], Apar[KTP][4];
    auto pack_store = [&](int kth) {
      Aown[kth][0] = pack_bf16(H[2 * kth][0], H[2 * kth][1]);
      Aown[kth][1] = pack_bf16(H[2 * kth][2], H[2 * kth][3]);
      Aown[kth][2] = pack_bf16(H[2 * kth + 1][0], H[2 * kth + 1][1]);
      Aown[kth][3] = pack_bf16(H[2 * kth + 1][2], H[2 * kth + 1][3]);
      asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(xslot(par, hf) + 512u * kth), "r"(Aown[kth][0]), "r"(Aown[kth][1]),
                   "r"(Aown[kth][2]), "r"(Aown[kth][3]) : "memory");
    };
    auto readout = [&](int kth) {   // accumulator tiles 2 kth and 2 kth + 1
      mma_bf16_16816_zero(Y[2 * kth], Aq, movmatrix_trans(Aown[kth][0]), movmatrix_trans(Aown[kth][1]));
      mma_bf16_16816_zero(Y[2 * kth + 1], Aq, movmatrix_trans(Aown[kth][2]), movmatrix_trans(Aown[kth][3]));
    };
    // The MMAs of own k-tile kth are issued between the units of the next k-tile's two
    // accumulator tiles, so that the tensor pipe and the tanh unit work at the same time
    // inside one in-order warp.
#pragma unroll
    for (int u = 0; u < 4; ++u) unit(u);
    pack_store(0);
#pragma unroll
    for (int kth = 0; kth < KTH; ++kth) {
#pragma unroll
      for (int nt = 0; nt < NTH; ++nt) {
        mma_bf16_16816(Pn[nt], Aown[kth], Wr[kth][nt][0], Wr[kth][nt][1]);
        if (kth + 1 < KTH) {
#pragma unroll
          for (int u = 4 * nt / NTH; u < 4 * (nt + 1) / NTH; ++u) unit(4 * (kth + 1) + u);
        }
      }
      readout(kth);
      if (kth + 1 < KTH) pack_store(kth + 1);
    }
    pair_sync();
    xload(par, Apar);
    mma_partner(Pn, Apar);
    // row 0 of the products: lanes 0-3 hold the slab's sums over its 16 rows, two adjacent memory
    // columns per accumulator tile
    if (g == 0) {
#pragma unroll
      for (int nt = 0; nt < NTH; ++nt) sts64(ydst + 4u * (col0 + 2 * nt), make_float2(Y[nt][0], Y[nt][1]));
    }
  };

  float P0[NTH][4], P1[NTH][4];
  int ck_left = 0, ck_idx = 0;
  auto maybe_checkpoint = [&](int steps) {
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
  constexpr uint32_t oK = 4u * TC * K, oV = 2 * oK, oF = oV + 4u * TC * V, oY = oF + 4u * TC;

  if (T > 0) {
    if (!mbar_wait(&full[0], 0)) { report_timeout(a.dev_status); return; }
    // prologue: the first step's product from the initial state (exchange parity 1 is free until step 1)
    seed(P0, stages_sa + oK, stages_sa + oV);
    uint32_t Aown[KTH][4], Apar[KTP][4];
    pack_own(Aown);
    xstore(1, Aown);
    mma_own(P0, Aown);
    pair_sync();
    xload(1, Apar);
    mma_partner(P0, Apar);
    pair_sync();   // the partner has read slot 1 before step 1 overwrites it
  }
  auto pair = [&](uint32_t st, int tl, uint32_t k2, uint32_t v2) {
    const uint32_t yp = st + oY + 4u * ((tl * NW + slab) * V);
    step(P0, P1, lds32(st + oF + 4u * tl), st + 4u * (tl * K), yp, st + oK + 4u * ((tl + 1) * K), st + oV + 4u * ((tl + 1) * V), 0);
    step(P1, P0, lds32(st + oF + 4u * (tl + 1)), st + 4u * ((tl + 1) * K), yp + 4u * (NW * V), k2, v2, 1);
  };
  for (int ch = 0, s = 0; ch < nchunks; ++ch) {
    const int sn = s + 1 == kStages ? 0 : s + 1;
    const uint32_t st = stage_sa(s);
    const int len = min(TC, T - ch * TC);
    uint32_t kN = st + oK, vN = st + oV;
    if (ch + 1 < nchunks) {
      if (!mbar_wait(&full[sn], ((ch + 1) / kStages) & 1)) { report_timeout(a.dev_status); return; }
      kN = stage_sa(sn) + oK;
      vN = stage_sa(sn) + oV;
    }
    if (len == TC) {
      // groups of kUnroll steps with compile-time offsets from one base address
#pragma unroll 1
      for (int t0 = 0; t0 < TC - kUnroll; t0 += kUnroll) {
        const uint32_t sg = st + 4u * (uint32_t)t0;   // unused: offsets below take t0 into account through tl
        (void)sg;
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
        step(P0, P1, lds32(st + oF + 4u * tl), st + 4u * (tl * K), st + oY + 4u * ((tl * NW + slab) * V),
             st + oK + 4u * (tl * K), st + oV + 4u * (tl * V), 0);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&done[s]);
    s = sn;
  }
  if (a.hT) store_state(a.hT + bn * KV);
}

template <int V, int SP, int NW, bool CKPT, int OCC>
cudaError_t launch_cs(const ScanArgs &a, cudaStream_t s) {
  const size_t smem = CsSmem<V>::bytes(16 * NW);
  cudaError_t e = cudaFuncSetAttribute(fwd_bf16_cs_kernel<V, SP, NW, CKPT, OCC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  fwd_bf16_cs_kernel<V, SP, NW, CKPT, OCC><<<a.B * a.N * (a.K / (16 * NW)), (SP * NW + cs_service_warps(SP * NW)) * 32, smem, s>>>(a);
  return cudaGetLastError();
}

template <int V, int SP, int NW>
cudaError_t launch_cs_v(const ScanArgs &a, cudaStream_t s) {
  return a.ckpt ? launch_cs<V, SP, NW, true, 1>(a, s) : launch_cs<V, SP, NW, false, 1>(a, s);
}

}  // namespace

// slabs per CTA this variant supports for a V: the register file holds (parts * slabs + 1) warps
bool fwd_cs_supported(const ScanArgs &a) {
  if (a.V == 128) return a.KCf <= 32;
  return (a.V == 32 || a.V == 64) && a.KCf <= 64;
}

// The slab count is a template parameter so that every shared-memory offset of a step is a
// compile-time constant.  Four warps per slab where the CTA would otherwise leave schedulers idle
// (one slab) and at V = 128 (a quarter of W per warp fits in registers), two elsewhere.
cudaError_t launch_fwd_bf16_cs(const ScanArgs &a, cudaStream_t s) {
  const int nw = a.KCf / 16;
  switch (a.V) {
    case 32:
      switch (nw) {
        case 1: return launch_cs_v<32, 2, 1>(a, s);
        case 2: return launch_cs_v<32, 2, 2>(a, s);
        case 3: return launch_cs_v<32, 2, 3>(a, s);
        case 4: return launch_cs_v<32, 2, 4>(a, s);
      }
      break;
    case 64:
      switch (nw) {
        case 1: return launch_cs_v<64, 4, 1>(a, s);
        case 2: return launch_cs_v<64, 2, 2>(a, s);
        case 3: return launch_cs_v<64, 2, 3>(a, s);
        case 4: return launch_cs_v<64, 2, 4>(a, s);
      }
      break;
    case 128:
      switch (nw) {
        case 1: return launch_cs_v<128, 4, 1>(a, s);
        case 2: return launch_cs_v<128, 4, 2>(a, s);
      }
      break;
  }
  return cudaErrorInvalidValue;
}

}  // namespace m2rnn

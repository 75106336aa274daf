// bf16 tensor-core backward through time (Algorithm 2 with the carried state gradient) for sm_100a.
//
// One CTA per (b, n, row slab): the K rows of a state are independent recurrences, so a CTA owns
// KC = 16*NWC of them.  Time is walked in chunks of C steps (the checkpoint interval), last chunk
// first, by four kinds of warps that overlap through shared memory:
//
//   recompute warps (NWC)  start from the checkpoint of the chunk and redo its forward steps
//                          (Eq. 1-2, the same arithmetic as the forward kernel), leaving for every
//                          step H_{t-1} as a bf16 row-major tile and Z_t as fp16 fragments;
//   reverse warps   (NWC)  carry C = dL/dH in registers and walk the chunk backwards:
//                          G = C + q dy^T, df, dX = (1-f) G (1 - Z^2),
//                          C <- f G + dX W^T  (mma.sync, bf16 operands, fp32 accumulate);
//                          dq = H_t dy and dk = dX v are small MMAs on fragments that are in
//                          registers anyway (H_t is the H_{t-1} tile of the step handled just
//                          before); dX is also left as a bf16 row-major tile;
//   dW warps        (V/16) accumulate dW += H_{t-1}^T dX on tensor cores from the two tiles
//                          (ldmatrix.trans operands), one 16-row slab of dW per warp, off the chain,
//                          and take dv = dX^T k along as one more row of the same product;
//   loader warp     (1)    stages q, k, v, dy and the gate of coming chunks;
//   writer warp     (1)    reduces and writes dq, dk, dv, dgate of finished ones.
//
// While the reverse warps sweep chunk c the recompute warps already work on chunk c-1 (two state
// buffers).  Hand-over is by mbarriers; every wait is bounded and reports through dev_status.
// Sums over rows that span CTAs (dv, dgate, dW) and over batch (dW) or shared heads (dq, dk) are
// finished by fixed-order second-stage kernels.
#include <cuda_fp16.h>

#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"
#include "tile.cuh"

namespace m2rnn {
namespace {

constexpr int kRing = 4;         // chunk slots of staged inputs / outputs in flight
constexpr int kBarBytes = 256;   // room for the mbarriers below

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float2 unpack_f16(uint32_t x) {
  return __half22float2(*reinterpret_cast<const __half2 *>(&x));
}
__device__ __forceinline__ float2 unpack_bf16(uint32_t x) {
  return make_float2(__uint_as_float(x << 16), __uint_as_float(x & 0xffff0000u));
}

// B fragment (kt, nt) of W^T under the column relabelling of mma_tile.cuh: B[k = j][n = l] = W[l][j].
template <int V>
__device__ __forceinline__ void load_wt_fragment(const __nv_bfloat16 *__restrict__ Wn, int kt, int nt, int lane,
                                                 uint32_t &b0, uint32_t &b1) {
  using G = TileGeom<V>;
  const int g = lane >> 2, c = lane & 3;
  const int l = G::mem_col(8 * nt + g);
  const int j0 = G::mem_col(16 * kt + 2 * c), j1 = G::mem_col(16 * kt + 2 * c + 1);
  const int j2 = G::mem_col(16 * kt + 8 + 2 * c), j3 = G::mem_col(16 * kt + 8 + 2 * c + 1);
  const uint16_t *w = reinterpret_cast<const uint16_t *>(Wn);
  b0 = (uint32_t)w[l * V + j0] | ((uint32_t)w[l * V + j1] << 16);
  b1 = (uint32_t)w[l * V + j2] | ((uint32_t)w[l * V + j3] << 16);
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}

// Register re-balancing between warpgroups (4 aligned warps): the kernel is compiled for an even
// split (128 per thread here), then the chain warps take registers that the dW and service warps
// give up.  An increase waits until the CTA's own pool holds enough released registers, so the
// increases must not ask for more than the decreases release:
//   V = 64:  +40*128 (recompute) + 80*128 (reverse) = 15360  <=  56*128 (dW) + 72*128 (service group) = 16384
//   V = 128: +120*128 (both kinds of chain warps)   = 15360  <=  24*256 (dW) + 72*128 (service group) = 15360.
// The instruction is warpgroup-wide, so only complete warpgroups may execute it: where it is used
// the CTA is padded to 16 warps, and the three spare warps join the service warp's decrease and
// leave.
template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

struct BwdLayout {
  // all byte offsets from the start of dynamic shared memory
  uint32_t wf, wtf, state, state_stride, ztile, dx, hfin, ring, slot_bytes, total;
  // word offsets inside a ring slot.  In: q, k, v, dy as fp32, f and df/dgate, and k, v, dy once
  // more as the raw bf16 pairs that serve as MMA operands.  Out: dq, dk, dv, per-lane df partials.
  uint32_t oQ, oK, oV, oDY, oF, oDF, oKB, oVB, oDYB, oDQ, oDK, oDV, oDFP;
};

template <int V>
__host__ __device__ inline BwdLayout bwd_layout(int KC, int C, bool w_in_smem) {
  BwdLayout L{};
  const int NWC = KC / 16;
  uint32_t off = kBarBytes;
  L.wf = off;
  if (w_in_smem) off += (V / 16) * (V / 8) * 32 * 8;
  L.wtf = off;
  if (w_in_smem) off += (V / 16) * (V / 8) * 32 * 8;
  L.state = off;                               // [2][C] x { H tile (bf16) | Z fragments (fp16) }
  L.ztile = (uint32_t)KC * V * 2;              // offset of the Z part inside one step's block
  L.state_stride = (uint32_t)KC * V * 4;       // bytes per step
  off += 2u * C * L.state_stride;
  L.dx = off;                                  // [2] dX tiles (bf16)
  off += 2u * KC * V * 2;
  L.hfin = off;                                // [2] H_t of a chunk's last step, as a tile (dq of that step): chunk j reads tile j & 1
  off += 2u * KC * V * 2;
  L.ring = off;
  const uint32_t Cp = (uint32_t)((C + 3) & ~3);  // keeps every array of a slot 16-byte aligned
  L.oQ = 0; L.oK = L.oQ + C * KC; L.oV = L.oK + C * KC; L.oDY = L.oV + C * V; L.oF = L.oDY + C * V;
  L.oDF = L.oF + Cp; L.oKB = L.oDF + Cp; L.oVB = L.oKB + C * KC / 2; L.oDYB = L.oVB + C * V / 2;
  L.oDQ = L.oDYB + C * V / 2; L.oDK = L.oDQ + C * KC; L.oDV = L.oDK + C * KC;
  L.oDFP = L.oDV + C * V;
  L.slot_bytes = (L.oDFP + C * NWC * 32) * 4;
  L.slot_bytes = (L.slot_bytes + 15u) & ~15u;
  off += kRing * L.slot_bytes;
  L.total = off;
  return L;
}

// Shapes whose warp roles fill whole warpgroups and whose chain warps need more than an even share
// of the registers: 4+4 chain warps + 4 dW warps (V = 64), 2+2 chain warps + 8 dW warps (V = 128).
template <int V, int NWC>
__host__ __device__ constexpr bool bwd_rebalance() { return (NWC == 4 && V == 64) || (NWC == 2 && V == 128); }
template <int V, int NWC>
__host__ __device__ constexpr int bwd_threads() { return bwd_rebalance<V, NWC>() ? 512 : (2 * NWC + V / 16 + 2) * 32; }

template <int V, int NWC>
__global__ void __launch_bounds__(bwd_threads<V, NWC>(), V == 16 ? (NWC == 2 ? 3 : 2) : 1) bwd_bf16_kernel(ScanArgs a) {
  using G = TileGeom<V>;
  constexpr int NT = G::NT, KT = G::KT, SEG = G::SEG;
  constexpr int KC = 16 * NWC, NDW = V / 16;
  constexpr bool kWInSmem = V > 64;
  // roles coincide with warpgroups only in this shape (4 + 4 + 4 + 1 warps), the one that needs it
  constexpr bool kRebalance = bwd_rebalance<V, NWC>();
  // running operand addresses and per-lane tile offsets worked out once (an add per step instead of
  // a multiply per use) where they measured faster; the 32-row V = 64 shape is short of registers
  // and works them out at every use
  constexpr bool kWalk = !(V == 64 && NWC == 2);
  // packed fp32x2 element-wise arithmetic where it measured faster (elsewhere its register pairs spill)
  constexpr bool kPacked = V <= 32 || (V == 64 && NWC == 4);
  constexpr int NSET = 1;   // accumulator sets of the state x W product, as in the forward kernel
  // Who computes dq = H_t dy and dk = dX v (small MMAs): the dW warps from the tiles, where they have
  // the time (more dW warps than row slabs: sweep64 backward 7.13 -> 5.76 ms, sweep32 2.65 -> 2.43),
  // else the reverse warps from the fragments they hold (with as many slabs as dW warps the dW
  // warps would set the pace: bptt_bf16 8.37 -> 9.00 ms, the paper's layer shape 3.13 -> 3.41)
  constexpr bool kDqDw = NDW >= 2 * NWC || (NDW == 1 && NWC == 1), kDkDw = kDqDw;
  extern __shared__ __align__(128) unsigned char smem[];

  const int K = a.K, N = a.N, C = a.C;
  const int RS = K / KC;
  // (the warp index through a shuffle: the compiler then knows it is the same in all lanes, keeps
  // what derives from it -- the role dispatch, the slab's addresses -- in uniform registers and
  // branches on it without a vote: 3 to 11 % faster across the shapes)
  const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  const int unit = blockIdx.x / RS, rs = blockIdx.x % RS;
  const int b = unit / N, n = unit % N;
  const UnitSpan span = unit_span(a, b);   // this batch entry's tokens (a slice of a packed batch, or b T ..)
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int nch = (T + C - 1) / C;             // chunks of this unit (a.nchunks is the checkpoint tensor's extent)
  const int rbase = rs * KC;                   // first state row of this CTA
  const size_t KV = (size_t)K * V;
  const BwdLayout L = bwd_layout<V>(KC, C, kWInSmem);

  uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
  uint64_t *in_full = bars;             // [kRing]
  uint64_t *out_full = bars + kRing;    // [kRing]
  uint64_t *st_ready = bars + 2 * kRing;      // [2]
  uint64_t *st_free = st_ready + 2;           // [2]
  uint64_t *dx_full = st_free + 2;            // [2]
  uint64_t *dx_free = dx_full + 2;            // [2] (unused: see dx_read)
  uint64_t *slot_free = dx_free + 2;          // [kRing] chunk slot written out, free for the loader
  // steps whose dX tile the dW warps are through with, summed over those warps.  A plain counter
  // instead of an mbarrier: the reverse warps read it at the top of a step and look at the value
  // only where they overwrite the tile, so the read's latency is off their dependency chain (an
  // mbarrier wait at that point cost up to 10 % of a V = 16 step, 2 % at V = 64).  The dW warps
  // add to it with release semantics after their last read of the tile; the overwrite of the tile
  // is control-dependent on the value read (a store is never issued speculatively), and the slow
  // path re-reads with acquire semantics
  uint32_t *dx_read = reinterpret_cast<uint32_t *>(slot_free + kRing);
  static_assert((3 * kRing + 8) * 8 + 4 <= kBarBytes, "barrier area");
  if (tid == 0) {
    *dx_read = 0u;
    for (int s = 0; s < kRing; ++s) { mbar_init(&in_full[s], 1); mbar_init(&out_full[s], NWC + NDW); mbar_init(&slot_free[s], 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&st_ready[s], NWC); mbar_init(&st_free[s], NWC + NDW);
      mbar_init(&dx_full[s], NWC);
    }
    fence_mbar_init();
  }
  const __nv_bfloat16 *Wn = static_cast<const __nv_bfloat16 *>(a.W) + (size_t)n * V * V;
  uint2 *Wf = reinterpret_cast<uint2 *>(smem + L.wf), *WTf = reinterpret_cast<uint2 *>(smem + L.wtf);
  if constexpr (kWInSmem) {
    for (int x = tid; x < KT * NT * 32; x += blockDim.x) {
      uint32_t b0, b1;
      load_w_fragment<V>(Wn, x / (NT * 32), (x / 32) % NT, x & 31, b0, b1);
      Wf[x] = make_uint2(b0, b1);
      load_wt_fragment<V>(Wn, x / (NT * 32), (x / 32) % NT, x & 31, b0, b1);
      WTf[x] = make_uint2(b0, b1);
    }
  }
  __syncthreads();

  const uint32_t sm0 = smem_u32(smem);
  auto slot_f = [&](int j) { return reinterpret_cast<float *>(smem + L.ring + (uint32_t)(j & (kRing - 1)) * L.slot_bytes); };
  auto slot_sa = [&](int j) { return sm0 + L.ring + (uint32_t)(j & (kRing - 1)) * L.slot_bytes; };
  auto state_sa = [&](int j, int s) { return sm0 + L.state + (uint32_t)((j & 1) * C + s) * L.state_stride; };
  // chunk j of the sweep covers steps [t0, t0 + len) of time chunk nch-1-j
  auto chunk_t0 = [&](int j) { return (nch - 1 - j) * C; };
  auto chunk_len = [&](int j) { return min(C, T - chunk_t0(j)); };

  // Thread (g,c) of chain warp w owns state rows r0 = 16w+g and r0+8 (MMA rows g, g+8) and the
  // SEG memory columns SEG*c .. SEG*c+SEG-1 (MMA columns 8nt+2c+e <-> memory column SEG*c+2nt+e).
  auto tile_store = [&](uint32_t tile_sa, int w, const uint32_t (&p)[NT][2]) { m2rnn::tile_store<V>(tile_sa, w, lane, p); };
  auto tile_load = [&](uint32_t tile_sa, int w, uint32_t (&p)[NT][2]) { m2rnn::tile_load<V>(tile_sa, w, lane, p); };
  // The same with the lane's byte offsets inside a tile worked out once per warp (they do not depend
  // on the step): toff[h][x] for row g + 8h of slab w and the thread's x-th 16-byte chunk.
  constexpr int CPRT = (SEG * 2 / 16) > 0 ? (SEG * 2 / 16) : 1;
  auto tile_offsets = [&](int w, uint32_t (&toff)[2][CPRT]) {
    if constexpr (!kWalk) return;
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int x = 0; x < CPRT; ++x) {
        const int row = 16 * w + g + 8 * h;
        if constexpr (SEG * 2 / 16 == 0) toff[h][x] = tile_off<V>(row, c >> 1) + 8u * (c & 1);
        else toff[h][x] = tile_off<V>(row, CPRT * c + x);
      }
  };
  auto tile_store_at = [&](uint32_t tile_sa, int w, const uint32_t (&toff)[2][CPRT], const uint32_t (&p)[NT][2]) {
    if constexpr (!kWalk) { m2rnn::tile_store<V>(tile_sa, w, lane, p); return; }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if constexpr (SEG * 2 / 16 == 0) {
        asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(tile_sa + toff[h][0]), "r"(p[0][h]), "r"(p[1][h]) : "memory");
      } else {
#pragma unroll
        for (int x = 0; x < CPRT; ++x)
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(tile_sa + toff[h][x]), "r"(p[4 * x][h]), "r"(p[4 * x + 1][h]),
                       "r"(p[4 * x + 2][h]), "r"(p[4 * x + 3][h]) : "memory");
      }
    }
  };
  auto tile_load_at = [&](uint32_t tile_sa, int w, const uint32_t (&toff)[2][CPRT], uint32_t (&p)[NT][2]) {
    if constexpr (!kWalk) { m2rnn::tile_load<V>(tile_sa, w, lane, p); return; }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if constexpr (SEG * 2 / 16 == 0) {
        asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(p[0][h]), "=r"(p[1][h]) : "r"(tile_sa + toff[h][0]));
      } else {
#pragma unroll
        for (int x = 0; x < CPRT; ++x)
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(p[4 * x][h]), "=r"(p[4 * x + 1][h]), "=r"(p[4 * x + 2][h]), "=r"(p[4 * x + 3][h]) : "r"(tile_sa + toff[h][x]));
      }
    }
  };
  // Z fragments: private to the (warp, lane) pair that wrote them, 2*NT words per thread kept as
  // NT/2 groups of 16 bytes (group x of lane l at word ((w*NT/2 + x)*32 + l)*4)
  constexpr int ZG = NT / 2;
  auto zfrag_sa = [&](uint32_t step_sa, int w) { return step_sa + L.ztile + (uint32_t)(w * ZG * 32 + lane) * 16u; };

  // (each setmaxnreg below is one instruction executed by every warp of its warpgroup, at the top
  // of the code it governs)
  if constexpr (kRebalance && V == 128) {
    if (warp < 2 * NWC) reg_inc<248>();
  }
  if (warp < NWC) {
    // ================================================================= recompute warps
    if constexpr (kRebalance && V == 64) reg_inc<168>();
    const int w = warp, r0 = 16 * w + g;
    uint32_t toff[2][CPRT];
    tile_offsets(w, toff);
    const uint32_t zoff = L.ztile + (uint32_t)(w * ZG * 32 + lane) * 16u;   // this lane's Z fragments inside a step's block
    uint32_t Wr[kWInSmem ? 1 : KT][kWInSmem ? 1 : NT][2];
    if constexpr (!kWInSmem) {
#pragma unroll
      for (int kt = 0; kt < KT; ++kt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) load_w_fragment<V>(Wn, kt, nt, lane, Wr[kt][nt][0], Wr[kt][nt][1]);
    }
    for (int j = 0; j < nch; ++j) {
      const int len = chunk_len(j);
      // the chunk's starting state: ckpt[b][n][chunk] = H before step t0 (fp32)
      float H[NT][4];
      const float *ck = a.ckpt + ((size_t)unit * a.nchunks + (nch - 1 - j)) * KV;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float *src = ck + (size_t)(rbase + r0 + 8 * h) * V + SEG * c;
#pragma unroll
        for (int x = 0; x < SEG / 4; ++x) {
          const float4 t4 = *reinterpret_cast<const float4 *>(src + 4 * x);
          H[2 * x][2 * h] = t4.x; H[2 * x][2 * h + 1] = t4.y; H[2 * x + 1][2 * h] = t4.z; H[2 * x + 1][2 * h + 1] = t4.w;
        }
      }
      if (!mbar_wait(&in_full[j & (kRing - 1)], (j / kRing) & 1)) { report_timeout(a.dev_status); return; }
      if (j >= 2 && !mbar_wait(&st_free[j & 1], ((j >> 1) - 1) & 1)) { report_timeout(a.dev_status); return; }
      const uint32_t sl = slot_sa(j);
      // addresses of the step's operands: walked (one add per step) or worked out from s
      struct Ptrs { uint32_t st, k, f, v; };
      auto ptrs_at = [&](int s) {
        return Ptrs{state_sa(j, s), sl + 4u * (L.oK + s * KC + r0), sl + 4u * (L.oF + s), sl + 4u * (L.oV + s * V + SEG * c)};
      };
      Ptrs run = ptrs_at(0);
      for (int s = 0; s < len; ++s) {
        // (worked out at the place of use when not walked: short live ranges)
        const uint32_t st = kWalk ? run.st : state_sa(j, s);
#define pK (kWalk ? run.k : sl + 4u * (L.oK + s * KC + r0))
#define pF (kWalk ? run.f : sl + 4u * (L.oF + s))
#define pV (kWalk ? run.v : sl + 4u * (L.oV + s * V + SEG * c))
        // H_{t-1} as bf16: the A operand of this step and the tile the dW and reverse warps read
        uint32_t hp[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { hp[nt][0] = pack_bf16(H[nt][0], H[nt][1]); hp[nt][1] = pack_bf16(H[nt][2], H[nt][3]); }
        tile_store_at(st, w, toff, hp);
        // P = k v^T + H W   (Eq. 1 before the non-linearity)
        const float k0 = lds32(pK), k1 = lds32(pK + 32u);
        const float f = lds32(pF);
        // (two accumulator sets, as in the one-warp-per-slab forward kernel)
        float P[NSET][NT][4];
#pragma unroll
        for (int x = 0; x < SEG / 4; ++x) {
          const float4 v4 = lds128(pV + 16u * x);
          if constexpr (kPacked) {   // packed fp32 pairs: one instruction per two products
            const float2 k02 = make_float2(k0, k0), k12 = make_float2(k1, k1);
            const float2 a0 = __fmul2_rn(k02, make_float2(v4.x, v4.y)), a1 = __fmul2_rn(k12, make_float2(v4.x, v4.y));
            const float2 b0 = __fmul2_rn(k02, make_float2(v4.z, v4.w)), b1 = __fmul2_rn(k12, make_float2(v4.z, v4.w));
            P[0][2 * x][0] = a0.x; P[0][2 * x][1] = a0.y; P[0][2 * x][2] = a1.x; P[0][2 * x][3] = a1.y;
            P[0][2 * x + 1][0] = b0.x; P[0][2 * x + 1][1] = b0.y; P[0][2 * x + 1][2] = b1.x; P[0][2 * x + 1][3] = b1.y;
          } else {
            P[0][2 * x][0] = k0 * v4.x; P[0][2 * x][1] = k0 * v4.y; P[0][2 * x][2] = k1 * v4.x; P[0][2 * x][3] = k1 * v4.y;
            P[0][2 * x + 1][0] = k0 * v4.z; P[0][2 * x + 1][1] = k0 * v4.w; P[0][2 * x + 1][2] = k1 * v4.z; P[0][2 * x + 1][3] = k1 * v4.w;
          }
        }
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
          const uint32_t Ak[4] = {hp[2 * kt][0], hp[2 * kt][1], hp[2 * kt + 1][0], hp[2 * kt + 1][1]};
          const int set = kt % NSET;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            uint2 wv;
            if constexpr (kWInSmem) wv = Wf[(kt * NT + nt) * 32 + lane];
            else wv = make_uint2(Wr[kt][nt][0], Wr[kt][nt][1]);
            if (kt >= 1 && kt < NSET) mma_bf16_16816_zero(P[set][nt], Ak, wv.x, wv.y);
            else mma_bf16_16816(P[set][nt], Ak, wv.x, wv.y);
          }
        }
        // Z = tanh(P), kept as fp16 for the reverse sweep; H <- f H + (1-f) Z  (Eq. 2)
        const uint32_t zs = kWalk ? st + zoff : zfrag_sa(st, w);
#pragma unroll
        for (int x = 0; x < ZG; ++x) {
          uint32_t zw[4];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int nt = 2 * x + u;
            float z[4];
            if constexpr (kPacked) {
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                float2 xin = make_float2(P[0][nt][2 * h], P[0][nt][2 * h + 1]);
                if constexpr (NSET == 2) xin = __fadd2_rn(xin, make_float2(P[1][nt][2 * h], P[1][nt][2 * h + 1]));
                const float2 z2 = make_float2(tanh_approx(xin.x), tanh_approx(xin.y));
                const float2 d2 = __ffma2_rn(z2, make_float2(-1.f, -1.f), make_float2(H[nt][2 * h], H[nt][2 * h + 1]));
                const float2 h2 = __ffma2_rn(make_float2(f, f), d2, z2);
                z[2 * h] = z2.x; z[2 * h + 1] = z2.y;
                H[nt][2 * h] = h2.x; H[nt][2 * h + 1] = h2.y;
              }
            } else {
#pragma unroll
              for (int r = 0; r < 4; ++r) {
                float xin = P[0][nt][r];
                if constexpr (NSET == 2) xin += P[1][nt][r];
                z[r] = tanh_approx(xin);
                H[nt][r] = fmaf(f, H[nt][r] - z[r], z[r]);
              }
            }
            zw[2 * u] = pack_f16(z[0], z[1]);
            zw[2 * u + 1] = pack_f16(z[2], z[3]);
          }
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(zs + 512u * x), "r"(zw[0]), "r"(zw[1]), "r"(zw[2]), "r"(zw[3]) : "memory");
        }
        if constexpr (kWalk) { run.st += L.state_stride; run.k += 4u * KC; run.f += 4u; run.v += 4u * V; }
      }
#undef pK
#undef pF
#undef pV
      if (j == 0) {   // the state after the last step of the scan: H_t of the first reverse step
        uint32_t hp[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { hp[nt][0] = pack_bf16(H[nt][0], H[nt][1]); hp[nt][1] = pack_bf16(H[nt][2], H[nt][3]); }
        tile_store_at(sm0 + L.hfin, w, toff, hp);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&st_ready[j & 1]);
    }
    return;
  }

  if (warp < 2 * NWC) {
    // ================================================================= reverse warps
    if constexpr (kRebalance && V == 64) reg_inc<208>();
    const int w = warp - NWC, r0 = 16 * w + g;
    uint32_t toff[2][CPRT];
    tile_offsets(w, toff);
    const uint32_t zoff = L.ztile + (uint32_t)(w * ZG * 32 + lane) * 16u;
    uint32_t WTr[kWInSmem ? 1 : KT][kWInSmem ? 1 : NT][2];
    if constexpr (!kWInSmem) {
#pragma unroll
      for (int kt = 0; kt < KT; ++kt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) load_wt_fragment<V>(Wn, kt, nt, lane, WTr[kt][nt][0], WTr[kt][nt][1]);
    }
    float Cg[NT][4];   // carried dL/dH_t
    if (a.d_hT) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float *src = a.d_hT + (size_t)unit * KV + (size_t)(rbase + r0 + 8 * h) * V + SEG * c;
#pragma unroll
        for (int x = 0; x < SEG / 4; ++x) {
          const float4 t4 = *reinterpret_cast<const float4 *>(src + 4 * x);
          Cg[2 * x][2 * h] = t4.x; Cg[2 * x][2 * h + 1] = t4.y; Cg[2 * x + 1][2 * h] = t4.z; Cg[2 * x + 1][2 * h + 1] = t4.w;
        }
      }
    } else {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) Cg[nt][0] = Cg[nt][1] = Cg[nt][2] = Cg[nt][3] = 0.f;
    }
    const float clip = a.dh_clip;
    int nstep = 0;   // steps taken so far: picks the dX tile
    // B operand of the small MMAs: the thread's SEG columns of a vector as bf16 pairs; every
    // column n of B holds the same vector, so every column of the result holds the product
    auto load_pairs = [&](uint32_t row_sa, uint32_t (&pr)[NT]) {
      if constexpr (NT == 2) {
        asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(pr[0]), "=r"(pr[1]) : "r"(row_sa + 4u * (SEG / 2) * c));
      } else {
#pragma unroll
        for (int x = 0; x < NT / 4; ++x)
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(pr[4 * x]), "=r"(pr[4 * x + 1]), "=r"(pr[4 * x + 2]), "=r"(pr[4 * x + 3])
                       : "r"(row_sa + 4u * ((SEG / 2) * c + 4 * x)));
      }
    };
    // (A . vec), A given as packed pairs in accumulator layout: rows g and g+8 end up in
    // d[.][0] and d[.][2], split over two accumulators that the caller adds when it stores them
    // (late in the step, so that the warp never waits on these off-chain products)
    auto matvec = [&](const uint32_t (&Ap)[NT][2], const uint32_t (&pr)[NT], float (&d)[2][4]) {
#pragma unroll
      for (int kt = 0; kt < KT; ++kt) {
        const uint32_t Ak[4] = {Ap[2 * kt][0], Ap[2 * kt][1], Ap[2 * kt + 1][0], Ap[2 * kt + 1][1]};
        if (kt < 2) mma_bf16_16816_zero(d[kt & 1], Ak, pr[2 * kt], pr[2 * kt + 1]);
        else mma_bf16_16816(d[kt & 1], Ak, pr[2 * kt], pr[2 * kt + 1]);
      }
      if constexpr (KT == 1) d[1][0] = d[1][2] = 0.f;
    };
    const uint32_t dx_read_sa = smem_u32(dx_read);
    uint32_t hn[NT][2];   // H_t of the step at hand as bf16 pairs = the H_{t-1} tile of the step done before
    for (int j = 0; j < nch; ++j) {
      const int len = chunk_len(j);
      if (!mbar_wait(&in_full[j & (kRing - 1)], (j / kRing) & 1)) { report_timeout(a.dev_status); return; }
      if (!mbar_wait(&st_ready[j & 1], (j >> 1) & 1)) { report_timeout(a.dev_status); return; }
      if constexpr (!kDqDw) { if (j == 0) tile_load_at(sm0 + L.hfin, w, toff, hn); }
      const uint32_t sl = slot_sa(j);
      // addresses of the step's operands: walked backwards (one add per step) or worked out from s
      struct Ptrs { uint32_t st, f, q, dyb, vb, dy, dfp, dq, dk; };
      auto ptrs_at = [&](int s) {
        return Ptrs{state_sa(j, s), sl + 4u * (L.oF + s), sl + 4u * (L.oQ + s * KC + r0), sl + 4u * (L.oDYB + s * (V / 2)),
                    sl + 4u * (L.oVB + s * (V / 2)), sl + 4u * (L.oDY + s * V + SEG * c),
                    sl + 4u * (L.oDFP + (s * NWC + w) * 32 + lane), sl + 4u * (L.oDQ + s * KC + r0), sl + 4u * (L.oDK + s * KC + r0)};
      };
      Ptrs run = ptrs_at(len - 1);
      for (int s = len - 1; s >= 0; --s, ++nstep) {
        const uint32_t st = kWalk ? run.st : state_sa(j, s);
#define pF (kWalk ? run.f : sl + 4u * (L.oF + s))
#define pQ (kWalk ? run.q : sl + 4u * (L.oQ + s * KC + r0))
#define pDYB (kWalk ? run.dyb : sl + 4u * (L.oDYB + s * (V / 2)))
#define pVB (kWalk ? run.vb : sl + 4u * (L.oVB + s * (V / 2)))
#define pDY (kWalk ? run.dy : sl + 4u * (L.oDY + s * V + SEG * c))
#define pDFP (kWalk ? run.dfp : sl + 4u * (L.oDFP + (s * NWC + w) * 32 + lane))
#define pDQ (kWalk ? run.dq : sl + 4u * (L.oDQ + s * KC + r0))
#define pDK (kWalk ? run.dk : sl + 4u * (L.oDK + s * KC + r0))
        uint32_t dx_seen;
        asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(dx_seen) : "r"(dx_read_sa) : "memory");
        uint32_t hp[NT][2];
        tile_load_at(st, w, toff, hp);
        const uint32_t zs = kWalk ? st + zoff : zfrag_sa(st, w);
        const float f = lds32(pF);
        const float q0 = lds32(pQ), q1 = lds32(pQ + 32u);
        const float omf = 1.f - f;
        // dq = H_t dy on the tensor cores (Algorithm 2, query-gradient line)
        float dqd[2][4], dkd[2][4];
        if constexpr (!kDqDw) {
          uint32_t dyp[NT];
          load_pairs(pDYB, dyp);
          matvec(hn, dyp, dqd);
        } else {
          // H_{t-1} of a chunk's first step is H_t of the last step of the chunk swept next; its
          // state buffer may be overwritten by then, so it is kept as a tile for the dW warps
          if (s == 0) tile_store_at(sm0 + L.hfin + (uint32_t)((j + 1) & 1) * (KC * V * 2), w, toff, hp);
        }
        float df = 0.f;
        float2 df2 = make_float2(0.f, 0.f);   // packed path: even and odd elements summed apart
        uint32_t xp[NT][2];   // dX as bf16 pairs: the A operand of dX W^T and the tile of the dW warps
#pragma unroll
        for (int x = 0; x < SEG / 4; ++x) {
          const float4 dy4 = lds128(pDY + 16u * x);
          const float dyv[4] = {dy4.x, dy4.y, dy4.z, dy4.w};
          uint32_t zw[4];
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(zw[0]), "=r"(zw[1]), "=r"(zw[2]), "=r"(zw[3]) : "r"(zs + 512u * x));
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int nt = 2 * x + u;
            const float2 za = unpack_f16(zw[2 * u]), zb = unpack_f16(zw[2 * u + 1]);
            const float2 ha = unpack_bf16(hp[nt][0]), hb = unpack_bf16(hp[nt][1]);
            const float z[4] = {za.x, za.y, zb.x, zb.y}, hprev[4] = {ha.x, ha.y, hb.x, hb.y};
            float dX[4];
            if constexpr (kPacked) {
              const float2 dy2 = make_float2(dyv[2 * u], dyv[2 * u + 1]);
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const float2 z2 = make_float2(z[2 * h], z[2 * h + 1]), hp2 = make_float2(hprev[2 * h], hprev[2 * h + 1]);
                const float qh = h ? q1 : q0;
                const float2 G2 = __ffma2_rn(make_float2(qh, qh), dy2, make_float2(Cg[nt][2 * h], Cg[nt][2 * h + 1]));   // G = C + q dy^T
                df2 = __ffma2_rn(G2, __ffma2_rn(z2, make_float2(-1.f, -1.f), hp2), df2);                                    // df = sum G (.) (H_{t-1} - Z)
                const float2 x2 = __fmul2_rn(__fmul2_rn(make_float2(-omf, -omf), G2), __ffma2_rn(z2, z2, make_float2(-1.f, -1.f)));   // (1-f) G (1 - Z^2)
                const float2 c2 = __fmul2_rn(make_float2(f, f), G2);                                                        // gated path into H_{t-1}
                dX[2 * h] = x2.x; dX[2 * h + 1] = x2.y;
                Cg[nt][2 * h] = c2.x; Cg[nt][2 * h + 1] = c2.y;
              }
            } else {
#pragma unroll
              for (int r = 0; r < 4; ++r) {
                const float dyc = dyv[2 * u + (r & 1)];
                const float qr = (r & 2) ? q1 : q0;
                const float Gv = fmaf(qr, dyc, Cg[nt][r]);        // G = C + q dy^T
                df = fmaf(Gv, hprev[r] - z[r], df);               // df = sum G (.) (H_{t-1} - Z)
                dX[r] = omf * Gv * fmaf(-z[r], z[r], 1.f);        // through the gate and tanh
                Cg[nt][r] = f * Gv;                               // gated path into H_{t-1}
              }
            }
            xp[nt][0] = pack_bf16(dX[0], dX[1]);
            xp[nt][1] = pack_bf16(dX[2], dX[3]);
          }
        }
        if constexpr (kPacked) df = df2.x + df2.y;
        // hand dX to the dW warps
        const int xb = nstep & 1;
        if (nstep >= 2) {   // the dW warps must be through with the tile written two steps ago
          const uint32_t need = (uint32_t)NDW * (uint32_t)(nstep - 1);
          bool ok = (int32_t)(dx_seen - need) >= 0;
          if (!ok) {
            const long long t0 = clock64();
            do {
              __nanosleep(20);
              asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(dx_seen) : "r"(dx_read_sa) : "memory");
              ok = (int32_t)(dx_seen - need) >= 0;
            } while (!ok && clock64() - t0 < kWaitCycles);
          }
          if (!__all_sync(0xffffffffu, ok)) { report_timeout(a.dev_status); return; }
        }
        tile_store_at(sm0 + L.dx + (uint32_t)xb * (KC * V * 2), w, toff, xp);
        __syncwarp();
        if (lane == 0) mbar_arrive(&dx_full[xb]);
        // C_{t-1} = f G + dX W^T
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
          const uint32_t Ak[4] = {xp[2 * kt][0], xp[2 * kt][1], xp[2 * kt + 1][0], xp[2 * kt + 1][1]};
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            if constexpr (kWInSmem) {
              const uint2 wv = WTf[(kt * NT + nt) * 32 + lane];
              mma_bf16_16816(Cg[nt], Ak, wv.x, wv.y);
            } else {
              mma_bf16_16816(Cg[nt], Ak, WTr[kt][nt][0], WTr[kt][nt][1]);
            }
          }
        }
        // dk = dX v on the tensor cores (Algorithm 2, key-gradient line)
        if constexpr (!kDkDw) {
          uint32_t vp[NT];
          load_pairs(pVB, vp);
          matvec(xp, vp, dkd);
        }
        if (clip > 0.f) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int r = 0; r < 4; ++r) Cg[nt][r] = fminf(fmaxf(Cg[nt][r], -clip), clip);
        }
        sts32(pDFP, df);   // summed by the service warp
        if (c == 0) {
          if constexpr (!kDqDw) { sts32(pDQ, dqd[0][0] + dqd[1][0]); sts32(pDQ + 32u, dqd[0][2] + dqd[1][2]); }
          if constexpr (!kDkDw) { sts32(pDK, dkd[0][0] + dkd[1][0]); sts32(pDK + 32u, dkd[0][2] + dkd[1][2]); }
        }
        if constexpr (!kDqDw) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) { hn[nt][0] = hp[nt][0]; hn[nt][1] = hp[nt][1]; }
        }
        if constexpr (kWalk) {
          run.st -= L.state_stride; run.f -= 4u; run.q -= 4u * KC; run.dyb -= 2u * V; run.vb -= 2u * V;
          run.dy -= 4u * V; run.dfp -= 4u * NWC * 32; run.dq -= 4u * KC; run.dk -= 4u * KC;
        }
      }
#undef pF
#undef pQ
#undef pDYB
#undef pVB
#undef pDY
#undef pDFP
#undef pDQ
#undef pDK
      __syncwarp();
      if (lane == 0) { mbar_arrive(&st_free[j & 1]); mbar_arrive(&out_full[j & (kRing - 1)]); }
    }
    if (a.dh0) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float *dst = a.dh0 + (size_t)unit * KV + (size_t)(rbase + r0 + 8 * h) * V + SEG * c;
#pragma unroll
        for (int x = 0; x < SEG / 4; ++x)
          *reinterpret_cast<float4 *>(dst + 4 * x) =
              make_float4(Cg[2 * x][2 * h], Cg[2 * x][2 * h + 1], Cg[2 * x + 1][2 * h], Cg[2 * x + 1][2 * h + 1]);
      }
    }
    return;
  }

  if (warp < 2 * NWC + NDW) {
    // ================================================================= dW warps
    // warp d owns dW rows l in [16d, 16d+16): acc += H_{t-1}[:, l]^T dX, contraction over the CTA's rows
    if constexpr (kRebalance) { if constexpr (V == 64) reg_dec<72>(); else reg_dec<104>(); }
    const int d = warp - 2 * NWC;
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    const int mi = lane >> 3, mr = lane & 7;   // ldmatrix: lane supplies row mr of matrix mi
    // Per-lane byte offsets of the ldmatrix rows inside a tile, without the slab term (16 rows =
    // 32 V bytes per kt, added as an immediate): rows of 128 bytes or more keep their chunk swizzle
    // (row & 7 = mr) when 16 rows are added, so the offsets are worked out once.
    constexpr bool kPreOff = kWalk && 2 * V >= 128;
    uint32_t offA = 0, offDv = 0, offB[NT / 2];
    if constexpr (kPreOff) {
      offA = tile_off<V>(mr + 8 * (mi >> 1), 2 * d + (mi & 1));
      offDv = tile_off<V>(mr + 8 * (mi & 1), 2 * d + (mi >> 1));
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) offB[np] = tile_off<V>(mr + 8 * (mi & 1), 2 * np + (mi >> 1));
    }
    int nstep = 0;
    for (int j = 0; j < nch; ++j) {
      const int len = chunk_len(j);
      if (!mbar_wait(&st_ready[j & 1], (j >> 1) & 1)) { report_timeout(a.dev_status); return; }
      for (int s = len - 1; s >= 0; --s, ++nstep) {
        const int xb = nstep & 1;
        if (!mbar_wait(&dx_full[xb], (nstep >> 1) & 1)) { report_timeout(a.dev_status); return; }
        const uint32_t ht = state_sa(j, s), xt = sm0 + L.dx + (uint32_t)xb * (KC * V * 2);
        // dv = dX^T k (Algorithm 2, value-gradient line) rides along as one more row of the product:
        // an A tile whose row 0 is k and whose other rows are zero; this warp takes columns 16d..16d+15
        float dvacc[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) dvacc[u][0] = dvacc[u][1] = dvacc[u][2] = dvacc[u][3] = 0.f;
        const uint32_t kb = slot_sa(j) + 4u * (L.oKB + s * (KC / 2));
#pragma unroll
        for (int kt = 0; kt < NWC; ++kt) {
          // A = H_{t-1}^T: matrices (i 0-7, l 0-7), (i 0-7, l 8-15), (i 8-15, l 0-7), (i 8-15, l 8-15)
          uint32_t A[4];
          if constexpr (kPreOff) ldmatrix_x4_trans(ht + offA + (uint32_t)(kt * 32 * V), A[0], A[1], A[2], A[3]);
          else ldmatrix_x4_trans(ht + tile_off<V>(16 * kt + mr + 8 * (mi >> 1), 2 * d + (mi & 1)), A[0], A[1], A[2], A[3]);
#pragma unroll
          for (int np = 0; np < NT / 2; ++np) {
            // B = dX: matrices (i 0-7, j-tile 2np), (i 8-15, 2np), (i 0-7, 2np+1), (i 8-15, 2np+1)
            uint32_t b0, b1, b2, b3;
            if constexpr (kPreOff) ldmatrix_x4_trans(xt + offB[np] + (uint32_t)(kt * 32 * V), b0, b1, b2, b3);
            else ldmatrix_x4_trans(xt + tile_off<V>(16 * kt + mr + 8 * (mi & 1), 2 * np + (mi >> 1)), b0, b1, b2, b3);
            mma_bf16_16816(acc[2 * np], A, b0, b1);
            mma_bf16_16816(acc[2 * np + 1], A, b2, b3);
          }
        }
#pragma unroll
        for (int kt = 0; kt < NWC; ++kt) {
          uint32_t Ak[4] = {0u, 0u, 0u, 0u}, b0, b1, b2, b3;
          if (g == 0) {
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(Ak[0]) : "r"(kb + 4u * (8 * kt + c)));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(Ak[2]) : "r"(kb + 4u * (8 * kt + 4 + c)));
          }
          if constexpr (kPreOff) ldmatrix_x4_trans(xt + offDv + (uint32_t)(kt * 32 * V), b0, b1, b2, b3);
          else ldmatrix_x4_trans(xt + tile_off<V>(16 * kt + mr + 8 * (mi & 1), 2 * d + (mi >> 1)), b0, b1, b2, b3);
          mma_bf16_16816(dvacc[0], Ak, b0, b1);
          mma_bf16_16816(dvacc[1], Ak, b2, b3);
        }
        if (g == 0) {
          const uint32_t dst = slot_sa(j) + 4u * (L.oDV + s * V + 16 * d + 2 * c);
          sts64(dst, make_float2(dvacc[0][0], dvacc[0][1]));
          sts64(dst + 32u, make_float2(dvacc[1][0], dvacc[1][1]));
        }
        // dq = H_t dy and dk = dX v (Algorithm 2, query- and key-gradient lines) for the 16-row
        // slabs this warp takes in turn: A fragments by ldmatrix from the H_t tile (the H_{t-1} tile
        // of the step after this one; for a chunk's last step the tile the reverse warps kept) and
        // from the dX tile, B = the vector as bf16 pairs in every column, so that every column of
        // the result holds the product
        if constexpr (kDqDw || kDkDw) {
          const uint32_t hnext = s + 1 < len ? state_sa(j, s + 1) : sm0 + L.hfin + (uint32_t)(j & 1) * (KC * V * 2);
          const uint32_t dyb = slot_sa(j) + 4u * (L.oDYB + s * (V / 2)), vb = slot_sa(j) + 4u * (L.oVB + s * (V / 2));
          auto pair_of = [&](uint32_t vec_sa, int kt, uint32_t &b0, uint32_t &b1) {
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(b0) : "r"(vec_sa + 4u * (8 * kt + c)));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(b1) : "r"(vec_sa + 4u * (8 * kt + 4 + c)));
          };
          for (int mt = d; mt < NWC; mt += NDW) {
            float dq[4] = {0.f, 0.f, 0.f, 0.f}, dk[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
              // matrices (rows 0-7, chunk 2kt), (rows 8-15, 2kt), (rows 0-7, 2kt+1), (rows 8-15, 2kt+1)
              const uint32_t off = tile_off<V>(16 * mt + mr + 8 * (mi & 1), 2 * kt + (mi >> 1));
              uint32_t A[4], b0, b1;
              if constexpr (kDqDw) {
                ldmatrix_x4(hnext + off, A);
                pair_of(dyb, kt, b0, b1);
                mma_bf16_16816(dq, A, b0, b1);
              }
              if constexpr (kDkDw) {
                ldmatrix_x4(xt + off, A);
                pair_of(vb, kt, b0, b1);
                mma_bf16_16816(dk, A, b0, b1);
              }
            }
            if (c == 0) {
              const uint32_t o = slot_sa(j) + 4u * (s * KC + 16 * mt + g);
              if constexpr (kDqDw) { sts32(o + 4u * L.oDQ, dq[0]); sts32(o + 4u * (L.oDQ + 8), dq[2]); }
              if constexpr (kDkDw) { sts32(o + 4u * L.oDK, dk[0]); sts32(o + 4u * (L.oDK + 8), dk[2]); }
            }
          }
        }
        __syncwarp();
        if (lane == 0) asm volatile("red.release.cta.shared.add.u32 [%0], 1;" ::"r"(smem_u32(dx_read)) : "memory");
      }
      __syncwarp();
      if (lane == 0) { mbar_arrive(&st_free[j & 1]); mbar_arrive(&out_full[j & (kRing - 1)]); }
    }
    float *dWp = a.dW_part + ((size_t)(b * RS + rs) * N + n) * V * V;   // one partial per CTA, [b][slab][n]
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      *reinterpret_cast<float2 *>(dWp + (size_t)(16 * d + g) * V + 8 * nt + 2 * c) = make_float2(acc[nt][0], acc[nt][1]);
      *reinterpret_cast<float2 *>(dWp + (size_t)(16 * d + g + 8) * V + 8 * nt + 2 * c) = make_float2(acc[nt][2], acc[nt][3]);
    }
    return;
  }

  // =================================================================== loader and writer warps
  if constexpr (kRebalance) reg_dec<56>();
  if (warp > 2 * NWC + NDW + 1) return;   // spare warps of a padded CTA
  const bool is_loader = warp == 2 * NWC + NDW;
  {
    const int hq = n / (N / a.Nq), hk = n / (N / a.Nk);
    const float al = a.alpha ? a.alpha[n] : 1.f, be = a.beta ? a.beta[n] : 0.f;
    const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(a.q), *kg = static_cast<const __nv_bfloat16 *>(a.k);
    const __nv_bfloat16 *vg = static_cast<const __nv_bfloat16 *>(a.v), *dyg = static_cast<const __nv_bfloat16 *>(a.dy);
    const __nv_bfloat16 *wr = static_cast<const __nv_bfloat16 *>(a.w_r);
    const size_t BT = (size_t)a.TT;
    auto fill = [&](int j) {
      float *sf = slot_f(j);
      const int t0 = chunk_t0(j), len = chunk_len(j);
      const size_t bt0 = tok0 + t0;
      const int kc8 = KC / 8, v8 = V / 8;
      uint4 *kb = reinterpret_cast<uint4 *>(sf + L.oKB), *vb = reinterpret_cast<uint4 *>(sf + L.oVB);
      uint4 *dyb = reinterpret_cast<uint4 *>(sf + L.oDYB);
      float gt = 0.f;
      if (lane < len) gt = a.gate[(bt0 + lane) * N + n];
      // 32 rows of 16 bytes of each tensor per pass, every load of a pass issued before its first use
      const int nk = len * kc8, nv = len * v8;
      for (int x0 = 0; x0 < max(nk, nv); x0 += 32) {
        const int x = x0 + lane;
        uint4 qr, kr, vr, dr;
        if (x < nk) {
          const int t = x / kc8, i = (x % kc8) * 8;
          qr = *reinterpret_cast<const uint4 *>(qg + (bt0 + t) * a.qs + hq * K + rbase + i);
          kr = *reinterpret_cast<const uint4 *>(kg + (bt0 + t) * a.ks + hk * K + rbase + i);
        }
        if (x < nv) {
          const int t = x / v8, i = (x % v8) * 8;
          vr = *reinterpret_cast<const uint4 *>(vg + (bt0 + t) * a.vs + n * V + i);
          dr = *reinterpret_cast<const uint4 *>(dyg + ((bt0 + t) * N + n) * V + i);
        }
        if (x < nk) {
          const int t = x / kc8, i = (x % kc8) * 8;
          store8_bf16_as_f32(sf + L.oQ + t * KC + i, qr);
          store8_bf16_as_f32(sf + L.oK + t * KC + i, kr);
          kb[x] = kr;
        }
        if (x < nv) {
          const int t = x / v8, i = (x % v8) * 8;
          store8_bf16_as_f32(sf + L.oV + t * V + i, vr);
          store8_bf16_as_f32(sf + L.oDY + t * V + i, dr);
          vb[x] = vr;
          dyb[x] = dr;
        }
      }
      if (lane < len) {
        float dfdx;
        sf[L.oF + lane] = gate_value(a.gate_kind, gt, al, be, &dfdx);
        sf[L.oDF + lane] = dfdx;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&in_full[j & (kRing - 1)]);
    };
    auto flush = [&](int j) {
      const float *sf = slot_f(j);
      const int t0 = chunk_t0(j), len = chunk_len(j);
      const size_t bt0 = tok0 + t0;
      // dq, dk: this CTA's rows
      for (int x = lane; x < len * (KC / 2); x += 32) {
        const int t = x / (KC / 2), i = (x % (KC / 2)) * 2;
        const float2 dq2 = *reinterpret_cast<const float2 *>(sf + L.oDQ + t * KC + i);
        const float2 dk2 = *reinterpret_cast<const float2 *>(sf + L.oDK + t * KC + i);
        if (a.dq_part) *reinterpret_cast<float2 *>(a.dq_part + ((bt0 + t) * N + n) * K + rbase + i) = dq2;
        else *reinterpret_cast<uint32_t *>(static_cast<__nv_bfloat16 *>(a.dq) + ((bt0 + t) * a.Nq + hq) * K + rbase + i) = pack_bf16(dq2.x, dq2.y);
        if (a.dk_part) *reinterpret_cast<float2 *>(a.dk_part + ((bt0 + t) * N + n) * K + rbase + i) = dk2;
        else *reinterpret_cast<uint32_t *>(static_cast<__nv_bfloat16 *>(a.dk) + ((bt0 + t) * a.Nk + hk) * K + rbase + i) = pack_bf16(dk2.x, dk2.y);
      }
      // dv of this CTA's rows (+ w_r (.) dy from Eq. 3, added by the first row slab only)
      for (int x = lane; x < len * (V / 2); x += 32) {
        const int t = x / (V / 2), jj = (x % (V / 2)) * 2;
        const float2 p = *reinterpret_cast<const float2 *>(sf + L.oDV + t * V + jj);
        float s0 = p.x, s1 = p.y;
        if (wr && rs == 0) {
          s0 = fmaf(__bfloat162float(wr[(size_t)n * V + jj]), sf[L.oDY + t * V + jj], s0);
          s1 = fmaf(__bfloat162float(wr[(size_t)n * V + jj + 1]), sf[L.oDY + t * V + jj + 1], s1);
        }
        const size_t o = ((bt0 + t) * N + n) * V + jj;
        if (a.dv_part) *reinterpret_cast<float2 *>(a.dv_part + (size_t)rs * BT * N * V + o) = make_float2(s0, s1);
        else *reinterpret_cast<uint32_t *>(static_cast<__nv_bfloat16 *>(a.dv) + o) = pack_bf16(s0, s1);
      }
      // dgate: the reverse warps leave one df partial per lane; fixed-order sum, then the gate's slope
      for (int t = 0; t < len; ++t) {
        float sdf = 0.f;
        for (int w = 0; w < NWC; ++w) sdf += sf[L.oDFP + (t * NWC + w) * 32 + lane];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sdf += __shfl_xor_sync(0xffffffffu, sdf, off);
        if (lane == 0) {
          sdf *= sf[L.oDF + t];
          const size_t o = (bt0 + t) * N + n;
          if (a.dgate_part) a.dgate_part[(size_t)rs * BT * N + o] = sdf;
          else a.dgate[o] = sdf;
        }
      }
    };
    if (is_loader) {
      for (int j = 0; j < nch; ++j) {   // runs up to kRing chunks ahead of the writer
        if (j >= kRing && !mbar_wait<1000>(&slot_free[j & (kRing - 1)], ((j / kRing) - 1) & 1)) { report_timeout(a.dev_status); return; }
        fill(j);
      }
    } else {
      for (int j = 0; j < nch; ++j) {
        if (!mbar_wait<1000>(&out_full[j & (kRing - 1)], (j / kRing) & 1)) { report_timeout(a.dev_status); return; }
        flush(j);
        __syncwarp();
        if (lane == 0) mbar_arrive(&slot_free[j & (kRing - 1)]);
      }
    }
  }
}

template <int V, int NWC>
cudaError_t launch_bwd_t(const ScanArgs &a, cudaStream_t s) {
  const BwdLayout L = bwd_layout<V>(16 * NWC, a.C, V > 64);
  cudaError_t e = cudaFuncSetAttribute(bwd_bf16_kernel<V, NWC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total);
  if (e != cudaSuccess) return e;
  const int RS = a.K / (16 * NWC);
  bwd_bf16_kernel<V, NWC><<<a.B * a.N * RS, bwd_threads<V, NWC>(), L.total, s>>>(a);
  return cudaGetLastError();
}

template <int V>
cudaError_t launch_bwd_v(const ScanArgs &a, cudaStream_t s) {
  switch (a.KC) {
    case 16: return launch_bwd_t<V, 1>(a, s);
    case 32: return launch_bwd_t<V, 2>(a, s);
    case 64: return launch_bwd_t<V, 4>(a, s);
    default: return cudaErrorInvalidValue;
  }
}

template <int V>
size_t bwd_smem(int KC, int C) { return bwd_layout<V>(KC, C, V > 64).total; }

}  // namespace

size_t bwd_bf16_smem_bytes(int KC, int V, int C) {
  switch (V) {
    case 16: return bwd_smem<16>(KC, C);
    case 32: return bwd_smem<32>(KC, C);
    case 64: return bwd_smem<64>(KC, C);
    default: return bwd_smem<128>(KC, C);
  }
}

cudaError_t launch_bwd_bf16(const ScanArgs &a, cudaStream_t s) {
  switch (a.V) {
    case 16: return launch_bwd_v<16>(a, s);
    case 32: return launch_bwd_v<32>(a, s);
    case 64: return launch_bwd_v<64>(a, s);
    case 128: return launch_bwd_v<128>(a, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace m2rnn

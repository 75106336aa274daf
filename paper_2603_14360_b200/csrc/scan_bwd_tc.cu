// bf16 backward through time (Algorithm 2 with the carried state gradient) for V = 128 on the
// 5th-generation tensor cores: every product of a step is a tcgen05.mma with its accumulator in
// tensor memory.
//
// At V = 128 the register kernels are bound by the legacy mma.sync path (W and W^T fragments no
// longer fit in registers, 130-150 MMAs and as many shared-memory loads per chain warp and step);
// here W^T and W sit in tensor memory for the whole scan and the products are issued by one thread.
// As in the tcgen05 forward kernel the products are computed transposed, M = 128 lanes = state
// columns, N = 32 state rows of the CTA, K = 128:
//     recompute   P^T  = W^T . H_{t-1}^T      (A = W^T in tensor memory, B = H_{t-1} slab, bf16, shared memory)
//     reverse     (dX W^T)^T = W . dX^T        (A = W   in tensor memory, B = dX slab)
//     dW += H_{t-1}^T dX                      (both slabs read MN-major from shared memory, one MMA per
//                                              step, accumulator 128 x 128 in tensor memory until the end)
// A thread owns one state column and 8 rows, so v_t[j], dy_t[j], f_t are per-thread scalars, k_t[i],
// q_t[i] warp-uniform broadcasts, and dv_j = sum_i dX[i][j] k_i is a sum over a thread's registers.
// Sums over columns (dq = H_t dy, dk = dX v) are small mma.sync products that helper warps take
// from the same shared-memory slabs, off the chain.
//
// One CTA per (b, n, 32-row slab).  Time is walked in chunks of C steps, last chunk first:
//   chain warps  (16)  run BOTH dependency chains, interleaved step by step: the recompute of chunk
//                      c-1 (forward steps from its checkpoint; per step the H_{t-1} slab -- bf16, the
//                      B operand -- and, per thread, Z_t as fp16) and the reverse sweep of chunk c
//                      (C = dL/dH in registers: G = C + q dy^T, df, dX = (1-f) G (1 - Z^2),
//                      C <- f G + dX W^T; dv; the dX slab).  While one chain's product is in the
//                      tensor core the warps do the other chain's arithmetic: a tcgen05 round trip
//                      is several hundred cycles, and two separate sets of warps (the first form of
//                      this kernel: 25 ms on sweep128) only waited on each other's products;
//   MMA warp      (1)  issues both chains' products as their slabs complete.  The issuing thread
//                      stalls while the tensor core is busy, so it is none of the chain warps (with
//                      a chain warp issuing behind CTA-wide barriers: 24.9 ms; this way 22.7 ms);
//   helper warps  (4)  issue the dW product, compute dq and dk;
//   loader, writer (2) stage q, k, v, dy and the gate of coming chunks / reduce and write dq, dk,
//                      dv, dgate of finished ones.
// Two state buffers: the recompute writes one while the reverse sweep, the helpers and the dW
// product read the other.  Hand-over is by mbarriers; every wait is bounded and reports through
// dev_status; a common exit frees the tensor memory.  Row-slab sums (dv, dgate, dW) are finished
// by the second-stage kernels.
#include <cuda_fp16.h>

#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"
#include "tc_common.cuh"
#include "tile.cuh"

namespace m2rnn {
namespace {

constexpr int kV = 128;
constexpr int kNR = 32;              // state rows per CTA = N of the MMAs
constexpr int kNT = 8;               // state rows per thread
constexpr int kChainWarps = 16;      // lane quarter (warp % 4) x row group (warp / 4)
constexpr int kRowGroups = kNR / kNT;
constexpr int kHelpWarps = 4;
constexpr int kWarps = kChainWarps + kHelpWarps + 3;   // + loader, writer, MMA issuer
constexpr int kThreads = kWarps * 32;
constexpr int kRingTc = 4;           // chunk slots of staged inputs / outputs in flight
constexpr int kCTc = 4;              // steps per chunk = checkpoint interval of this kernel
// tensor-memory columns: W^T, W (two bf16 per column), the two chain accumulators, dW
constexpr uint32_t kColWT = 0, kColW = 64, kColP = 128, kColC = 160, kColDW = 256, kTmemColsBwd = 512;

constexpr uint32_t kTileBytes = kNR * 256;                   // a 32 x 128 bf16 slab: 128 columns of 64 bytes
constexpr uint32_t kPrivBytes = kChainWarps * 32 * 16;       // per thread 8 x fp16 = 16 bytes of Z
constexpr uint32_t kStepBytes = kTileBytes + kPrivBytes;     // 16 384: keeps every tile on a 1024-byte boundary

struct TcBwdSmem {
  // byte offsets from the 1024-byte aligned base
  static constexpr uint32_t oBar = 0, oState = 1024;
  // [2] x { C step blocks (slab + Z), one more slab: the state after the chunk's last step }
  static constexpr uint32_t buf_bytes = kCTc * kStepBytes + kTileBytes, state_bytes = 2u * buf_bytes;
  static constexpr uint32_t oDx = oState + state_bytes, oRing = oDx + 2 * kTileBytes;
  // words of a ring slot.  In: q, k [C][32] as fp32, f and its slope [C], v and dy [C][128] as the
  // raw bf16 (a chain thread widens its own element; the helper products take them as pairs).
  // Out: the helpers' shares of dq and dk [C][4][32], dv per row group [C][4][128], one df partial
  // per chain warp [C][16].
  static constexpr uint32_t oQ = 0, oK = oQ + kCTc * kNR, oF = oK + kCTc * kNR, oDF = oF + 4, oDYB = oDF + 4,
                            oVB = oDYB + kCTc * kV / 2, oDQ = oVB + kCTc * kV / 2, oDK = oDQ + kCTc * kHelpWarps * kNR,
                            oDV = oDK + kCTc * kHelpWarps * kNR, oDFP = oDV + kCTc * kRowGroups * kV,
                            slot_words = oDFP + kCTc * kChainWarps;
  static constexpr uint32_t slot_bytes = slot_words * 4;
  static constexpr uint32_t total = oRing + kRingTc * slot_bytes + 1024;      // + slack to align the base
};
static_assert(kCTc == 4, "the slot layout keeps f and its slope in four words each");

// A slab holds 32 state rows x 128 columns of bf16 COLUMN by column: column l is a row of 64 bytes
// (the 32 state rows, contiguous), 64-byte swizzled: the 16-byte chunk (i / 8) of column l sits at
// chunk (i / 8) ^ ((l / 2) % 4).  A chain thread's 8 rows of its column are one 16-byte access; the
// tensor core reads the slab N-major (N = state rows) as the B operand of the chain products and
// K-major (K = state rows) as either operand of the dW product.
__device__ __forceinline__ uint32_t slab_off(int i, int l) {
  return (uint32_t)l * 64u + ((((uint32_t)i >> 3) ^ (((uint32_t)l >> 1) & 3u)) << 4) + (uint32_t)(i & 7) * 2u;
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float2 unpack_f16x2(uint32_t x) { return __half22float2(*reinterpret_cast<const __half2 *>(&x)); }

__global__ void __launch_bounds__(kThreads, 1) bwd_tc_kernel(ScanArgs a) {
  using S = TcBwdSmem;
  constexpr int V = kV;
  const int C = a.C;                 // steps per chunk (<= kCTc, which sizes the buffers)
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base_sa = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char *base = smem_dyn + (base_sa - smem_u32(smem_dyn));
  uint64_t *bars = reinterpret_cast<uint64_t *>(base + S::oBar);
  uint64_t *in_full = bars;                    // [kRingTc] a chunk's inputs are staged
  uint64_t *out_full = in_full + kRingTc;      // [kRingTc] its dq, dk, dv, df shares are in the slot
  uint64_t *slot_free = out_full + kRingTc;    // [kRingTc] ... and written out
  uint64_t *st_ready = slot_free + kRingTc;    // [2] a chunk's recomputed steps are in the state buffer
  uint64_t *st_free = st_ready + 2;            // [2] ... and read by everybody
  uint64_t *dx_full = st_free + 2;             // [2] a step's dX slab is written
  uint64_t *dx_free = dx_full + 2;             // [2] ... and read by the helpers and the dW product
  uint64_t *rec_done = dx_free + 2;            // the recompute product has landed in tensor memory
  uint64_t *rev_done = rec_done + 1;           // the reverse product has landed
  uint64_t *dw_done = rev_done + 1;            // every dW product has landed
  uint64_t *rec_slab = dw_done + 1;            // the recompute's H_{t-1} slab of a step is written (all chain warps)
  uint64_t *rev_slab = rec_slab + 1;           // the reverse sweep's dX slab of a step is written
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(rev_slab + 1);

  const int K = a.K, N = a.N;
  const int tid = threadIdx.x, warp = __shfl_sync(0xffffffffu, tid >> 5, 0), lane = tid & 31;
  const int RS = K / kNR;
  const int unit = blockIdx.x / RS, rs = blockIdx.x % RS, b = unit / N, n = unit % N;
  const int rbase = rs * kNR;
  const UnitSpan span = unit_span(a, b);
  const int T = span.T;
  const size_t tok0 = span.tok0;
  const int nch = (T + C - 1) / C;
  const size_t KV = (size_t)K * V;
  auto chunk_t0 = [&](int j) { return (nch - 1 - j) * C; };      // chunk j of the sweep = time chunk nch-1-j
  auto chunk_len = [&](int j) { return min(C, T - chunk_t0(j)); };
  auto slot_f = [&](int j) { return reinterpret_cast<float *>(base + S::oRing + (uint32_t)(j & (kRingTc - 1)) * S::slot_bytes); };
  auto step_sa = [&](int j, int s) { return base_sa + S::oState + (uint32_t)(j & 1) * S::buf_bytes + (uint32_t)s * kStepBytes; };

  if (tid == 0) {
    for (int s = 0; s < kRingTc; ++s) { mbar_init(&in_full[s], 1); mbar_init(&out_full[s], kChainWarps + kHelpWarps); mbar_init(&slot_free[s], 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(&st_ready[s], kChainWarps);
      mbar_init(&st_free[s], kHelpWarps + 1);                   // helpers and the dW product's commit
      mbar_init(&dx_full[s], kChainWarps);
      mbar_init(&dx_free[s], kHelpWarps + 1);
    }
    mbar_init(rec_done, 1); mbar_init(rev_done, 1); mbar_init(dw_done, 1);
    mbar_init(rec_slab, kChainWarps); mbar_init(rev_slab, kChainWarps);
    fence_mbar_init();
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemColsBwd) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);
  if (warp < 8) {
    // W^T (warps 0-3) and W (warps 4-7) into tensor memory, lane = row, column c = elements 2c, 2c+1:
    // W^T row j = W[:, j]; W row l = W[l, :]
    const int r = 32 * (warp & 3) + lane;
    const uint16_t *w = reinterpret_cast<const uint16_t *>(a.W) + (size_t)n * V * V;
    const bool transposed = warp < 4;
#pragma unroll 1
    for (int c0 = 0; c0 < 64; c0 += 8) {
      uint32_t v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int x = 2 * (c0 + e);
        v[e] = transposed ? ((uint32_t)w[(size_t)x * V + r] | ((uint32_t)w[(size_t)(x + 1) * V + r] << 16))
                          : *reinterpret_cast<const uint32_t *>(w + (size_t)r * V + x);
      }
      tmem_st8(tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (transposed ? kColWT : kColW) + (uint32_t)c0, v);
    }
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  bool failed = false;

  if (warp < kChainWarps) {
    // ================================================================= chain warps
    const int quarter = warp & 3, rg = warp >> 2;
    const int j = 32 * quarter + lane;                 // this thread's state column = tensor-memory lane
    const int i0 = kNT * rg;                           // its first row inside the CTA's slab
    static_assert(kNT == 8, "a thread's rows of its column are one 16-byte chunk of a slab");
    const uint32_t own = slab_off(i0, j);              // its 16 bytes inside a slab
    const uint32_t priv = kTileBytes + (uint32_t)(128 * rg + j) * 16u;   // its 16 bytes of Z inside a step block
    const uint32_t lane_tm = tmem_base + ((uint32_t)(32 * quarter) << 16) + (uint32_t)i0;
    auto store_slab = [&](uint32_t slab_sa, const float (&x)[kNT]) {
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(slab_sa + own), "r"(pack_bf16(x[0], x[1])), "r"(pack_bf16(x[2], x[3])),
                   "r"(pack_bf16(x[4], x[5])), "r"(pack_bf16(x[6], x[7])) : "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> visible to the tensor core
    };
    // a slab is complete when every chain warp has said so; the MMA warp takes it from there (its
    // issue stalls while the tensor core is busy, which must not hold up the chain warps)
    auto slab_done = [&](uint64_t *bar) {
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar);
    };
    auto load_ckpt = [&](int jc, float (&h)[kNT]) {      // the state before chunk jc's first step (fp32)
      const float *ck = a.ckpt + ((size_t)unit * a.nchunks + (nch - 1 - jc)) * KV + (size_t)(rbase + i0) * V + j;
#pragma unroll
      for (int x = 0; x < kNT; ++x) h[x] = ck[(size_t)x * V];
    };

    float H[kNT], Hn[kNT], Cg[kNT];      // recompute state, the next chunk's checkpoint (fetched a chunk ahead), dL/dH
    if (a.d_hT) {
#pragma unroll
      for (int x = 0; x < kNT; ++x) Cg[x] = a.d_hT[(size_t)unit * KV + (size_t)(rbase + i0 + x) * V + j];
    } else {
#pragma unroll
      for (int x = 0; x < kNT; ++x) Cg[x] = 0.f;
    }
    if (nch > 0) load_ckpt(0, Hn);
    const float clip = a.dh_clip;
    uint32_t nrec = 0, nrev = 0;   // products issued so far by either chain: phases of rec_done / rev_done, dX slab in turn
    bool pending = false;          // a product dX W^T is in flight and not yet added to Cg
    auto absorb = [&]() -> bool {   // Cg <- f G (already there) + dX W^T
      if (!mbar_wait(rev_done, (nrev - 1u) & 1u)) return false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float Pp[kNT];
      tmem_ld(lane_tm + kColC, Pp);
#pragma unroll
      for (int x = 0; x < kNT; x += 2) {
        const float2 c = __fadd2_rn(make_float2(Cg[x], Cg[x + 1]), make_float2(Pp[x], Pp[x + 1]));
        Cg[x] = c.x; Cg[x + 1] = c.y;
      }
      if (clip > 0.f) {
#pragma unroll
        for (int x = 0; x < kNT; ++x) Cg[x] = fminf(fmaxf(Cg[x], -clip), clip);
      }
      pending = false;
      return true;
    };
    // iteration `it` recomputes chunk it and sweeps chunk it - 1 backwards
    for (int it = 0; it <= nch && !failed; ++it) {
      const bool do_rec = it < nch, do_rev = it >= 1;
      const int lenR = do_rec ? chunk_len(it) : 0, lenV = do_rev ? chunk_len(it - 1) : 0;
      const float *sfR = slot_f(it);
      float *sfV = slot_f(it - 1);
      if (do_rec) {
#pragma unroll
        for (int x = 0; x < kNT; ++x) H[x] = Hn[x];
        if (it + 1 < nch) load_ckpt(it + 1, Hn);        // lands while this chunk is computed
        if (!mbar_wait(&in_full[it & (kRingTc - 1)], (it / kRingTc) & 1)) { failed = true; break; }
        if (it >= 2 && !mbar_wait(&st_free[it & 1], ((it >> 1) - 1) & 1)) { failed = true; break; }
      }
      for (int x = 0; x < C; ++x) {
        const bool rec_on = x < lenR, rev_on = x < lenV;
        const int sv = lenV - 1 - x;                      // the reverse sweep's step inside its chunk
        const uint32_t blkR = step_sa(it, x), blkV = step_sa(it - 1, sv);
        // ---- recompute: H_{t-1} -> slab (this step's B operand, and what dW and dq read later)
        if (rec_on) { store_slab(blkR, H); slab_done(rec_slab); ++nrec; }
        // ---- reverse step, while the recompute product is in the tensor core
        const int xb = nrev & 1u;
        const uint32_t dx_sa = base_sa + S::oDx + (uint32_t)xb * kTileBytes;
        if (rev_on) {
          const uint4 z0 = *reinterpret_cast<const uint4 *>(base + (blkV - base_sa) + priv);
          const uint32_t zw[kNT / 2] = {z0.x, z0.y, z0.z, z0.w};
          const float dyj = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(sfV + S::oDYB)[sv * V + j] << 16);
          const float f = sfV[S::oF + sv], omf = 1.f - f;
          uint32_t hw[kNT / 2];   // H_{t-1}, this thread's own chunk of the slab it wrote a chunk ago
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(hw[0]), "=r"(hw[1]), "=r"(hw[2]), "=r"(hw[3]) : "r"(blkV + own));
          if (pending && !absorb()) { failed = true; break; }
          float dX[kNT];
          float2 df2 = make_float2(0.f, 0.f), dv2 = make_float2(0.f, 0.f);
          float q8[kNT], k8[kNT];
#pragma unroll
          for (int r = 0; r < kNT; r += 4) {
            *reinterpret_cast<float4 *>(q8 + r) = *reinterpret_cast<const float4 *>(sfV + S::oQ + sv * kNR + i0 + r);
            *reinterpret_cast<float4 *>(k8 + r) = *reinterpret_cast<const float4 *>(sfV + S::oK + sv * kNR + i0 + r);
          }
#pragma unroll
          for (int r = 0; r < kNT; r += 2) {
            const float2 qq = make_float2(q8[r], q8[r + 1]), kk = make_float2(k8[r], k8[r + 1]);
            const float2 hp = make_float2(__uint_as_float(hw[r / 2] << 16), __uint_as_float(hw[r / 2] & 0xffff0000u));
            const float2 z = unpack_f16x2(zw[r / 2]);
            const float2 G = __ffma2_rn(qq, make_float2(dyj, dyj), make_float2(Cg[r], Cg[r + 1]));                             // G = C + q dy^T
            df2 = __ffma2_rn(G, __ffma2_rn(z, make_float2(-1.f, -1.f), hp), df2);                                          // df = sum G (.) (H_{t-1} - Z)
            const float2 x2 = __fmul2_rn(__fmul2_rn(make_float2(-omf, -omf), G), __ffma2_rn(z, z, make_float2(-1.f, -1.f)));   // (1-f) G (1 - Z^2)
            const float2 c2 = __fmul2_rn(make_float2(f, f), G);                                                            // gated path into H_{t-1}
            dv2 = __ffma2_rn(x2, kk, dv2);                                                                                 // dv = dX^T k, this thread's rows
            dX[r] = x2.x; dX[r + 1] = x2.y;
            Cg[r] = c2.x; Cg[r + 1] = c2.y;
          }
          // df: summed over the warp here, over the warps by the writer; dv: one share per row group,
          // added by the writer
          float df = df2.x + df2.y;
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) df += __shfl_xor_sync(0xffffffffu, df, off);
          if (lane == 0) sfV[S::oDFP + sv * kChainWarps + warp] = df;
          sfV[S::oDV + (sv * kRowGroups + rg) * V + j] = dv2.x + dv2.y;
          // (the buffer is free: the MMA warp issued the previous step's product, whose result was
          // added above, only after the helpers and the dW product were through with it)
          store_slab(dx_sa, dX);
          slab_done(rev_slab);
          ++nrev;
          pending = true;
          if (lane == 0) mbar_arrive(&dx_full[xb]);
        }
        // ---- recompute epilogue, while the reverse product is in the tensor core
        if (rec_on) {
          const float vj = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t *>(sfR + S::oVB)[x * V + j] << 16), f = sfR[S::oF + x];
          if (!mbar_wait(rec_done, (nrec - 1u) & 1u)) { failed = true; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          float P[kNT];
          tmem_ld(lane_tm + kColP, P);
          uint32_t zw[kNT / 2];
          float k8[kNT];
#pragma unroll
          for (int r = 0; r < kNT; r += 4) *reinterpret_cast<float4 *>(k8 + r) = *reinterpret_cast<const float4 *>(sfR + S::oK + x * kNR + i0 + r);
#pragma unroll
          for (int r = 0; r < kNT; r += 2) {
            const float2 kk = make_float2(k8[r], k8[r + 1]);
            const float2 pre = __ffma2_rn(kk, make_float2(vj, vj), make_float2(P[r], P[r + 1]));
            const float2 z = make_float2(tanh_approx(pre.x), tanh_approx(pre.y));                            // Eq. 1
            const float2 d = __ffma2_rn(z, make_float2(-1.f, -1.f), make_float2(H[r], H[r + 1]));             // H_{t-1} - Z
            const float2 h = __ffma2_rn(make_float2(f, f), d, z);                                           // Eq. 2
            H[r] = h.x; H[r + 1] = h.y;
            zw[r / 2] = pack_f16x2(z.x, z.y);
          }
          *reinterpret_cast<uint4 *>(base + (blkR - base_sa) + priv) = make_uint4(zw[0], zw[1], zw[2], zw[3]);
        }
      }
      if (failed) break;
      if (do_rec) {
        store_slab(step_sa(it, lenR), H);                // the state after the chunk's last step: H_t of its last step's dq
        __syncwarp();
        if (lane == 0) mbar_arrive(&st_ready[it & 1]);
      }
      if (do_rev) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&out_full[(it - 1) & (kRingTc - 1)]);
      }
    }
    if (!failed && pending && !absorb()) failed = true;   // the last step's product
    if (a.dh0 && !failed) {
#pragma unroll
      for (int x = 0; x < kNT; ++x) a.dh0[(size_t)unit * KV + (size_t)(rbase + i0 + x) * V + j] = Cg[x];
    }
  } else if (warp < kChainWarps + kHelpWarps) {
    // ================================================================= helper warps
    const int h = warp - kChainWarps, g = lane >> 2, c = lane & 3;
    // transposing ldmatrix of a 16 x 16 A fragment (state rows 16 mt .., columns 16 kt ..) of a slab:
    // lane supplies column 16 kt + 8 (lane / 16) + lane % 8, rows 16 mt + 8 ((lane / 8) % 2) .. + 7
    uint32_t aoff[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int x = 0; x < 2; ++x) aoff[mt][x] = slab_off(16 * mt + 8 * ((lane >> 3) & 1), 16 * (2 * h + x) + 8 * (lane >> 4) + (lane & 7));
    constexpr uint32_t idesc_dw = idesc_bf16(128, V);
    uint32_t nstep = 0;
    for (int jc = 0; jc < nch && !failed; ++jc) {
      const int len = chunk_len(jc);
      if (!mbar_wait(&st_ready[jc & 1], (jc >> 1) & 1)) { failed = true; break; }
      float *sf = slot_f(jc);
      for (int s = len - 1; s >= 0; --s, ++nstep) {
        const int xb = nstep & 1u;
        if (!mbar_wait(&dx_full[xb], (nstep >> 1) & 1u)) { failed = true; break; }
        const uint32_t ht = step_sa(jc, s), hn = step_sa(jc, s + 1), xt = base_sa + S::oDx + (uint32_t)xb * kTileBytes;
        if (h == 0 && elect_one()) {
          // dW += H_{t-1}^T dX: M = l and N = j are the slabs' columns, K = their 32 state rows (K-major),
          // in two MMAs of 16 rows = 32 bytes of every column
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int kt = 0; kt < kNR / 16; ++kt)
            umma_bf16_ss(tmem_base + kColDW, smem_desc_sw64(ht + 32u * kt), smem_desc_sw64(xt + 32u * kt), idesc_dw,
                         (nstep > 0 || kt > 0) ? 1u : 0u);
          umma_commit_tc(&dx_free[xb]);
          if (s == 0) umma_commit_tc(&st_free[jc & 1]);
        }
        __syncwarp();
        // dq = H_t dy and dk = dX v over this warp's 32 columns (two k-tiles); rows 16 mt + g, + 8
        float dq[2][4], dk[2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) dq[mt][0] = dq[mt][1] = dq[mt][2] = dq[mt][3] = dk[mt][0] = dk[mt][1] = dk[mt][2] = dk[mt][3] = 0.f;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const int kt = 2 * h + x;
          const float *dyb = sf + S::oDYB + s * (V / 2) + 8 * kt, *vb = sf + S::oVB + s * (V / 2) + 8 * kt;
          const uint32_t bq0 = __float_as_uint(dyb[c]), bq1 = __float_as_uint(dyb[4 + c]);
          const uint32_t bk0 = __float_as_uint(vb[c]), bk1 = __float_as_uint(vb[4 + c]);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            uint32_t A[4];
            ldmatrix_x4_trans(hn + aoff[mt][x], A);
            mma_bf16_16816(dq[mt], A, bq0, bq1);
            ldmatrix_x4_trans(xt + aoff[mt][x], A);
            mma_bf16_16816(dk[mt], A, bk0, bk1);
          }
        }
        if (c == 0) {
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            float *pq = sf + S::oDQ + (s * kHelpWarps + h) * kNR + 16 * mt + g, *pk = sf + S::oDK + (s * kHelpWarps + h) * kNR + 16 * mt + g;
            pq[0] = dq[mt][0]; pq[8] = dq[mt][2];
            pk[0] = dk[mt][0]; pk[8] = dk[mt][2];
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&dx_free[xb]);
      }
      if (failed) break;
      __syncwarp();
      if (lane == 0) { mbar_arrive(&st_free[jc & 1]); mbar_arrive(&out_full[jc & (kRingTc - 1)]); }
    }
    // the dW accumulator (lane = row l, column = j) goes to this CTA's partial sum
    if (h == 0 && elect_one()) umma_commit_tc(dw_done);
    __syncwarp();
    const bool landed = mbar_wait(dw_done, 0);
    if (!landed) failed = true;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    float *row = a.dW_part + ((size_t)(b * RS + rs) * N + n) * V * V + (size_t)(32 * h + lane) * V;
#pragma unroll 1
    for (int x = 0; x < V / 8; ++x) {
      float r[8];
      if (landed && !failed && nstep > 0) {
        tmem_ld(tmem_base + ((uint32_t)(32 * h) << 16) + kColDW + 8u * x, r);
      } else {   // no step at all (an empty sequence): the sum is empty
#pragma unroll
        for (int e = 0; e < 8; ++e) r[e] = 0.f;
      }
      *reinterpret_cast<float4 *>(row + 8 * x) = make_float4(r[0], r[1], r[2], r[3]);
      *reinterpret_cast<float4 *>(row + 8 * x + 4) = make_float4(r[4], r[5], r[6], r[7]);
    }
  } else if (warp == kChainWarps + kHelpWarps + 2) {
    // ================================================================= MMA warp
    // Follows the chain warps' schedule: per iteration and step first the recompute product, then
    // the reverse product, each as soon as its slab is complete.  Eight MMAs of 16 K indices: 8
    // columns of A in tensor memory, 16 columns = 1024 bytes of the slab, read N-major.
    constexpr uint32_t idesc = idesc_bf16(128, kNR) | (1u << 16);
    auto issue = [&](uint32_t d_col, uint32_t a_col, uint32_t slab_sa, uint64_t *bar) {
      if (elect_one()) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          umma_bf16_ts(tmem_base + d_col, tmem_base + a_col + 8u * kk,
                       smem_desc_sw64(slab_sa + 1024u * kk), idesc, kk > 0);
        umma_commit_tc(bar);
      }
      __syncwarp();
    };
    uint32_t nrec = 0, nrev = 0;
    for (int it = 0; it <= nch && !failed; ++it) {
      const int lenR = it < nch ? chunk_len(it) : 0, lenV = it >= 1 ? chunk_len(it - 1) : 0;
      for (int x = 0; x < C; ++x) {
        if (x < lenR) {
          if (!mbar_wait(rec_slab, nrec & 1u)) { failed = true; break; }
          issue(kColP, kColWT, step_sa(it, x), rec_done);
          ++nrec;
        }
        if (x < lenV) {
          if (!mbar_wait(rev_slab, nrev & 1u)) { failed = true; break; }
          // the NEXT step's dX goes into the other buffer as soon as this product has been added to
          // the carried gradient: hold the product back until that buffer's last readers (the
          // helpers and the dW product of the step before this one) are through
          if (nrev >= 1 && !mbar_wait(&dx_free[(nrev + 1u) & 1u], ((nrev - 1u) >> 1) & 1u)) { failed = true; break; }
          issue(kColC, kColW, base_sa + S::oDx + (uint32_t)(nrev & 1u) * kTileBytes, rev_done);
          ++nrev;
        }
      }
    }
  } else {
    // ================================================================= loader and writer warps
    const bool is_loader = warp == kChainWarps + kHelpWarps;
    const int hq = n / (N / a.Nq), hk = n / (N / a.Nk);
    const float al = a.alpha ? a.alpha[n] : 1.f, be = a.beta ? a.beta[n] : 0.f;
    const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(a.q), *kg = static_cast<const __nv_bfloat16 *>(a.k);
    const __nv_bfloat16 *vg = static_cast<const __nv_bfloat16 *>(a.v), *dyg = static_cast<const __nv_bfloat16 *>(a.dy);
    const __nv_bfloat16 *wr = static_cast<const __nv_bfloat16 *>(a.w_r);
    const size_t TT = (size_t)a.TT;
    if (is_loader) {
      for (int jc = 0; jc < nch; ++jc) {   // runs up to kRingTc chunks ahead of the writer
        if (jc >= kRingTc && !mbar_wait<1000>(&slot_free[jc & (kRingTc - 1)], ((jc / kRingTc) - 1) & 1)) { failed = true; break; }
        float *sf = slot_f(jc);
        const int t0 = chunk_t0(jc), len = chunk_len(jc);
        const size_t bt0 = tok0 + t0;
        // q, k: 32 rows = 4 chunks of 16 bytes per step; v, dy: 16 chunks per step
        if (lane < 4 * len) {
          const int t = lane >> 2, i = (lane & 3) * 8;
          const uint4 qr = *reinterpret_cast<const uint4 *>(qg + (bt0 + t) * a.qs + (size_t)hq * K + rbase + i);
          const uint4 kr = *reinterpret_cast<const uint4 *>(kg + (bt0 + t) * a.ks + (size_t)hk * K + rbase + i);
          store8_bf16_as_f32(sf + S::oQ + t * kNR + i, qr);
          store8_bf16_as_f32(sf + S::oK + t * kNR + i, kr);
        }
        for (int x = lane; x < 16 * len; x += 32) {
          const int t = x >> 4, i = (x & 15) * 8;
          const uint4 vr = *reinterpret_cast<const uint4 *>(vg + (bt0 + t) * a.vs + (size_t)n * V + i);
          const uint4 dr = *reinterpret_cast<const uint4 *>(dyg + ((bt0 + t) * N + n) * V + i);
          reinterpret_cast<uint4 *>(sf + S::oVB)[x] = vr;
          reinterpret_cast<uint4 *>(sf + S::oDYB)[x] = dr;
        }
        if (lane < len) {
          float dfdx;
          sf[S::oF + lane] = gate_value(a.gate_kind, a.gate[(bt0 + lane) * N + n], al, be, &dfdx);
          sf[S::oDF + lane] = dfdx;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&in_full[jc & (kRingTc - 1)]);
      }
    } else {
      for (int jc = 0; jc < nch; ++jc) {
        if (!mbar_wait<1000>(&out_full[jc & (kRingTc - 1)], (jc / kRingTc) & 1)) { failed = true; break; }
        const float *sf = slot_f(jc);
        const int t0 = chunk_t0(jc), len = chunk_len(jc);
        const size_t bt0 = tok0 + t0;
        // dq, dk: the four helpers' shares of this CTA's 32 rows, one row per lane
        {
          for (int t = 0; t < len; ++t) {
            float sq = 0.f, sk = 0.f;
#pragma unroll
            for (int hh = 0; hh < kHelpWarps; ++hh) {
              sq += sf[S::oDQ + (t * kHelpWarps + hh) * kNR + lane];
              sk += sf[S::oDK + (t * kHelpWarps + hh) * kNR + lane];
            }
            if (a.dq_part) a.dq_part[((bt0 + t) * N + n) * K + rbase + lane] = sq;
            else static_cast<__nv_bfloat16 *>(a.dq)[((bt0 + t) * a.Nq + hq) * K + rbase + lane] = __float2bfloat16_rn(sq);
            if (a.dk_part) a.dk_part[((bt0 + t) * N + n) * K + rbase + lane] = sk;
            else static_cast<__nv_bfloat16 *>(a.dk)[((bt0 + t) * a.Nk + hk) * K + rbase + lane] = __float2bfloat16_rn(sk);
          }
        }
        // dv of this CTA's rows (+ w_r (.) dy from Eq. 3, added by the first row slab only)
        for (int x = lane; x < len * (V / 2); x += 32) {
          const int t = x / (V / 2), jj = (x % (V / 2)) * 2;
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int r = 0; r < kRowGroups; ++r) {
            const float2 p = *reinterpret_cast<const float2 *>(sf + S::oDV + (t * kRowGroups + r) * V + jj);
            s0 += p.x; s1 += p.y;
          }
          if (wr && rs == 0) {
            const uint32_t dyp = __float_as_uint(sf[S::oDYB + t * (V / 2) + jj / 2]);
            s0 = fmaf(__bfloat162float(wr[(size_t)n * V + jj]), __uint_as_float(dyp << 16), s0);
            s1 = fmaf(__bfloat162float(wr[(size_t)n * V + jj + 1]), __uint_as_float(dyp & 0xffff0000u), s1);
          }
          const size_t o = ((bt0 + t) * N + n) * V + jj;
          if (a.dv_part) *reinterpret_cast<float2 *>(a.dv_part + (size_t)rs * TT * N * V + o) = make_float2(s0, s1);
          else *reinterpret_cast<uint32_t *>(static_cast<__nv_bfloat16 *>(a.dv) + o) = pack_bf16(s0, s1);
        }
        // dgate: one df partial per chain warp; fixed-order sum, then the gate's slope
        for (int t = 0; t < len; ++t) {
          if (lane == 0) {
            float sdf = 0.f;
#pragma unroll
            for (int x = 0; x < kChainWarps; ++x) sdf += sf[S::oDFP + t * kChainWarps + x];
            sdf *= sf[S::oDF + t];
            const size_t o = (bt0 + t) * N + n;
            if (a.dgate_part) a.dgate_part[(size_t)rs * TT * N + o] = sdf;
            else a.dgate[o] = sdf;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&slot_free[jc & (kRingTc - 1)]);
      }
    }
  }
  if (failed) report_timeout(a.dev_status);
  // common exit: every loop above ends after a bounded time
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemColsBwd) : "memory");
  }
}

}  // namespace

int bwd_tc_rows_per_cta() { return kNR; }
int bwd_tc_chunk() { return kCTc; }

cudaError_t launch_bwd_bf16_tc(const ScanArgs &a, cudaStream_t s) {
  if (a.V != kV || a.KC != kNR || a.C < 1 || a.C > kCTc) return cudaErrorInvalidValue;
  const size_t smem = TcBwdSmem::total;
  cudaError_t e = cudaFuncSetAttribute(bwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  bwd_tc_kernel<<<a.B * a.N * (a.K / kNR), kThreads, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace m2rnn

// bf16 decoding step (Eq. 1-3 once on a cached fp32 state) on the 5th-generation tensor cores.
//
// At decode time the K rows of every (b,n) state are independent rows of one product per head:
// [B*K, V] x [V, V].  A CTA stacks the states of 128/K units of one head into an M = 128 tile and
// runs H W as tcgen05.mma (kind::tf32, operands from shared memory, fp32 accumulator in tensor
// memory), which leaves the SM's issue slots and register file to the streaming part of the step:
//   - the states of the next task arrive by TMA (cp.async.bulk.tensor, 32-column boxes landing in
//     128-byte-swizzled rows, completion on an mbarrier) while the current task is computed;
//   - the staged fp32 tile is already the canonical K-major 128-byte-swizzled layout of a 32-bit
//     operand, so it is the A operand as it stands (the tensor core reads it as tf32, which keeps
//     three more mantissa bits of the state than a bf16 copy would, and no conversion pass runs);
//   - one thread issues the V/8 MMAs and commits them to an mbarrier;
//   - every thread then owns one state row and half of its columns: tcgen05.ld, + k_i v^T, tanh,
//     gate against the staged fp32 row, write H_t back in place (global) and into the stage;
//   - the readout y = H_t^T q is a column sum over the stage.
// Persistent CTAs walk (head, batch) tasks in head-major order; W_n^T is rebuilt in shared memory
// (K-major B tile) only when the head changes.  Every wait is bounded; a wait that runs out ends
// the CTA through the common exit, which frees the tensor memory.
#include <cuda.h>

#include "device_common.cuh"
#include "internal.h"
#include "mma_tile.cuh"
#include "pipeline.cuh"

namespace m2rnn {
namespace {

constexpr int kM = 128;   // rows of the MMA tile = threads that own a row each

__device__ __forceinline__ void mbar_expect_tx_tc(uint64_t *bar, uint32_t bytes) {
  asm volatile("{\n .reg .b64 st;\n mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// One box of a tiled (2-D) tensor map, global -> shared, no multicast.  x (innermost) times the
// element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst_sa, const CUtensorMap *map, int x, int y, uint64_t *bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst_sa), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// One box, shared -> global; completion is tracked by the issuing thread's bulk-async group.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int x, int y, uint32_t src_sa) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(src_sa) : "memory");
}

// Shared-memory matrix descriptor of a K-major operand in the 128-byte-swizzled canonical
// layout: rows of 128 bytes (32 tf32 elements), groups of 8 rows 1024 bytes apart, 16-byte chunks
// of a row XOR-ed with the row index modulo 8.
//   bits  0-13 start address >> 4     bits 32-45 stride between 8-row groups >> 4
//   bits 16-29 leading offset >> 4 (not used by swizzled K-major layouts)
//   bits 46-47 descriptor version 1   bits 61-63 swizzle mode (2 = 128 bytes)
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t sa) {
  return (uint64_t)((sa & 0x3ffffu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}
// Instruction descriptor of kind::tf32: fp32 accumulator (bits 4-5 = 1), tf32 A and B (bits 7-9 and
// 10-12 = 2), both K-major (bits 15, 16 = 0), N >> 3 in bits 17-22, M >> 4 in bits 24-28.
__host__ __device__ constexpr uint32_t umma_idesc_tf32(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[128 x N] (+)= A[128 x 8] B[N x 8]^T, both operands tf32
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7]), "=f"(r[8]),
        "=f"(r[9]), "=f"(r[10]), "=f"(r[11]), "=f"(r[12]), "=f"(r[13]), "=f"(r[14]), "=f"(r[15]), "=f"(r[16]),
        "=f"(r[17]), "=f"(r[18]), "=f"(r[19]), "=f"(r[20]), "=f"(r[21]), "=f"(r[22]), "=f"(r[23]), "=f"(r[24]),
        "=f"(r[25]), "=f"(r[26]), "=f"(r[27]), "=f"(r[28]), "=f"(r[29]), "=f"(r[30]), "=f"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// A staged fp32 state tile: V/32 blocks of [128 rows][32 columns = 128 bytes], the 16-byte chunks of
// a row XOR-ed with the row index modulo 8 (what the tensor map's 128-byte swizzle writes), so
// that a thread walking along its own row and a warp walking down a column both spread over all
// banks.  Offset in floats of element (i, j):
template <int V>
__device__ __forceinline__ uint32_t stage_off(int i, int j) {
  return (uint32_t)(j >> 5) * (kM * 32) + (uint32_t)i * 32 + (uint32_t)(((((j & 31) >> 2) ^ (i & 7)) << 2) | (j & 3));
}

template <int V>
struct TcSmem {
  static constexpr uint32_t b_bytes = V * V * 4;              // B tile (W^T as fp32): V/32 blocks of [V rows][128 bytes]
  static constexpr uint32_t stage_bytes = kM * V * 4;         // a stage = the A tile: V/32 blocks of [128 rows][128 bytes]
  // offsets from the 1024-byte aligned base
  static constexpr uint32_t oB = 0, oStage = oB + b_bytes, oVec = oStage + 2 * stage_bytes;
  // vectors (two buffers, the next task's are fetched a task ahead): k [128], q [128], f [128] per
  // row, v [128/K <= 8][V]; then the warps' readout partials [8][V]
  static constexpr uint32_t vec_floats = 3 * kM + 8 * V;
  static constexpr uint32_t vec_bytes = (2 * vec_floats + 8 * V) * 4;
  static constexpr uint32_t oBar = oVec + vec_bytes;          // 8 mbarriers, tmem slot, flag
  static constexpr uint32_t total = oBar + 128 + 1024;         // + slack for the alignment of the base
};

constexpr int kComputeThreads = 256;            // 8 compute warps ...
constexpr int kThreads = kComputeThreads + 32;   // ... and one warp that moves the states

// Barrier 1: the compute warps only (the mover never joins it), plain or with an AND over a
// per-thread predicate.
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory"); }
__device__ __forceinline__ bool compute_sync_and(bool pred) {
  uint32_t r;
  asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 q, %1, 0;\n bar.red.and.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}"
               : "=r"(r) : "r"((uint32_t)pred), "n"(kComputeThreads) : "memory");
  return r != 0;
}

template <int V>
__global__ void __launch_bounds__(kThreads, 1) decode_tc_kernel(ScanArgs a, int GPI, int tasks_per_head,
                                                                const __grid_constant__ CUtensorMap state_map) {
  using S = TcSmem<V>;
  constexpr int HC = V / 2;             // columns per thread in the epilogue
  extern __shared__ unsigned char smem_dyn[];
  // the swizzled tiles want a 1024-byte aligned base
  const uint32_t base_sa = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char *base = smem_dyn + (base_sa - smem_u32(smem_dyn));
  float *stage = reinterpret_cast<float *>(base + S::oStage);
  float *vecs = reinterpret_cast<float *>(base + S::oVec);
  float *ypart = vecs + 2 * S::vec_floats;                  // [8 warps][V]
  uint64_t *full = reinterpret_cast<uint64_t *>(base + S::oBar);   // [2] a task's states have landed in the stage
  uint64_t *mma_done = full + 2;                                    // [2] one per accumulator
  uint64_t *epi_done = mma_done + 2;                                // [2] H_t of the task is in the stage (8 warps arrive)
  uint64_t *stage_free = epi_done + 2;                              // [2] no compute warp reads the stage any more (8 arrive)
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(stage_free + 2);
  volatile uint32_t *early_flag = tmem_slot + 1;   // the next task's MMAs are already in flight

  const int K = a.K, N = a.N, B = a.B;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const __nv_bfloat16 *qg = static_cast<const __nv_bfloat16 *>(a.q), *kg = static_cast<const __nv_bfloat16 *>(a.k);
  const __nv_bfloat16 *vg = static_cast<const __nv_bfloat16 *>(a.v), *wr = static_cast<const __nv_bfloat16 *>(a.w_r);
  __nv_bfloat16 *yg = static_cast<__nv_bfloat16 *>(a.y);

  if (tid == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&mma_done[s], 1);
      mbar_init(&epi_done[s], kComputeThreads / 32);
      mbar_init(&stage_free[s], kComputeThreads / 32);
    }
    *early_flag = 0u;
    fence_mbar_init();
  }
  if (warp == 0) {   // 2 x V columns of tensor memory: two accumulators, used by alternate tasks
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * V) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  // Persistent CTA: tasks [t_begin, t_end) in head-major order; task -> (head n, batch group tb),
  // stepped without divisions
  const long ntasks = (long)N * tasks_per_head;
  const long t_begin = ntasks * blockIdx.x / gridDim.x, t_end = ntasks * (blockIdx.x + 1) / gridDim.x;
  const int n0 = (int)(t_begin / tasks_per_head), tb0 = (int)(t_begin % tasks_per_head);
  auto advance = [&](int &n, int &tb) { if (++tb == tasks_per_head) { tb = 0; ++n; } };

  if (warp == kComputeThreads / 32) {
    // ================================================================ the warp that moves states
    // Per task and 32-column block one box of [K rows][32 columns] per unit of the state viewed as
    // a [B*N*K, V] matrix.  Loads run two tasks ahead, into the stage whose store has drained.
    auto load_task = [&](int n, int tb, int st) {
      const int b0 = tb * GPI, units = min(GPI, B - b0);
      if (lane == 0) mbar_expect_tx_tc(&full[st], (uint32_t)(units * K) * (uint32_t)(V * 4));
      __syncwarp();
      const uint32_t dst0 = base_sa + S::oStage + (uint32_t)st * S::stage_bytes;
      for (int x = lane; x < units * (V / 32); x += 32) {
        const int u = x / (V / 32), cb = x % (V / 32);
        tma_load_2d(dst0 + (uint32_t)cb * (kM * 128) + (uint32_t)(u * K) * 128, &state_map, 32 * cb, ((b0 + u) * N + n) * K, &full[st]);
      }
    };
    auto store_task = [&](int n, int tb, int st) {
      const int b0 = tb * GPI, units = min(GPI, B - b0);
      const uint32_t src0 = base_sa + S::oStage + (uint32_t)st * S::stage_bytes;
      for (int x = lane; x < units * (V / 32); x += 32) {
        const int u = x / (V / 32), cb = x % (V / 32);
        tma_store_2d(&state_map, 32 * cb, ((b0 + u) * N + n) * K, src0 + (uint32_t)cb * (kM * 128) + (uint32_t)(u * K) * 128);
      }
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    };
    int nl = n0, tbl = tb0, ns = n0, tbs = tb0;   // next task to load / to store
    long loaded = t_begin;
    for (int st = 0; st < 2 && loaded < t_end; ++st, ++loaded) { load_task(nl, tbl, st); advance(nl, tbl); }
    bool ok = true;
    int it = 0;
    for (long task = t_begin; task < t_end; ++task, ++it) {
      const int st = it & 1;
      const uint32_t par = (uint32_t)(it >> 1) & 1u;
      // H_t is in the stage (written through the generic proxy, fenced by its writers): store it
      if (!mbar_wait(&epi_done[st], par)) { ok = false; break; }
      store_task(ns, tbs, st);
      advance(ns, tbs);
      if (loaded < t_end) {
        // the stage is free for the task after next once the readout no longer reads it and the
        // store has read it
        if (!mbar_wait(&stage_free[st], par)) { ok = false; break; }
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        load_task(nl, tbl, st);
        advance(nl, tbl);
        ++loaded;
      }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // the last stores
    if (!ok) report_timeout(a.dev_status);
  } else {
    // ================================================================ compute warps
    // Per-row scalars (threads 0..127: k_i, q_i, f of the row's unit) and the units' v vectors
    // (threads 128..255) of a task, fetched into registers a task ahead and parked in shared
    // memory when the current task no longer reads that buffer.
    constexpr int kVPer = 8 * V / 128;   // v entries per thread at most (8 units)
    const int dq = N / a.Nq, dk = N / a.Nk;
    const int my_u = (tid & (kM - 1)) / K, my_r = (tid & (kM - 1)) % K;
    // raw values only: nothing may depend on a load before the task that issued it is over
    struct VecRegs { uint16_t k, q; float gate; uint16_t v[kVPer]; int n; };
    auto fetch_vecs = [&](int n, int tb, VecRegs &o) {
      const int b0 = tb * GPI;
      o.n = n;
      o.k = o.q = 0; o.gate = 0.f;
      if (tid < kM) {
        const int bb = b0 + my_u;
        if (my_u < GPI && bb < B) {
          o.k = reinterpret_cast<const uint16_t *>(kg)[((size_t)bb * a.Nk + n / dk) * K + my_r];
          o.q = reinterpret_cast<const uint16_t *>(qg)[((size_t)bb * a.Nq + n / dq) * K + my_r];
          o.gate = a.gate[(size_t)bb * N + n];
        }
      } else {
#pragma unroll
        for (int m = 0; m < kVPer; ++m) {
          const int x = tid - kM + m * kM, u = x / V, bb = b0 + u;
          o.v[m] = (x < GPI * V && bb < B) ? reinterpret_cast<const uint16_t *>(vg)[((size_t)bb * N + n) * V + (x % V)] : (uint16_t)0;
        }
      }
    };
    const float *alpha = a.alpha, *beta = a.beta;
    auto park_vecs = [&](int buf, const VecRegs &o) {
      float *vb = vecs + (size_t)buf * S::vec_floats;
      if (tid < kM) {
        vb[tid] = __uint_as_float((uint32_t)o.k << 16);
        vb[kM + tid] = __uint_as_float((uint32_t)o.q << 16);
        // rows of absent units carry gate 0 -> some f; their results are never used
        vb[2 * kM + tid] = gate_value(a.gate_kind, o.gate, alpha ? alpha[o.n] : 1.f, beta ? beta[o.n] : 0.f, nullptr);
      } else {
#pragma unroll
        for (int m = 0; m < kVPer; ++m) {
          const int x = tid - kM + m * kM;
          if (x < GPI * V) vb[3 * kM + x] = __uint_as_float((uint32_t)o.v[m] << 16);
        }
      }
    };
    if (t_begin < t_end) {
      VecRegs first;
      fetch_vecs(n0, tb0, first);
      park_vecs(0, first);
    }

    constexpr uint32_t idesc = umma_idesc_tf32(kM, V);
    // the V/8 MMAs of the task whose states sit in stage st, into accumulator st (one thread)
    auto issue_mmas = [&](int st) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a_sa = base_sa + S::oStage + (uint32_t)st * S::stage_bytes;
#pragma unroll
      for (int ks = 0; ks < V / 8; ++ks) {
        // 8 elements (32 bytes) per step inside a 128-byte block, then the next block
        const uint32_t koff = (uint32_t)(ks / 4) * 128u * kM + (uint32_t)(ks % 4) * 32u;
        const uint32_t koffb = (uint32_t)(ks / 4) * 128u * V + (uint32_t)(ks % 4) * 32u;
        umma_tf32(tmem_base + (uint32_t)st * V, umma_desc_sw128(a_sa + koff), umma_desc_sw128(base_sa + S::oB + koffb), idesc, ks > 0);
      }
      umma_commit(&mma_done[st]);
    };
    int cur_head = -1, it = 0, n = n0, tb = tb0;
    bool failed = false;
    bool early = false;   // this task's MMAs were issued during the previous one
    for (long task = t_begin; task < t_end; ++task, ++it) {
      const int st = it & 1;
      const uint32_t par = (uint32_t)(it >> 1) & 1u;
      const int b0 = tb * GPI;
      const int rows = min(GPI, B - b0) * K;     // live rows of the tile
      const bool has_next = task + 1 < t_end;
      int n1 = n, tb1 = tb;
      advance(n1, tb1);
      VecRegs next;
      if (has_next) fetch_vecs(n1, tb1, next);   // lands while this task is computed
      if (n != cur_head) {
        // B tile = W_n^T widened to fp32, K-major: row j holds W[:, j]; element (j, l) sits in block
        // l/32 at row j, 16-byte chunk ((l%32)/4) ^ (j%8), like the rows of a stage
        const uint16_t *w = reinterpret_cast<const uint16_t *>(a.W) + (size_t)n * V * V;
        for (int x = tid; x < V * V / 4; x += kComputeThreads) {
          const int j = x % V, l0 = (x / V) * 4;
          uint32_t p[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) p[e] = (uint32_t)w[(l0 + e) * V + j] << 16;
          const uint32_t off = S::oB + (uint32_t)(l0 / 32) * (V * 128) + (uint32_t)j * 128 + ((((l0 % 32) / 4) ^ (j & 7)) << 4);
          *reinterpret_cast<uint4 *>(base + off) = make_uint4(p[0], p[1], p[2], p[3]);
        }
        cur_head = n;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the tensor core
      }
      const float *kvec = vecs + (size_t)st * S::vec_floats, *qvec = kvec + kM, *fvec = qvec + kM, *vvec = fvec + kM;
      // the task's states have landed (this barrier also orders the B tile's writes before the MMAs)
      if (!compute_sync_and(mbar_wait(&full[st], par))) { failed = true; break; }
      float *sg = stage + (size_t)st * (kM * V);
      if (tid == 0 && !early) issue_mmas(st);
      if (!compute_sync_and(mbar_wait(&mma_done[st], par))) { failed = true; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

      // epilogue: thread = (row i, column half)
      {
        const int i = 32 * (warp & 3) + lane, half = warp >> 2;
        const int u = i / K;
        const bool live = i < rows;
        const float ki = kvec[i], f = fvec[i];
        const float *vrow = vvec + (size_t)(live ? u : 0) * V + half * HC;
#pragma unroll
        for (int cb = 0; cb < HC / 32; ++cb) {
          float P[32];
          tmem_ld32(tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(st * V + half * HC + 32 * cb), P);
          if (live) {
#pragma unroll
            for (int x = 0; x < 8; ++x) {
              float4 *sp = reinterpret_cast<float4 *>(sg + stage_off<V>(i, half * HC + 32 * cb + 4 * x));
              const float4 h4 = *sp;
              const float4 v4 = *reinterpret_cast<const float4 *>(vrow + 32 * cb + 4 * x);
              float hn[4];
              const float hv[4] = {h4.x, h4.y, h4.z, h4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float z = tanh_approx(fmaf(ki, vv[e], P[4 * x + e]));   // Eq. 1
                hn[e] = fmaf(f, hv[e] - z, z);                               // Eq. 2
              }
              *sp = make_float4(hn[0], hn[1], hn[2], hn[3]);
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // H_t in the stage -> visible to the TMA store
      __syncwarp();
      if (lane == 0) mbar_arrive(&epi_done[st]);
      compute_sync();
      if (warp == 0) {
        // The next task's product does not depend on this one: start it now, into the other
        // accumulator, so that the tensor core works while the readout runs (unless the head
        // changes, which rebuilds the B tile first).  The outcome reaches every thread through
        // shared memory at the next barrier.
        bool go = has_next && n1 == n;
        if (go) go = mbar_wait(&full[st ^ 1], (uint32_t)((it + 1) >> 1) & 1u);
        if (go && lane == 0) issue_mmas(st ^ 1);
        if (lane == 0) *early_flag = go ? 1u : 0u;
      }
      // readout (Eq. 3): y[u][j] = sum over the unit's rows of q_i H_t[i][j].  Each warp sums 16 rows
      // (all of one unit, K >= 16); then the warps of a unit are added.
      {
        // lane = (row group, 32-column block, 16-byte chunk): one 128-byte row of a block per 8 lanes
        constexpr int NB = V / 32, RG = 4 / NB;
        const int c8 = lane & 7, m = (lane >> 3) % NB, rg = lane / (8 * NB);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int rr = 0; rr < 16 / RG; ++rr) {
          const int i = 16 * warp + rg * (16 / RG) + rr;
          const float qi = qvec[i];
          const float4 h4 = *reinterpret_cast<const float4 *>(sg + (uint32_t)m * (kM * 32) + (uint32_t)i * 32 + (uint32_t)((c8 ^ (i & 7)) << 2));
          acc.x = fmaf(qi, h4.x, acc.x); acc.y = fmaf(qi, h4.y, acc.y); acc.z = fmaf(qi, h4.z, acc.z); acc.w = fmaf(qi, h4.w, acc.w);
        }
        if constexpr (RG == 2) {
          acc.x += __shfl_xor_sync(0xffffffffu, acc.x, 16); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, 16);
          acc.z += __shfl_xor_sync(0xffffffffu, acc.z, 16); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, 16);
        }
        if (rg == 0) *reinterpret_cast<float4 *>(ypart + warp * V + 32 * m + 4 * c8) = acc;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&stage_free[st]);   // this warp has read the stage for the last time
      compute_sync();
      for (int x = tid; x < GPI * V; x += kComputeThreads) {
        const int u = x / V, j = x % V, bb = b0 + u;
        if (bb < B) {
          float s = 0.f;
          for (int w = u * K / 16; w < (u + 1) * K / 16; ++w) s += ypart[w * V + j];
          if (wr) s = fmaf(__bfloat162float(wr[(size_t)n * V + j]), vvec[x], s);
          yg[((size_t)bb * N + n) * V + j] = __float2bfloat16_rn(s);
        }
      }
      if (has_next) park_vecs(st ^ 1, next);
      early = *early_flag != 0u;   // written before the barrier in front of the final sum
      compute_sync();   // vectors and partial sums are free again
      n = n1; tb = tb1;
    }
    if (failed) report_timeout(a.dev_status);
  }
  // common exit: every loop above ends after a bounded time
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * V) : "memory");
  }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against libcuda)
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

template <int V>
cudaError_t launch_tc(const ScanArgs &a, cudaStream_t s) {
  // the state as a [B*N*K, V] fp32 matrix, boxes of [K rows][32 columns], 128-byte swizzle
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return cudaErrorNotSupported;
  CUtensorMap map;
  const cuuint64_t dims[2] = {(cuuint64_t)V, (cuuint64_t)a.B * a.N * a.K};
  const cuuint64_t strides[1] = {(cuuint64_t)V * 4};
  const cuuint32_t box[2] = {32u, (cuuint32_t)a.K}, estr[2] = {1u, 1u};
  if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, a.hT, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  const int GPI = kM / a.K;
  const int tasks_per_head = (a.B + GPI - 1) / GPI;
  const long ntasks = (long)a.N * tasks_per_head;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = (int)(ntasks < sms ? ntasks : sms);
  const size_t smem = TcSmem<V>::total;
  cudaError_t e = cudaFuncSetAttribute(decode_tc_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  decode_tc_kernel<V><<<grid, kThreads, smem, s>>>(a, GPI, tasks_per_head, map);
  return cudaGetLastError();
}

}  // namespace

bool decode_tc_supported(const ScanArgs &a) {
  return (a.V == 64 || a.V == 128) && (a.K == 16 || a.K == 32 || a.K == 64 || a.K == 128);
}

cudaError_t launch_decode_tc_bf16(const ScanArgs &a, cudaStream_t s) {
  return a.V == 64 ? launch_tc<64>(a, s) : launch_tc<128>(a, s);
}

}  // namespace m2rnn

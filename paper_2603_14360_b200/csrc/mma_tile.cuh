// Register-resident 16-row state tile for the bf16 tensor-core path.
//
// A warp owns 16 rows of H (all V columns).  The state x W product of Eq. 1 is issued as
// mma.sync.m16n8k16 (bf16 x bf16 -> fp32): the accumulator fragment of step t has exactly the
// thread<->element map of the A operand of step t+1, so H never leaves registers.
//
// Fragment geometry (g = lane/4, c = lane%4):
//   accumulator tile nt (16 x 8): d[0],d[1] = row g,   MMA cols 8nt+2c, 8nt+2c+1
//                                 d[2],d[3] = row g+8, same cols
//   A tile kt (16 x 16) = accumulator tiles 2kt and 2kt+1 packed to bf16 pairs.
// Rows and columns of the state may be relabelled freely as long as W is relabelled with them,
// so the MMA indices are mapped to memory so that every thread's data is contiguous:
//   MMA row g + 8h      <-> memory row  16*warp + 2g + h
//   MMA col 8nt + 2c + e <-> memory col (V/4)*c + 2nt + e
// i.e. a thread holds two adjacent rows x V/4 adjacent columns.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace m2rnn {

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// d = a * b with a fresh (zero) accumulator
__device__ __forceinline__ void mma_bf16_16816_zero(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

__device__ __forceinline__ float tanh_approx(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// lower 16 bits <- lo, upper 16 bits <- hi (round to nearest even)
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

template <int V>
struct TileGeom {
  static constexpr int NT = V / 8;    // accumulator tiles per warp
  static constexpr int KT = V / 16;   // k tiles of the V x V transition matrix
  static constexpr int SEG = V / 4;   // contiguous memory columns per thread
  // memory column of MMA column m
  __host__ __device__ static constexpr int mem_col(int m) { return SEG * ((m & 7) >> 1) + 2 * (m >> 3) + (m & 1); }
};

// B fragment (kt, nt) of the relabelled W for this lane, read from W in memory (row-major bf16).
template <int V>
__device__ __forceinline__ void load_w_fragment(const __nv_bfloat16 *__restrict__ Wn, int kt, int nt, int lane,
                                                uint32_t &b0, uint32_t &b1) {
  using G = TileGeom<V>;
  const int g = lane >> 2, c = lane & 3;
  const int col = G::mem_col(8 * nt + g);
  const int r0 = G::mem_col(16 * kt + 2 * c), r1 = G::mem_col(16 * kt + 2 * c + 1);
  const int r2 = G::mem_col(16 * kt + 8 + 2 * c), r3 = G::mem_col(16 * kt + 8 + 2 * c + 1);
  const uint16_t *w = reinterpret_cast<const uint16_t *>(Wn);
  b0 = (uint32_t)w[r0 * V + col] | ((uint32_t)w[r1 * V + col] << 16);
  b1 = (uint32_t)w[r2 * V + col] | ((uint32_t)w[r3 * V + col] << 16);
}

// Sum, over the 8 lane groups g of a warp, of per-thread partials p[idx] (idx = 2nt+e, i.e. the
// thread's SEG memory columns in order), by recursive halving: each round a lane keeps one half
// of its values and hands the other half to its partner.  Afterwards lane (g,c) holds
// SEG >> R sums for the memory columns  SEG*c + sel*(SEG>>R) + j,  with R = min(3, log2 SEG)
// and sel = g >> (3 - R).  If R < 3 the remaining lane bits are folded with full exchanges.
template <int NVAL>
__device__ __forceinline__ void reduce_over_rows(float (&p)[NVAL], int lane) {
  if constexpr (NVAL >= 2) {
    constexpr int H = NVAL / 2;
    const bool up = lane & 16;
#pragma unroll
    for (int i = 0; i < H; ++i) {
      const float send = up ? p[i] : p[H + i];
      const float keep = up ? p[H + i] : p[i];
      p[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
  } else {
    p[0] += __shfl_xor_sync(0xffffffffu, p[0], 16);
  }
  if constexpr (NVAL >= 4) {
    constexpr int H = NVAL / 4;
    const bool up = lane & 8;
#pragma unroll
    for (int i = 0; i < H; ++i) {
      const float send = up ? p[i] : p[H + i];
      const float keep = up ? p[H + i] : p[i];
      p[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
  } else {
#pragma unroll
    for (int i = 0; i < (NVAL >= 2 ? NVAL / 2 : 1); ++i) p[i] += __shfl_xor_sync(0xffffffffu, p[i], 8);
  }
  if constexpr (NVAL >= 8) {
    constexpr int H = NVAL / 8;
    const bool up = lane & 4;
#pragma unroll
    for (int i = 0; i < H; ++i) {
      const float send = up ? p[i] : p[H + i];
      const float keep = up ? p[H + i] : p[i];
      p[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
  } else {
#pragma unroll
    for (int i = 0; i < (NVAL >= 4 ? NVAL / 4 : 1); ++i) p[i] += __shfl_xor_sync(0xffffffffu, p[i], 4);
  }
}

// Number of values a lane holds after reduce_over_rows, their first memory column, and whether
// this lane is the one that should store them (duplicates exist when SEG < 8).
template <int V>
struct RowReduceOut {
  static constexpr int SEG = V / 4;
  static constexpr int R = SEG >= 8 ? 3 : (SEG >= 4 ? 2 : 1);
  static constexpr int CNT = SEG >> R;
  __device__ static int first_col(int lane) {
    const int g = lane >> 2, c = lane & 3;
    return SEG * c + (g >> (3 - R)) * CNT;
  }
  __device__ static bool owner(int lane) { return ((lane >> 2) & ((1 << (3 - R)) - 1)) == 0; }
};

}  // namespace m2rnn

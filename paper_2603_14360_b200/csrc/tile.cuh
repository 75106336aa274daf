// bf16 [rows][V] tiles in shared memory that the chain warps write fragment-wise and other warps
// read back as MMA operands with ldmatrix.
#pragma once

#include <stdint.h>

#include "mma_tile.cuh"

namespace m2rnn {

// Byte offset of 16-byte chunk `chunk` of row `row`.  Chunks are XOR-swizzled within 128-byte lines
// so that both the fragment-wise stores (8 rows x 4 lanes per instruction) and the ldmatrix reads
// (8 rows, same column chunk) spread over all banks.
template <int V>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
  constexpr int RB = 2 * V;
  if constexpr (RB >= 128) {
    return (uint32_t)(row * RB + ((chunk ^ (row & 7)) << 4));
  } else {
    const uint32_t lin = (uint32_t)(row * RB + (chunk << 4));
    const uint32_t line = lin >> 7;
    return (line << 7) | ((((lin >> 4) & 7u) ^ (line & 7u)) << 4);
  }
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}

// A warp's 16 x V slab as packed bf16 pairs in accumulator layout: p[nt][h] = (row g + 8h of the
// slab, memory columns SEG*c + 2nt, +1), g = lane/4, c = lane%4, SEG = V/4.  `slab` is the slab's
// index in the tile (rows 16*slab ..).
template <int V>
__device__ __forceinline__ void tile_store(uint32_t tile_sa, int slab, int lane, const uint32_t (&p)[V / 8][2]) {
  constexpr int SEG = V / 4, CPR = SEG * 2 / 16;   // 16-byte chunks per thread-row (0 when V == 16)
  const int g = lane >> 2, c = lane & 3;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = 16 * slab + g + 8 * h;
    if constexpr (CPR == 0) {   // V == 16: 8 bytes per thread-row
      const uint32_t addr = tile_sa + tile_off<V>(row, c >> 1) + 8u * (c & 1);
      asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(addr), "r"(p[0][h]), "r"(p[1][h]) : "memory");
    } else {
#pragma unroll
      for (int x = 0; x < CPR; ++x) {
        const uint32_t addr = tile_sa + tile_off<V>(row, CPR * c + x);
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(p[4 * x][h]), "r"(p[4 * x + 1][h]),
                     "r"(p[4 * x + 2][h]), "r"(p[4 * x + 3][h]) : "memory");
      }
    }
  }
}

template <int V>
__device__ __forceinline__ void tile_load(uint32_t tile_sa, int slab, int lane, uint32_t (&p)[V / 8][2]) {
  constexpr int SEG = V / 4, CPR = SEG * 2 / 16;
  const int g = lane >> 2, c = lane & 3;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = 16 * slab + g + 8 * h;
    if constexpr (CPR == 0) {
      const uint32_t addr = tile_sa + tile_off<V>(row, c >> 1) + 8u * (c & 1);
      asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(p[0][h]), "=r"(p[1][h]) : "r"(addr));
    } else {
#pragma unroll
      for (int x = 0; x < CPR; ++x) {
        const uint32_t addr = tile_sa + tile_off<V>(row, CPR * c + x);
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(p[4 * x][h]), "=r"(p[4 * x + 1][h]), "=r"(p[4 * x + 2][h]), "=r"(p[4 * x + 3][h]) : "r"(addr));
      }
    }
  }
}

}  // namespace m2rnn

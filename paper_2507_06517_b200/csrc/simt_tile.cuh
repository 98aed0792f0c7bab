// 64x64 dot-product tile on CUDA cores (fp32 FMA), used by the fp32 paths of the window-score
// and similarity kernels.  256 threads; thread (ty, tx) = (tid / 16, tid % 16) owns rows
// ty*4..ty*4+3 and columns tx*4..tx*4+3 of the tile.  Operands are staged through shared memory
// in slabs of 32 elements along head_dim, transposed so that the inner loop reads float4s.
#pragma once

#include "common.cuh"

namespace skv {

constexpr int kTile = 64;
constexpr int kSlab = 32;
constexpr int kPad = 68;  // row pitch of a slab in floats (multiple of 4 keeps float4 reads aligned)

struct TileSmem {
  float a[kSlab][kPad];
  float b[kSlab][kPad];
};

// RowA / RowB: callables int -> const T* (row within the tile -> pointer to its head_dim elements,
// or nullptr for a row that does not exist, which then reads as zeros).
template <typename T, int D, typename RowA, typename RowB>
__device__ __forceinline__ void dot_tile_64x64(TileSmem& sm, RowA row_a, RowB row_b, float (&acc)[4][4]) {
  const int tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  const int lrow = tid >> 2, lseg = (tid & 3) * 8;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const T* pa = row_a(lrow);
  const T* pb = row_b(lrow);
  for (int k0 = 0; k0 < D; k0 += kSlab) {
    float va[8], vb[8];
    if (pa) load8(pa + k0 + lseg, va); else {
#pragma unroll
      for (int i = 0; i < 8; ++i) va[i] = 0.f;
    }
    if (pb) load8(pb + k0 + lseg, vb); else {
#pragma unroll
      for (int i = 0; i < 8; ++i) vb[i] = 0.f;
    }
    __syncthreads();  // previous slab fully consumed
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      sm.a[lseg + i][lrow] = va[i];
      sm.b[lseg + i][lrow] = vb[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSlab; ++kk) {
      float4 a4 = *reinterpret_cast<const float4*>(&sm.a[kk][ty * 4]);
      float4 b4 = *reinterpret_cast<const float4*>(&sm.b[kk][tx * 4]);
      float av[4] = {a4.x, a4.y, a4.z, a4.w};
      float bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
  }
}

}  // namespace skv

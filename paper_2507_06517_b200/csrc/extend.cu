// Decode-time merging of new tokens into an existing CodeBook (Section 3.4, last paragraph): every new
// token first looks for a suitable entry, i.e. one whose cosine similarity with it exceeds theta (the
// most similar one, ties to the lower entry number); the tokens that find none are listed so that
// Algorithm 1 can build entries for them, which are then appended.
#include "common.cuh"
#include "simt_tile.cuh"

namespace skv {

struct MatchParams {
  View G, C;              // new tokens, CodeBook rows
  Batch batch;            // describes the new tokens (max_len = most new tokens of a unit)
  int n_heads, c_rows;    // c_rows: row capacity of a unit's CodeBook
  float theta;
  const int32_t* n_entries;    // [layers][B][H]
  unsigned long long* best;    // [layers][H][T] (similarity image << 32) | ~entry, 0: none suitable so far
  float* mag;                  // [layers][H][T]
  int32_t* ref;                // [layers][H][T]
  int32_t* left_idx;           // [layers][H][T]
  int32_t* left_cnt;           // [layers][B][H]
};

__device__ __forceinline__ uint32_t float_order(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// 64 new tokens x 64 entries per block: dot products on CUDA cores, norms of both sides from the rows
// themselves, one atomic maximum per token and tile.
template <typename T, int D>
__global__ void __launch_bounds__(256) match_tile_kernel(MatchParams p) {
  __shared__ TileSmem sm;
  __shared__ float nr[kTile], nc[kTile];
  const int unit = blockIdx.z;
  const int h = unit % p.n_heads;
  const int ls = unit / p.n_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int t_new = seq_len(p.batch, layer, s, h);
  const int n_ent = min(p.n_entries[(layer * p.batch.n_seqs + s) * p.n_heads + h], p.c_rows);
  const int r0 = blockIdx.y * kTile, c0 = blockIdx.x * kTile;
  if (r0 >= t_new) return;
  const T* gbase = reinterpret_cast<const T*>(p.G.ptr) + unit_offset(p.G, p.batch, layer, s, h);
  const T* cbase = reinterpret_cast<const T*>(p.C.ptr) + unit_offset(p.C, p.batch, layer, s, h);
  const int64_t orow = ((int64_t)layer * p.n_heads + h) * p.batch.total_len + tok_base(p.batch, s);
  // norms of the tile's rows and columns: four threads per vector
  {
    const int v = threadIdx.x >> 2, part = threadIdx.x & 3;
#pragma unroll
    for (int side = 0; side < 2; ++side) {
      const int idx = (side ? c0 : r0) + v;
      const bool ok = idx < (side ? n_ent : t_new);
      const T* src = (side ? cbase + (int64_t)idx * p.C.st : gbase + (int64_t)idx * p.G.st) + part * (D / 4);
      float ss = 0.f;
      if (ok) {
#pragma unroll
        for (int k = 0; k < D / 4; k += 8) {
          float x[8];
          load8(src + k, x);
#pragma unroll
          for (int i = 0; i < 8; ++i) ss = fmaf(x[i], x[i], ss);
        }
      }
      ss += __shfl_xor_sync(0xffffffffu, ss, 1);
      ss += __shfl_xor_sync(0xffffffffu, ss, 2);
      if (part == 0) (side ? nc : nr)[v] = sqrtf(ss);
    }
  }
  __syncthreads();
  if (blockIdx.x == 0 && threadIdx.x < kTile && r0 + threadIdx.x < t_new) p.mag[orow + r0 + threadIdx.x] = nr[threadIdx.x];
  if (c0 >= n_ent) return;
  float acc[4][4];
  auto row_a = [&](int r) -> const T* { return r0 + r < t_new ? gbase + (int64_t)(r0 + r) * p.G.st : nullptr; };
  auto row_b = [&](int r) -> const T* { return c0 + r < n_ent ? cbase + (int64_t)(c0 + r) * p.C.st : nullptr; };
  dot_tile_64x64<T, D>(sm, row_a, row_b, acc);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int a = r0 + ty * 4 + i;
    // a zero vector has similarity 0 with everything: magnitude 1 keeps the comparison "0 > theta"
    const float ma = nr[ty * 4 + i] > 0.f ? nr[ty * 4 + i] : 1.f;
    unsigned long long best = 0ull;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int e = c0 + tx * 4 + c;
      const float mc = nc[tx * 4 + c] > 0.f ? nc[tx * 4 + c] : 1.f;
      const float den = ma * mc;
      if (a < t_new && e < n_ent && acc[i][c] > p.theta * den) {
        const unsigned long long key = ((unsigned long long)float_order(acc[i][c] / den) << 32) |
                                       (unsigned long long)(0xFFFFFFFFu - (uint32_t)e);
        best = key > best ? key : best;
      }
    }
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other > best ? other : best;
    }
    if (tx == 0 && best) atomicMax(&p.best[orow + a], best);
  }
}

// One block per unit: entry numbers of the matched tokens, ascending list of the others.
__global__ void __launch_bounds__(1024) match_finish_kernel(MatchParams p) {
  __shared__ int warp_sums[33];
  const int unit = blockIdx.x;
  const int h = unit % p.n_heads;
  const int ls = unit / p.n_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int t_new = seq_len(p.batch, layer, s, h);
  const int64_t orow = ((int64_t)layer * p.n_heads + h) * p.batch.total_len + tok_base(p.batch, s);
  int base = 0;
  for (int t0 = 0; t0 < t_new; t0 += 1024) {
    const int t = t0 + threadIdx.x;
    int left = 0;
    if (t < t_new) {
      const unsigned long long key = p.best[orow + t];
      left = key == 0ull;
      p.ref[orow + t] = left ? -1 : (int32_t)(0xFFFFFFFFu - (uint32_t)(key & 0xFFFFFFFFull));
    }
    int total;
    const int pos = block_exclusive_scan(left, warp_sums, total) + base;
    if (left) p.left_idx[orow + pos] = t;
    base += total;
  }
  if (threadIdx.x == 0) p.left_cnt[(layer * p.batch.n_seqs + s) * p.n_heads + h] = base;
}

size_t match_workspace_bytes(const spindlekv_batch& b, int n_heads) {
  return kHeaderBytes + align_up((size_t)b.n_layers * n_heads * b.total_len * sizeof(unsigned long long), 256);
}

spindlekv_status match_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& G,
                            const spindlekv_tensor& C, const int32_t* n_entries, int c_rows, float theta, float* mag,
                            int32_t* ref, int32_t* left_idx, int32_t* left_cnt, void* ws, size_t ws_bytes, cudaStream_t st) {
  if (ws_bytes < match_workspace_bytes(b, n_heads)) return SPINDLEKV_WORKSPACE_TOO_SMALL;
  const int units = b.n_layers * b.n_seqs * n_heads;
  if (units > 65535) return SPINDLEKV_UNSUPPORTED;
  MatchParams p;
  p.G = make_view(G);
  p.C = make_view(C);
  p.batch = make_batch(b);
  p.n_heads = n_heads;
  p.c_rows = c_rows;
  p.theta = theta;
  p.n_entries = n_entries;
  p.best = reinterpret_cast<unsigned long long*>(reinterpret_cast<char*>(ws) + kHeaderBytes);
  p.mag = mag;
  p.ref = ref;
  p.left_idx = left_idx;
  p.left_cnt = left_cnt;
  if (cudaMemsetAsync(ws, 0, match_workspace_bytes(b, n_heads), st) != cudaSuccess) return SPINDLEKV_CUDA;
  dim3 grid(ceil_div(c_rows, kTile), ceil_div(b.max_len, kTile), units);
  const bool bf = G.dtype == SPINDLEKV_BF16;
  {
    LaunchScope ls(KC_SIM, st);
    if (head_dim == 64) {
      if (bf) match_tile_kernel<__nv_bfloat16, 64><<<grid, 256, 0, st>>>(p); else match_tile_kernel<float, 64><<<grid, 256, 0, st>>>(p);
    } else {
      if (bf) match_tile_kernel<__nv_bfloat16, 128><<<grid, 256, 0, st>>>(p); else match_tile_kernel<float, 128><<<grid, 256, 0, st>>>(p);
    }
  }
  {
    LaunchScope ls(KC_FINAL, st);
    match_finish_kernel<<<units, 1024, 0, st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

// ---- appending the entries built for the unmatched tokens ------------------------------------------
struct AppendParams {
  View L, C;              // rows of the unmatched tokens (gathered), CodeBook rows
  Batch batch;            // describes the new tokens
  int n_heads, c_rows;
  const float* mag_left;          // [layers][H][T] magnitudes of the gathered rows
  const int32_t* ref_left;        // [layers][H][T] entry (among the new ones) of each gathered row
  const int32_t* centre_left;     // [layers][H][T] gathered-row number of each new entry
  const int32_t* n_left_entries;  // [layers][B][H]
  const int32_t* left_idx;        // [layers][H][T]
  const int32_t* left_cnt;        // [layers][B][H]
  int32_t* n_entries;             // [layers][B][H] in: entries before, out: entries after
  int32_t* ref_new;               // [layers][H][T]
};

template <typename T, int D>
__global__ void __launch_bounds__(256) append_kernel(AppendParams p) {
  constexpr int EPT = 16 / sizeof(T);
  constexpr int TPR = D / EPT;
  constexpr int RPB = 256 / TPR;
  const int unit = blockIdx.x;
  const int h = unit % p.n_heads;
  const int ls = unit / p.n_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int cu = (layer * p.batch.n_seqs + s) * p.n_heads + h;
  const int n_old = p.n_entries[cu], n_add = p.n_left_entries[cu], n_left = p.left_cnt[cu];
  const int64_t orow = ((int64_t)layer * p.n_heads + h) * p.batch.total_len + tok_base(p.batch, s);
  for (int q = threadIdx.x; q < n_left; q += 256) p.ref_new[orow + p.left_idx[orow + q]] = n_old + p.ref_left[orow + q];
  const T* lbase = reinterpret_cast<const T*>(p.L.ptr) + unit_offset(p.L, p.batch, layer, s, h);
  T* cbase = reinterpret_cast<T*>(const_cast<void*>(p.C.ptr)) + unit_offset(p.C, p.batch, layer, s, h);
  const int seg = threadIdx.x % TPR;
  for (int e = threadIdx.x / TPR; e < n_add && n_old + e < p.c_rows; e += RPB) {
    const int a = p.centre_left[orow + e];
    const float m = p.mag_left[orow + a];
    uint4 v = *reinterpret_cast<const uint4*>(lbase + (int64_t)a * p.L.st + seg * EPT);
    if (sizeof(T) == 4) {
      float* f = reinterpret_cast<float*>(&v);
#pragma unroll
      for (int i = 0; i < 4; ++i) f[i] = m > 0.f ? f[i] / m : 0.f;
    } else {
      uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xFFFF0000u);
        lo = m > 0.f ? lo / m : 0.f;
        hi = m > 0.f ? hi / m : 0.f;
        __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
        w[i] = *reinterpret_cast<uint32_t*>(&pk);
      }
    }
    *reinterpret_cast<uint4*>(cbase + (int64_t)(n_old + e) * p.C.st + seg * EPT) = v;
  }
  __syncthreads();
  if (threadIdx.x == 0) p.n_entries[cu] = n_old + n_add;
}

spindlekv_status append_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& Lt,
                             const float* mag_left, const int32_t* ref_left, const int32_t* centre_left,
                             const int32_t* n_left_entries, const int32_t* left_idx, const int32_t* left_cnt,
                             const spindlekv_tensor& C, int c_rows, int32_t* n_entries, int32_t* ref_new, cudaStream_t st) {
  AppendParams p;
  p.L = make_view(Lt);
  p.C = make_view(C);
  p.batch = make_batch(b);
  p.n_heads = n_heads;
  p.c_rows = c_rows;
  p.mag_left = mag_left;
  p.ref_left = ref_left;
  p.centre_left = centre_left;
  p.n_left_entries = n_left_entries;
  p.left_idx = left_idx;
  p.left_cnt = left_cnt;
  p.n_entries = n_entries;
  p.ref_new = ref_new;
  const int units = b.n_layers * b.n_seqs * n_heads;
  LaunchScope ls(KC_GATHER, st);
  const bool bf = C.dtype == SPINDLEKV_BF16;
  if (head_dim == 64) {
    if (bf) append_kernel<__nv_bfloat16, 64><<<units, 256, 0, st>>>(p); else append_kernel<float, 64><<<units, 256, 0, st>>>(p);
  } else {
    if (bf) append_kernel<__nv_bfloat16, 128><<<units, 256, 0, st>>>(p); else append_kernel<float, 128><<<units, 256, 0, st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

// Gather of kept tokens / CodeBook centres into the output cache (Eq. (7) second line, Eq. (11)):
// 16-byte loads and stores, one row per group of head_dim*elem/16 threads, eight rows of every group in
// flight, rows of a unit contiguous in the destination.
#include "common.cuh"

namespace skv {

struct CompactParams {
  View src, dst;
  Batch batch;
  int n_heads;
  const int32_t* idx;     // [layers][H][T]
  const int32_t* cnt;     // [layers][B][H]
  const float* divide_by; // optional [layers][H][T]
  const int32_t* dst_cu;  // optional [B+1]
};

constexpr int kGatherRows = 8;   // rows per thread group, all of their loads in flight before any is used

template <typename T, int D>
__global__ void __launch_bounds__(256) compact_kernel(CompactParams p) {
  constexpr int EPT = 16 / sizeof(T);       // elements per thread
  constexpr int TPR = D / EPT;              // threads per row
  constexpr int RPB = 256 / TPR;            // rows per sweep of the block
  const int unit = blockIdx.y;
  const int h = unit % p.n_heads;
  const int ls = unit / p.n_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int n = p.cnt[(layer * p.batch.n_seqs + s) * p.n_heads + h];
  const int64_t orow = ((int64_t)layer * p.n_heads + h) * p.batch.total_len + tok_base(p.batch, s);
  const T* sbase = reinterpret_cast<const T*>(p.src.ptr) + unit_offset(p.src, p.batch, layer, s, h);
  T* dbase = reinterpret_cast<T*>(const_cast<void*>(p.dst.ptr)) + (int64_t)layer * p.dst.sl + (int64_t)h * p.dst.sh;
  if (p.dst_cu) dbase += (int64_t)p.dst_cu[s] * p.dst.st;
  else if (p.batch.cu) dbase += (int64_t)p.batch.cu[s] * p.dst.st;
  else dbase += (int64_t)s * p.dst.ss;
  const int seg = threadIdx.x % TPR;
  // a block owns kGatherRows * RPB consecutive output rows
  for (int r0 = blockIdx.x * (RPB * kGatherRows) + threadIdx.x / TPR; r0 < n; r0 += gridDim.x * (RPB * kGatherRows)) {
    int a[kGatherRows];
    uint4 v[kGatherRows];
    float rc[kGatherRows];
#pragma unroll
    for (int i = 0; i < kGatherRows; ++i) {
      const int r = r0 + i * RPB;
      a[i] = r < n ? p.idx[orow + r] : -1;
    }
#pragma unroll
    for (int i = 0; i < kGatherRows; ++i) {
      if (a[i] < 0) continue;
      v[i] = *reinterpret_cast<const uint4*>(sbase + (int64_t)a[i] * p.src.st + seg * EPT);
      if (p.divide_by) rc[i] = p.divide_by[orow + a[i]];
    }
#pragma unroll
    for (int i = 0; i < kGatherRows; ++i) {
      if (a[i] < 0) continue;
      if (p.divide_by) {
        // one correctly rounded reciprocal per row, then a product per element; a zero row stays zero
        const float m = rc[i] > 0.f ? __frcp_rn(rc[i]) : 0.f;
        if (sizeof(T) == 4) {
          float* f = reinterpret_cast<float*>(&v[i]);
#pragma unroll
          for (int q = 0; q < 4; ++q) f[q] *= m;
        } else {
          uint32_t* w = reinterpret_cast<uint32_t*>(&v[i]);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float lo = __uint_as_float(w[q] << 16), hi = __uint_as_float(w[q] & 0xFFFF0000u);
            __nv_bfloat162 pk = __floats2bfloat162_rn(lo * m, hi * m);
            w[q] = *reinterpret_cast<uint32_t*>(&pk);
          }
        }
      }
      *reinterpret_cast<uint4*>(dbase + (int64_t)(r0 + i * RPB) * p.dst.st + seg * EPT) = v[i];
    }
  }
}

// ---- Eq. (14): Gamma_r = C[r] (x) m --------------------------------------------------------------
// One group of head_dim*elem/16 threads per token: reads the token's entry row, scales it by the
// token's magnitude in fp32, writes the row.
struct ReconstructParams {
  View C, dst;
  Batch batch;
  int n_heads;
  const int32_t* ref;   // [layers][H][T]
  const float* mag;     // [layers][H][T]
};

template <typename T, int D>
__global__ void __launch_bounds__(256) reconstruct_kernel(ReconstructParams p) {
  constexpr int EPT = 16 / sizeof(T);
  constexpr int TPR = D / EPT;
  constexpr int RPB = 256 / TPR;
  const int unit = blockIdx.y;
  const int h = unit % p.n_heads;
  const int ls = unit / p.n_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int l = seq_len(p.batch, layer, s, h);
  const int64_t orow = ((int64_t)layer * p.n_heads + h) * p.batch.total_len + tok_base(p.batch, s);
  const T* cbase = reinterpret_cast<const T*>(p.C.ptr) + unit_offset(p.C, p.batch, layer, s, h);
  T* dbase = reinterpret_cast<T*>(const_cast<void*>(p.dst.ptr)) + unit_offset(p.dst, p.batch, layer, s, h);
  const int seg = threadIdx.x % TPR;
  for (int t = blockIdx.x * RPB + threadIdx.x / TPR; t < l; t += gridDim.x * RPB) {
    const int r = p.ref[orow + t];
    const float m = p.mag[orow + t];
    uint4 v = *reinterpret_cast<const uint4*>(cbase + (int64_t)r * p.C.st + seg * EPT);
    if (sizeof(T) == 4) {
      float* f = reinterpret_cast<float*>(&v);
#pragma unroll
      for (int i = 0; i < 4; ++i) f[i] *= m;
    } else {
      uint32_t* w = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float lo = __uint_as_float(w[i] << 16) * m, hi = __uint_as_float(w[i] & 0xFFFF0000u) * m;
        __nv_bfloat162 pk = __floats2bfloat162_rn(lo, hi);
        w[i] = *reinterpret_cast<uint32_t*>(&pk);
      }
    }
    *reinterpret_cast<uint4*>(dbase + (int64_t)t * p.dst.st + seg * EPT) = v;
  }
}

spindlekv_status reconstruct_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& C,
                                  const int32_t* ref, const float* mag, const spindlekv_tensor& dst, cudaStream_t st) {
  ReconstructParams p;
  p.C = make_view(C);
  p.dst = make_view(dst);
  p.batch = make_batch(b);
  p.n_heads = n_heads;
  p.ref = ref;
  p.mag = mag;
  const int units = b.n_layers * b.n_seqs * n_heads;
  if (units > 65535) return SPINDLEKV_UNSUPPORTED;
  dim3 grid(ceil_div(b.max_len, 64), units);
  LaunchScope ls(KC_GATHER, st);
  const bool bf = C.dtype == SPINDLEKV_BF16;
  if (head_dim == 64) {
    if (bf) reconstruct_kernel<__nv_bfloat16, 64><<<grid, 256, 0, st>>>(p); else reconstruct_kernel<float, 64><<<grid, 256, 0, st>>>(p);
  } else {
    if (bf) reconstruct_kernel<__nv_bfloat16, 128><<<grid, 256, 0, st>>>(p); else reconstruct_kernel<float, 128><<<grid, 256, 0, st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

// ---- lists of several passes over the same heads, one after the other ------------------------------
// GQA "repeat": every query head of a group selects tokens of the group's KV head on its own; the
// CodeBook of the KV head is then built from all of them.  out list of (layer, seq, head) = list of
// pass 0, then pass 1, ...; its count is the sum of the counts.
struct UnionParams {
  int n_layers, n_seqs, n_heads, n_lists;
  int lists_inner;             // 0: idx_in [n_lists][layers][H][t_in]; 1: [layers][H][n_lists][t_in] (cnt alike)
  int t_in, t_out;             // row length of one (layer, head) in idx_in / idx_out
  int seq_in, seq_out;         // start of sequence s within a row: s * seq_in, s * seq_out
  const int32_t* idx_in;       // [n_lists][layers][H][t_in]
  const int32_t* cnt_in;       // [n_lists][layers][B][H]
  int32_t* idx_out;            // [layers][H][t_out]
  int32_t* cnt_out;            // [layers][B][H]
};

__global__ void __launch_bounds__(256) union_lists_kernel(UnionParams p) {
  const int unit = blockIdx.x;
  const int h = unit % p.n_heads;
  const int ls = unit / p.n_heads;
  const int s = ls % p.n_seqs;
  const int layer = ls / p.n_seqs;
  const int64_t per_list_idx = (int64_t)p.n_layers * p.n_heads * p.t_in;
  const int64_t per_list_cnt = (int64_t)p.n_layers * p.n_seqs * p.n_heads;
  const int64_t in_row = ((int64_t)layer * p.n_heads + h) * p.t_in + (int64_t)s * p.seq_in;
  const int64_t out_row = ((int64_t)layer * p.n_heads + h) * p.t_out + (int64_t)s * p.seq_out;
  const int64_t cnt_at = ((int64_t)layer * p.n_seqs + s) * p.n_heads + h;
  int base = 0;
  for (int g = 0; g < p.n_lists; ++g) {
    const int n = p.lists_inner ? p.cnt_in[cnt_at * p.n_lists + g] : p.cnt_in[g * per_list_cnt + cnt_at];
    const int32_t* src = p.lists_inner
        ? p.idx_in + (((int64_t)layer * p.n_heads + h) * p.n_lists + g) * p.t_in + (int64_t)s * p.seq_in
        : p.idx_in + g * per_list_idx + in_row;
    for (int r = threadIdx.x; r < n && base + r < p.seq_out; r += blockDim.x) p.idx_out[out_row + base + r] = src[r];
    base += n;
  }
  if (threadIdx.x == 0) p.cnt_out[cnt_at] = min(base, p.seq_out);
}

spindlekv_status union_lists_impl(int n_layers, int n_seqs, int n_heads, int n_lists, int lists_inner, int t_in, int seq_in,
                                  const int32_t* idx_in, const int32_t* cnt_in, int t_out, int seq_out,
                                  int32_t* idx_out, int32_t* cnt_out, cudaStream_t st) {
  UnionParams p{n_layers, n_seqs, n_heads, n_lists, lists_inner, t_in, t_out, seq_in, seq_out, idx_in, cnt_in, idx_out, cnt_out};
  LaunchScope ls(KC_GATHER, st);
  union_lists_kernel<<<n_layers * n_seqs * n_heads, 256, 0, st>>>(p);
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

spindlekv_status compact_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& src,
                              const int32_t* idx, const int32_t* cnt, const float* divide_by,
                              const spindlekv_tensor& dst, const int32_t* dst_cu, cudaStream_t st) {
  CompactParams p;
  p.src = make_view(src);
  p.dst = make_view(dst);
  p.batch = make_batch(b);
  p.n_heads = n_heads;
  p.idx = idx;
  p.cnt = cnt;
  p.divide_by = divide_by;
  p.dst_cu = dst_cu;
  const int units = b.n_layers * b.n_seqs * n_heads;
  if (units > 65535) return SPINDLEKV_UNSUPPORTED;
  // enough blocks along x to cover the longest possible row list in one sweep (128 rows per block at 16 threads per row)
  const int gx = ceil_div(b.max_len, 16 * kGatherRows);
  dim3 grid(gx, units);
  LaunchScope ls(KC_GATHER, st);
  const bool bf = src.dtype == SPINDLEKV_BF16;
  if (head_dim == 64) {
    if (bf) compact_kernel<__nv_bfloat16, 64><<<grid, 256, 0, st>>>(p); else compact_kernel<float, 64><<<grid, 256, 0, st>>>(p);
  } else {
    if (bf) compact_kernel<__nv_bfloat16, 128><<<grid, 256, 0, st>>>(p); else compact_kernel<float, 128><<<grid, 256, 0, st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

// Deep-layer eviction: window scores (Eq. (1)(2)(3)) and per-head top-k (Eq. (7)).
//
// Window scores are computed in two passes over the keys because the column sums of Eq. (2)
// need each window row's final softmax maximum and denominator:
//   pass A  per (unit, key tile): partial row max and row sum of exp;   combine -> (max, 1/sum)
//   pass B  per (unit, key tile): recompute the logits, form the probabilities, sum each key column
//           over all h_n * l_w rows of the group, divide by h_n (Eq. (3)) and by (l - a) (Eq. (2)).
// A unit is one (layer, sequence, KV head); its rows are r = g * l_w + t for query head h_n*j+g and
// window query t (position b = l_c + t).  All reductions run in a fixed order: results are
// bit-reproducible from run to run.
#include <math_constants.h>

#include "common.cuh"
#include "simt_tile.cuh"

namespace skv {

struct EvictParams {
  View K, Q;
  Batch batch;
  int n_q_heads, n_kv_heads, window, h_n;   // n_kv_heads: heads that get a score row; h_n: query heads summed into one
  int kv_div;           // head j reads KV head j / kv_div (1, or h_n when every query head has its own row)
  int n_tiles;          // key tiles per unit = ceil(max_len / 64)
  int score_norm;
  float scale;          // 1 / sqrt(d_h)
  float2* part;         // [units][M][n_tiles] partial (max, sum)
  float2* rowstat;      // [units][M] (max, 1/sum)
  float* scores;        // [layers][H_kv][T]
};

__device__ __forceinline__ void decode_unit(const EvictParams& p, int unit, int& layer, int& s, int& j) {
  j = unit % p.n_kv_heads;
  int ls = unit / p.n_kv_heads;
  s = ls % p.batch.n_seqs;
  layer = ls / p.batch.n_seqs;
}

// logits of a 64(rows) x 64(keys) tile, masked entries marked by `valid`
template <typename T, int D>
__device__ __forceinline__ void logits_tile(const EvictParams& p, TileSmem& sm, int layer, int s, int j, int l,
                                            int row0, int key0, float (&acc)[4][4]) {
  const T* kbase = reinterpret_cast<const T*>(p.K.ptr) + unit_offset(p.K, p.batch, layer, s, j / p.kv_div);
  const T* qbase = reinterpret_cast<const T*>(p.Q.ptr) + (int64_t)layer * p.Q.sl + (int64_t)s * p.Q.ss;
  const int M = p.h_n * p.window;
  auto row_q = [&](int r) -> const T* {
    int row = row0 + r;
    if (row >= M) return nullptr;
    int g = row / p.window, t = row - g * p.window;
    return qbase + (int64_t)(p.h_n * j + g) * p.Q.sh + (int64_t)t * p.Q.st;
  };
  auto row_k = [&](int r) -> const T* {
    int a = key0 + r;
    return a < l ? kbase + (int64_t)a * p.K.st : nullptr;
  };
  dot_tile_64x64<T, D>(sm, row_q, row_k, acc);
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[i][c] *= p.scale;
}

template <typename T, int D>
__global__ void __launch_bounds__(256) win_stats_kernel(EvictParams p) {
  __shared__ TileSmem sm;
  int layer, s, j;
  decode_unit(p, blockIdx.y, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int key0 = blockIdx.x * kTile;
  if (key0 >= l) return;
  const int l_c = l - p.window;
  const int M = p.h_n * p.window;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  for (int row0 = 0; row0 < M; row0 += kTile) {
    float acc[4][4];
    logits_tile<T, D>(p, sm, layer, s, j, l, row0, key0, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int row = row0 + ty * 4 + i;
      int b = l_c + (row % p.window);
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int a = key0 + tx * 4 + c;
        if (a <= b && a < l) mx = fmaxf(mx, acc[i][c]);
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int a = key0 + tx * 4 + c;
        if (a <= b && a < l) sum += expf(acc[i][c] - mx);
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (tx == 0 && row < M) p.part[((int64_t)blockIdx.y * M + row) * p.n_tiles + blockIdx.x] = make_float2(mx, sum);
    }
  }
}

// one warp per (unit, row): merge the per-tile partials
__global__ void win_combine_kernel(EvictParams p, int n_units) {
  const int M = p.h_n * p.window;
  int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  if (gw >= n_units * M) return;
  int unit = gw / M;
  int layer, s, j;
  decode_unit(p, unit, layer, s, j);
  int nt = (seq_len(p.batch, layer, s, j) + kTile - 1) / kTile;
  const float2* src = p.part + (int64_t)gw * p.n_tiles;
  float mx = -CUDART_INF_F;
  for (int t = lane; t < nt; t += 32) mx = fmaxf(mx, src[t].x);
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int t = lane; t < nt; t += 32) {
    float2 v = src[t];
    if (v.y > 0.f) sum += v.y * expf(v.x - mx);
  }
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) p.rowstat[gw] = make_float2(mx, 1.0f / sum);
}

template <typename T, int D>
__global__ void __launch_bounds__(256) win_colsum_kernel(EvictParams p) {
  __shared__ TileSmem sm;
  __shared__ float colred[16][kTile];
  int layer, s, j;
  decode_unit(p, blockIdx.y, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int l_c = l - p.window;
  const int key0 = blockIdx.x * kTile;
  if (key0 >= l_c) return;  // only context columns are scored
  const int M = p.h_n * p.window;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  float col[4] = {0.f, 0.f, 0.f, 0.f};
  for (int row0 = 0; row0 < M; row0 += kTile) {
    float acc[4][4];
    logits_tile<T, D>(p, sm, layer, s, j, l, row0, key0, acc);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int row = row0 + ty * 4 + i;
      if (row >= M) continue;
      float2 st = p.rowstat[(int64_t)blockIdx.y * M + row];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int a = key0 + tx * 4 + c;
        if (a < l_c) col[c] += expf(acc[i][c] - st.x) * st.y;  // context keys are visible to every window query
      }
    }
  }
#pragma unroll
  for (int c = 0; c < 4; ++c) colred[ty][tx * 4 + c] = col[c];
  __syncthreads();
  if (threadIdx.x < kTile) {
    int a = key0 + threadIdx.x;
    if (a < l_c) {
      float sum = 0.f;
#pragma unroll
      for (int r = 0; r < 16; ++r) sum += colred[r][threadIdx.x];
      float v = sum / (float)p.h_n;
      if (p.score_norm == 0) v = v / (float)(l - a);
      p.scores[((int64_t)layer * p.n_kv_heads + j) * p.batch.total_len + tok_base(p.batch, s) + a] = v;
    }
  }
}

// ---- top-k ------------------------------------------------------------------------------------
// One block per unit.  Radix select (4 passes of 8 bits, most significant first) finds the k-th
// largest key; then one ordered sweep writes, in ascending position, every score above the
// threshold plus the first `need` scores equal to it, which is the lower-index tie-break.

struct TopkParams {
  Batch batch;
  int n_kv_heads, window;
  const float* scores;   // [layers][H_kv][T]
  const int32_t* k_ctx;  // [layers][B]
  int32_t* keep_idx;     // [layers][H_kv][T]
  int32_t* keep_cnt;     // [layers][B][H_kv]
};

__device__ __forceinline__ uint32_t order_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kTopkThreads = 1024;
constexpr int kTopkItems = 16;                                // scores per thread loaded together
constexpr int kTopkChunk = kTopkThreads * kTopkItems;         // scores per sweep of the block

// One block per unit.  Four 8-bit radix passes find the k-th largest key and how many of its equals are
// taken; one ordered pass writes the kept positions in ascending order (ties to the lower position).
// A thread loads its kTopkItems scores of a sweep (positions `i * kTopkThreads + tid`) before using any.
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(TopkParams p) {
  __shared__ int hist[256];
  __shared__ int warp_sums[33];
  __shared__ int cnt_gt[kTopkItems * 32], cnt_eq[kTopkItems * 32];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_need;
  const int unit = blockIdx.x;
  const int j = unit % p.n_kv_heads;
  const int ls = unit / p.n_kv_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int l = seq_len(p.batch, layer, s, j);
  const int l_c = l - p.window;
  int k = p.k_ctx[layer * p.batch.n_seqs + s];
  k = max(0, min(k, l_c));
  const int64_t row = ((int64_t)layer * p.n_kv_heads + j) * p.batch.total_len + tok_base(p.batch, s);
  const float* sc = p.scores + row;
  int32_t* out = p.keep_idx + row;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  uint32_t prefix = 0, mask = 0;
  int need = k;
  if (k > 0 && k < l_c) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      for (int a0 = 0; a0 < l_c; a0 += kTopkChunk) {
        uint32_t key[kTopkItems];
#pragma unroll
        for (int i = 0; i < kTopkItems; ++i) {
          const int a = a0 + i * kTopkThreads + tid;
          key[i] = a < l_c ? order_key(sc[a]) : 0u;
        }
#pragma unroll
        for (int i = 0; i < kTopkItems; ++i) {
          const int a = a0 + i * kTopkThreads + tid;
          const bool part = a < l_c && (key[i] & mask) == prefix;
          const int bin = (key[i] >> shift) & 255;
          if (shift == 24) {
            // the leading byte (sign and exponent) takes few values: one atomic per value and warp
            const uint32_t peers = __match_any_sync(0xffffffffu, part ? bin : 256);
            if (part && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
          } else if (part) {
            atomicAdd(&hist[bin], 1);
          }
        }
      }
      __syncthreads();
      if (wid == 0) {
        // the bin that holds the `need`-th largest: lane t owns bins 8t .. 8t+7
        int h[8], mine = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          h[i] = hist[lane * 8 + i];
          mine += h[i];
        }
        int incl = mine;   // sum over lanes >= this one
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int n = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += n;
        }
        int above = incl - mine;
        // the highest lane whose inclusive sum reaches `need` holds the bin; none does only if fewer than
        // `need` keys carry the prefix, which the previous pass excludes; bin 0 is the guard
        const uint32_t reach = __ballot_sync(0xffffffffu, incl >= need);
        const int owner = reach ? 31 - __clz(reach) : 0;
        if (lane == owner) {
          int bin = 7;
          for (; bin > 0; --bin) {
            if (above + h[bin] >= need) break;
            above += h[bin];
          }
          sh_prefix = prefix | ((uint32_t)(lane * 8 + bin) << shift);
          sh_need = need - above;
        }
      }
      __syncthreads();
      prefix = sh_prefix;
      need = sh_need;
      mask |= 0xFFu << shift;
    }
  }
  // ordered pass: counts of every (sweep, warp) by ballot, one block scan over them per kTopkChunk positions
  int base_gt = 0, base_eq = 0;
  for (int a0 = 0; a0 < l_c; a0 += kTopkChunk) {
    uint32_t key[kTopkItems], bg[kTopkItems], be[kTopkItems];
#pragma unroll
    for (int i = 0; i < kTopkItems; ++i) {
      const int a = a0 + i * kTopkThreads + tid;
      key[i] = (a < l_c && k > 0 && k < l_c) ? order_key(sc[a]) : 0u;
    }
#pragma unroll
    for (int i = 0; i < kTopkItems; ++i) {
      const int a = a0 + i * kTopkThreads + tid;
      const bool in = a < l_c;
      bool gt = false, eq = false;
      if (in) {
        if (k >= l_c) gt = true;
        else if (k > 0) {
          gt = key[i] > prefix;
          eq = key[i] == prefix;
        }
      }
      bg[i] = __ballot_sync(0xffffffffu, gt);
      be[i] = __ballot_sync(0xffffffffu, eq);
      if (lane == 0) {
        cnt_gt[i * 32 + wid] = __popc(bg[i]);
        cnt_eq[i * 32 + wid] = __popc(be[i]);
      }
    }
    __syncthreads();
    int tot_gt, tot_eq;
    {
      const bool has = tid < kTopkItems * 32;
      const int vg = has ? cnt_gt[tid] : 0, ve = has ? cnt_eq[tid] : 0;
      const int eg = block_exclusive_scan(vg, warp_sums, tot_gt);
      const int ee = block_exclusive_scan(ve, warp_sums, tot_eq);
      if (has) {
        cnt_gt[tid] = eg;
        cnt_eq[tid] = ee;
      }
      __syncthreads();
    }
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll
    for (int i = 0; i < kTopkItems; ++i) {
      const int a = a0 + i * kTopkThreads + tid;
      const bool gt = (bg[i] >> lane) & 1u, eq = (be[i] >> lane) & 1u;
      if (!gt && !eq) continue;
      // kept before this position: every larger key, and the first `need` of the equal ones
      const int gt_before = base_gt + cnt_gt[i * 32 + wid] + __popc(bg[i] & below);
      const int eq_before = base_eq + cnt_eq[i * 32 + wid] + __popc(be[i] & below);
      if (gt || eq_before < need) out[gt_before + min(eq_before, need)] = a;
    }
    base_gt += tot_gt;
    base_eq += tot_eq;
    __syncthreads();
  }
  for (int t = tid; t < p.window; t += kTopkThreads) out[k + t] = l_c + t;
  if (tid == 0) p.keep_cnt[(layer * p.batch.n_seqs + s) * p.n_kv_heads + j] = k + p.window;
}

// ---- host side ----------------------------------------------------------------------------------

size_t evict_workspace_bytes(const spindlekv_config& cfg, const spindlekv_batch& b) {
  size_t units = (size_t)b.n_layers * b.n_seqs * cfg.n_kv_heads;
  size_t M = (size_t)(cfg.n_q_heads / cfg.n_kv_heads) * cfg.window;
  size_t nt = ceil_div(b.max_len, kTile);
  return kHeaderBytes + align_up(units * M * nt * sizeof(float2), 256) + align_up(units * M * sizeof(float2), 256);
}

bool win_tc_supported(const spindlekv_config& cfg, int dtype);

// Scratch the call really uses: the tensor-core window-score kernel keeps its row statistics on chip and
// needs the status block only; the CUDA-core kernels keep per-tile row statistics in the workspace.
size_t evict_scratch_needed(const spindlekv_config& cfg, const spindlekv_batch& b, int dtype) {
  return win_tc_supported(cfg, dtype) ? (size_t)kHeaderBytes : evict_workspace_bytes(cfg, b);
}

template <typename T, int D>
static void launch_window(const EvictParams& p, int units, cudaStream_t st) {
  dim3 grid(p.n_tiles, units);
  { LaunchScope ls(KC_WINDOW, st); win_stats_kernel<T, D><<<grid, 256, 0, st>>>(p); }
  int rows = units * p.h_n * p.window;
  { LaunchScope ls(KC_WINDOW, st); win_combine_kernel<<<ceil_div(rows * 32, 256), 256, 0, st>>>(p, units); }
  { LaunchScope ls(KC_WINDOW, st); win_colsum_kernel<T, D><<<grid, 256, 0, st>>>(p); }
}

spindlekv_status launch_win_tc(const spindlekv_config& cfg, const spindlekv_batch& b, const spindlekv_tensor& K,
                               const spindlekv_tensor& Q, float* scores, uint32_t* hdr, cudaStream_t st);

spindlekv_status evict_deep_impl(const spindlekv_config& cfg, const spindlekv_batch& b, const spindlekv_tensor& K,
                                 const spindlekv_tensor& Q, const int32_t* k_ctx, int32_t* keep_idx,
                                 int32_t* keep_cnt, float* scores, void* ws, size_t ws_bytes, cudaStream_t st) {
  if (ws_bytes < evict_scratch_needed(cfg, b, K.dtype)) return SPINDLEKV_WORKSPACE_TOO_SMALL;
  // per_query_head: every query head is a unit of its own (one head per "group") that reads its group's KV head
  const bool per_head = cfg.per_query_head != 0;
  const int out_heads = per_head ? cfg.n_q_heads : cfg.n_kv_heads;
  const int units = b.n_layers * b.n_seqs * out_heads;
  const int h_n = per_head ? 1 : cfg.n_q_heads / cfg.n_kv_heads;
  const size_t M = (size_t)h_n * cfg.window;
  EvictParams p;
  p.K = make_view(K);
  p.Q = make_view(Q);
  p.batch = make_batch(b);
  p.n_q_heads = cfg.n_q_heads;
  p.n_kv_heads = out_heads;
  p.window = cfg.window;
  p.h_n = h_n;
  p.kv_div = per_head ? cfg.n_q_heads / cfg.n_kv_heads : 1;
  p.n_tiles = ceil_div(b.max_len, kTile);
  p.score_norm = cfg.score_norm;
  p.scale = 1.0f / sqrtf((float)cfg.head_dim);
  char* w = reinterpret_cast<char*>(ws);
  if (cudaMemsetAsync(w, 0, kHeaderBytes, st) != cudaSuccess) return SPINDLEKV_CUDA;
  p.part = reinterpret_cast<float2*>(w + kHeaderBytes);
  p.rowstat = reinterpret_cast<float2*>(w + kHeaderBytes + align_up((size_t)units * M * p.n_tiles * sizeof(float2), 256));
  p.scores = scores;
  const bool bf = K.dtype == SPINDLEKV_BF16;
  if (win_tc_supported(cfg, K.dtype)) {
    // bf16 with a window that tiles 128 rows: both passes on the tensor cores, one launch
    spindlekv_status rs = launch_win_tc(cfg, b, K, Q, scores, reinterpret_cast<uint32_t*>(w), st);
    if (rs != SPINDLEKV_OK) return rs;
  } else if (cfg.head_dim == 64) {
    if (bf) launch_window<__nv_bfloat16, 64>(p, units, st); else launch_window<float, 64>(p, units, st);
  } else {
    if (bf) launch_window<__nv_bfloat16, 128>(p, units, st); else launch_window<float, 128>(p, units, st);
  }
  TopkParams t;
  t.batch = p.batch;
  t.n_kv_heads = out_heads;
  t.window = cfg.window;
  t.scores = scores;
  t.k_ctx = k_ctx;
  t.keep_idx = keep_idx;
  t.keep_cnt = keep_cnt;
  { LaunchScope ls(KC_TOPK, st); topk_kernel<<<units, kTopkThreads, 0, st>>>(t); }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

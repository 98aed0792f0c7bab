// Decode-time attention over the replaced cache (Section 3.4 after Eq. (14)): the new token's queries
// attend to K = C_K[r_K] (x) m_K and V = C_V[r_V] (x) m_V without the rebuilt rows ever being written to
// memory.  The CodeBooks hold pre-RoPE keys, so every rebuilt key is rotated at its token's original
// position on the fly (rotary embedding of Eq. (1): element i paired with element i + d/2, angle
// position * base^(-2i/d)), with cosines and sines taken from a table the caller prepares once.
//
// One unit is (layer, sequence, KV head); the h_n query heads of its GQA group are served together, so a
// key is rebuilt and rotated once for all of them.  A unit's tokens are split into chunks of kDecChunk;
// one block per (chunk, unit):
//   1. scores: 16 threads per token gather the token's CodeBook row (16-byte pieces), scale it by the
//      token's magnitude, rotate it, and form the dot products with the rotated queries (kept in shared
//      memory); the 16 partial sums meet through shuffles.  Scores of the chunk stay in shared memory.
//   2. the chunk's maximum and exp-sum per query head (fixed-order block reductions);
//   3. values: every thread owns one pair of output elements for all query heads and a share of the chunk's
//      tokens, adding weight * magnitude * CodeBook row; the row pieces of a token are read by consecutive
//      threads, once for the whole group; the shares are then added up in a fixed order.
// A second kernel merges the chunks of a unit (log-sum-exp weights) in chunk order.  All sums run in a
// fixed order: the result is bit-reproducible from run to run.
#include <math_constants.h>

#include "common.cuh"

namespace skv {

constexpr int kDecChunk = 512;     // tokens per block
constexpr int kDecThreads = 256;
constexpr int kDecMaxGroup = 8;    // query heads per KV head

struct DecodeParams {
  View q, CK, CV;         // q: [layer][seq][q head][d]; CodeBook rows [layer][seq][kv head][entry][d]
  Batch batch;            // describes the cached tokens (per-layer / per-head lengths allowed)
  int n_q_heads, n_kv_heads, h_n, n_chunks;
  const int32_t* pos_q;   // [B]
  const int32_t* ref_k; const float* mag_k;   // [layers][H][T]
  const int32_t* ref_v; const float* mag_v;
  const int32_t* positions;                   // [layers][H][T] or null: token t sits at position t
  const float2* table;    // [table_positions][d/2] (cos, sin)
  int table_positions;
  float scale;            // 1 / sqrt(d)
  float* part;            // [units][n_chunks][h_n][d + 2]: (max, sum, weighted value sums)
  float* out;             // [layers][B][n_q_heads][d]
};

template <typename T, int N>
__device__ __forceinline__ void load_row_piece(const T* p, float (&out)[N]) {
  if constexpr (sizeof(T) == 4) {
    if constexpr (N == 4) {
      const float4 v = *reinterpret_cast<const float4*>(p);
      out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    } else {
      const float2 v = *reinterpret_cast<const float2*>(p);
      out[0] = v.x; out[1] = v.y;
    }
  } else {
    uint32_t w[N / 2];
    if constexpr (N == 4) {
      const uint2 v = *reinterpret_cast<const uint2*>(p);
      w[0] = v.x; w[1] = v.y;
    } else {
      w[0] = *reinterpret_cast<const uint32_t*>(p);
    }
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
}

// HN: query heads per KV head the instantiation is unrolled for (the group's actual size h_n <= HN)
template <typename T, int D, int HN>
__global__ void __launch_bounds__(kDecThreads) decode_chunk_kernel(DecodeParams p) {
  constexpr int H = D / 2;            // rotation pairs
  constexpr int PPT = D / 32;         // pairs per thread of a 16-thread token group
  extern __shared__ float sm[];
  const int unit = blockIdx.y, chunk = blockIdx.x;
  const int j = unit % p.n_kv_heads;
  const int ls = unit / p.n_kv_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int n = seq_len(p.batch, layer, s, j);
  const int t0 = chunk * kDecChunk;
  const int h_n = p.h_n;
  float* part = p.part + (((int64_t)unit * p.n_chunks + chunk) * h_n) * (D + 2);
  const int tid = threadIdx.x;
  if (t0 >= n) {
    // an empty chunk contributes nothing: weight exp(-inf) in the merge
    for (int i = tid; i < h_n * (D + 2); i += kDecThreads) part[i] = (i % (D + 2)) == 0 ? -CUDART_INF_F : 0.f;
    return;
  }
  const int nt = min(kDecChunk, n - t0);
  float* sq = sm;                                 // [h_n][D] rotated queries
  float* sc = sq + kDecMaxGroup * D;              // [h_n][kDecChunk] scores, then weights
  int32_t* srv = reinterpret_cast<int32_t*>(sc + kDecMaxGroup * kDecChunk);   // [kDecChunk] value references
  float* smv = reinterpret_cast<float*>(srv + kDecChunk);                     // [kDecChunk] value magnitudes
  float* red = smv + kDecChunk;                   // [kDecMaxGroup][8] reduction scratch
  const int64_t orow = ((int64_t)layer * p.n_kv_heads + j) * p.batch.total_len + tok_base(p.batch, s);
  const T* ck = reinterpret_cast<const T*>(p.CK.ptr) + unit_offset(p.CK, p.batch, layer, s, j);
  const T* cv = reinterpret_cast<const T*>(p.CV.ptr) + unit_offset(p.CV, p.batch, layer, s, j);
  // the group's queries, rotated at the new token's position
  {
    const int pq = min(max(p.pos_q[s], 0), p.table_positions - 1);
    const float2* tq = p.table + (int64_t)pq * H;
    const T* qb = reinterpret_cast<const T*>(p.q.ptr) + (int64_t)layer * p.q.sl + (int64_t)s * p.q.ss;
    for (int i = tid; i < h_n * H; i += kDecThreads) {
      const int g = i / H, k = i - g * H;
      const T* qr = qb + (int64_t)(h_n * j + g) * p.q.sh;
      const float a = to_f32(qr[k]), b = to_f32(qr[k + H]);
      const float2 cs = tq[k];
      sq[g * D + k] = a * cs.x - b * cs.y;
      sq[g * D + k + H] = b * cs.x + a * cs.y;
    }
  }
  for (int t = tid; t < nt; t += kDecThreads) {
    srv[t] = p.ref_v[orow + t0 + t];
    smv[t] = p.mag_v[orow + t0 + t];
  }
  __syncthreads();
  // ---- 1. scores: two tokens per 16-thread group and sweep, all their loads in flight before any is used ----
  {
    constexpr int kTok = 2;
    const int sub = tid & 15, grp = tid >> 4;     // 16 token groups per sweep
    // this thread's part of the rotated queries stays in registers for the whole chunk
    float qlo[HN][PPT], qhi[HN][PPT];
#pragma unroll
    for (int g = 0; g < HN; ++g)
#pragma unroll
      for (int k = 0; k < PPT; ++k) {
        qlo[g][k] = g < h_n ? sq[g * D + sub * PPT + k] : 0.f;
        qhi[g][k] = g < h_n ? sq[g * D + H + sub * PPT + k] : 0.f;
      }
    for (int tb = 0; tb < nt; tb += kTok * (kDecThreads / 16)) {
      float lo[kTok][PPT], hi[kTok][PPT], m[kTok];
      float2 cs[kTok][PPT];
      int tk[kTok];
#pragma unroll
      for (int x = 0; x < kTok; ++x) {
        const int t = tb + x * (kDecThreads / 16) + grp;
        tk[x] = t;
        const bool has = t < nt;
        const int r = has ? p.ref_k[orow + t0 + t] : 0;
        m[x] = has ? p.mag_k[orow + t0 + t] : 0.f;
        const int pos = (has && p.positions) ? p.positions[orow + t0 + t] : t0 + t;
        const float2* tab = p.table + (int64_t)min(max(pos, 0), p.table_positions - 1) * H + sub * PPT;
        const T* row = ck + (int64_t)r * p.CK.st;
        load_row_piece<T, PPT>(row + sub * PPT, lo[x]);
        load_row_piece<T, PPT>(row + H + sub * PPT, hi[x]);
#pragma unroll
        for (int k = 0; k < PPT; k += 2) {
          const float4 v = *reinterpret_cast<const float4*>(tab + k);
          cs[x][k] = make_float2(v.x, v.y);
          cs[x][k + 1] = make_float2(v.z, v.w);
        }
      }
#pragma unroll
      for (int x = 0; x < kTok; ++x) {
        float acc[HN];
#pragma unroll
        for (int g = 0; g < HN; ++g) acc[g] = 0.f;
#pragma unroll
        for (int k = 0; k < PPT; ++k) {
          const float a = lo[x][k] * m[x], b = hi[x][k] * m[x];               // Eq. (14)
          const float ra = a * cs[x][k].x - b * cs[x][k].y, rb = b * cs[x][k].x + a * cs[x][k].y;
#pragma unroll
          for (int g = 0; g < HN; ++g)
            if (g < h_n) acc[g] = fmaf(qlo[g][k], ra, fmaf(qhi[g][k], rb, acc[g]));
        }
#pragma unroll
        for (int g = 0; g < HN; ++g) {
          if (g < h_n) {
#pragma unroll
            for (int o = 8; o >= 1; o >>= 1) acc[g] += __shfl_xor_sync(0xffffffffu, acc[g], o);
            if (sub == 0 && tk[x] < nt) sc[g * kDecChunk + tk[x]] = acc[g] * p.scale;
          }
        }
      }
    }
  }
  __syncthreads();
  // ---- 2. maximum and exp-sum per query head: warp w of eight takes head w (and w + 8 never: h_n <= 8) ----
  {
    const int w = tid >> 5, lane = tid & 31;
    if (w < h_n) {
      float mx = -CUDART_INF_F;
      for (int t = lane; t < nt; t += 32) mx = fmaxf(mx, sc[w * kDecChunk + t]);
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float sum = 0.f;
      for (int t = lane; t < nt; t += 32) {
        const float e = expf(sc[w * kDecChunk + t] - mx);
        sc[w * kDecChunk + t] = e * smv[t];          // weight of the CodeBook row: probability share times magnitude
        sum += e;
      }
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        red[w * 2] = mx;
        red[w * 2 + 1] = sum;
      }
    }
  }
  __syncthreads();
  // ---- 3. values: a thread owns one pair of output elements for all query heads and every kParts-th token, so a
  // CodeBook row piece is loaded once for the whole group; the kParts partial sums meet in shared memory ----
  {
    constexpr int kParts = kDecThreads / H;
    constexpr int kUnroll = 8;
    const int pr = tid % H, tq = tid / H;
    float o[HN][2];
#pragma unroll
    for (int g = 0; g < HN; ++g) o[g][0] = o[g][1] = 0.f;
    for (int tb = tq; tb < nt; tb += kParts * kUnroll) {
      float x[kUnroll][2];
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        const int t = tb + i * kParts;
        const int r = t < nt ? srv[t] : 0;
        if constexpr (sizeof(T) == 4) {
          const float2 v = *reinterpret_cast<const float2*>(cv + (int64_t)r * p.CV.st + 2 * pr);
          x[i][0] = v.x; x[i][1] = v.y;
        } else {
          const uint32_t v = *reinterpret_cast<const uint32_t*>(cv + (int64_t)r * p.CV.st + 2 * pr);
          x[i][0] = __uint_as_float(v << 16); x[i][1] = __uint_as_float(v & 0xFFFF0000u);
        }
      }
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        const int t = tb + i * kParts;
        if (t >= nt) continue;
#pragma unroll
        for (int g = 0; g < HN; ++g)
          if (g < h_n) {
            const float wv = sc[g * kDecChunk + t];
            o[g][0] = fmaf(wv, x[i][0], o[g][0]);
            o[g][1] = fmaf(wv, x[i][1], o[g][1]);
          }
      }
    }
    __syncthreads();                         // every thread is done with the weights: their place takes the partial sums
    float* ps = sc;                          // [kParts][h_n][D]
#pragma unroll
    for (int g = 0; g < HN; ++g)
      if (g < h_n) {
        ps[(tq * h_n + g) * D + 2 * pr] = o[g][0];
        ps[(tq * h_n + g) * D + 2 * pr + 1] = o[g][1];
      }
    __syncthreads();
    for (int i = tid; i < h_n * D; i += kDecThreads) {
      float sum = 0.f;
#pragma unroll
      for (int q = 0; q < kParts; ++q) sum += ps[q * h_n * D + i];   // fixed order
      part[(i / D) * (D + 2) + 2 + (i % D)] = sum;
    }
  }
  if (tid < h_n) {
    part[tid * (D + 2)] = red[tid * 2];
    part[tid * (D + 2) + 1] = red[tid * 2 + 1];
  }
}

// chunks of a unit -> output rows of its query heads
template <int D>
__global__ void __launch_bounds__(kDecThreads) decode_merge_kernel(DecodeParams p) {
  const int unit = blockIdx.x;
  const int j = unit % p.n_kv_heads;
  const int ls = unit / p.n_kv_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int h_n = p.h_n;
  const float* part = p.part + (int64_t)unit * p.n_chunks * h_n * (D + 2);
  for (int i = threadIdx.x; i < h_n * D; i += kDecThreads) {
    const int g = i / D, e = i - g * D;
    float mx = -CUDART_INF_F;
    for (int c = 0; c < p.n_chunks; ++c) mx = fmaxf(mx, part[((int64_t)c * h_n + g) * (D + 2)]);
    float num = 0.f, den = 0.f;
    for (int c = 0; c < p.n_chunks; ++c) {
      const float* q = part + ((int64_t)c * h_n + g) * (D + 2);
      const float w = q[0] == -CUDART_INF_F ? 0.f : expf(q[0] - mx);
      num = fmaf(w, q[2 + e], num);
      den = fmaf(w, q[1], den);
    }
    p.out[(((int64_t)layer * p.batch.n_seqs + s) * p.n_q_heads + (h_n * j + g)) * D + e] = den > 0.f ? num / den : 0.f;
  }
}

// cos and sin of position * base^(-2i/d), in double precision, rounded once to fp32
__global__ void rope_table_kernel(float2* table, int half, int n_pos, double base, int d) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (int64_t)n_pos * half) return;
  const int pos = (int)(i / half), k = (int)(i - (int64_t)pos * half);
  const double omega = pow(base, -2.0 * (double)k / (double)d);
  double sn, cs;
  sincos((double)pos * omega, &sn, &cs);
  table[i] = make_float2((float)cs, (float)sn);
}

spindlekv_status rope_table_impl(int head_dim, int n_pos, double base, void* table, cudaStream_t st) {
  const int64_t n = (int64_t)n_pos * (head_dim / 2);
  LaunchScope ls(KC_GATHER, st);
  rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(reinterpret_cast<float2*>(table), head_dim / 2, n_pos, base, head_dim);
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

size_t decode_workspace_bytes(const spindlekv_batch& b, int n_q_heads, int n_kv_heads, int head_dim) {
  const size_t units = (size_t)b.n_layers * b.n_seqs * n_kv_heads;
  const size_t chunks = (size_t)ceil_div(b.max_len, kDecChunk);
  return align_up(units * chunks * (size_t)(n_q_heads / n_kv_heads) * (head_dim + 2) * sizeof(float), 256);
}

static size_t decode_smem_bytes(int head_dim) {
  return (size_t)(kDecMaxGroup * head_dim + kDecMaxGroup * kDecChunk + 2 * kDecChunk + kDecMaxGroup * 8) * 4;
}

template <typename T, int D, int HN>
static spindlekv_status launch_decode_hn(const DecodeParams& p, int units, cudaStream_t st) {
  static PerDeviceOnce once;
  const int dev = PerDeviceOnce::current();
  if (dev < 0) return SPINDLEKV_CUDA;
  const size_t smem = decode_smem_bytes(D);
  if (!once.done[dev]) {
    if (cudaFuncSetAttribute(decode_chunk_kernel<T, D, HN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SPINDLEKV_CUDA;
    once.done[dev] = true;
  }
  { LaunchScope ls(KC_DECODE, st); decode_chunk_kernel<T, D, HN><<<dim3(p.n_chunks, units), kDecThreads, smem, st>>>(p); }
  { LaunchScope ls(KC_DECODE, st); decode_merge_kernel<D><<<units, kDecThreads, 0, st>>>(p); }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

template <typename T, int D>
static spindlekv_status launch_decode(const DecodeParams& p, int units, cudaStream_t st) {
  if (p.h_n <= 1) return launch_decode_hn<T, D, 1>(p, units, st);
  if (p.h_n <= 2) return launch_decode_hn<T, D, 2>(p, units, st);
  if (p.h_n <= 4) return launch_decode_hn<T, D, 4>(p, units, st);
  return launch_decode_hn<T, D, kDecMaxGroup>(p, units, st);
}

spindlekv_status decode_attend_impl(const spindlekv_batch& b, int n_q_heads, int n_kv_heads, int head_dim,
                                    const spindlekv_tensor& q, const int32_t* pos_q, const spindlekv_tensor& CK,
                                    const int32_t* ref_k, const float* mag_k, const spindlekv_tensor& CV,
                                    const int32_t* ref_v, const float* mag_v, const int32_t* positions,
                                    const void* table, int table_positions, float* out, void* ws, size_t ws_bytes,
                                    cudaStream_t st) {
  if (ws_bytes < decode_workspace_bytes(b, n_q_heads, n_kv_heads, head_dim)) return SPINDLEKV_WORKSPACE_TOO_SMALL;
  const int units = b.n_layers * b.n_seqs * n_kv_heads;
  if (units > 65535) return SPINDLEKV_UNSUPPORTED;
  DecodeParams p;
  p.q = make_view(q);
  p.CK = make_view(CK);
  p.CV = make_view(CV);
  p.batch = make_batch(b);
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = n_kv_heads;
  p.h_n = n_q_heads / n_kv_heads;
  p.n_chunks = ceil_div(b.max_len, kDecChunk);
  p.pos_q = pos_q;
  p.ref_k = ref_k; p.mag_k = mag_k;
  p.ref_v = ref_v; p.mag_v = mag_v;
  p.positions = positions;
  p.table = reinterpret_cast<const float2*>(table);
  p.table_positions = table_positions;
  p.scale = 1.0f / sqrtf((float)head_dim);
  p.part = reinterpret_cast<float*>(ws);
  p.out = out;
  const bool bf = CK.dtype == SPINDLEKV_BF16;
  if (head_dim == 64) return bf ? launch_decode<__nv_bfloat16, 64>(p, units, st) : launch_decode<float, 64>(p, units, st);
  return bf ? launch_decode<__nv_bfloat16, 128>(p, units, st) : launch_decode<float, 128>(p, units, st);
}

}  // namespace skv

// Decode-time attention over the replaced cache (Section 3.4 after Eq. (14)): the new token's queries
// attend to K = C_K[r_K] (x) m_K and V = C_V[r_V] (x) m_V without the rebuilt rows ever being written to
// memory.  The CodeBooks hold pre-RoPE keys, so every rebuilt key is rotated at its token's original
// position on the fly (rotary embedding of Eq. (1): element i paired with element i + d/2, angle
// position * base^(-2i/d)), with cosines and sines taken from a table the caller prepares once.
//
// One unit is (layer, sequence, KV head); the h_n query heads of its GQA group are served together, so a
// key is rebuilt and rotated once for all of them.  A unit's tokens are split into chunks of kDecChunk;
// one block per (chunk, unit):
//   0. the chunk's references, magnitudes and positions are copied into shared memory, so that no row load
//      waits for the load of its own address;
//   1. scores: 16 threads per token gather the token's CodeBook row, scale it by the token's magnitude, rotate
//      it, and form the dot products with the rotated queries (each thread's part of them in registers); the
//      16 partial sums meet through shuffles.  Scores of the chunk stay in shared memory.
//   2. the chunk's maximum and exp-sum per query head (fixed-order reductions);
//   3. values: a 16-byte piece of a CodeBook row per thread and token (the threads of a row side by side, the
//      chunk's tokens dealt out over the rows of threads), weight * magnitude * piece added for all query heads
//      at once; the partial sums meet by shuffles inside a warp and through shared memory across warps, in a
//      fixed order.
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

// Sum of acc[g] over the 16 threads of a token, for all HN heads at once: at every step a thread keeps half of its
// values and hands the other half to its partner, so HN heads cost HN - 1 + (4 - log2 HN) shuffles instead of
// 4 HN.  Returns the total of head `head` in the threads whose low 4 - log2(HN) bits of `sub` are zero (all
// threads of the token hold some head's total; those are the ones that store it).  Fixed order of additions.
template <int HN>
__device__ __forceinline__ float reduce_heads(const float (&acc)[HN], int sub, int& head) {
  float v[HN];
#pragma unroll
  for (int g = 0; g < HN; ++g) v[g] = acc[g];
  head = 0;
  int n = HN;
#pragma unroll
  for (int bit = 8; bit >= 1; bit >>= 1) {
    if (n > 1) {
      const bool up = (sub & bit) != 0;
      const int half = n >> 1;
#pragma unroll
      for (int i = 0; i < HN / 2; ++i) {
        if (i < half) {
          const float keep = up ? v[half + i] : v[i];
          const float send = up ? v[i] : v[half + i];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
        }
      }
      head += up ? half : 0;
      n = half;
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], bit);
    }
  }
  return v[0];
}

template <int HN>
__device__ __forceinline__ void load_heads(const float* p, float (&w)[HN]) {
  if constexpr (HN == 1) {
    w[0] = p[0];
  } else if constexpr (HN == 2) {
    const float2 v = *reinterpret_cast<const float2*>(p);
    w[0] = v.x; w[1] = v.y;
  } else {
#pragma unroll
    for (int i = 0; i < HN; i += 4) {
      const float4 v = *reinterpret_cast<const float4*>(p + i);
      w[i] = v.x; w[i + 1] = v.y; w[i + 2] = v.z; w[i + 3] = v.w;
    }
  }
}

// HN: query heads per KV head the instantiation is unrolled for (the group's actual size h_n <= HN)
template <typename T, int D, int HN>
__global__ void __launch_bounds__(kDecThreads, HN <= 4 ? 4 : 2) decode_chunk_kernel(DecodeParams p) {
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
  float* sc = sq + h_n * D;                       // [kDecChunk][HN] scores, then weights (a token's heads side by side)
  // per token, read with one 16-byte load: key reference, key magnitude (bits), position clamped to the table,
  // value reference
  int4* stok = reinterpret_cast<int4*>(sc + HN * kDecChunk);                  // [kDecChunk]
  float* smv = reinterpret_cast<float*>(stok + kDecChunk);                    // [kDecChunk] value magnitudes
  float* red = smv + kDecChunk;                                               // [2][warps][HN] reduction scratch
  float* ps = red + 2 * kDecMaxGroup * (kDecThreads / 32);             // [warps][h_n][D] partial value sums
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
    smv[t] = p.mag_v[orow + t0 + t];
    stok[t] = make_int4(p.ref_k[orow + t0 + t], __float_as_int(p.mag_k[orow + t0 + t]),
                        min(max(p.positions ? p.positions[orow + t0 + t] : t0 + t, 0), p.table_positions - 1),
                        p.ref_v[orow + t0 + t]);
  }
  __syncthreads();
  // ---- 1. scores: two tokens per 16-thread group and sweep, all their loads in flight before any is used ----
  {
    constexpr int kTok = 2;
    const int sub = tid & 15, grp = tid >> 4;     // 16 token groups per sweep
    // this thread's part of the rotated queries stays in registers for the whole chunk, two pairs to a register
    // pair: the arithmetic below is packed (two fp32 lanes per instruction)
    static_assert(PPT % 2 == 0, "pairs are handled two at a time");
    float2 qlo[HN][PPT / 2], qhi[HN][PPT / 2];
#pragma unroll
    for (int g = 0; g < HN; ++g)
#pragma unroll
      for (int k = 0; k < PPT / 2; ++k) {
        const float* q0 = sq + g * D + sub * PPT + 2 * k;
        qlo[g][k] = g < h_n ? make_float2(q0[0], q0[1]) : make_float2(0.f, 0.f);
        qhi[g][k] = g < h_n ? make_float2(q0[H], q0[H + 1]) : make_float2(0.f, 0.f);
      }
    for (int tb = 0; tb < nt; tb += kTok * (kDecThreads / 16)) {
      float lo[kTok][PPT], hi[kTok][PPT], m[kTok];
      float4 cs[kTok][PPT / 2];          // (cos, sin) of two pairs
      int tk[kTok];
#pragma unroll
      for (int x = 0; x < kTok; ++x) {
        const int t = tb + x * (kDecThreads / 16) + grp;
        tk[x] = t;
        const bool has = t < nt;
        const int4 tk4 = has ? stok[t] : make_int4(0, 0, 0, 0);
        const int r = tk4.x;
        m[x] = __int_as_float(tk4.y);
        const float2* tab = p.table + (int64_t)tk4.z * H + sub * PPT;
        const T* row = ck + (int64_t)r * p.CK.st;
        load_row_piece<T, PPT>(row + sub * PPT, lo[x]);
        load_row_piece<T, PPT>(row + H + sub * PPT, hi[x]);
#pragma unroll
        for (int k = 0; k < PPT / 2; ++k) cs[x][k] = *reinterpret_cast<const float4*>(tab + 2 * k);
      }
#pragma unroll
      for (int x = 0; x < kTok; ++x) {
        float2 acc2[HN];
#pragma unroll
        for (int g = 0; g < HN; ++g) acc2[g] = make_float2(0.f, 0.f);
        const float2 m2 = make_float2(m[x], m[x]);
#pragma unroll
        for (int k = 0; k < PPT / 2; ++k) {
          const float2 c2 = make_float2(cs[x][k].x, cs[x][k].z), s2 = make_float2(cs[x][k].y, cs[x][k].w);
          const float2 a2 = __fmul2_rn(make_float2(lo[x][2 * k], lo[x][2 * k + 1]), m2);    // Eq. (14)
          const float2 b2 = __fmul2_rn(make_float2(hi[x][2 * k], hi[x][2 * k + 1]), m2);
          // (a, b) -> (a cos - b sin, b cos + a sin)
          const float2 ra = __ffma2_rn(make_float2(-b2.x, -b2.y), s2, __fmul2_rn(a2, c2));
          const float2 rb = __ffma2_rn(a2, s2, __fmul2_rn(b2, c2));
#pragma unroll
          for (int g = 0; g < HN; ++g)
            if (g < h_n) acc2[g] = __ffma2_rn(qlo[g][k], ra, __ffma2_rn(qhi[g][k], rb, acc2[g]));
        }
        float acc[HN];
#pragma unroll
        for (int g = 0; g < HN; ++g) acc[g] = acc2[g].x + acc2[g].y;
        int head;
        const float total = reduce_heads<HN>(acc, sub, head);
        if ((sub & (16 / HN - 1)) == 0 && head < h_n && tk[x] < nt) sc[tk[x] * HN + head] = total * p.scale;
      }
    }
  }
  __syncthreads();
  // ---- 2. maximum and exp-sum per query head: a thread takes every kDecThreads-th token with all its heads; the
  // partial results meet by shuffles inside a warp and through shared memory across the warps, in a fixed order ----
  {
    const int w = tid >> 5, lane = tid & 31;
    constexpr int NW = kDecThreads / 32;
    float mx[HN];
#pragma unroll
    for (int g = 0; g < HN; ++g) mx[g] = -CUDART_INF_F;
    for (int t = tid; t < nt; t += kDecThreads) {
      float v[HN];
      load_heads<HN>(sc + t * HN, v);
#pragma unroll
      for (int g = 0; g < HN; ++g) mx[g] = fmaxf(mx[g], v[g]);
    }
#pragma unroll
    for (int g = 0; g < HN; ++g) {
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xffffffffu, mx[g], o));
      if (lane == 0) red[w * HN + g] = mx[g];
    }
    __syncthreads();
#pragma unroll
    for (int g = 0; g < HN; ++g) {
      float v = red[g];
#pragma unroll
      for (int q = 1; q < NW; ++q) v = fmaxf(v, red[q * HN + g]);
      mx[g] = v;
    }
    float sum[HN];
#pragma unroll
    for (int g = 0; g < HN; ++g) sum[g] = 0.f;
    for (int t = tid; t < nt; t += kDecThreads) {
      float v[HN];
      load_heads<HN>(sc + t * HN, v);
      const float mv = smv[t];
#pragma unroll
      for (int g = 0; g < HN; ++g) {
        const float e = g < h_n ? expf(v[g] - mx[g]) : 0.f;
        sum[g] += e;
        sc[t * HN + g] = e * mv;                   // weight of the CodeBook row: probability share times magnitude
      }
    }
#pragma unroll
    for (int g = 0; g < HN; ++g) {
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) sum[g] += __shfl_xor_sync(0xffffffffu, sum[g], o);
      if (lane == 0) red[kDecMaxGroup * NW + w * HN + g] = sum[g];
    }
    __syncthreads();
    if (tid < h_n) {
      float vm = red[tid], v = 0.f;
#pragma unroll
      for (int q = 1; q < NW; ++q) vm = fmaxf(vm, red[q * HN + tid]);
#pragma unroll
      for (int q = 0; q < NW; ++q) v += red[kDecMaxGroup * NW + q * HN + tid];     // fixed order
      part[tid * (D + 2)] = vm;
      part[tid * (D + 2) + 1] = v;
    }
  }
  // ---- 3. values: TPR threads side by side read a CodeBook row in 16-byte pieces, once for the whole group; the
  // chunk's tokens are dealt out over the kDecThreads / TPR rows of threads ----
  {
    constexpr int EPT = 16 / (int)sizeof(T);     // elements per piece
    constexpr int TPR = D / EPT;                 // threads per row
    constexpr int G = kDecThreads / TPR;         // rows of threads
    constexpr int kUnroll = 4;
    static_assert(TPR <= 32 && 32 % TPR == 0, "a row of threads lies inside a warp");
    const int sub = tid % TPR, grp = tid / TPR;
    float2 o[HN][EPT / 2];
#pragma unroll
    for (int g = 0; g < HN; ++g)
#pragma unroll
      for (int e = 0; e < EPT / 2; ++e) o[g][e] = make_float2(0.f, 0.f);
    for (int tb = grp; tb < nt; tb += G * kUnroll) {
      uint4 raw[kUnroll];
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        const int t = tb + i * G;
        const int r = t < nt ? stok[t].w : 0;
        raw[i] = *reinterpret_cast<const uint4*>(cv + (int64_t)r * p.CV.st + sub * EPT);
      }
#pragma unroll
      for (int i = 0; i < kUnroll; ++i) {
        const int t = tb + i * G;
        if (t >= nt) continue;
        float x[EPT];
        if constexpr (sizeof(T) == 4) {
          x[0] = __uint_as_float(raw[i].x); x[1] = __uint_as_float(raw[i].y);
          x[2] = __uint_as_float(raw[i].z); x[3] = __uint_as_float(raw[i].w);
        } else {
          const uint32_t w4[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            x[2 * e] = __uint_as_float(w4[e] << 16);
            x[2 * e + 1] = __uint_as_float(w4[e] & 0xFFFF0000u);
          }
        }
        float wv[HN];
        load_heads<HN>(sc + t * HN, wv);
#pragma unroll
        for (int g = 0; g < HN; ++g) {
          const float2 w2 = make_float2(wv[g], wv[g]);
#pragma unroll
          for (int e = 0; e < EPT / 2; ++e) o[g][e] = __ffma2_rn(w2, make_float2(x[2 * e], x[2 * e + 1]), o[g][e]);
        }
      }
    }
    // the rows of threads of a warp first (lanes that hold the same piece), then the warps in order
#pragma unroll
    for (int off = TPR; off < 32; off <<= 1)
#pragma unroll
      for (int g = 0; g < HN; ++g)
#pragma unroll
        for (int e = 0; e < EPT / 2; ++e) {
          o[g][e].x += __shfl_xor_sync(0xffffffffu, o[g][e].x, off);
          o[g][e].y += __shfl_xor_sync(0xffffffffu, o[g][e].y, off);
        }
    const int wp = tid >> 5, lane = tid & 31;
    if (lane < TPR) {
#pragma unroll
      for (int g = 0; g < HN; ++g)
        if (g < h_n) {
#pragma unroll
          for (int e = 0; e < EPT / 2; ++e)
            *reinterpret_cast<float2*>(ps + (wp * h_n + g) * D + sub * EPT + 2 * e) = o[g][e];
        }
    }
    __syncthreads();
    for (int i = tid; i < h_n * D; i += kDecThreads) {
      float sum = 0.f;
#pragma unroll
      for (int q = 0; q < kDecThreads / 32; ++q) sum += ps[q * h_n * D + i];   // fixed order
      part[(i / D) * (D + 2) + 2 + (i % D)] = sum;
    }
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

// hn_slots: the group size the kernel instantiation is unrolled for (a token's scores take that many floats)
static size_t decode_smem_bytes(int head_dim, int h_n, int hn_slots) {
  // rotated queries, scores, five per-token arrays, reduction scratch, per-warp partial value sums
  return (size_t)(h_n * head_dim + hn_slots * kDecChunk + 5 * kDecChunk + 2 * kDecMaxGroup * (kDecThreads / 32) + (kDecThreads / 32) * h_n * head_dim) * 4;
}

template <typename T, int D, int HN>
static spindlekv_status launch_decode_hn(const DecodeParams& p, int units, cudaStream_t st) {
  static PerDeviceOnce once;
  const int dev = PerDeviceOnce::current();
  if (dev < 0) return SPINDLEKV_CUDA;
  const size_t smem = decode_smem_bytes(D, p.h_n, HN);
  if (!once.done[dev]) {
    if (cudaFuncSetAttribute(decode_chunk_kernel<T, D, HN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)decode_smem_bytes(D, HN, HN)) != cudaSuccess)
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

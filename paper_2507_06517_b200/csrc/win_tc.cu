// Window scores of the evicting layers (Eq. (1)(2)(3)) on the 5th-generation tensor cores, bf16.
//
// One CTA owns one unit (layer, sequence, KV head): its M = h_n * l_w window-query rows (row
// r = g * l_w + t: query head h_n*j + g, window query t at position b = l_c + t) stay in shared memory,
// the keys stream through a ring of 128-row tiles, twice:
//
//   pass A   S = Q K^T  (tcgen05.mma, rows = queries).  A thread owns one query row and keeps the
//            running maximum and the running sum of exp of that row over the keys 0..b (causal mask,
//            Eq. (1)), in the base-2 domain: y = s * log2(e) / sqrt(d_h).
//   between  lse_r = max_r + log2(sum_r); L_r = lse_r / (log2(e)/sqrt(d_h)) is split into three bf16
//            pieces and written, negated, into a 16-element operand row.
//   pass B   S^T = K Q^T (rows = keys) with one extra K-step that adds -L_r to column r: the
//            accumulator holds q_r . k_a - L_r, so exp2 of it (times the scale) is the softmax weight
//            A[r, a] itself.  A thread owns one key a and sums its M columns: Eq. (2)'s sum over the
//            window queries and Eq. (3)'s sum over the group in one go, then divides by h_n and by
//            (l - a).  No value crosses a lane in either pass.
//
// Roles: warp 0 issues TMA loads, warp 1 issues the MMAs, warps 2..9 are two epilogue groups of
// four warps (one per TMEM lane quarter); group e handles the tiles that land in TMEM stage e, so
// the two groups never wait for each other inside a pass.  Every wait is bounded.
#include <math_constants.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace skv {

struct WinTcParams {
  Batch batch;
  int n_kv_heads, h_n, window;
  int m_rows;            // h_n * window
  int score_norm;
  int per_head;          // 1: one score row per query head (Eq. (2)), no group mean; scores are then [layers][H_q][T]
  float c;               // log2(e) / sqrt(d_h)
  float* scores;         // [layers][H_kv][T]
  uint32_t* hdr;
};

constexpr int kWinTile = 128;                 // keys per tile
constexpr int kWinStages = 4;                 // K ring
// Epilogue groups of four warps (one per lane quarter of tensor memory); group g takes the tiles i with i % G == g.
// With one block of query rows an accumulator is 128 columns wide: four stages, four groups.  With two blocks it is
// 256 columns wide: two stages, two groups.
template <int QB> struct WinShape {
  static constexpr int G = QB == 1 ? 4 : 2;
  static constexpr int EPI_WARPS = 4 * G;
  static constexpr int THREADS = 32 * (2 + EPI_WARPS);
};

template <int D, int QB>
struct WinSmem {
  static constexpr int KH = D / 64;
  static constexpr int NQ = QB * 128;                 // query rows held (padded to whole 128-row blocks)
  static constexpr int Q_BYTES = KH * NQ * 128;
  static constexpr int K_BYTES = KH * kWinTile * 128;
  static constexpr int EA_BYTES = 2 * kWinTile * 16;  // ones operand, two 16-byte column chunks
  static constexpr int EB_BYTES = 2 * NQ * 16;        // -L operand
  static constexpr int ST_BYTES = (WinShape<QB>::G - 1) * NQ * 8;   // (max, sum) of the epilogue groups after the first
  static constexpr int OFF_K = Q_BYTES;
  static constexpr int OFF_EA = OFF_K + kWinStages * K_BYTES;
  static constexpr int OFF_EB = OFF_EA + EA_BYTES;
  static constexpr int OFF_ST = OFF_EB + EB_BYTES;
  static constexpr int OFF_BAR = OFF_ST + ST_BYTES;
  static constexpr int USED = OFF_BAR + 256 + 1024;
  // more than half of an SM's shared memory, so that two blocks never share an SM (each takes all of TMEM)
  static constexpr int TOTAL = USED > 120 * 1024 ? USED : 120 * 1024;
  static_assert(TOTAL <= 227 * 1024, "shared memory budget");
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D, int QB>
__global__ void __launch_bounds__(WinShape<QB>::THREADS, 1) win_tc_kernel(const __grid_constant__ CUtensorMap kmap,
                                                                const __grid_constant__ CUtensorMap qmap,
                                                                WinTcParams p) {
  using L = WinSmem<D, QB>;
  constexpr int NQ = L::NQ;
  const int unit = blockIdx.x;
  const int j = unit % p.n_kv_heads;
  const int ls = unit / p.n_kv_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int l = seq_len(p.batch, layer, s, j);
  const int l_c = l - p.window;
  // accumulator ring in tensor memory: four stages of 128 columns when one block of query rows is held, else two
  // of 256; the epilogue group of tile i is i & 1, so a stage always belongs to one group
  constexpr int AS = WinShape<QB>::G;
  constexpr int AS_COLS = 512 / AS;
  constexpr int G = WinShape<QB>::G;
  constexpr int kWinEpiWarps = WinShape<QB>::EPI_WARPS;
  constexpr int kWinThreads = WinShape<QB>::THREADS;
  const int T = (l + kWinTile - 1) / kWinTile;      // tiles of pass A (all keys)
  const int Tc = (l_c + kWinTile - 1) / kWinTile;   // tiles of pass B (context keys)

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                  // [kh][NQ rows][128 B], 128-byte swizzle
  uint8_t* sK = smem + L::OFF_K;       // [stage][kh][128 rows][128 B]
  uint8_t* sEA = smem + L::OFF_EA;     // [chunk][128 rows][16 B], no swizzle
  uint8_t* sEB = smem + L::OFF_EB;     // [chunk][NQ rows][16 B], no swizzle
  float2* sST = reinterpret_cast<float2*>(smem + L::OFF_ST);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  uint64_t* q_full = bars + 0;
  uint64_t* k_full = bars + 1;                 // [kWinStages]
  uint64_t* k_empty = bars + 1 + kWinStages;   // [kWinStages]
  uint64_t* acc_full = bars + 1 + 2 * kWinStages;   // [AS]
  uint64_t* acc_empty = acc_full + 4;               // [AS]
  uint64_t* ext_full = acc_empty + 4;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ext_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ext_full + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    ptx::mbar_init(q_full, 1);
    for (int i = 0; i < kWinStages; ++i) { ptx::mbar_init(k_full + i, 1); ptx::mbar_init(k_empty + i, 1); }
    for (int i = 0; i < AS; ++i) { ptx::mbar_init(acc_full + i, 1); ptx::mbar_init(acc_empty + i, 4); }
    ptx::mbar_init(ext_full, kWinEpiWarps);
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  // the constant operand of the extra K-step: three ones per key row (they pick up the three pieces of -L)
  for (int i = threadIdx.x; i < L::EA_BYTES / 16; i += kWinThreads) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (i < kWinTile) { v.x = 0x3F803F80u; v.y = 0x00003F80u; }   // bf16 1.0 in slots 0, 1, 2 of chunk 0
    reinterpret_cast<uint4*>(sEA)[i] = v;
  }
  ptx::fence_proxy_async();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int tok0 = p.batch.cu ? p.batch.cu[s] : 0;
  const int sdim = p.batch.cu ? 0 : s;

  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&kmap);
      ptx::prefetch_tensormap(&qmap);
      ptx::mbar_expect_tx(q_full, L::Q_BYTES);
      const int heads_per_block = 128 / p.window;
      for (int kh = 0; kh < L::KH; ++kh)
        for (int qb = 0; qb < QB; ++qb)
          ptx::tma_load_5d(sQ + kh * NQ * 128 + qb * 128 * 128, &qmap, q_full, kh * 64, 0,
                           p.h_n * j + qb * heads_per_block, s, layer);
      for (int i = 0; i < T + Tc; ++i) {
        const int tile = i < T ? i : i - T;
        const int st = i % kWinStages;
        if (!ptx::mbar_wait(k_empty + st, ((i / kWinStages) & 1) ^ 1, abort_flag)) break;
        ptx::mbar_expect_tx(k_full + st, L::K_BYTES);
        for (int kh = 0; kh < L::KH; ++kh)
          ptx::tma_load_5d(sK + st * L::K_BYTES + kh * kWinTile * 128, &kmap, k_full + st, kh * 64,
                           tok0 + tile * kWinTile, j, sdim, layer);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc_a = ptx::idesc_bf16_f32(128, kWinTile);   // queries x keys
      constexpr uint32_t idesc_b = ptx::idesc_bf16_f32(kWinTile, NQ);    // keys x queries
      const uint32_t q_addr = ptx::smem_u32(sQ);
      bool ok = ptx::mbar_wait(q_full, 0, abort_flag);
      int i = 0;
      for (; ok && i < T; ++i) {
        const int st = i % kWinStages, as = i % AS;
        if (!ptx::mbar_wait(k_full + st, (i / kWinStages) & 1, abort_flag)) { ok = false; break; }
        if (!ptx::mbar_wait(acc_empty + as, ((i / AS) & 1) ^ 1, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t k_addr = ptx::smem_u32(sK + st * L::K_BYTES);
#pragma unroll
        for (int qb = 0; qb < QB; ++qb)
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const int kh = k >> 2, kk = k & 3;
            const uint64_t da = ptx::smem_desc_sw128(q_addr + kh * NQ * 128 + qb * 128 * 128 + kk * 32);
            const uint64_t db = ptx::smem_desc_sw128(k_addr + kh * kWinTile * 128 + kk * 32);
            ptx::umma_bf16(tmem_base + as * AS_COLS + qb * 128, da, db, idesc_a, k > 0 ? 1u : 0u);
          }
        ptx::umma_commit(k_empty + st);
        ptx::umma_commit(acc_full + as);
      }
      if (ok) ok = ptx::mbar_wait(ext_full, 0, abort_flag);
      const uint64_t dea = ptx::smem_desc_interleaved(ptx::smem_u32(sEA), kWinTile * 16, 128);
      const uint64_t deb = ptx::smem_desc_interleaved(ptx::smem_u32(sEB), NQ * 16, 128);
      for (; ok && i < T + Tc; ++i) {
        const int st = i % kWinStages, as = i % AS;
        if (!ptx::mbar_wait(k_full + st, (i / kWinStages) & 1, abort_flag)) break;
        if (!ptx::mbar_wait(acc_empty + as, ((i / AS) & 1) ^ 1, abort_flag)) break;
        ptx::tc_fence_after();
        const uint32_t k_addr = ptx::smem_u32(sK + st * L::K_BYTES);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const int kh = k >> 2, kk = k & 3;
          const uint64_t da = ptx::smem_desc_sw128(k_addr + kh * kWinTile * 128 + kk * 32);
          const uint64_t db = ptx::smem_desc_sw128(q_addr + kh * NQ * 128 + kk * 32);
          ptx::umma_bf16(tmem_base + as * AS_COLS, da, db, idesc_b, k > 0 ? 1u : 0u);
        }
        ptx::umma_bf16(tmem_base + as * AS_COLS, dea, deb, idesc_b, 1u);   // - L_r on column r
        ptx::umma_commit(k_empty + st);
        ptx::umma_commit(acc_full + as);
      }
    }
  } else {
    const int q = warp & 3;                 // TMEM lane quarter of this warp
    const int eg = (warp - 2) >> 2;         // epilogue group = TMEM stage it serves
    const uint32_t tquarter = tmem_base + ((uint32_t)(q * 32) << 16);
    const float c = p.c;
    // ---- pass A: running (max, sum) of this thread's query rows, base-2 domain ----
    float rmax[QB], rsum[QB];
    int brow[QB];                           // position of the query of row qb*128 + q*32 + lane
#pragma unroll
    for (int qb = 0; qb < QB; ++qb) {
      rmax[qb] = -CUDART_INF_F;
      rsum[qb] = 0.f;
      brow[qb] = l_c + (qb * 128 + q * 32 + lane) % p.window;
    }
    bool ok = true;
    for (int i = eg; i < T; i += G) {
      const int as = i % AS;
      const uint32_t tlane = tquarter + as * AS_COLS;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(acc_full + as, (i / AS) & 1, abort_flag))) { ok = false; break; }
      ptx::tc_fence_after();
      const int key0 = i * kWinTile;
      const bool masked = key0 + kWinTile > l_c;     // window keys or the ragged end are in this tile
      // 32 columns at a time; the next 32 are on their way from tensor memory while these are worked on
      auto chunk_a = [&](const uint32_t (&raw)[32], int qb, int ch) {
        float v[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(raw[e]);
        if (masked) {
          const int a0 = key0 + ch * 32;
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (a0 + e > brow[qb]) v[e] = -CUDART_INF_F;   // causal: query b sees keys 0..b (b < l)
        }
        float mx = v[0];
#pragma unroll
        for (int e = 1; e < 32; ++e) mx = fmaxf(mx, v[e]);
        const float m_new = fmaxf(rmax[qb], mx * c);
        // a row that has seen no visible key yet keeps max = -inf and sum = 0 (exp2(-inf) = 0)
        const float m_ref = m_new == -CUDART_INF_F ? 0.f : m_new;
        float acc = rsum[qb] * ex2_approx(rmax[qb] - m_ref);
#pragma unroll
        for (int e = 0; e < 32; ++e) acc += ex2_approx(fmaf(v[e], c, -m_ref));
        rsum[qb] = acc;
        rmax[qb] = m_new;
      };
      constexpr int CPT = kWinTile / 32;   // chunks per 128 query rows
#pragma unroll
      for (int qb = 0; qb < QB; ++qb) {
#pragma unroll 1
        for (int ch = 0; ch < CPT; ++ch) {
          uint32_t raw[32];
          ptx::tmem_ld_32x32(tlane + qb * 128 + ch * 32, raw);
          ptx::tmem_ld_wait(raw);
          chunk_a(raw, qb, ch);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(acc_empty + as);
    }
    // ---- merge the groups' statistics; write the -L operand of pass B ----
    if (eg > 0) {
#pragma unroll
      for (int qb = 0; qb < QB; ++qb) sST[(eg - 1) * NQ + qb * 128 + q * 32 + lane] = make_float2(rmax[qb], rsum[qb]);
    }
    asm volatile("bar.sync 1, %0;" ::"n"(32 * kWinEpiWarps) : "memory");
    if (eg == 0) {
#pragma unroll
      for (int qb = 0; qb < QB; ++qb) {
        const int r = qb * 128 + q * 32 + lane;
        float m = rmax[qb];
        float2 o[G - 1];
#pragma unroll
        for (int g = 0; g < G - 1; ++g) {
          o[g] = sST[g * NQ + r];
          m = fmaxf(m, o[g].x);
        }
        // a group that saw no visible key of this row has (max, sum) = (-inf, 0): its term is 0 * exp2(-inf) = 0
        const float m_ref = m == -CUDART_INF_F ? 0.f : m;
        float sum = rsum[qb] * ex2_approx(rmax[qb] - m_ref);
#pragma unroll
        for (int g = 0; g < G - 1; ++g) sum += o[g].y * ex2_approx(o[g].x - m_ref);
        // rows beyond M (padding, or heads of the next group) get a huge L: their weights vanish
        float Lr = r < p.m_rows ? (m + lg2_approx(sum)) / c : 1e30f;
        uint32_t pc[3];
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const __nv_bfloat16 h = __float2bfloat16_rn(Lr);
          Lr -= __bfloat162float(h);
          pc[t] = (uint32_t)__bfloat16_as_ushort(h) ^ 0x8000u;   // negated piece
        }
        reinterpret_cast<uint4*>(sEB)[r] = make_uint4(pc[0] | (pc[1] << 16), pc[2], 0u, 0u);
        reinterpret_cast<uint4*>(sEB)[NQ + r] = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(ext_full);
    // ---- pass B: this thread's key, summed over all query rows (group mean) or over each head's rows ----
    const float inv_hn = 1.0f / (float)p.h_n;
    const bool per_head = p.per_head != 0;
    const int out_heads = per_head ? p.n_kv_heads * p.h_n : p.n_kv_heads;
    float* out = p.scores + ((int64_t)layer * out_heads + (per_head ? p.h_n * j : j)) * p.batch.total_len + tok_base(p.batch, s);
    const int cph = p.window >= 32 ? p.window / 32 : 1;   // 32-column chunks per query head (a window of 16: two heads per chunk)
    // the first pass-B item whose stage belongs to this group
    for (int i = T + ((eg - T % G + G) % G); ok && i < T + Tc; i += G) {
      const int as = i % AS;
      const uint32_t tlane = tquarter + as * AS_COLS;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(acc_full + as, (i / AS) & 1, abort_flag))) break;
      ptx::tc_fence_after();
      const int a = (i - T) * kWinTile + q * 32 + lane;
      float colsum = 0.f, headsum = 0.f;
      // Eq. (2) for one query head: its window rows summed, divided by the distance to the end
      auto write_head = [&](int g, float v) {
        if (g < p.h_n && a < l_c) out[(int64_t)g * p.batch.total_len + a] = p.score_norm == 0 ? v / (float)(l - a) : v;
      };
      auto chunk_b = [&](const uint32_t (&raw)[32], int ch) {
        float lo = 0.f, hi = 0.f;
#pragma unroll
        for (int e = 0; e < 16; ++e) lo += ex2_approx(__uint_as_float(raw[e]) * c);
#pragma unroll
        for (int e = 16; e < 32; ++e) hi += ex2_approx(__uint_as_float(raw[e]) * c);
        colsum += lo + hi;
        if (per_head) {
          if (p.window == 16) {
            write_head(2 * ch, lo);
            write_head(2 * ch + 1, hi);
          } else {
            headsum += lo + hi;
            if ((ch + 1) % cph == 0) {
              write_head(ch / cph, headsum);
              headsum = 0.f;
            }
          }
        }
      };
      if constexpr (QB == 1) {
        // eighteen warps share the register file: one load at a time, the other warps of the scheduler fill in
#pragma unroll 1
        for (int ch = 0; ch < NQ / 32; ++ch) {
          uint32_t raw[32];
          ptx::tmem_ld_32x32(tlane + ch * 32, raw);
          ptx::tmem_ld_wait(raw);
          chunk_b(raw, ch);
        }
      } else {
        // groups of four chunks in straight-line code, the next 32 columns on their way while these are worked on:
        // registers with a load in flight are not carried around a loop edge
#pragma unroll 1
        for (int g = 0; g < NQ / 128; ++g) {
          uint32_t r0[32], r1[32];
          ptx::tmem_ld_32x32(tlane + g * 128, r0);
#pragma unroll
          for (int ch = 0; ch < 4; ch += 2) {
            ptx::tmem_ld_wait(r0);
            ptx::tmem_ld_32x32(tlane + g * 128 + (ch + 1) * 32, r1);
            chunk_b(r0, g * 4 + ch);
            ptx::tmem_ld_wait(r1);
            if (ch + 2 < 4) ptx::tmem_ld_32x32(tlane + g * 128 + (ch + 2) * 32, r0);
            chunk_b(r1, g * 4 + ch + 1);
          }
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(acc_empty + as);
      if (!per_head && a < l_c) {
        float v = colsum * inv_hn;
        if (p.score_norm == 0) v = v / (float)(l - a);
        out[a] = v;
      }
    }
  }
  // teardown: every role ends here, also after a wait that gave up
  __syncwarp();
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicExch(&p.hdr[kHdrStatus], (uint32_t)SPINDLEKV_TIMEOUT);
    __nanosleep(100000);  // let any bulk copy still in flight land before the block retires
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// ---- host -----------------------------------------------------------------------------------------

bool make_tensor_map_bf16(CUtensorMap* map, const spindlekv_tensor& t, const spindlekv_batch& b, int n_heads,
                          int head_dim, int box_rows);
bool make_query_map_bf16(CUtensorMap* map, const spindlekv_tensor& q, const spindlekv_batch& b, int n_q_heads,
                         int head_dim, int window);
bool sim_tc_available();

// Shapes the tensor-core path takes: bf16, window a divisor of 128 (16, 32, 64, 128), at most 256
// query rows per KV head.
bool win_tc_supported(const spindlekv_config& cfg, int dtype) {
  if (dtype != SPINDLEKV_BF16 || !sim_tc_available()) return false;
  const int w = cfg.window;
  if (w != 16 && w != 32 && w != 64 && w != 128) return false;
  if (cfg.n_q_heads < 128 / w) return false;   // the query box spans 128 / w heads
  const int m = (cfg.n_q_heads / cfg.n_kv_heads) * w;
  return m <= 256;
}

template <int D, int QB>
static spindlekv_status launch_one(const CUtensorMap& kmap, const CUtensorMap& qmap, const WinTcParams& p, int units,
                                   cudaStream_t st) {
  using L = WinSmem<D, QB>;
  static PerDeviceOnce once;
  const int dev = PerDeviceOnce::current();
  if (dev < 0) return SPINDLEKV_CUDA;
  if (!once.done[dev]) {
    if (cudaFuncSetAttribute(win_tc_kernel<D, QB>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL) != cudaSuccess)
      return SPINDLEKV_CUDA;
    once.done[dev] = true;
  }
  win_tc_kernel<D, QB><<<units, WinShape<QB>::THREADS, L::TOTAL, st>>>(kmap, qmap, p);
  return SPINDLEKV_OK;
}

spindlekv_status launch_win_tc(const spindlekv_config& cfg, const spindlekv_batch& b, const spindlekv_tensor& K,
                               const spindlekv_tensor& Q, float* scores, uint32_t* hdr, cudaStream_t st) {
  CUtensorMap kmap, qmap;
  if (!make_tensor_map_bf16(&kmap, K, b, cfg.n_kv_heads, cfg.head_dim, kWinTile)) return SPINDLEKV_CUDA;
  if (!make_query_map_bf16(&qmap, Q, b, cfg.n_q_heads, cfg.head_dim, cfg.window)) return SPINDLEKV_CUDA;
  WinTcParams p;
  p.batch = make_batch(b);
  p.n_kv_heads = cfg.n_kv_heads;
  p.h_n = cfg.n_q_heads / cfg.n_kv_heads;
  p.window = cfg.window;
  p.m_rows = p.h_n * cfg.window;
  p.score_norm = cfg.score_norm;
  p.per_head = cfg.per_query_head ? 1 : 0;
  p.c = 1.4426950408889634f / sqrtf((float)cfg.head_dim);
  p.scores = scores;
  p.hdr = hdr;
  const int units = b.n_layers * b.n_seqs * cfg.n_kv_heads;
  const int qb = p.m_rows > 128 ? 2 : 1;
  LaunchScope ls(KC_WINDOW, st);
  spindlekv_status rs;
  if (cfg.head_dim == 128) rs = qb == 2 ? launch_one<128, 2>(kmap, qmap, p, units, st) : launch_one<128, 1>(kmap, qmap, p, units, st);
  else rs = qb == 2 ? launch_one<64, 2>(kmap, qmap, p, units, st) : launch_one<64, 1>(kmap, qmap, p, units, st);
  if (rs != SPINDLEKV_OK) return rs;
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

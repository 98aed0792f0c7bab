// Thresholded cosine similarity (Eq. (4)(9)) on the 5th-generation tensor cores, bf16 inputs.
//
// The adjacency is symmetric, so only pairs (a, b) with a < b are computed and each decision is
// written twice: into row a and, mirrored, into row b.
//
// One CTA owns a block of 128 token rows of one (layer, sequence, head) unit: the block is loaded
// once by TMA and stays in shared memory as operand A; tiles of 256 token rows, from the tile that
// holds the diagonal onwards, stream through a two-stage ring as operand B.  One elected thread
// issues tcgen05.mma (128 x 256 x 16, fp32 accumulation in TMEM) for the raw bf16 dot products.
// Eight epilogue warps read the accumulators back with tcgen05.ld while the tensor cores work on
// the other TMEM stage.  A thread owns one row a; per pair it evaluates
//     x = fma(-dot, rinv_b, theta * |a|)        (rinv = 1/|gamma|, 0 for a zero vector)
// whose sign bit is the decision dot/(|a||b|) > theta, and shifts that bit into a 32-bit word.
// The word goes to row a as is; a 32x32 bit transpose across the warp turns the 32 words of a
// sub-block into the words of the mirrored rows, which are staged in shared memory and written
// 16 bytes per row.  Nothing but bits leaves the SM: N*N/8 bytes per unit.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace skv {

struct SimTcParams {
  Batch batch;
  int n_kv_heads, row_words;
  float theta;
  const float* rinv;   // [units][row_words*32], zero beyond the sequence
  uint32_t* adj;       // [units][max_len][row_words]
  uint32_t* hdr;
};

constexpr int kBM = 128;          // rows of the resident block (UMMA M)
constexpr int kBN = 256;          // rows of a streamed tile (UMMA N)
constexpr int kStages = 2;
constexpr int kEpiWarps = 16;
constexpr int kColsPerWarp = kBN / (kEpiWarps / 4);   // tile columns handled by one epilogue warp
constexpr int kChunks = kColsPerWarp / 32;
constexpr int kEpiThreads = 32 * kEpiWarps;
constexpr int kSimThreads = 32 * (2 + kEpiWarps);

template <int D>
struct SimSmem {
  static constexpr int KH = D / 64;                  // 64-element (128-byte) swizzle atoms along head_dim
  static constexpr int A_BYTES = KH * kBM * 128;
  static constexpr int B_BYTES = KH * kBN * 128;
  static constexpr int RC_BYTES = 2 * kBN * 4;       // inverse norms of the tile's 256 tokens, two slots
  static constexpr int T_BYTES = 2 * 4 * kBN * 4;    // mirrored words [slot][row quarter][tile column]
  static constexpr int USED = A_BYTES + kStages * B_BYTES + RC_BYTES + T_BYTES + 256 /*barriers*/ + 1024 /*alignment*/;
  // at least 120 KB so that two blocks never share an SM: each block allocates all 512 TMEM columns
  static constexpr int TOTAL = USED > 120 * 1024 ? USED : 120 * 1024;
};

// 32x32 bit transpose across a warp: in: lane r holds bits (r, c) at bit c; out: lane c holds bit r
__device__ __forceinline__ uint32_t warp_transpose32(uint32_t x, int lane) {
  uint32_t m = 0x0000FFFFu;
#pragma unroll
  for (int j = 16; j >= 1; j >>= 1) {
    const uint32_t y = __shfl_xor_sync(0xffffffffu, x, j);
    const bool hi = (lane & j) != 0;
    const uint32_t keep = hi ? ~m : m;
    const uint32_t sh = hi ? (y >> j) : (y << j);
    x = (x & keep) | (sh & ~keep);
    m ^= m << (j >> 1);
  }
  return x;
}

// four transposes at once: the shuffles of one stage are independent of each other
__device__ __forceinline__ void warp_transpose32x4(uint32_t (&x)[4], int lane) {
  uint32_t m = 0x0000FFFFu;
#pragma unroll
  for (int j = 16; j >= 1; j >>= 1) {
    const bool hi = (lane & j) != 0;
    const uint32_t keep = hi ? ~m : m;
    uint32_t y[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) y[i] = __shfl_xor_sync(0xffffffffu, x[i], j);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t sh = hi ? (y[i] >> j) : (y[i] << j);
      x[i] = (x[i] & keep) | (sh & ~keep);
    }
    m ^= m << (j >> 1);
  }
}

__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); }

template <int D>
__global__ void __launch_bounds__(kSimThreads, 1) sim_tc_kernel(const __grid_constant__ CUtensorMap tmap, SimTcParams p) {
  using L = SimSmem<D>;
  const int unit = blockIdx.y;
  const int j = unit % p.n_kv_heads;
  const int ls = unit / p.n_kv_heads;
  const int s = ls % p.batch.n_seqs;
  const int layer = ls / p.batch.n_seqs;
  const int l = seq_len(p.batch, s);
  const int row0 = blockIdx.x * kBM;
  if (row0 >= l) return;
  const int n_tiles = (p.row_words * 32 + kBN - 1) / kBN;
  const int tile0 = row0 / kBN;   // the tile that holds this block's diagonal; earlier tiles are mirrored by other blocks

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + L::A_BYTES;
  float* sRC = reinterpret_cast<float*>(smem + L::A_BYTES + kStages * L::B_BYTES);
  uint32_t* sT = reinterpret_cast<uint32_t*>(smem + L::A_BYTES + kStages * L::B_BYTES + L::RC_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::A_BYTES + kStages * L::B_BYTES + L::RC_BYTES + L::T_BYTES);
  uint64_t* a_full = bars + 0;
  uint64_t* b_full = bars + 1;      // [kStages]
  uint64_t* b_empty = bars + 3;     // [kStages]
  uint64_t* acc_full = bars + 5;    // [2]
  uint64_t* acc_empty = bars + 7;   // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 9);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 10);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    ptx::mbar_init(a_full, 1);
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(b_full + i, 1); ptx::mbar_init(b_empty + i, 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(acc_full + i, 1); ptx::mbar_init(acc_empty + i, kEpiWarps); }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int tok0 = p.batch.cu ? p.batch.cu[s] : 0;
  const int sdim = p.batch.cu ? 0 : s;

  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap);
      ptx::mbar_expect_tx(a_full, L::A_BYTES);
      for (int kh = 0; kh < L::KH; ++kh)
        ptx::tma_load_5d(sA + kh * kBM * 128, &tmap, a_full, kh * 64, tok0 + row0, j, sdim, layer);
      for (int it = 0; tile0 + it < n_tiles; ++it) {
        const int st = it & 1;
        if (!ptx::mbar_wait(b_empty + st, ((it >> 1) & 1) ^ 1, abort_flag)) break;
        ptx::mbar_expect_tx(b_full + st, L::B_BYTES);
        uint8_t* dst = sB + st * L::B_BYTES;
        for (int kh = 0; kh < L::KH; ++kh)
          for (int half = 0; half < 2; ++half)
            ptx::tma_load_5d(dst + kh * kBN * 128 + half * 128 * 128, &tmap, b_full + st, kh * 64,
                             tok0 + (tile0 + it) * kBN + half * 128, j, sdim, layer);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(kBM, kBN);
      const uint32_t a_addr = ptx::smem_u32(sA);
      bool ok = ptx::mbar_wait(a_full, 0, abort_flag);
      for (int it = 0; ok && tile0 + it < n_tiles; ++it) {
        const int st = it & 1;
        const uint32_t ph = (it >> 1) & 1;
        if (!ptx::mbar_wait(b_full + st, ph, abort_flag)) break;
        if (!ptx::mbar_wait(acc_empty + st, ph ^ 1, abort_flag)) break;
        ptx::tc_fence_after();
        const uint32_t b_addr = ptx::smem_u32(sB + st * L::B_BYTES);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const int kh = k >> 2, kk = k & 3;
          uint64_t da = ptx::smem_desc_sw128(a_addr + kh * kBM * 128 + kk * 32);
          uint64_t db = ptx::smem_desc_sw128(b_addr + kh * kBN * 128 + kk * 32);
          ptx::umma_bf16(tmem_base + st * kBN, da, db, idesc, k > 0 ? 1u : 0u);
        }
        ptx::umma_commit(b_empty + st);   // shared-memory stage may be refilled
        ptx::umma_commit(acc_full + st);  // accumulator ready for the epilogue
      }
    }
  } else {
    const int q = warp & 3;               // TMEM lane quarter this warp may read
    const int cg = (warp - 2) >> 2;       // which group of kColsPerWarp tile columns
    const int et = threadIdx.x - 64;      // index within the epilogue group
    const int R = row0 + q * 32;          // first row of this warp's 32-row strip
    const int row = R + lane;
    const float* rinv = p.rinv + (int64_t)unit * p.row_words * 32;
    const int ncols = p.row_words * 32;
    // threshold scaled by this row's norm; a zero row has similarity 0 with everything
    float thr;
    {
      const float rr = row < l ? rinv[row] : 0.f;
      thr = rr > 0.f ? p.theta / rr : p.theta;
    }
    uint32_t* adj_unit = p.adj + (int64_t)unit * p.batch.max_len * p.row_words;
    uint32_t* out = adj_unit + (int64_t)row * p.row_words;
    if (et < kBN) {
      const int c = tile0 * kBN + et;
      sRC[et] = c < ncols ? rinv[c] : 0.f;
    }
    epi_bar_sync();
    for (int it = 0; tile0 + it < n_tiles; ++it) {
      const int st = it & 1;
      const int c0 = (tile0 + it) * kBN;
      const bool fast = c0 >= row0 + kBM;      // whole tile strictly above the diagonal
      float rc_next = 0.f;
      if (et < kBN) {
        const int c = c0 + kBN + et;
        if (tile0 + it + 1 < n_tiles && c < ncols) rc_next = __ldg(rinv + c);
      }
      // one lane polls, the warp follows
      int ok = 1;
      if (lane == 0) ok = ptx::mbar_wait(acc_full + st, (it >> 1) & 1, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      ptx::tc_fence_after();
      const float* rcs = sRC + st * kBN + cg * kColsPerWarp;
      const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + st * kBN + cg * kColsPerWarp;
      uint32_t words[kChunks];
#pragma unroll
      for (int ch = 0; ch < kChunks; ++ch) {
        const int col0 = c0 + cg * kColsPerWarp + ch * 32;
        uint32_t acc[32];
        ptx::tmem_ld_32x32(tbase + ch * 32, acc);
        ptx::tmem_ld_wait(acc);
        // four independent 8-bit groups keep the shift chains short
        uint32_t wg[4] = {0, 0, 0, 0};
#pragma unroll
        for (int v = 7; v >= 0; --v) {
          float4 t = *reinterpret_cast<const float4*>(rcs + ch * 32 + v * 4);
          const float rc4[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
          for (int e = 3; e >= 0; --e) {
            const int c = v * 4 + e;
            float x = fmaf(-__uint_as_float(acc[c]), rc4[e], thr);
            wg[c >> 3] = __funnelshift_l(__float_as_uint(x), wg[c >> 3], 1);
          }
        }
        uint32_t w = __byte_perm(__byte_perm(wg[0], wg[1], 0x0040), __byte_perm(wg[2], wg[3], 0x0040), 0x5410);
        const int nvalid = l - col0;  // columns of this word that exist
        if (nvalid < 32) w &= nvalid > 0 ? ((1u << nvalid) - 1u) : 0u;
        if (row >= l) w = 0;
        words[ch] = w;
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(acc_empty + st);
      const int widx = (c0 >> 5) + cg * kChunks;
      if (fast) {
        if (row < l && widx < p.row_words) {
          if (kChunks == 2) *reinterpret_cast<uint2*>(out + widx) = make_uint2(words[0], words[kChunks - 1]);
          else
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch) out[widx + ch] = words[ch];
        }
        uint32_t* tq = sT + (st * 4 + q) * kBN + cg * kColsPerWarp;
#pragma unroll
        for (int ch = 0; ch < kChunks; ++ch) tq[ch * 32 + lane] = warp_transpose32(words[ch], lane);
      } else {
#pragma unroll
        for (int ch = 0; ch < kChunks; ++ch) {
          const int col0 = c0 + cg * kColsPerWarp + ch * 32;
          if (col0 + 32 <= R) continue;                      // below the diagonal: another block mirrors it
          if (col0 == R) {
            // diagonal sub-block: upper triangle as computed, lower triangle mirrored from it, unit diagonal
            const uint32_t upper = lane == 31 ? 0u : (0xFFFFFFFFu << (lane + 1));
            const uint32_t wu = words[ch] & upper;
            const uint32_t wt = warp_transpose32(wu, lane);
            if (row < l) out[widx + ch] = wu | wt | (1u << lane);
          } else {
            if (row < l && widx + ch < p.row_words) out[widx + ch] = words[ch];
            const uint32_t wt = warp_transpose32(words[ch], lane);
            if (col0 + lane < l) adj_unit[(int64_t)(col0 + lane) * p.row_words + (R >> 5)] = wt;
          }
        }
      }
      if (et < kBN) sRC[(st ^ 1) * kBN + et] = rc_next;
      epi_bar_sync();  // mirrored words of this tile and the next tile's inverse norms are in shared memory
      if (fast && et < kBN) {
        const int b = c0 + et;
        if (b < l) {
          const uint32_t* t0 = sT + st * 4 * kBN + et;
          *reinterpret_cast<uint4*>(adj_unit + (int64_t)b * p.row_words + (row0 >> 5)) =
              make_uint4(t0[0], t0[kBN], t0[2 * kBN], t0[3 * kBN]);
        }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 tensor [layer][seq][head][token][d] -> 5-D map (d, token, head, seq, layer), box 64 x 128 rows
bool make_tensor_map_bf16(CUtensorMap* map, const spindlekv_tensor& t, const spindlekv_batch& b, int n_heads,
                          int head_dim, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const bool packed = b.cu_seqlens != nullptr;
  auto bytes = [](int64_t elems) { return (cuuint64_t)(elems > 0 ? elems : 8) * 2; };
  cuuint64_t dims[5] = {(cuuint64_t)head_dim, (cuuint64_t)(packed ? b.total_len : b.max_len), (cuuint64_t)n_heads,
                        (cuuint64_t)(packed ? 1 : b.n_seqs), (cuuint64_t)b.n_layers};
  cuuint64_t strides[4] = {bytes(t.stride_tok), bytes(t.stride_head), bytes(packed ? t.stride_tok : t.stride_seq),
                           bytes(t.stride_layer)};
  for (int i = 1; i < 5; ++i) {
    const int64_t st_el[5] = {1, t.stride_tok, t.stride_head, packed ? t.stride_tok : t.stride_seq, t.stride_layer};
    if (dims[i] > 1 && st_el[i] <= 0) return false;
  }
  cuuint32_t box[5] = {64, (cuuint32_t)box_rows, 1, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, t.ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool sim_tc_available() {
  static int ok = -1;
  if (ok < 0) {
    int dev = 0, major = 0;
    ok = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess && major == 10 &&
        encode_fn() != nullptr)
      ok = 1;
  }
  return ok == 1;
}

spindlekv_status launch_sim_tc(const spindlekv_tensor& Gamma, const spindlekv_batch& b, int n_kv_heads, int head_dim,
                               float theta, const float* rinv, uint32_t* adj, uint32_t* hdr, cudaStream_t st) {
  CUtensorMap map;
  if (!make_tensor_map_bf16(&map, Gamma, b, n_kv_heads, head_dim, 128)) return SPINDLEKV_CUDA;
  SimTcParams p;
  p.batch = make_batch(b);
  p.n_kv_heads = n_kv_heads;
  p.row_words = row_words_for(b.max_len);
  p.theta = theta;
  p.rinv = rinv;
  p.adj = adj;
  p.hdr = hdr;
  const int units = b.n_layers * b.n_seqs * n_kv_heads;
  dim3 grid(ceil_div(b.max_len, kBM), units);
  LaunchScope ls(KC_SIM, st);
  if (head_dim == 128) {
    static bool set = false;
    if (!set) {
      if (cudaFuncSetAttribute(sim_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, SimSmem<128>::TOTAL) != cudaSuccess)
        return SPINDLEKV_CUDA;
      set = true;
    }
    sim_tc_kernel<128><<<grid, kSimThreads, SimSmem<128>::TOTAL, st>>>(map, p);
  } else {
    static bool set = false;
    if (!set) {
      if (cudaFuncSetAttribute(sim_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SimSmem<64>::TOTAL) != cudaSuccess)
        return SPINDLEKV_CUDA;
      set = true;
    }
    sim_tc_kernel<64><<<grid, kSimThreads, SimSmem<64>::TOTAL, st>>>(map, p);
  }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

// Shallow-layer CodeBook construction (Algorithm 1): magnitudes (Eq. (8)), thresholded cosine
// similarity as a bit matrix (Eq. (4)(9)), exact parallel form of the greedy cover (Eq. (10)-(13)),
// and the numbering of the entries.
//
// Greedy cover in parallel.  Algorithm 1 picks one centre per iteration: the live node with the
// largest live degree, lowest index on ties, i.e. the largest key (degree, -index).  A live node whose
// key is the largest among all live nodes within graph distance 2 can be picked at once with its
// current degree and neighbours: a pick elsewhere changes this node's degree only if it lies within
// distance 2, and any such node has a smaller key now and a key that can only fall later, so the
// sequential arg-max reaches this node first.  Every round picks all such nodes together; neighbours
// of two picks of one round cannot coincide (the picks would be within distance 2 of each other).
// Pick-time keys equal those of the sequential run and strictly decrease along it, so entry numbers
// are the ranks of the picks by key.  The result is bit-identical to the one-at-a-time loop.
#include <algorithm>

#include "common.cuh"
#include "simt_tile.cuh"

namespace skv {

struct CodebookParams {
  View G;                // Gamma
  Batch batch;
  int n_kv_heads, n_units, row_words;
  float theta;
  float* mag;            // [layers][H][T]
  __nv_bfloat16* ext;    // [2][units][row_words*32][16]: the extra K-step of the tensor-core similarity
                         // ([0]: theta*|gamma|, [1]: |gamma|, each in three bf16 pieces; zero beyond the sequence)
  uint32_t* adj;         // [units][max_len][row_words]
  int32_t* deg;          // [units][max_len]
  uint32_t* live0;       // [units][row_words] tokens that have a neighbour: live when the greedy cover starts
  int32_t* owner;        // [units][max_len]
  int32_t* pickdeg;      // [units][max_len], -1 = not a centre
  int32_t* rank;         // [units][max_len] entry number of a centre
  int32_t* lists;        // [units][list_cap] neighbour lists, one contiguous run per row, starting at lbase[row]
  int32_t* ell_cnt;      // [units][max_len] list length n <= kEll; -1: use the bit row; -1 - n: a list of n > kEll neighbours
  int32_t* dense_rows;   // [units][max_len] tokens with more than kEll neighbours, in no particular order
  int32_t* dense_cnt;    // [units] how many
  uint32_t* flags;       // [units][row_words][row_words/2] bit r of word [w][c]: chunk c (64 columns) of row 32w+r may hold a bit
  uint32_t* hdr;
  int32_t* ref;          // [layers][H][T]
  int32_t* centre_idx;   // [layers][H][T]
  int32_t* n_entries;    // [layers][B][H]
  // candidate records of the tensor-core similarity kernel and what is built from them
  const uint2* rec;      // [units][unit_rec_cap]
  const int32_t* rec_cnt;   // [units][n_blocks]
  int32_t* ovf;          // [units] != 0: the unit goes through the bit matrix (records did not fit, or no records at all)
  int rec_per_tile, n_blocks;
  long long unit_rec_cap;
  int32_t* lbase;        // [units][max_len] start of a row's list within its unit's part of `lists`
  int list_cap;          // entries per unit (at least kEll per row: the bit-matrix path gives every row kEll slots)
  int round_cap;         // rounds after which the greedy cover gives up
};

__device__ __forceinline__ void cb_decode(const CodebookParams& p, int unit, int& layer, int& s, int& j) {
  j = unit % p.n_kv_heads;
  int ls = unit / p.n_kv_heads;
  s = ls % p.batch.n_seqs;
  layer = ls / p.batch.n_seqs;
}
__device__ __forceinline__ int64_t cb_out_row(const CodebookParams& p, int layer, int s, int j) {
  return ((int64_t)layer * p.n_kv_heads + j) * p.batch.total_len + tok_base(p.batch, s);
}

// ---- Eq. (8): magnitudes.  8 lanes per row of 64 elements, 16 lanes per row of 128. -----------
// x = p0 + p1 + p2 exactly, each piece a bf16 (8 significant bits each, 24 in all)
__device__ __forceinline__ void split3_bf16(float x, __nv_bfloat16 (&pc)[3]) {
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    pc[i] = __float2bfloat16_rn(x);
    x -= __bfloat162float(pc[i]);
  }
}

constexpr int kNormRows = 4;   // rows per thread group: their loads are all in flight before any is used

template <typename T, int D>
__global__ void __launch_bounds__(256) norms_kernel(CodebookParams p) {
  constexpr int LPR = D / 8;  // lanes per row
  constexpr int RPB = 256 / LPR;
  constexpr int ROWS = RPB * kNormRows;   // consecutive rows of one block
  __shared__ float sm_m[ROWS];
  int layer, s, j;
  cb_decode(p, blockIdx.y, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int seg = threadIdx.x % LPR;
  const int block_row0 = blockIdx.x * ROWS;
  const int local_first = threadIdx.x / LPR;
  const T* base = reinterpret_cast<const T*>(p.G.ptr) + unit_offset(p.G, p.batch, layer, s, j) + seg * 8;
  float v[kNormRows][8];
#pragma unroll
  for (int r = 0; r < kNormRows; ++r) {
    const int row = block_row0 + local_first + r * RPB;
    if (row < l) load8(base + (int64_t)row * p.G.st, v[r]);
    else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[r][i] = 0.f;
    }
  }
#pragma unroll
  for (int r = 0; r < kNormRows; ++r) {
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) ss = fmaf(v[r][i], v[r][i], ss);
#pragma unroll
    for (int o = LPR / 2; o >= 1; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if (seg == 0) sm_m[local_first + r * RPB] = sqrtf(ss);
  }
  __syncthreads();
  // magnitudes and operand rows leave in whole lines: consecutive threads, consecutive addresses
  if (threadIdx.x < ROWS && block_row0 + threadIdx.x < l)
    p.mag[cb_out_row(p, layer, s, j) + block_row0 + threadIdx.x] = sm_m[threadIdx.x];
  if (p.ext) {
    // Operand [op] of the extra K-step, row `row`: slots 0..8 hold the pieces so that the nine products of
    // an A row with a B row add up to -theta*|a| * |b|: the similarity kernel negates operand A in every MMA
    // (one instruction descriptor for the whole tile), which turns a.b into -a.b and this into +theta*|a|*|b|.
    // A zero vector takes magnitude 1: its dot products are 0, so the accumulator keeps the sign of theta, as
    // "0 > theta" demands.
    for (int t = threadIdx.x; t < ROWS * 4; t += 256) {
      const int op = t / (ROWS * 2), r = (t % (ROWS * 2)) >> 1, hi = t & 1;
      const int row = block_row0 + r;
      if (row >= p.row_words * 32) continue;
      const float m = sm_m[r];
      const float n = m > 0.f ? m : 1.f;
      __nv_bfloat16 pc[3];
      split3_bf16(op == 0 ? -(p.theta * n) : n, pc);
      __align__(16) __nv_bfloat16 out[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int slot = hi * 8 + i;
        out[i] = (row < l && slot < 9) ? (op == 0 ? pc[slot / 3] : pc[slot % 3]) : __float2bfloat16_rn(0.f);
      }
      uint4* dst = reinterpret_cast<uint4*>(p.ext + (((int64_t)op * p.n_units + blockIdx.y) * p.row_words * 32 + row) * 16);
      dst[hi] = *reinterpret_cast<const uint4*>(out);
    }
  }
}

// ---- Eq. (4)(9) on CUDA cores: 64x64 tiles, decision dot > theta * (|a| * |b|) ------------------
template <typename T, int D>
__global__ void __launch_bounds__(256) sim_simt_kernel(CodebookParams p) {
  __shared__ TileSmem sm;
  int layer, s, j;
  cb_decode(p, blockIdx.z, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int r0 = blockIdx.y * kTile, c0 = blockIdx.x * kTile;
  if (r0 >= l || c0 >= row_words_for(p.batch.max_len) * 32) return;
  const T* base = reinterpret_cast<const T*>(p.G.ptr) + unit_offset(p.G, p.batch, layer, s, j);
  const float* mag = p.mag + cb_out_row(p, layer, s, j);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  uint32_t bits[4] = {0, 0, 0, 0};
  if (c0 < l) {
    float acc[4][4];
    auto row_a = [&](int r) -> const T* { return r0 + r < l ? base + (int64_t)(r0 + r) * p.G.st : nullptr; };
    auto row_b = [&](int r) -> const T* { return c0 + r < l ? base + (int64_t)(c0 + r) * p.G.st : nullptr; };
    dot_tile_64x64<T, D>(sm, row_a, row_b, acc);
    float mr[4], mc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int a = r0 + ty * 4 + i, b = c0 + tx * 4 + i;
      mr[i] = a < l ? mag[a] : 0.f;
      mc[i] = b < l ? mag[b] : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int a = r0 + ty * 4 + i, b = c0 + tx * 4 + c;
        bool on = (a < l && b < l) && (a == b || acc[i][c] > p.theta * (mr[i] * mc[c]));
        bits[i] |= (on ? 1u : 0u) << ((tx & 7) * 4 + c);
      }
  }
  // eight neighbouring threads hold the 32 columns of one word
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int o = 1; o <= 4; o <<= 1) bits[i] |= __shfl_xor_sync(0xffffffffu, bits[i], o);
    int a = r0 + ty * 4 + i;
    if ((tx & 7) == 0 && a < l)
      p.adj[((int64_t)blockIdx.z * p.batch.max_len + a) * p.row_words + (c0 >> 5) + (tx >> 3)] = bits[i];
  }
}

// ---- neighbour lists ------------------------------------------------------------------------------
// One thread per row.  The similarity kernel left one bit per (row, 64-column chunk) that says
// whether the chunk may hold a set bit (a word holds the bits of 32 rows: a warp reads the words of 256
// chunks, eight per lane, and transposes them into per-row occupancy words); only those chunks of the bit
// row are read, several at a time.  Written per row:
// the initial degree (Eq. (10)), and, for rows with at most kEll neighbours (the row itself
// not counted), the ascending list of those neighbours in the row's kEll slots of `lists`.
// Rows with more neighbours keep using their bit row
// and are appended to a list of dense rows.  A token with no neighbour at all is settled here: it is
// a centre with pick degree 1 (Algorithm 1 reaches it with exactly that degree, whenever it does).
constexpr int kEll = 32;
constexpr int kChunkBatch = 8;    // occupied chunks of a row fetched together
constexpr int kFlagGroup = 8;     // flag words fetched together (256 chunks = 16384 columns)

__global__ void __launch_bounds__(256, 5) extract_kernel(CodebookParams p) {
  const int lane = threadIdx.x & 31;
  const int RW = p.row_words, NP = RW * 32, NC = RW >> 1, ML = p.batch.max_len;
  const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // over units x padded rows
  if (g >= (int64_t)p.n_units * NP) return;                           // whole warps: NP is a multiple of 32
  const int unit = (int)(g / NP), u = (int)(g - (int64_t)unit * NP);
  if (!p.ovf[unit]) return;                                           // built from candidate records instead
  if (u == 0) atomicAdd(&p.hdr[kHdrBitUnits], 1u);
  int layer, s, j;
  cb_decode(p, unit, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const bool exists = u < l;
  const int64_t idx = (int64_t)unit * ML + (exists ? u : 0);
  const int own = u >> 6;   // the chunk that holds the token's own bit
  const uint32_t* fl = p.flags + ((int64_t)unit * RW + (u >> 5)) * NC;
  const uint2* row2 = reinterpret_cast<const uint2*>(p.adj + idx * RW);
  int32_t* my_list = p.lists + (int64_t)unit * p.list_cap + (int64_t)(exists ? u : 0) * kEll;   // kEll slots per row
  TransposeLane tr;
  tr.init(lane);
  int cnt = 1, k = 0;
  const int nc = (l + 63) >> 6;   // chunks of this sequence (flags and bit rows beyond it are not written)
  __shared__ uint32_t occ_sh[kFlagGroup][256];   // per thread: occupancy of its row, 32 chunks per word
  for (int cb = 0; cb < nc; cb += 32 * kFlagGroup) {
    uint32_t fw[kFlagGroup];
#pragma unroll
    for (int i = 0; i < kFlagGroup; ++i) {
      const int c = cb + 32 * i + lane;
      fw[i] = c < nc ? fl[c] : 0u;
    }
    // lane c held the flags of chunk cb + 32 i + c for the warp's 32 rows; after the transpose lane r holds
    // the flags of its own row for these 32 chunks
#pragma unroll
    for (int i = 0; i < kFlagGroup; ++i) {
      const uint32_t occ = tr.apply(fw[i]);
      occ_sh[i][threadIdx.x] = exists ? occ : 0u;
    }
    // the row's occupied chunks in ascending order, kChunkBatch at a time across all flag words, loaded
    // before any of them is looked at: a row costs a round trip per batch, not one per flag word
    int wi = 0;
    uint32_t cur = occ_sh[0][threadIdx.x];
    for (;;) {
      int cs[kChunkBatch];
      uint2 av[kChunkBatch];
#pragma unroll
      for (int i = 0; i < kChunkBatch; ++i) {
        while (cur == 0u && wi < kFlagGroup - 1) cur = occ_sh[++wi][threadIdx.x];
        cs[i] = cur ? cb + 32 * wi + __ffs(cur) - 1 : -1;
        cur &= cur - 1;   // 0 stays 0
      }
      if (cs[0] < 0) break;
#pragma unroll
      for (int i = 0; i < kChunkBatch; ++i) av[i] = cs[i] >= 0 ? row2[cs[i]] : make_uint2(0, 0);
#pragma unroll
      for (int i = 0; i < kChunkBatch; ++i) {
        if (cs[i] < 0) continue;
        const uint32_t wd[2] = {av[i].x, av[i].y};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          uint32_t m = wd[q];
          if (cs[i] == own && q == ((u >> 5) & 1)) m &= ~(1u << (u & 31));   // the token itself is not listed
          cnt += __popc(m);
          while (m && k < kEll) {
            const int b = __ffs(m) - 1;
            m &= m - 1;
            my_list[k] = cs[i] * 64 + q * 32 + b;
            ++k;
          }
        }
      }
    }
  }
  bool live = false;
  if (exists) {
    p.deg[idx] = cnt;
    p.ell_cnt[idx] = cnt - 1 <= kEll ? cnt - 1 : -1;
    p.lbase[idx] = u * kEll;
    p.pickdeg[idx] = cnt == 1 ? 1 : -1;   // -1: not a centre (until the greedy cover picks it)
    if (cnt == 1) {
      p.owner[idx] = u;
    } else {
      live = true;
      if (cnt - 1 > kEll) p.dense_rows[(int64_t)unit * ML + atomicAdd(&p.dense_cnt[unit], 1)] = u;
    }
  }
  // all tokens that still have a neighbour start live
  const uint32_t word = __ballot_sync(0xffffffffu, live);
  if (lane == 0) p.live0[(int64_t)unit * RW + (u >> 5)] = word;
}

// ---- neighbour lists from candidate records ------------------------------------------------------
// One block per unit that fitted its record pool.  A record is a non-zero word of the strict upper
// triangle: every set bit is a pair (a, b), a < b, and is entered into both tokens' lists.  First the
// degrees are counted in shared memory (one word per token), then a prefix sum turns the counts into the
// start of every token's list within the unit's part of `lists`, then the pairs are entered, the shared
// word of a token serving as its fill cursor.  The lists of a unit are contiguous and small (two entries
// per pair), so the scattered 4-byte stores of the last step meet in the L2 cache.  The order inside a
// list depends on the order in which the atomics land; nothing downstream depends on it (maxima, counts
// and ownership by the single centre within reach are all independent of it).  Everything else the
// bit-matrix path's extraction pass leaves behind is written here too: degree, live mask, settled
// isolated tokens, the list of rows with more than kEll neighbours (which the greedy kernels walk a warp
// per row).  A unit whose lists do not fit `list_cap` raises its overflow flag and goes through the bit
// matrix instead.
constexpr int kBuildThreads = 1024;

template <typename F>
__device__ __forceinline__ void for_each_record(const CodebookParams& p, int unit, F f) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int T = p.n_blocks >> 1;
  const uint2* pool = p.rec + (long long)unit * p.unit_rec_cap;
  for (int blk = wid; blk < p.n_blocks; blk += kBuildThreads / 32) {
    const int n = p.rec_cnt[(long long)unit * p.n_blocks + blk];
    const uint2* r = pool + rec_region_offset(blk, T, p.rec_per_tile);
    for (int i0 = 0; i0 < n; i0 += 128) {
      uint2 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + k * 32 + lane;
        v[k] = i < n ? r[i] : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (v[k].y) f((int)(v[k].x >> kRecRowShift), (int)(v[k].x & ((1u << kRecRowShift) - 1u)) * 32, v[k].y);
    }
  }
}

__global__ void __launch_bounds__(kBuildThreads) build_lists_kernel(CodebookParams p) {
  extern __shared__ uint32_t cur[];   // [row_words * 32]: degree, then start of the list, then fill cursor
  __shared__ int warp_total[32];
  const int unit = blockIdx.x;
  if (p.ovf[unit]) return;
  int layer, s, j;
  cb_decode(p, unit, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int RW = p.row_words, NP = RW * 32, ML = p.batch.max_len;
  const int64_t row0 = (int64_t)unit * ML;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  for (int u = tid; u < NP; u += kBuildThreads) cur[u] = 0u;
  __syncthreads();
  // Eq. (10) without the token itself: both ends of every pair
  for_each_record(p, unit, [&](int a, int b0, uint32_t bits) {
    atomicAdd(&cur[a], (uint32_t)__popc(bits));
    while (bits) {
      atomicAdd(&cur[b0 + __ffs(bits) - 1], 1u);
      bits &= bits - 1;
    }
  });
  __syncthreads();
  // prefix sum of the degrees: warp w owns the rows [w * seg, (w + 1) * seg) and walks them 32 at a time;
  // first the warps' totals (and the decision whether the lists fit), then the starts and all per-row outputs
  const int seg = ((NP + 1023) / 1024) * 32;   // rows per warp, a multiple of 32
  const int u_end = min((wid + 1) * seg, NP);
  {
    int run = 0;
    for (int u0 = wid * seg; u0 < u_end; u0 += 32) run += (int)cur[u0 + lane];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) run += __shfl_xor_sync(0xffffffffu, run, o);
    if (lane == 0) warp_total[wid] = run;
  }
  __syncthreads();
  int run = 0, total = 0;
  for (int w = 0; w < 32; ++w) {
    const int t = warp_total[w];
    if (w < wid) run += t;
    total += t;
  }
  if (total > p.list_cap) {            // the same decision in every thread
    if (tid == 0) p.ovf[unit] = 1;
    return;
  }
  if (tid == 0) atomicAdd(&p.hdr[kHdrListEntries], (uint32_t)total);
  for (int u0 = wid * seg; u0 < u_end; u0 += 32) {
    const int u = u0 + lane;
    const bool exists = u < l;
    const int d = (int)cur[u];         // 0 beyond the sequence
    int inc = d;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += n;
    }
    const int start = run + inc - d;
    run += __shfl_sync(0xffffffffu, inc, 31);
    cur[u] = (uint32_t)start;
    const int64_t idx = row0 + u;
    if (exists) {
      const int cnt = d + 1;
      p.deg[idx] = cnt;
      p.ell_cnt[idx] = d <= kEll ? d : -1 - d;
      p.lbase[idx] = start;
      p.pickdeg[idx] = cnt == 1 ? 1 : -1;   // a token without a neighbour is a centre of pick degree 1
      if (cnt == 1) p.owner[idx] = u;
      if (d > kEll) p.dense_rows[row0 + atomicAdd(&p.dense_cnt[unit], 1)] = u;
    }
    const uint32_t word = __ballot_sync(0xffffffffu, exists && d > 0);   // tokens with a neighbour start live
    if (lane == 0) p.live0[(int64_t)unit * RW + (u0 >> 5)] = word;
  }
  __syncthreads();
  int32_t* lists = p.lists + (int64_t)unit * p.list_cap;
  for_each_record(p, unit, [&](int a, int b0, uint32_t bits) {
    uint32_t at_a = atomicAdd(&cur[a], (uint32_t)__popc(bits));
    while (bits) {
      const int b = b0 + __ffs(bits) - 1;
      bits &= bits - 1;
      lists[at_a++] = b;
      lists[atomicAdd(&cur[b], 1u)] = a;
    }
  });
}

// The units whose overflow flag is set, in ascending order, for the bit-matrix pass of the similarity kernel.
__global__ void __launch_bounds__(1024) list_overflowed_kernel(const int32_t* ovf, int n_units, int32_t* work_list, int32_t* n_work) {
  __shared__ int warp_sums[33];
  int base = 0;
  for (int u0 = 0; u0 < n_units; u0 += 1024) {
    const int u = u0 + threadIdx.x;
    const int flag = (u < n_units && ovf[u]) ? 1 : 0;
    int total;
    const int at = block_exclusive_scan(flag, warp_sums, total);
    if (flag) work_list[base + at] = u;
    base += total;
  }
  if (threadIdx.x == 0) *n_work = base;
}

// Flag words of the units that go through the bit matrix start at zero (the similarity kernel writes only
// the words that hold a set bit).
__global__ void __launch_bounds__(256) clear_flags_kernel(CodebookParams p) {
  const int unit = blockIdx.y;
  if (!p.ovf[unit]) return;
  const int64_t n = (int64_t)(p.row_words >> 1) * p.row_words;
  uint32_t* f = p.flags + (int64_t)unit * n;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) f[i] = 0u;
}

// The adjacency bit matrix of the units that were built from records, for callers that ask for it: unit
// diagonal, every recorded pair and its mirror image.  The caller has cleared the matrix.
__global__ void __launch_bounds__(kBuildThreads) expand_records_kernel(CodebookParams p, uint32_t* adj) {
  const int unit = blockIdx.x;
  if (p.ovf[unit]) return;
  int layer, s, j;
  cb_decode(p, unit, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int RW = p.row_words;
  uint32_t* a_unit = adj + (int64_t)unit * p.batch.max_len * RW;
  for (int u = threadIdx.x; u < l; u += kBuildThreads) atomicOr(&a_unit[(int64_t)u * RW + (u >> 5)], 1u << (u & 31));
  for_each_record(p, unit, [&](int a, int b0, uint32_t bits) {
    atomicOr(&a_unit[(int64_t)a * RW + (b0 >> 5)], bits);
    while (bits) {
      const int b = b0 + __ffs(bits) - 1;
      bits &= bits - 1;
      atomicOr(&a_unit[(int64_t)b * RW + (a >> 5)], 1u << (a & 31));
    }
  });
}

// ---- greedy cover: one block per unit, its state on chip ----------------------------------------------
// Units are independent graphs, so a block runs all rounds of its unit with block barriers between the three
// phases of a round and stops as soon as the unit has no live token left, whatever the other units still do.
// What the phases gather from at random sits in shared memory: the two live masks, the key of every token
// (live degree in the high half, 0xFFFF - index in the low half: larger degree first, lower index on ties) and,
// per token, the index of the largest key in its closed live neighbourhood.  What stays in global memory is
// read once per row and phase: the row's list (or, on the bit-matrix path, its bit row).
//
// Round 0 finds every token with a neighbour live and its degree known from the list building; the rounds after
// it first collect the tokens that are left into a list (as a rule a few per cent) and work on that list, one
// thread per token, instead of sweeping the live mask.  Rows with more than kEll neighbours are taken a warp
// per row from the unit's list of such rows.
__device__ __forceinline__ bool is_live(const uint32_t* lv, int v) { return (lv[v >> 5] >> (v & 31)) & 1u; }

// The flag words of token u's group of 32 rows, one per 64-column chunk.  A chunk of a bit row whose flag bit is
// clear holds no set bit and may never have been written: readers of whole bit rows skip it.
__device__ __forceinline__ const uint32_t* flag_row(const CodebookParams& p, int unit, int u) {
  return p.flags + ((int64_t)unit * p.row_words + (u >> 5)) * (p.row_words >> 1);
}
__device__ __forceinline__ bool chunk_flagged(const uint32_t* fr, int chunk, int u) { return (fr[chunk] >> (u & 31)) & 1u; }

// Eight entries of a row's neighbour list at a time: the loads of one batch do not depend on each
// other, so a row costs a few memory round trips instead of one per neighbour.
constexpr int kBatch = 8;
__device__ __forceinline__ void load_batch(const int32_t* list, int k0, int ec, int (&v)[kBatch]) {
#pragma unroll
  for (int i = 0; i < kBatch; ++i) v[i] = k0 + i < ec ? list[k0 + i] : -1;
}
// keeps only the entries that are live (others become -1)
__device__ __forceinline__ void keep_live(const uint32_t* lv, int (&v)[kBatch]) {
#pragma unroll
  for (int i = 0; i < kBatch; ++i)
    if (v[i] >= 0 && !is_live(lv, v[i])) v[i] = -1;
}

struct CoverState {        // shared memory of one unit's block
  uint32_t* key;           // [tokens] (live degree << 16) | (0xFFFF - token)
  uint16_t* best;          // [tokens] token with the largest key in the closed live neighbourhood
  uint32_t* live0;         // [row_words] live masks: rounds alternate between the two
  uint32_t* live1;
  uint16_t* left;          // [kLeftCap] tokens still live at the start of a round
};
constexpr int kLeftCap = 4096;
constexpr int kCoverMaxTokens = 32768;   // 16-bit token numbers, and 6 bytes of shared memory per token

__device__ __forceinline__ uint32_t make_key(int cnt, int u) { return ((uint32_t)cnt << 16) | (uint32_t)(0xFFFF - u); }
__device__ __forceinline__ int key_token(uint32_t k) { return 0xFFFF - (int)(k & 0xFFFFu); }

// ---- rows with a list of at most kEll neighbours, one thread per row --------------------------------
// phase 1: live degree (Eq. (10)) and key
__device__ __forceinline__ void degree_of_row(const CodebookParams& p, const CoverState& st, const uint32_t* lv, int64_t row0, int u) {
  const int ec = p.ell_cnt[row0 + u];
  if (ec < 0) return;                             // rows with many neighbours: separately
  const int32_t* list = p.lists + p.lbase[row0 + u];
  int cnt = 1;
  for (int k0 = 0; k0 < ec; k0 += kBatch) {
    int v[kBatch];
    load_batch(list, k0, ec, v);
    keep_live(lv, v);
#pragma unroll
    for (int i = 0; i < kBatch; ++i) cnt += v[i] >= 0 ? 1 : 0;
  }
  st.key[u] = make_key(cnt, u);
}

// phase 2: largest key in the closed live neighbourhood.  `kAllLive`: every listed neighbour is known to be live
// (round 0: a token with a neighbour is live).
template <bool kAllLive>
__device__ __forceinline__ void best_of_row(const CodebookParams& p, const CoverState& st, const uint32_t* lv, int64_t row0, int u) {
  const int ec = p.ell_cnt[row0 + u];
  if (ec < 0) return;
  const int32_t* list = p.lists + p.lbase[row0 + u];
  uint32_t best = st.key[u];                      // the token itself belongs to its closed neighbourhood
  for (int k0 = 0; k0 < ec; k0 += kBatch) {
    int v[kBatch];
    load_batch(list, k0, ec, v);
    if (!kAllLive) keep_live(lv, v);
#pragma unroll
    for (int i = 0; i < kBatch; ++i) best = max(best, v[i] >= 0 ? st.key[v[i]] : 0u);
  }
  st.best[u] = (uint16_t)key_token(best);
}

// phase 3: a token that is the maximum of every live neighbour's neighbourhood is a centre (Eq. (11)); its live
// neighbours take it as owner (Eq. (12)) and leave the graph (Eq. (13))
template <bool kAllLive>
__device__ __forceinline__ void pick_row(const CodebookParams& p, const CoverState& st, const uint32_t* lv, uint32_t* nx, int64_t row0,
                                         int u) {
  const int ec = p.ell_cnt[row0 + u];
  if (ec < 0) return;
  if (st.best[u] != (uint16_t)u) return;
  const int32_t* list = p.lists + p.lbase[row0 + u];
  bool ok = true;
  for (int k0 = 0; k0 < ec && ok; k0 += kBatch) {
    int v[kBatch];
    load_batch(list, k0, ec, v);
    if (!kAllLive) keep_live(lv, v);
#pragma unroll
    for (int i = 0; i < kBatch; ++i) ok = ok && (v[i] < 0 || st.best[v[i]] == (uint16_t)u);
  }
  if (!ok) return;
  int32_t* owner = p.owner + row0;
  for (int k0 = 0; k0 < ec; k0 += kBatch) {
    int v[kBatch];
    load_batch(list, k0, ec, v);
    if (!kAllLive) keep_live(lv, v);
#pragma unroll
    for (int i = 0; i < kBatch; ++i)
      if (v[i] >= 0) {
        owner[v[i]] = u;
        atomicAnd(&nx[v[i] >> 5], ~(1u << (v[i] & 31)));
      }
  }
  p.pickdeg[row0 + u] = (int)(st.key[u] >> 16);
  owner[u] = u;
  atomicAnd(&nx[u >> 5], ~(1u << (u & 31)));
}

// ---- rows with more than kEll neighbours, one warp per row: the neighbours come from the row's list (record
// path, ell_cnt = -1 - n) or from its bit row masked by the occupancy flags (bit-matrix path, ell_cnt = -1) ----
template <typename F>
__device__ __forceinline__ void for_each_live_neighbour(const CodebookParams& p, const uint32_t* lv, int unit, int64_t row0, int u,
                                                        int lane, F f) {
  const int ec = p.ell_cnt[row0 + u];
  if (ec == -1) {
    const int RW = p.row_words;
    const uint32_t* row = p.adj + (row0 + u) * RW;
    const uint32_t* fr = flag_row(p, unit, u);
    for (int w = lane; w < RW; w += 32) {
      uint32_t m = chunk_flagged(fr, w >> 1, u) ? row[w] & lv[w] : 0u;
      while (m) {
        const int b = __ffs(m) - 1;
        m &= m - 1;
        if (w * 32 + b != u) f(w * 32 + b);
      }
    }
  } else {
    const int n = -1 - ec;
    const int32_t* list = p.lists + p.lbase[row0 + u];
    for (int k = lane; k < n; k += 32) {
      const int v = list[k];
      if (is_live(lv, v)) f(v);
    }
  }
}

__device__ __forceinline__ void degree_of_big_row(const CodebookParams& p, const CoverState& st, const uint32_t* lv, int unit,
                                                  int64_t row0, int u, int lane) {
  if (!is_live(lv, u)) return;
  int cnt = 0;
  for_each_live_neighbour(p, lv, unit, row0, u, lane, [&](int) { ++cnt; });
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if (lane == 0) st.key[u] = make_key(cnt + 1, u);
}

__device__ __forceinline__ void best_of_big_row(const CodebookParams& p, const CoverState& st, const uint32_t* lv, int unit,
                                                int64_t row0, int u, int lane) {
  if (!is_live(lv, u)) return;
  uint32_t best = lane == 0 ? st.key[u] : 0u;
  for_each_live_neighbour(p, lv, unit, row0, u, lane, [&](int v) { best = max(best, st.key[v]); });
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, o));
  if (lane == 0) st.best[u] = (uint16_t)key_token(best);
}

__device__ __forceinline__ void pick_big_row(const CodebookParams& p, const CoverState& st, const uint32_t* lv, uint32_t* nx, int unit,
                                             int64_t row0, int u, int lane) {
  if (!is_live(lv, u)) return;
  if (st.best[u] != (uint16_t)u) return;
  bool ok = true;
  for_each_live_neighbour(p, lv, unit, row0, u, lane, [&](int v) { ok = ok && st.best[v] == (uint16_t)u; });
  if (!__all_sync(0xffffffffu, ok)) return;
  int32_t* owner = p.owner + row0;
  for_each_live_neighbour(p, lv, unit, row0, u, lane, [&](int v) {
    owner[v] = u;
    atomicAnd(&nx[v >> 5], ~(1u << (v & 31)));
  });
  if (lane == 0) {
    p.pickdeg[row0 + u] = (int)(st.key[u] >> 16);
    owner[u] = u;
    atomicAnd(&nx[u >> 5], ~(1u << (u & 31)));
  }
}

constexpr int kCoverThreads = 1024;

__global__ void __launch_bounds__(kCoverThreads) cover_kernel(CodebookParams p) {
  extern __shared__ uint32_t cover_sm[];
  __shared__ int n_left;
  const int unit = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  constexpr int NW = kCoverThreads / 32;
  const int ML = p.batch.max_len, RW = p.row_words, NP = RW * 32;
  const int64_t row0 = (int64_t)unit * ML;
  CoverState st;
  st.key = cover_sm;
  st.live0 = st.key + NP;
  st.live1 = st.live0 + RW;
  st.best = reinterpret_cast<uint16_t*>(st.live1 + RW);
  st.left = st.best + NP;
  {
    int layer, s, j;
    cb_decode(p, unit, layer, s, j);
    const int l = seq_len(p.batch, layer, s, j);
    for (int u = tid; u < NP; u += kCoverThreads) st.key[u] = make_key(u < l ? p.deg[row0 + u] : 0, u);
    for (int w = tid; w < RW; w += kCoverThreads) st.live0[w] = st.live1[w] = p.live0[(int64_t)unit * RW + w];
  }
  // the lists of this unit are addressed from the unit's part of the list buffer
  p.lists += (int64_t)unit * p.list_cap;
  const int32_t* big = p.dense_rows + row0;
  const int n_big = p.dense_cnt[unit];
  const int round_cap = min(ML, p.round_cap);
  __syncthreads();
  int round = 0;
  bool gave_up = false;
  for (;; ++round) {
    const uint32_t* lv = (round & 1) ? st.live1 : st.live0;
    uint32_t* nx = (round & 1) ? st.live0 : st.live1;
    bool listed = false;                 // the live tokens of this round are in st.left
    if (round > 0) {
      if (round > round_cap) { gave_up = true; break; }
      // phase 1: `next` becomes a copy of `live`; the tokens that are left, their number, their live degrees
      if (tid == 0) n_left = 0;
      __syncthreads();
      for (int w = wid; w < RW; w += NW) {
        const uint32_t lvw = lv[w];
        if (lane == 0) nx[w] = lvw;
        if (!lvw) continue;
        int at = 0;
        if (lane == 0) at = atomicAdd(&n_left, __popc(lvw));
        at = __shfl_sync(0xffffffffu, at, 0) + __popc(lvw & ((1u << lane) - 1u));
        if (((lvw >> lane) & 1u) && at < kLeftCap) st.left[at] = (uint16_t)(w * 32 + lane);
      }
      __syncthreads();
      const int nl = n_left;
      if (nl == 0) break;
      listed = nl <= kLeftCap;
      if (listed) {
        for (int i = tid; i < nl; i += kCoverThreads) degree_of_row(p, st, lv, row0, st.left[i]);
      } else {
        for (int w = wid; w < RW; w += NW)
          if ((lv[w] >> lane) & 1u) degree_of_row(p, st, lv, row0, w * 32 + lane);
      }
      for (int d = wid; d < n_big; d += NW) degree_of_big_row(p, st, lv, unit, row0, big[d], lane);
      __syncthreads();
    }
    // phase 2: largest key in each closed live neighbourhood
    if (round == 0) {
      for (int w = wid; w < RW; w += NW)
        if ((lv[w] >> lane) & 1u) best_of_row<true>(p, st, lv, row0, w * 32 + lane);
    } else if (listed) {
      for (int i = tid; i < n_left; i += kCoverThreads) best_of_row<false>(p, st, lv, row0, st.left[i]);
    } else {
      for (int w = wid; w < RW; w += NW)
        if ((lv[w] >> lane) & 1u) best_of_row<false>(p, st, lv, row0, w * 32 + lane);
    }
    for (int d = wid; d < n_big; d += NW) best_of_big_row(p, st, lv, unit, row0, big[d], lane);
    __syncthreads();
    // phase 3: picks
    if (round == 0) {
      for (int w = wid; w < RW; w += NW)
        if ((lv[w] >> lane) & 1u) pick_row<true>(p, st, lv, nx, row0, w * 32 + lane);
    } else if (listed) {
      for (int i = tid; i < n_left; i += kCoverThreads) pick_row<false>(p, st, lv, nx, row0, st.left[i]);
    } else {
      for (int w = wid; w < RW; w += NW)
        if ((lv[w] >> lane) & 1u) pick_row<false>(p, st, lv, nx, row0, w * 32 + lane);
    }
    for (int d = wid; d < n_big; d += NW) pick_big_row(p, st, lv, nx, unit, row0, big[d], lane);
    __syncthreads();
  }
  if (tid == 0) {
    atomicMax(&p.hdr[kHdrRounds], (uint32_t)round);
    if (gave_up) {
      // the round that was not run: its live tokens are the ones left without a centre
      const uint32_t* lv = (round & 1) ? st.live1 : st.live0;
      uint32_t left = 0;
      for (int w = 0; w < RW; ++w) left += __popc(lv[w]);
      atomicAdd(&p.hdr[kHdrLive], max(left, 1u));
      atomicExch(&p.hdr[kHdrStatus], (uint32_t)SPINDLEKV_TIMEOUT);
    }
  }
}

static size_t cover_smem_bytes(int row_words) {
  const size_t NP = (size_t)row_words * 32;
  return NP * 4 + 2 * (size_t)row_words * 4 + NP * 2 + kLeftCap * 2;
}

// ---- entry numbering ------------------------------------------------------------------------------
// One block per unit.  Entries are numbered by decreasing pick-time key (degree, then lower index):
// a counting sort on the degree, stable in the index.  hist[] lives in dynamic shared memory.
// Centres of degree 1 are placed by all threads (ballots and a block scan); centres of larger degree by
// one warp that walks, in index order, only the 32-token chunks that hold one.
constexpr int kFinalThreads = 512;     // two blocks fit an SM: the K and the V call of a pass run side by side
constexpr int kFinalWarps = kFinalThreads / 32;
constexpr int kFinalBatch = 16;        // tokens per thread loaded together
constexpr int kFinalChunkWords = 64;   // chunk map for 64 * 32 * 32 = 65536 tokens (longer sequences: every chunk is visited)

__global__ void __launch_bounds__(kFinalThreads, 2) finalize_kernel(CodebookParams p) {
  extern __shared__ int hist[];  // [l + 2]
  __shared__ int warp_sums[33];
  __shared__ uint32_t busy[kFinalChunkWords];   // bit per 32-token chunk: holds a centre of pick degree >= 2
  __shared__ uint16_t busy_list[kFinalChunkWords * 32];
  __shared__ int cnt_sh[kFinalBatch * kFinalWarps];
  static_assert(kFinalBatch * kFinalWarps <= kFinalThreads, "one thread per count in the scan");
  const int unit = blockIdx.x;
  int layer, s, j;
  cb_decode(p, unit, layer, s, j);
  const int l = seq_len(p.batch, layer, s, j);
  const int ML = p.batch.max_len;
  const int32_t* pickdeg = p.pickdeg + (int64_t)unit * ML;
  const int32_t* owner = p.owner + (int64_t)unit * ML;
  int32_t* rank = p.rank + (int64_t)unit * ML;
  const int64_t orow = cb_out_row(p, layer, s, j);
  const int tid = threadIdx.x, lane = tid & 31;

  for (int d = tid; d <= l + 1; d += kFinalThreads) hist[d] = 0;
  for (int c = tid; c < kFinalChunkWords; c += kFinalThreads) busy[c] = 0u;
  __syncthreads();
  // centres of pick degree 1 (tokens without a neighbour, as a rule the bulk) are counted by ballot: one
  // atomic per warp instead of 32 on one address.  A thread's kFinalBatch tokens are loaded before any is used.
  for (int base0 = 0; base0 < l; base0 += kFinalBatch * kFinalThreads) {
    int dr[kFinalBatch];
#pragma unroll
    for (int i = 0; i < kFinalBatch; ++i) {
      const int u = base0 + i * kFinalThreads + tid;
      dr[i] = u < l ? pickdeg[u] : -1;
    }
    int n_ones = 0;
#pragma unroll
    for (int i = 0; i < kFinalBatch; ++i) {
      const int u = base0 + i * kFinalThreads + tid;
      n_ones += __popc(__ballot_sync(0xffffffffu, dr[i] == 1));
      if (dr[i] >= 2) atomicAdd(&hist[dr[i]], 1);
      // 32-token chunks that hold a centre of degree >= 2: the only ones the ordered sweep below visits
      const uint32_t more = __ballot_sync(0xffffffffu, dr[i] >= 2);
      if (lane == 0 && more && (u >> 5) < kFinalChunkWords * 32) atomicOr(&busy[u >> 10], 1u << ((u >> 5) & 31));
    }
    if (lane == 0 && n_ones) atomicAdd(&hist[1], n_ones);
  }
  __syncthreads();
  // start[d] = number of centres with a larger degree: exclusive scan from the top, in place; a thread owns
  // `nb` consecutive degrees
  int n_entries;
  {
    const int nb = (l + 1 + kFinalThreads - 1) / kFinalThreads;
    const int hi = l - tid * nb;
    int sum = 0;
    for (int i = 0; i < nb; ++i) {
      const int d = hi - i;
      if (d >= 0) sum += hist[d];
    }
    int run = block_exclusive_scan(sum, warp_sums, n_entries);
    for (int i = 0; i < nb; ++i) {
      const int d = hi - i;
      if (d >= 0) {
        const int v = hist[d];
        hist[d] = run;
        run += v;
      }
    }
    __syncthreads();
  }
  // degree 1, stable in the index: position = start[1] + number of such centres before the token
  {
    int before = hist[1];
    for (int base0 = 0; base0 < l; base0 += kFinalBatch * kFinalThreads) {
      uint32_t ones[kFinalBatch];
      int dr[kFinalBatch];
#pragma unroll
      for (int i = 0; i < kFinalBatch; ++i) {
        const int u = base0 + i * kFinalThreads + tid;
        dr[i] = u < l ? pickdeg[u] : -1;
      }
#pragma unroll
      for (int i = 0; i < kFinalBatch; ++i) {
        ones[i] = __ballot_sync(0xffffffffu, dr[i] == 1);
        if (lane == 0) cnt_sh[i * kFinalWarps + (tid >> 5)] = __popc(ones[i]);   // in token order: sweep i, warp w
      }
      __syncthreads();
      int tot;
      {
        // exclusive scan of the kFinalBatch * kFinalWarps counts (threads beyond them count 0)
        const int v = tid < kFinalBatch * kFinalWarps ? cnt_sh[tid] : 0;
        const int ex = block_exclusive_scan(v, warp_sums, tot);
        if (tid < kFinalBatch * kFinalWarps) cnt_sh[tid] = ex;
        __syncthreads();
      }
#pragma unroll
      for (int i = 0; i < kFinalBatch; ++i) {
        if (dr[i] == 1) {
          const int u = base0 + i * kFinalThreads + tid;
          const int pos = before + cnt_sh[i * kFinalWarps + (tid >> 5)] + __popc(ones[i] & ((1u << lane) - 1u));
          rank[u] = pos;
          p.centre_idx[orow + pos] = u;
        }
      }
      before += tot;
      __syncthreads();
    }
  }
  // larger degrees: stable placement in index order by one warp over the chunks that hold such a centre,
  // eight chunks in flight
  if (tid < 32) {
    const int n_chunks = (l + 31) >> 5;
    // ascending list of those chunks (beyond the map every chunk is listed by its number at once)
    int n_busy = 0;
    for (int cw0 = 0; cw0 < kFinalChunkWords; cw0 += 32) {
      uint32_t wd = busy[cw0 + lane];
      const int c = __popc(wd);
      int inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      int at = n_busy + inc - c;
      while (wd) {
        busy_list[at++] = (uint16_t)((cw0 + lane) * 32 + __ffs(wd) - 1);
        wd &= wd - 1;
      }
      n_busy += __shfl_sync(0xffffffffu, inc, 31);
    }
    __syncwarp();
    const int extra0 = kFinalChunkWords * 32;   // first chunk that the map does not cover
    const int n_items = n_busy + (n_chunks > extra0 ? n_chunks - extra0 : 0);
    for (int i0 = 0; i0 < n_items; i0 += 8) {
      int cv[8], dv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int it = i0 + i;
        cv[i] = it < n_busy ? (int)busy_list[it] : (it < n_items ? extra0 + (it - n_busy) : -1);
        const int u = cv[i] * 32 + lane;
        dv[i] = (cv[i] >= 0 && u < l) ? pickdeg[u] : -1;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (cv[i] < 0) break;
        const int u = cv[i] * 32 + lane;
        const int d = dv[i] >= 2 ? dv[i] : -1;   // others share one value: the match costs a step per distinct value
        const uint32_t peers = __match_any_sync(0xffffffffu, d);
        if (d >= 2) {
          const int pos = hist[d] + __popc(peers & ((1u << lane) - 1u));
          rank[u] = pos;
          p.centre_idx[orow + pos] = u;
        }
        __syncwarp();
        if (d >= 2 && lane == (31 - __clz(peers))) hist[d] += __popc(peers);
        __syncwarp();
      }
    }
  }
  __syncthreads();
  // rank[] was written by this block: make the writes visible to all of its threads, then resolve the references
  // (eight independent owner -> rank chains per thread)
  for (int b0 = tid; b0 < l; b0 += 8 * kFinalThreads) {
    int o[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int b = b0 + i * kFinalThreads;
      o[i] = b < l ? owner[b] : -1;
    }
    int r[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = (o[i] >= 0 && o[i] < l) ? rank[o[i]] : 0;   // a cover that was cut short leaves owners unset
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int b = b0 + i * kFinalThreads;
      if (b < l) p.ref[orow + b] = r[i];
    }
  }
  if (tid == 0) p.n_entries[(layer * p.batch.n_seqs + s) * p.n_kv_heads + j] = n_entries;
}

// ---- host side ----------------------------------------------------------------------------------

struct CodebookLayout {
  size_t ext, ell, ell_cnt, dense_rows, flags, adj, deg, live0, owner, pickdeg, rank, total;
  size_t ovf, rec_cnt, dense_cnt, work_list, lbase, rec;   // candidate records (tensor-core path)
  int rec_per_tile, n_blocks, list_cap;
};

// Neighbour-list entries per unit: the bit-matrix path gives every row kEll slots; the record path may spend
// twice that on the whole unit, however the entries are spread over the rows.
static int list_capacity(int max_len) { return 2 * kEll * max_len; }
// The record path counts degrees in one 32-bit word per token in shared memory.
static bool record_path_fits(int max_len) { return row_words_for(max_len) * 32 <= 49152; }

static CodebookLayout codebook_layout(const spindlekv_config& cfg, const spindlekv_batch& b, bool adj_in_ws, int rec_per_tile) {
  size_t units = (size_t)b.n_layers * b.n_seqs * cfg.n_kv_heads;
  size_t ML = b.max_len, RW = row_words_for(b.max_len);
  CodebookLayout L;
  size_t off = kHeaderBytes;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
  L.deg = take(units * ML * 4);
  L.live0 = take(units * RW * 4);
  L.owner = take(units * ML * 4);
  L.pickdeg = take(units * ML * 4);
  L.rank = take(units * ML * 4);
  L.ext = take(2 * units * RW * 32 * 16 * 2);
  L.list_cap = list_capacity(b.max_len);
  L.ell = take(units * (size_t)L.list_cap * 4);
  L.ell_cnt = take(units * ML * 4);
  L.dense_rows = take(units * ML * 4);
  L.flags = take(units * (RW / 2) * RW * 4);
  // candidate records: the overflow flags and the per-block counts sit side by side (one clearing pass)
  L.rec_per_tile = record_path_fits(b.max_len) ? rec_per_tile : 0;
  L.n_blocks = 2 * ceil_div(b.max_len, 256);
  L.ovf = take(units * 4);
  L.rec_cnt = take(units * L.n_blocks * 4);
  L.dense_cnt = take(units * 4);
  L.work_list = take((units + 1) * 4);
  L.lbase = take(units * ML * 4);
  L.rec = take(L.rec_per_tile ? units * (size_t)rec_unit_capacity(L.n_blocks / 2, L.rec_per_tile) * 8 : 0);
  L.adj = off;
  if (adj_in_ws) take(units * ML * RW * 4);
  L.total = off;
  return L;
}

size_t codebook_workspace_bytes(const spindlekv_config& cfg, const spindlekv_batch& b) {
  // sized for the default record pool; tuning can only make the pool of a call smaller
  return codebook_layout(cfg, b, true, kDefaultRecPerTile).total;
}

bool sim_tc_available();
spindlekv_status launch_sim_tc(const spindlekv_tensor& Gamma, const spindlekv_batch& b, int n_kv_heads, int head_dim,
                               const void* ext, uint32_t* adj, uint32_t* flags, uint32_t* hdr, bool skip_empty,
                               const SimRecordPool* pool, bool emit, long long wait_cycles, cudaStream_t st);

template <typename T, int D>
static void launch_norms(const CodebookParams& p, cudaStream_t st) {
  constexpr int RPB = 256 / (D / 8);
  LaunchScope ls(KC_NORMS, st);
  norms_kernel<T, D><<<dim3(ceil_div(p.row_words * 32, RPB * kNormRows), p.n_units), 256, 0, st>>>(p);
}

template <typename T, int D>
static void launch_sim_simt(const CodebookParams& p, const spindlekv_batch& b, cudaStream_t st) {
  int ct = ceil_div(p.row_words * 32, kTile), rt = ceil_div(b.max_len, kTile);
  { LaunchScope ls(KC_SIM, st); sim_simt_kernel<T, D><<<dim3(ct, rt, p.n_units), 256, 0, st>>>(p); }
}

spindlekv_status codebook_shallow_impl(const spindlekv_config& cfg, const spindlekv_batch& b,
                                       const spindlekv_tensor& Gamma, float theta, float* mag, int32_t* ref,
                                       int32_t* centre_idx, int32_t* n_entries, uint32_t* adj_bits, void* ws,
                                       size_t ws_bytes, cudaStream_t st) {
  const bool adj_in_ws = adj_bits == nullptr;
  const Tuning tune = current_tuning();
  const bool bf = Gamma.dtype == SPINDLEKV_BF16;
  const bool tc = bf && sim_tc_available();   // bf16: tensor-core similarity (TMA + tcgen05)
  CodebookLayout L = codebook_layout(cfg, b, adj_in_ws, tc ? min(tune.rec_per_tile, kDefaultRecPerTile) : 0);
  if (ws_bytes < L.total) return SPINDLEKV_WORKSPACE_TOO_SMALL;
  if (row_words_for(b.max_len) * 32 > kCoverMaxTokens) return SPINDLEKV_UNSUPPORTED;   // the cover keeps a unit's state on chip
  const int units = b.n_layers * b.n_seqs * cfg.n_kv_heads;
  if (units > 65535) return SPINDLEKV_UNSUPPORTED;
  const bool records = L.rec_per_tile > 0;    // candidate records first, the bit matrix for units that overflow
  char* w = reinterpret_cast<char*>(ws);
  CodebookParams p;
  p.G = make_view(Gamma);
  p.batch = make_batch(b);
  p.n_kv_heads = cfg.n_kv_heads;
  p.n_units = units;
  p.row_words = row_words_for(b.max_len);
  p.theta = theta;
  p.mag = mag;
  p.adj = adj_in_ws ? reinterpret_cast<uint32_t*>(w + L.adj) : adj_bits;
  p.deg = reinterpret_cast<int32_t*>(w + L.deg);
  p.live0 = reinterpret_cast<uint32_t*>(w + L.live0);
  p.owner = reinterpret_cast<int32_t*>(w + L.owner);
  p.pickdeg = reinterpret_cast<int32_t*>(w + L.pickdeg);
  p.rank = reinterpret_cast<int32_t*>(w + L.rank);
  p.lists = reinterpret_cast<int32_t*>(w + L.ell);
  p.ell_cnt = reinterpret_cast<int32_t*>(w + L.ell_cnt);
  p.dense_rows = reinterpret_cast<int32_t*>(w + L.dense_rows);
  p.dense_cnt = reinterpret_cast<int32_t*>(w + L.dense_cnt);
  p.flags = reinterpret_cast<uint32_t*>(w + L.flags);
  p.hdr = reinterpret_cast<uint32_t*>(w);
  p.ref = ref;
  p.centre_idx = centre_idx;
  p.n_entries = n_entries;
  p.rec = reinterpret_cast<const uint2*>(w + L.rec);
  p.rec_cnt = reinterpret_cast<const int32_t*>(w + L.rec_cnt);
  p.ovf = reinterpret_cast<int32_t*>(w + L.ovf);
  p.rec_per_tile = L.rec_per_tile;
  p.n_blocks = L.n_blocks;
  p.unit_rec_cap = records ? rec_unit_capacity(L.n_blocks / 2, L.rec_per_tile) : 0;
  p.lbase = reinterpret_cast<int32_t*>(w + L.lbase);
  p.list_cap = L.list_cap;
  p.round_cap = tune.round_cap;
  if (cudaMemsetAsync(w, 0, kHeaderBytes, st) != cudaSuccess) return SPINDLEKV_CUDA;
  // overflow flags and record counts: all zero on the record path; without records every unit counts as overflowed;
  // the per-unit counts of rows with many neighbours start at zero
  if (cudaMemsetAsync(w + L.ovf, records ? 0 : 1, L.dense_cnt - L.ovf, st) != cudaSuccess) return SPINDLEKV_CUDA;
  if (cudaMemsetAsync(w + L.dense_cnt, 0, L.work_list - L.dense_cnt, st) != cudaSuccess) return SPINDLEKV_CUDA;
  p.ext = tc ? reinterpret_cast<__nv_bfloat16*>(w + L.ext) : nullptr;
  if (cfg.head_dim == 64) {
    if (bf) launch_norms<__nv_bfloat16, 64>(p, st); else launch_norms<float, 64>(p, st);
  } else {
    if (bf) launch_norms<__nv_bfloat16, 128>(p, st); else launch_norms<float, 128>(p, st);
  }
  const size_t flag_words = (size_t)(p.row_words / 2) * p.row_words;
  if (tc) {
    SimRecordPool pool{reinterpret_cast<uint2*>(w + L.rec), reinterpret_cast<int32_t*>(w + L.rec_cnt), p.ovf, L.rec_per_tile,
                       reinterpret_cast<int32_t*>(w + L.work_list) + 1, reinterpret_cast<int32_t*>(w + L.work_list)};
    if (records) {
      if (!adj_in_ws &&
          cudaMemsetAsync(adj_bits, 0, (size_t)units * b.max_len * p.row_words * 4, st) != cudaSuccess) return SPINDLEKV_CUDA;
      spindlekv_status rs = launch_sim_tc(Gamma, b, cfg.n_kv_heads, cfg.head_dim, p.ext, p.adj, p.flags, p.hdr, adj_in_ws, &pool,
                                          true, tune.mbar_wait_cycles, st);
      if (rs != SPINDLEKV_OK) return rs;
      static PerDeviceOnce once;
      const int dev0 = PerDeviceOnce::current();
      if (dev0 < 0) return SPINDLEKV_CUDA;
      if (!once.done[dev0]) {
        if (cudaFuncSetAttribute(build_lists_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 49152 * 4) != cudaSuccess)
          return SPINDLEKV_CUDA;
        once.done[dev0] = true;
      }
      LaunchScope ls(KC_DEGREE, st);
      build_lists_kernel<<<units, kBuildThreads, (size_t)p.row_words * 32 * 4, st>>>(p);
    }
    // units without usable records (all of them when the record path is off): bit matrix, occupancy flags, extraction
    if (records) {
      LaunchScope ls(KC_DEGREE, st);
      list_overflowed_kernel<<<1, 1024, 0, st>>>(p.ovf, units, pool.work_list, pool.n_work);
    }
    {
      LaunchScope ls(KC_DEGREE, st);
      clear_flags_kernel<<<dim3((unsigned)std::min<size_t>((flag_words + 255) / 256, 64), units), 256, 0, st>>>(p);
    }
    spindlekv_status rs = launch_sim_tc(Gamma, b, cfg.n_kv_heads, cfg.head_dim, p.ext, p.adj, p.flags, p.hdr, adj_in_ws, &pool,
                                        false, tune.mbar_wait_cycles, st);
    if (rs != SPINDLEKV_OK) return rs;
  } else if (cfg.head_dim == 64) {
    if (bf) launch_sim_simt<__nv_bfloat16, 64>(p, b, st); else launch_sim_simt<float, 64>(p, b, st);
  } else {
    if (bf) launch_sim_simt<__nv_bfloat16, 128>(p, b, st); else launch_sim_simt<float, 128>(p, b, st);
  }
  if (!tc) {
    // the CUDA-core similarity kernel writes no occupancy flags: every chunk counts as occupied
    if (cudaMemsetAsync(p.flags, 0xFF, (size_t)units * flag_words * 4, st) != cudaSuccess) return SPINDLEKV_CUDA;
  }
  {
    LaunchScope ls(KC_DEGREE, st);
    extract_kernel<<<(unsigned)(((size_t)units * p.row_words * 32 + 255) / 256), 256, 0, st>>>(p);
  }
  if (records && !adj_in_ws) {
    LaunchScope ls(KC_DEGREE, st);
    expand_records_kernel<<<units, kBuildThreads, 0, st>>>(p, adj_bits);
  }
  const int dev = PerDeviceOnce::current();
  if (dev < 0) return SPINDLEKV_CUDA;
  {
    static PerDeviceOnce once;
    if (!once.done[dev]) {
      if (cudaFuncSetAttribute(cover_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cover_smem_bytes(kCoverMaxTokens / 32)) != cudaSuccess)
        return SPINDLEKV_CUDA;
      once.done[dev] = true;
    }
    LaunchScope ls(KC_GREEDY, st);
    cover_kernel<<<units, kCoverThreads, cover_smem_bytes(p.row_words), st>>>(p);
  }
  {
    size_t smem = (size_t)(b.max_len + 2) * 4;
    static PerDeviceOnce once;
    if (!once.done[dev]) {
      if (cudaFuncSetAttribute(finalize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
        return SPINDLEKV_CUDA;
      once.done[dev] = true;
    }
    LaunchScope ls(KC_FINAL, st);
    finalize_kernel<<<units, kFinalThreads, smem, st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

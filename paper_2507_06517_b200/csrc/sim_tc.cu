// Thresholded cosine similarity (Eq. (4)(9)) on the 5th-generation tensor cores, bf16 inputs.
//
// The adjacency is symmetric, so only pairs (a, b) with a < b are computed and each decision is
// written twice: into row a and, mirrored, into row b.
//
// A pair of CTAs (a cluster) works on a 256-row span of one (layer, sequence, head) unit: each CTA's
// block of 128 token rows is loaded once by TMA and stays in shared memory as operand A; tiles of 256
// token rows, from the tile that holds the diagonal onwards, stream through a ring as operand B.  The
// two CTAs share one MMA stream: each loads only its half of every streamed tile, and threads of the
// first CTA issue tcgen05.mma.cta_group::2 (256 x 256 x 16, fp32 accumulation in both CTAs' TMEM, 128
// rows each), which halves the operand traffic per SM.
//
// The threshold is part of the contraction.  Every K-step runs with the negate-A flag: the main ones
// accumulate -gamma_a . gamma_b; one more K-step multiplies two 16-element rows prepared by the
// magnitude kernel: -theta*|gamma_a| and |gamma_b|, each split into three bf16 pieces, laid out so
// that the nine cross products add up to -theta*|gamma_a|*|gamma_b| (exact up to the fp32
// accumulation).  The accumulator then holds  theta*|a||b| - a.b , whose sign bit is the decision
// a.b / (|a||b|) > theta.  The epilogue therefore only collects sign bits: no per-column operand,
// no floating-point instruction.
//
// Two threads issue the MMAs, one the even tiles into the first accumulator, one the odd tiles into the
// second, taking turns tile by tile; while one issues, the other does the commits of its last tile and
// the barrier waits of its next one (with a single thread the tensor cores idled over those).
//
// Candidate emission (the first choice; the bit matrix below is the bounded fallback).  Graphs of real
// caches are sparse: a token is similar to a handful of others.  The launch is a fixed number of CTA
// pairs, as many as the device holds; they share out the items (unit, fold), a fold being the row spans
// f and n_tiles - 1 - f of a unit, which together always cost n_tiles + 1 tiles, and walk them with two
// resident blocks in shared memory, so that the next block loads while the current one is in use and
// rings, accumulators and barrier phases carry on from item to item.  All sixteen epilogue warps read
// every tile back with tcgen05.ld (a warp: 32 rows x 64 columns); a thread owns one row a and shifts the
// sign bits of 32 columns into a word.  A warp keeps the pairs with a < b only and writes nothing but
// the non-zero words, as records (row, word column, 32 bits): a ballot counts them, one shared-memory
// atomic reserves room in the block's own region of the unit's record pool, and the lanes store their
// records side by side.  No transpose, no staging: the next kernel mirrors the pairs when it builds
// the neighbour lists.  A block's region holds `rec_per_tile` records per tile it computes; a block
// that runs out of room raises the unit's overflow flag, and such units are computed again as a bit
// matrix.  The order of the records inside a region depends on warp timing; everything derived from
// them is independent of that order.
//
// Bit matrix (units that overflowed their record pool, or every unit when the caller passes no pool).
// One pair of CTAs per row span and slot; a slot walks the listed units with its fixed span.  Sixteen
// epilogue warps in two teams of eight; team e serves TMEM stage e, i.e. every other tile.  Inside a
// team a warp owns a 32-row strip and half of the tile's columns.  Direct words are staged in shared
// memory and leave in 32-byte pieces, two per row, after the team's two tiles of a four-tile span (the
// two warps of a strip meet for that); a 32x32 bit transpose across the warp turns the words of a
// sub-block into the words of the mirrored rows, which are staged too and written 16 bytes per row by
// the whole team.  Nothing but bits leaves the SM: N*N/8 bytes per unit, plus one bit per (row,
// 64-column chunk) that says whether the chunk may hold a set bit (0: certainly empty), so that the
// next kernel reads only the occupied part of a sparse graph.  The flags of 32 consecutive rows and
// one chunk form a word (`flags[row / 32][chunk]`) with exactly one writer: the rows' own block for
// chunks at or right of the block's own columns, the block that mirrors into the rows for chunks left
// of them.  The caller clears the flag words; only words with a set bit are written.
#include <algorithm>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace skv {

struct SimTcParams {
  Batch batch;
  int n_kv_heads, row_words;
  uint32_t* adj;       // [units][max_len][row_words]
  uint32_t* flags;     // [units][row_words][row_words / 2]
  uint32_t* hdr;
  int skip_empty;      // mirrored chunks without a set bit are not stored (their flag bit stays 0)
  // candidate emission
  uint2* rec;          // [units][unit_rec_cap] records: .x = row << kRecRowShift | word column, .y = bits (pairs a < b only)
  int32_t* rec_cnt;    // [units][blocks] records written by each row block (cleared by the caller)
  int32_t* ovf;        // [units] != 0: the unit does not fit the record pool and is computed as a bit matrix
  int rec_per_tile;    // a block's region holds rec_per_tile records per tile it computes
  long long unit_rec_cap;
  long long wait_cycles;   // bound of every mbarrier wait, in SM clock cycles
  // bit-matrix instantiation behind a record pool: the units to compute (those that overflowed), in ascending
  // order, and their number; a pair of blocks with blockIdx.y = k takes the units work_list[k], work_list[k +
  // gridDim.y], ...  Null: blockIdx.y is the unit.
  const int32_t* work_list;
  const int32_t* n_work;
  int n_units;         // units of the call
};

constexpr int kBM = 128;          // rows of the resident block (UMMA M)
constexpr int kBN = 256;          // rows of a streamed tile (UMMA N)
constexpr int kStages = 4;         // shared-memory ring of streamed half tiles (TMEM ring: 2 accumulators)
constexpr int kBH = kBN / 2;       // rows of a streamed tile that one CTA of the pair loads
constexpr int kEpiWarps = 16;                         // two teams of eight; team e serves TMEM stage e
constexpr int kTeamWarps = kEpiWarps / 2;
constexpr int kColsPerWarp = kBN / (kTeamWarps / 4);  // tile columns handled by one epilogue warp
constexpr int kChunks = kColsPerWarp / 32;
constexpr int kEmitCols = kBN / (kEpiWarps / 4);     // columns of a tile per warp when all warps share every tile
constexpr int kEmitChunks = kEmitCols / 32;
static_assert(kEmitChunks == 2, "the record epilogue keeps two words per lane");
constexpr int kIssueWarp2 = 2 + kEpiWarps;            // the warp of the second MMA-issuing thread
constexpr int kSimThreads = 32 * (3 + kEpiWarps);   // loads, MMAs of even tiles, epilogue warps, MMAs of odd tiles
constexpr int kTileWords = kBN / 32;                  // words of a row per tile
constexpr int kDPitch = 2 * kTileWords + 2;           // staging pitch: a team's two tiles of a four-tile span
static_assert(kChunks == 4 && kTileWords == 8, "epilogue layout assumes 128 columns per warp");

// kEmit: two resident blocks (the next one loads while the MMAs read the current one) and no staging of
// bit-matrix words; otherwise one resident block and the staging areas.
template <int D, bool kEmit>
struct SimSmem {
  static constexpr int KH = D / 64;                  // 64-element (128-byte) swizzle atoms along head_dim
  static constexpr int NA = kEmit ? 2 : 1;           // resident blocks in shared memory
  static constexpr int A_BYTES = KH * kBM * 128;
  static constexpr int B_BYTES = KH * kBH * 128;     // this CTA's half of a streamed tile
  static constexpr int EA_BYTES = kBM * 32;          // threshold rows of the block (one 16-element K-step)
  static constexpr int EB_BYTES = kBH * 32;          // magnitude rows of this CTA's half tile
  static constexpr int T_BYTES = kEmit ? 0 : 2 * 4 * kBN * 4;    // mirrored words [slot][row quarter][tile column]
  static constexpr int D_BYTES = kEmit ? 0 : 2 * 2 * kBM * kDPitch * 4;  // direct words [team][slot][row][word]
  static constexpr int OFF_B = NA * A_BYTES;
  static constexpr int OFF_EA = OFF_B + kStages * B_BYTES;
  static constexpr int OFF_EB = OFF_EA + NA * EA_BYTES;
  static constexpr int OFF_T = OFF_EB + kStages * EB_BYTES;
  static constexpr int OFF_D = OFF_T + T_BYTES;
  static constexpr int OFF_BAR = OFF_D + D_BYTES;
  static constexpr int USED = OFF_BAR + 256 /*barriers*/ + 1024 /*alignment*/;
  // at least 120 KB so that two blocks never share an SM: each block allocates all 512 TMEM columns
  static constexpr int TOTAL = USED > 120 * 1024 ? USED : 120 * 1024;
  static_assert(TOTAL <= 227 * 1024, "shared memory budget");
};

// Named barrier over some of the epilogue warps: ids 2, 3 for a whole team (256 threads), ids 4..11 for
// the two warps of a team that share a 32-row strip (64 threads).
__device__ __forceinline__ void epi_bar_n(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Waits until the shared counter `turn` reaches `want`; gives up like a barrier wait (false, abort flag set).
__device__ __forceinline__ bool wait_turn(volatile int* turn, int want, volatile int* abort_flag, long long limit_cycles) {
  if (*turn == want) return true;
  const long long t0 = clock64();
  for (uint32_t i = 0;; ++i) {
    if (*turn == want) return true;
    if ((i & 63u) == 63u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit_cycles) break;
    }
  }
  *abort_flag = 1;
  return false;
}

// sign bits of 32 accumulators -> one word, bit c = sign of column c
__device__ __forceinline__ uint32_t sign_word(const uint32_t (&acc)[32]) {
  // four independent 8-bit groups keep the shift chains short
  uint32_t wg[4] = {0, 0, 0, 0};
#pragma unroll
  for (int c = 31; c >= 0; --c) wg[c >> 3] = __funnelshift_l(acc[c], wg[c >> 3], 1);
  return __byte_perm(__byte_perm(wg[0], wg[1], 0x0040), __byte_perm(wg[2], wg[3], 0x0040), 0x5410);
}

// ---- CTA pairs ------------------------------------------------------------------------------------
// Two CTAs of a cluster (ranks 0 and 1) own the two 128-row blocks of a 256-row span and run one
// tcgen05.mma.cta_group::2 stream, issued by rank 0: each CTA holds its own block (operand A) and loads
// only its half of every streamed tile (operand B), which halves the operand traffic per SM.
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in the pair's rank-0 CTA
__device__ __forceinline__ uint32_t leader_addr(const void* p) { return ptx::smem_u32(p) & 0xFEFFFFFFu; }
__device__ __forceinline__ void mbar_arrive_leader(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(leader_addr(bar)) : "memory");
}
// tiled TMA loads into this CTA's shared memory whose completion is counted on the leader's barrier
__device__ __forceinline__ void tma_load_5d_pair(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                 int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(ptx::smem_u32(smem_dst)), "l"(map), "r"(leader_addr(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                                 int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(ptx::smem_u32(smem_dst)), "l"(map), "r"(leader_addr(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {  // warp 1 of both CTAs
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(smem_result)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the same barrier in both CTAs once all MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(ptx::smem_u32(bar)), "h"((uint16_t)3) : "memory");
}

// kEmit: candidate records for every unit; otherwise the bit matrix, for the units whose overflow flag is set
// (all units when the caller passes no flags).
template <int D, bool kEmit>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kSimThreads, 1) sim_tc_kernel(const __grid_constant__ CUtensorMap tmap,
                                                                const __grid_constant__ CUtensorMap emap,
                                                                SimTcParams p) {
  using L = SimSmem<D, kEmit>;
  const int n_work = p.work_list ? *p.n_work : p.n_units;
  const int rank = (int)cluster_ctarank();   // = blockIdx.x & 1
  // Work of a pair of blocks, walked in the same order by every role of both CTAs.  The roles count the tiles done
  // so far (`base`) and the pieces that had any (`ua`): ring stages, accumulator stages, resident blocks and barrier
  // phases carry on from one piece to the next.
  //  Bit matrix: a piece is (unit, the pair's own 256-row span blockIdx.x / 2); the pair takes the units with list
  //  index blockIdx.y, blockIdx.y + gridDim.y, ...
  //  Candidate records: the grid is a fixed number of pairs; item i = (unit i / F, fold f = i % F) holds the spans
  //  f and n_tiles - 1 - f of the unit, which together always cost n_tiles + 1 tiles, and the pair takes the items
  //  blockIdx.x / 2, + gridDim.x / 2, ...: neighbouring pairs work on the same few units at any time.
  constexpr int kHalves = kEmit ? 2 : 1;
  const int F = kEmit ? ((p.batch.max_len + kBN - 1) / kBN + 1) / 2 : 1;
  const int item0 = kEmit ? (int)(blockIdx.x >> 1) : (int)blockIdx.y;
  const int item_step = kEmit ? (int)(gridDim.x >> 1) : (int)gridDim.y;
  const int n_items = n_work * F;
  if (item0 >= n_items) return;              // both CTAs of a pair: nothing to compute
  struct Piece { int unit, j, s, layer, l, n_tiles, nt, span; };
  auto piece = [&](int i, int h) {
    Piece w;
    const int k = kEmit ? i / F : i;
    const int f = kEmit ? i - k * F : (int)(blockIdx.x >> 1);
    w.unit = p.work_list ? p.work_list[k] : k;
    w.j = w.unit % p.n_kv_heads;
    const int ls = w.unit / p.n_kv_heads;
    w.s = ls % p.batch.n_seqs;
    w.layer = ls / p.batch.n_seqs;
    w.l = seq_len(p.batch, w.layer, w.s, w.j);
    w.n_tiles = (w.l + kBN - 1) / kBN;         // tiles of this sequence: columns beyond its end are never produced
    w.span = h == 0 ? f : w.n_tiles - 1 - f;
    // a fold has work while its first span is not beyond its second (a sequence shorter than the longest has
    // fewer folds); the second span counts only where it is another one than the first
    const bool any = kEmit ? (h == 0 ? 2 * f <= w.n_tiles - 1 : 2 * f < w.n_tiles - 1) : w.span < w.n_tiles;
    w.nt = any ? w.n_tiles - w.span : 0;
    return w;
  };
  // bit matrix only: the pair's fixed rows
  const int row0 = blockIdx.x * kBM;
  const int tile0 = row0 / kBN;   // the tile that holds the pair's diagonal; earlier tiles are mirrored by other pairs

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + L::OFF_B;
  uint8_t* sEA = smem + L::OFF_EA;
  uint8_t* sEB = smem + L::OFF_EB;
  uint32_t* sT = reinterpret_cast<uint32_t*>(smem + L::OFF_T);
  uint32_t* sD = reinterpret_cast<uint32_t*>(smem + L::OFF_D);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
  // a_full, b_full and acc_empty are used in the leader (rank 0) only: both CTAs' loads and both CTAs'
  // epilogue warps signal them there; b_empty and acc_full are signalled in both CTAs by the leader's commits
  uint64_t* a_full = bars + 0;                  // [2]
  uint64_t* b_full = bars + 2;                  // [kStages]
  uint64_t* b_empty = bars + 2 + kStages;       // [kStages]
  uint64_t* acc_full = bars + 2 + 2 * kStages;  // [2]
  uint64_t* acc_empty = acc_full + 2;           // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(acc_empty + 3);
  uint64_t* a_empty = acc_empty + 4;            // [2] both CTAs: the MMAs of a piece have read its resident block
  int* rec_used = reinterpret_cast<int*>(acc_empty + 6);   // [2] records reserved for a piece; pieces alternate
  volatile int* turn = reinterpret_cast<volatile int*>(acc_empty + 7);   // the tile whose MMAs may be issued now
  const long long wait_cycles = p.wait_cycles;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(a_full + i, 1); ptx::mbar_init(a_empty + i, 2); }
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(b_full + i, 1); ptx::mbar_init(b_empty + i, 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(acc_full + i, 1); ptx::mbar_init(acc_empty + i, kEmit ? 2 * kEpiWarps : 2 * kTeamWarps); }
    *abort_flag = 0;
    rec_used[0] = rec_used[1] = 0;
    *turn = 0;
    ptx::fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  cluster_sync_all();   // barriers of both CTAs are initialised before either signals the other
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      ptx::prefetch_tensormap(&tmap);
      ptx::prefetch_tensormap(&emap);
      int base = 0, ua = 0;
      bool ok = true;
      for (int i = item0; ok && i < n_items; i += item_step) {
        for (int h = 0; ok && h < kHalves; ++h) {
          const Piece w = piece(i, h);
          if (w.nt == 0) continue;
          const int tok0 = p.batch.cu ? p.batch.cu[w.s] : 0;
          const int sdim = p.batch.cu ? 0 : w.s;
          const int ab = ua % L::NA;
          // the piece that used this resident block before must have been read by all of its MMAs
          if (ua >= L::NA && !ptx::mbar_wait(a_empty + ab, ((ua / L::NA) & 1) ^ 1, abort_flag, wait_cycles)) { ok = false; break; }
          if (rank == 0) ptx::mbar_expect_tx(a_full + ab, 2 * (L::A_BYTES + L::EA_BYTES));
          const int arow = w.span * kBN + rank * kBM;
          for (int kh = 0; kh < L::KH; ++kh)
            tma_load_5d_pair(sA + ab * L::A_BYTES + kh * kBM * 128, &tmap, a_full + ab, kh * 64, tok0 + arow, w.j, sdim, w.layer);
          tma_load_4d_pair(sEA + ab * L::EA_BYTES, &emap, a_full + ab, 0, arow, w.unit, 0);
          for (int it = 0; it < w.nt; ++it) {
            const int gi = base + it, st = gi % kStages;
            if (!ptx::mbar_wait(b_empty + st, ((gi / kStages) & 1) ^ 1, abort_flag, wait_cycles)) { ok = false; break; }
            if (rank == 0) ptx::mbar_expect_tx(b_full + st, 2 * (L::B_BYTES + L::EB_BYTES));
            uint8_t* dst = sB + st * L::B_BYTES;
            const int brow = (w.span + it) * kBN + rank * kBH;   // this CTA's half of the tile
            for (int kh = 0; kh < L::KH; ++kh)
              tma_load_5d_pair(dst + kh * kBH * 128, &tmap, b_full + st, kh * 64, tok0 + brow, w.j, sdim, w.layer);
            tma_load_4d_pair(sEB + st * L::EB_BYTES, &emap, b_full + st, 0, brow, w.unit, 1);
          }
          base += w.nt;
          ++ua;
        }
      }
    }
  } else if (warp == 1 || warp == kIssueWarp2) {
    // Two threads of the leader issue the MMAs, one the even tiles (first accumulator), one the odd tiles (second
    // accumulator), taking turns tile by tile.  Issuing an MMA holds its thread for about as long as the MMA runs,
    // and the commits and barrier waits around a tile come on top: with one thread the tensor cores sat idle over
    // those.  Here a thread does its waits while the other issues, takes the turn, issues its nine MMAs, hands the
    // turn on and only then commits.  (MMAs of two tiles issued in alternation ran far slower: hence the turns.)
    if (lane == 0 && rank == 0) {
      const int me = warp == 1 ? 0 : 1;
      constexpr uint32_t idesc_neg = ptx::idesc_bf16_f32(2 * kBM, kBN, true);
      int base = 0, ua = 0;
      bool ok = true;
      for (int i = item0; ok && i < n_items; i += item_step) {
        for (int h = 0; ok && h < kHalves; ++h) {
          const Piece w = piece(i, h);
          if (w.nt == 0) continue;
          const int ab = ua % L::NA;
          const uint32_t a_addr = ptx::smem_u32(sA + ab * L::A_BYTES);
          const uint64_t dea = ptx::smem_desc_sw32(ptx::smem_u32(sEA + ab * L::EA_BYTES));
          ok = ptx::mbar_wait(a_full + ab, (ua / L::NA) & 1, abort_flag, wait_cycles);
          for (int it = (me ^ base) & 1; ok && it < w.nt; it += 2) {
            const int gi = base + it, st = gi % kStages;   // gi & 1 == me: the accumulator of this thread
            if (!ptx::mbar_wait(b_full + st, (gi / kStages) & 1, abort_flag, wait_cycles)) { ok = false; break; }
            if (!ptx::mbar_wait(acc_empty + me, ((gi >> 1) & 1) ^ 1, abort_flag, wait_cycles)) { ok = false; break; }
            if (!wait_turn(turn, gi, abort_flag, wait_cycles)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t b_addr = ptx::smem_u32(sB + st * L::B_BYTES);
#pragma unroll
            for (int kk16 = 0; kk16 < D / 16; ++kk16) {
              const int kh = kk16 >> 2, kk = kk16 & 3;
              uint64_t da = ptx::smem_desc_sw128(a_addr + kh * kBM * 128 + kk * 32);
              uint64_t db = ptx::smem_desc_sw128(b_addr + kh * kBH * 128 + kk * 32);
              umma_bf16_pair(tmem_base + me * kBN, da, db, idesc_neg, kk16 > 0 ? 1u : 0u);
            }
            // + theta * |a| * |b|: the threshold rows of operand A are stored negated, so the same descriptor serves
            // (a change of descriptor between MMAs cost about twenty cycles each time)
            umma_bf16_pair(tmem_base + me * kBN, dea, ptx::smem_desc_sw32(ptx::smem_u32(sEB + st * L::EB_BYTES)), idesc_neg, 1u);
            *turn = gi + 1;                   // the other thread may issue the next tile
            umma_commit_pair(b_empty + st);   // both CTAs: the stage may be refilled
            umma_commit_pair(acc_full + me);  // both CTAs: accumulator ready for the epilogue
          }
          // both CTAs: the resident block may be replaced once both threads' MMAs of the piece have read it (a
          // thread without a tile in the piece arrives at once)
          if (ok) umma_commit_pair(a_empty + ab);
          base += w.nt;
          ++ua;
        }
      }
    }
  } else if constexpr (kEmit) {
    // ---- candidate emission ----
    // All sixteen warps work on every tile: a warp reads 64 columns of its 32 accumulator rows, so that an
    // accumulator is handed back to the MMAs well within the time the other one takes to fill.
    const int q = warp & 3;               // TMEM lane quarter this warp may read
    const int cg = (warp - 2) >> 2;       // which quarter of the tile's columns
    const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + cg * kEmitCols;
    const uint32_t below = (1u << lane) - 1u;
    const int T_max = (p.batch.max_len + kBN - 1) / kBN;
    int base = 0, ui = 0;
    // every piece of the pair, also after a wait that gave up: the warps meet at a barrier at the end of each
    for (int i = item0; i < n_items; i += item_step) {
      for (int h = 0; h < kHalves; ++h) {
        const Piece w = piece(i, h);
        if (w.nt == 0) continue;
        const int unit = w.unit, l = w.l;
        const int blk = 2 * w.span + rank;             // the 128-row block of the sequence this CTA holds
        const int R = blk * kBM + q * 32;              // first row of this warp's 32-row strip
        const int row = R + lane;
        const uint32_t key_row = (uint32_t)row << kRecRowShift;
        const int cap = p.rec_per_tile * (T_max - w.span);   // records the block's region holds
        int* used = rec_used + (ui & 1);               // pieces alternate between two counters
        const bool live_block = blk * kBM < l;         // the second CTA of a sequence's last span may own no row at all
#pragma unroll 1
        for (int it = 0; it < w.nt; ++it) {
          const int c0 = (w.span + it) * kBN;
          const int as = (base + it) & 1;              // accumulator stage of this tile
          bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(acc_full + as, ((base + it) >> 1) & 1, abort_flag, wait_cycles));
          if (!ok) break;                     // the barrier at the end of the piece is still met
          if (!live_block) {
            if (lane == 0) mbar_arrive_leader(acc_empty + as);
            continue;
          }
          ptx::tc_fence_after();
          uint32_t words[kEmitChunks];
          words[0] = words[1] = 0u;
          // This loop must stay a loop: unrolled, every pass gets 32 registers of its own for its accumulators
          // and the thread (96 registers with twenty warps in the block) spills, which costs more than all the rest.
#pragma unroll 1
          for (int ch = 0; ch < kEmitChunks; ++ch) {
            uint32_t acc[32];
            ptx::tmem_ld_32x32_sync(tcol + as * kBN + ch * 32, acc);   // load and wait in one statement
            const uint32_t sw = sign_word(acc);
            words[0] = ch == 0 ? sw : words[0];
            words[1] = ch == 1 ? sw : words[1];
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(acc_empty + as);
          const int wc0 = (c0 + cg * kEmitCols) >> 5;   // word column of this warp's first 32 columns
          if (c0 + kBN > l || R + 32 > l) {
            // ragged edge: columns and rows that do not exist carry no bits
#pragma unroll
            for (int ch = 0; ch < kEmitChunks; ++ch) {
              const int nvalid = l - (wc0 + ch) * 32;
              if (nvalid < 32) words[ch] &= nvalid > 0 ? ((1u << nvalid) - 1u) : 0u;
              if (row >= l) words[ch] = 0;
            }
          }
          if (it == 0) {
            // the tile that holds the diagonal: only pairs a < b are kept (the rest is their mirror image)
#pragma unroll
            for (int ch = 0; ch < kEmitChunks; ++ch) {
              const int col0 = (wc0 + ch) * 32;
              if (col0 + 32 <= R) words[ch] = 0u;
              else if (col0 == R) words[ch] &= lane == 31 ? 0u : (0xFFFFFFFFu << (lane + 1));
            }
          }
          uint32_t m[kEmitChunks];
          int n = 0;
#pragma unroll
          for (int ch = 0; ch < kEmitChunks; ++ch) {
            m[ch] = __ballot_sync(0xffffffffu, words[ch] != 0u);
            n += __popc(m[ch]);
          }
          if (n == 0) continue;
          int at = 0;
          if (lane == 0) at = atomicAdd(used, n);
          at = __shfl_sync(0xffffffffu, at, 0);
          if (at + n > cap) {
            if (lane == 0) p.ovf[unit] = 1;   // the unit is computed again as a bit matrix
            continue;
          }
          // the block's region of the unit's record pool (worked out here, where it is needed, to keep registers free)
          uint2* rec_blk = p.rec + (long long)unit * p.unit_rec_cap + rec_region_offset(blk, T_max, p.rec_per_tile);
#pragma unroll
          for (int ch = 0; ch < kEmitChunks; ++ch) {
            if (words[ch]) rec_blk[at + __popc(m[ch] & below)] = make_uint2(key_row | (uint32_t)(wc0 + ch), words[ch]);
            at += __popc(m[ch]);
          }
        }
        // all warps have reserved and written this piece's records: publish the count, clear the counter for the
        // piece after next
        epi_bar_n(2, 32 * kEpiWarps);
        if (warp == 2 && lane == 0) {
          p.rec_cnt[(long long)unit * (2 * T_max) + blk] = min(*used, cap);
          *used = 0;
        }
        base += w.nt;
        ++ui;
      }
    }
  } else {
    const int q = warp & 3;               // TMEM lane quarter this warp may read
    const int team = (warp - 2) >> 3;     // which TMEM stage this warp serves
    const int cg = ((warp - 2) >> 2) & 1; // which half of the tile's columns
    const int tt = ((warp - 2) & 7) * 32 + lane;   // thread index within the team
    const int rl = q * 32 + lane;         // row within the block
    const int R = row0 + q * 32;          // first row of this warp's 32-row strip
    const int row = R + lane;
    TransposeLane tr;
    tr.init(lane);
    int base = 0;
    // Every unit of the pair, also after a wait that gave up (every later wait then returns at once): the warps of
    // a team meet at named barriers inside, so none may leave early.
    for (int i = item0; i < n_items; i += item_step) {
      const Piece w = piece(i, 0);
      if (w.nt == 0) continue;
      const int unit = w.unit, l = w.l, n_tiles = w.n_tiles;
      const int RW = p.row_words;
      uint32_t* adj_unit = p.adj + (int64_t)unit * p.batch.max_len * RW;
      const int NC = RW >> 1;               // 64-column chunks per row
      const int blk = blockIdx.x;
      uint32_t* funit = p.flags + (int64_t)unit * NC * RW;
      // the second CTA of a sequence's last pair may own no row at all: it still loads its half tiles and
      // keeps the barrier protocol going, but reads and writes nothing
      const bool live_block = row0 < l;
      if (lane == 0 && live_block) {
        // The two chunks that hold the block's own 128 columns are flagged as occupied without looking:
        // for the block's rows (diagonal bit, and words mirrored inside the block), and, from an even
        // block, for the rows of the next block, which its diagonal tile mirrors into piecemeal.
        const int chunk = 2 * blk + cg;
        const int wb = (row0 >> 5) + team * 4 + q;   // team 0: own rows; team 1: the next block's rows
        if (chunk < NC && wb < RW && (team == 0 || !(blk & 1))) funit[(int64_t)wb * NC + chunk] = 0xFFFFFFFFu;
      }
      uint32_t* sD_team = sD + team * (2 * kBM * kDPitch);
      // mirrored rows: thread tt of the team writes row c0 + tt, 16 bytes at the block's column
      const uint32_t tcol = tmem_base + ((uint32_t)(q * 32) << 16) + team * kBN + cg * kColsPerWarp;
      uint32_t* tq = sT + (team * 4 + q) * kBN + cg * kColsPerWarp + lane;
      const uint32_t* tr0 = sT + team * 4 * kBN + tt;
      // No early exit from this loop: after a wait that gave up (every later wait then returns at once)
      // the warp still meets its partners at each barrier, with nothing to do in between.
      for (int it = (team ^ base) & 1; it < w.nt; it += 2) {
        const int tile = tile0 + it;
        const int c0 = tile * kBN;
        const bool fast = c0 >= row0 + kBM;      // whole tile strictly above the diagonal
        const int slot = (tile >> 1) & 1;        // which of the team's two tiles of the four-tile span
        uint32_t* sdbuf = sD_team + ((tile >> 2) & 1) * (kBM * kDPitch);
        uint32_t* sdw = sdbuf + rl * kDPitch + slot * kTileWords + cg * kChunks;
        bool ok = __all_sync(0xffffffffu, ptx::mbar_wait(acc_full + team, ((base + it) >> 1) & 1, abort_flag, wait_cycles));
        if (ok && !live_block) {
          if (lane == 0) mbar_arrive_leader(acc_empty + team);
          ok = false;
        }
        if (ok) {
          ptx::tc_fence_after();
          uint32_t words[kChunks];
  #pragma unroll
          for (int ch = 0; ch < kChunks; ++ch) {
            uint32_t acc[32];
            ptx::tmem_ld_32x32(tcol + ch * 32, acc);
            ptx::tmem_ld_wait(acc);
            words[ch] = sign_word(acc);
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_leader(acc_empty + team);
          if (c0 + kBN > l || R + 32 > l) {
            // ragged edge: columns and rows that do not exist carry no bits
  #pragma unroll
            for (int ch = 0; ch < kChunks; ++ch) {
              const int nvalid = l - (c0 + cg * kColsPerWarp + ch * 32);
              if (nvalid < 32) words[ch] &= nvalid > 0 ? ((1u << nvalid) - 1u) : 0u;
              if (row >= l) words[ch] = 0;
            }
          }
          if (c0 + cg * kColsPerWarp >= row0 + kBM) {
            // this warp's two 64-column chunks lie right of the block's own columns: their flags for the strip
            const uint32_t f0 = __ballot_sync(0xffffffffu, (words[0] | words[1]) != 0u);
            const uint32_t f1 = __ballot_sync(0xffffffffu, (words[2] | words[3]) != 0u);
            const int chunk = tile * 4 + cg * 2 + lane;
            const uint32_t fw = lane ? f1 : f0;   // the flag words start at zero: only occupied ones are written
            if (lane < 2 && chunk < NC && fw) funit[(int64_t)(R >> 5) * NC + chunk] = fw;
          }
          if (fast) {
            *reinterpret_cast<uint2*>(sdw) = make_uint2(words[0], words[1]);
            *reinterpret_cast<uint2*>(sdw + 2) = make_uint2(words[2], words[3]);
            // most 32 x 32 sub-blocks of a sparse graph are empty: their mirror image is too
  #pragma unroll
            for (int ch = 0; ch < kChunks; ++ch)
              tq[ch * 32] = __any_sync(0xffffffffu, words[ch] != 0u) ? tr.apply(words[ch]) : 0u;
          } else {
  #pragma unroll
            for (int ch = 0; ch < kChunks; ++ch) {
              const int col0 = c0 + cg * kColsPerWarp + ch * 32;
              if (col0 + 32 <= R) continue;                      // below the diagonal: another block mirrors it
              if (col0 == R) {
                // diagonal sub-block: upper triangle as computed, lower triangle mirrored from it, unit diagonal
                const uint32_t upper = lane == 31 ? 0u : (0xFFFFFFFFu << (lane + 1));
                const uint32_t wu = words[ch] & upper;
                const uint32_t wt = tr.apply(wu);
                sdw[ch] = row < l ? (wu | wt | (1u << lane)) : 0u;
              } else {
                sdw[ch] = words[ch];
                const uint32_t wt = tr.apply(words[ch]);
                if (col0 + lane < l) adj_unit[(int64_t)(col0 + lane) * RW + (R >> 5)] = wt;
              }
            }
          }
        }
        // the team's mirrored words of this tile are in shared memory
        epi_bar_n(2 + team, 32 * kTeamWarps);
        if (ok && fast) {
          const int b = c0 + tt;
          bool occ_lo = false, occ_hi = false;
          if (b < l) {
            const uint4 mv = make_uint4(tr0[0], tr0[kBN], tr0[2 * kBN], tr0[3 * kBN]);
            occ_lo = (mv.x | mv.y) != 0u;
            occ_hi = (mv.z | mv.w) != 0u;
            uint32_t* dst = adj_unit + (int64_t)b * RW + (row0 >> 5);
            if (!p.skip_empty) {
              *reinterpret_cast<uint4*>(dst) = mv;
            } else {
              // a reader consults the chunk's flag bit first: empty chunks need not reach memory
              if (occ_lo) *reinterpret_cast<uint2*>(dst) = make_uint2(mv.x, mv.y);
              if (occ_hi) *reinterpret_cast<uint2*>(dst + 2) = make_uint2(mv.z, mv.w);
            }
          }
          const uint32_t flo = __ballot_sync(0xffffffffu, occ_lo), fhi = __ballot_sync(0xffffffffu, occ_hi);
          const uint32_t fw = lane ? fhi : flo;
          if (lane < 2 && (b >> 5) < RW && fw) funit[(int64_t)(b >> 5) * NC + 2 * blk + lane] = fw;
        }
        if (slot == 1 || tile + 2 >= n_tiles) {
          // the two warps of the team that share this 32-row strip have staged their direct words of the
          // team's (up to) two tiles of this four-tile span: two 32-byte pieces per row, sixteen rows per
          // warp, two rows per store; words left of the strip's diagonal sub-block belong to mirrored writes
          epi_bar_n(4 + team * 4 + q, 64);
          const int half = lane >> 4, wl = lane & 15;           // row of the pair, word of the row's 16
          const int wtile = (tile & ~3) + (tile & 1) + 2 * (wl >> 3);   // the tile this word belongs to
          const int wi = wtile * kTileWords + (wl & 7);
          const int r0 = q * 32 + cg * 16 + half;
          if (wi >= (R >> 5) && wi < RW && wtile < n_tiles) {   // words of tiles beyond the sequence hold nothing of this unit
            uint32_t* dst = adj_unit + (int64_t)(row0 + r0) * RW + wi;
            const uint32_t* src = sdbuf + r0 * kDPitch + wl;
  #pragma unroll
            for (int i = 0; i < 16; i += 2)
              if (row0 + r0 + i < l) dst[(int64_t)i * RW] = src[i * kDPitch];
          }
        }
      }
      base += w.nt;
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
  cluster_sync_all();   // neither CTA leaves (or frees TMEM) while its partner may still signal it or use its memory
  if (warp == 1) {
    ptx::tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// Self-test of the bounded mbarrier wait: nobody ever arrives on the barrier, so the wait must run out
// after `wait_cycles`, and the block reports TIMEOUT the way the kernels above do.
__global__ void mbar_selftest_kernel(uint32_t* hdr, long long wait_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_sh;
  volatile int* abort_flag = &abort_sh;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_sh = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  const bool ok = ptx::mbar_wait(&bar, 0, abort_flag, wait_cycles);   // every thread waits; the first to give up releases the rest
  __syncthreads();
  if (threadIdx.x == 0) {
    if (*abort_flag) atomicExch(&hdr[kHdrStatus], (uint32_t)SPINDLEKV_TIMEOUT);
    if (ok) hdr[kHdrLive] = 0xBADu;   // must not happen
  }
}

spindlekv_status selftest_mbarrier_impl(uint32_t* hdr, long long wait_cycles, cudaStream_t st) {
  if (cudaMemsetAsync(hdr, 0, kHeaderBytes, st) != cudaSuccess) return SPINDLEKV_CUDA;
  mbar_selftest_kernel<<<1, 64, 0, st>>>(hdr, wait_cycles);
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
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

// bf16 window queries [layer][seq][q head][window row][d] -> 5-D map (d, row, head, seq, layer); one box is
// 64 elements x `window` rows x 128/window heads: 128 operand rows (head-major) of 128 bytes
bool make_query_map_bf16(CUtensorMap* map, const spindlekv_tensor& q, const spindlekv_batch& b, int n_q_heads,
                         int head_dim, int window) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || window <= 0 || 128 % window) return false;
  auto bytes = [](int64_t elems) { return (cuuint64_t)(elems > 0 ? elems : 8) * 2; };
  cuuint64_t dims[5] = {(cuuint64_t)head_dim, (cuuint64_t)window, (cuuint64_t)n_q_heads, (cuuint64_t)b.n_seqs,
                        (cuuint64_t)b.n_layers};
  cuuint64_t strides[4] = {bytes(q.stride_tok), bytes(q.stride_head), bytes(q.stride_seq), bytes(q.stride_layer)};
  const int64_t st_el[5] = {1, q.stride_tok, q.stride_head, q.stride_seq, q.stride_layer};
  for (int i = 1; i < 5; ++i)
    if (dims[i] > 1 && st_el[i] <= 0) return false;
  cuuint32_t box[5] = {64, (cuuint32_t)window, (cuuint32_t)(128 / window), 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, q.ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// threshold / magnitude rows [2][units][rows_padded][16] bf16 -> 4-D map, box 16 x 128 rows, 32-byte swizzle
static bool make_ext_map(CUtensorMap* map, const void* ext, int units, int rows_padded) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {16, (cuuint64_t)rows_padded, (cuuint64_t)units, 2};
  cuuint64_t strides[3] = {32, (cuuint64_t)rows_padded * 32, (cuuint64_t)units * rows_padded * 32};
  cuuint32_t box[4] = {16, 128, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ext), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool sim_tc_available() {
  static int ok[kMaxDevices] = {};   // 0: not asked yet, 1: yes, 2: no
  const int dev = PerDeviceOnce::current();
  if (dev < 0) return false;
  if (ok[dev] == 0) {
    int major = 0;
    ok[dev] = (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess && major == 10 &&
               encode_fn() != nullptr) ? 1 : 2;
  }
  return ok[dev] == 1;
}

template <int D, bool kEmit>
static bool sim_tc_prepare() {
  static PerDeviceOnce once;
  const int dev = PerDeviceOnce::current();
  if (dev < 0) return false;
  if (!once.done[dev]) {
    if (cudaFuncSetAttribute(sim_tc_kernel<D, kEmit>, cudaFuncAttributeMaxDynamicSharedMemorySize, SimSmem<D, kEmit>::TOTAL) != cudaSuccess)
      return false;
    once.done[dev] = true;
  }
  return true;
}

// Pairs of blocks of the candidate-record kernel that the device holds at once (one block per SM).
template <int D>
static int resident_pairs() {
  static int pairs[kMaxDevices] = {};
  const int dev = PerDeviceOnce::current();
  if (dev < 0 || !sim_tc_prepare<D, true>()) return 0;
  if (pairs[dev] == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (sms / 2), 1, 1);
    cfg.blockDim = dim3(kSimThreads, 1, 1);
    cfg.dynamicSmemBytes = SimSmem<D, true>::TOTAL;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, sim_tc_kernel<D, true>, &cfg) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = sms / 2;
    }
    pairs[dev] = std::min(n, sms / 2);
  }
  return pairs[dev];
}

template <int D, bool kEmit>
static spindlekv_status launch_sim_tc_one(const CUtensorMap& map, const CUtensorMap& emap, const SimTcParams& p, dim3 grid,
                                          cudaStream_t st) {
  if (!sim_tc_prepare<D, kEmit>()) return SPINDLEKV_CUDA;
  sim_tc_kernel<D, kEmit><<<grid, kSimThreads, SimSmem<D, kEmit>::TOTAL, st>>>(map, emap, p);
  return SPINDLEKV_OK;
}

// `pool`: where candidate records go.  emit = true: every unit's candidates are written as records (units that do
// not fit raise their overflow flag).  emit = false: the bit matrix, for the units whose overflow flag is set, or,
// without a pool, for every unit.
spindlekv_status launch_sim_tc(const spindlekv_tensor& Gamma, const spindlekv_batch& b, int n_kv_heads, int head_dim,
                               const void* ext, uint32_t* adj, uint32_t* flags, uint32_t* hdr, bool skip_empty,
                               const SimRecordPool* pool, bool emit, long long wait_cycles, cudaStream_t st) {
  const int units = b.n_layers * b.n_seqs * n_kv_heads;
  CUtensorMap map, emap;
  if (!make_tensor_map_bf16(&map, Gamma, b, n_kv_heads, head_dim, 128)) return SPINDLEKV_CUDA;
  if (!make_ext_map(&emap, ext, units, row_words_for(b.max_len) * 32)) return SPINDLEKV_CUDA;
  if (emit && !pool) return SPINDLEKV_INVALID_ARG;
  SimTcParams p;
  p.batch = make_batch(b);
  p.n_kv_heads = n_kv_heads;
  p.row_words = row_words_for(b.max_len);
  p.adj = adj;
  p.flags = flags;
  p.hdr = hdr;
  p.skip_empty = skip_empty ? 1 : 0;
  p.rec = pool ? pool->rec : nullptr;
  p.rec_cnt = pool ? pool->rec_cnt : nullptr;
  p.ovf = pool ? pool->ovf : nullptr;
  p.rec_per_tile = pool ? pool->rec_per_tile : 0;
  p.unit_rec_cap = pool ? rec_unit_capacity(ceil_div(b.max_len, kBN), pool->rec_per_tile) : 0;
  p.wait_cycles = wait_cycles;
  // behind a record pool the bit-matrix pass computes the overflowed units only: a few slots of blocks walk their list
  const bool listed = !emit && pool && pool->rec_per_tile > 0;
  p.work_list = listed ? pool->work_list : nullptr;
  p.n_work = listed ? pool->n_work : nullptr;
  p.n_units = units;
  const int spans = ceil_div(b.max_len, 2 * kBM);
  dim3 grid(2 * spans, listed ? std::min(units, kFallbackSlots) : units);   // whole pairs
  if (emit) {
    // as many pairs as the device runs at once, each walking its share of the (unit, fold) items
    int pairs = head_dim == 128 ? resident_pairs<128>() : resident_pairs<64>();
    if (pairs <= 0) return SPINDLEKV_CUDA;
    const Tuning tune = current_tuning();
    if (tune.sim_block_pairs > 0) pairs = std::min(pairs, tune.sim_block_pairs);
    const long long items = (long long)units * ((spans + 1) / 2);
    grid = dim3(2 * (unsigned)std::min<long long>(pairs, items), 1);
  }
  LaunchScope ls(listed ? KC_SIM_FALLBACK : KC_SIM, st);
  spindlekv_status rs;
  if (head_dim == 128) rs = emit ? launch_sim_tc_one<128, true>(map, emap, p, grid, st) : launch_sim_tc_one<128, false>(map, emap, p, grid, st);
  else rs = emit ? launch_sim_tc_one<64, true>(map, emap, p, grid, st) : launch_sim_tc_one<64, false>(map, emap, p, grid, st);
  if (rs != SPINDLEKV_OK) return rs;
  return cudaGetLastError() == cudaSuccess ? SPINDLEKV_OK : SPINDLEKV_CUDA;
}

}  // namespace skv

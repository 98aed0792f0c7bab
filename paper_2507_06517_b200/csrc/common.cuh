// Shared device/host helpers of the SpindleKV reduction library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spindlekv.h"

namespace skv {

// ---- status block at the start of every workspace -------------------------------------------
// word 0: device status, 1: greedy rounds used, 2: live tokens left, 3: units whose neighbour lists came from a bit matrix,
// 4: neighbour-list entries built from candidate records (both directions of every pair),
// the rest is unused.
constexpr int kHeaderBytes = 256;
constexpr int kHdrStatus = 0;
constexpr int kHdrRounds = 1;
constexpr int kHdrLive = 2;
constexpr int kHdrBitUnits = 3;
constexpr int kHdrListEntries = 4;

// kernel classes for launch counting / timing
enum KernelClass { KC_WINDOW = 0, KC_TOPK, KC_NORMS, KC_SIM, KC_DEGREE, KC_GREEDY, KC_FINAL, KC_GATHER, KC_SIM_FALLBACK, KC_DECODE, KC_COUNT };

struct View {  // device-side copy of spindlekv_tensor
  const void* ptr;
  int64_t sl, ss, sh, st;
};

inline View make_view(const spindlekv_tensor& t) { return View{t.ptr, t.stride_layer, t.stride_seq, t.stride_head, t.stride_tok}; }

struct Batch {  // device-side copy of spindlekv_batch
  int n_layers, n_seqs, max_len, total_len;
  const int32_t* cu;
  const int32_t* ll;   // lengths per layer [n_layers][n_seqs], or per unit [n_layers][n_seqs][ll_heads], or null
  int ll_heads;        // 0: `ll` is per layer and sequence; otherwise the number of heads it is indexed by
};

inline Batch make_batch(const spindlekv_batch& b) {
  return Batch{b.n_layers, b.n_seqs, b.max_len, b.total_len, b.cu_seqlens, b.layer_lens, b.layer_lens_heads};
}

// tokens of sequence s (head `head`) in layer `layer` of the call
__device__ __forceinline__ int seq_len(const Batch& b, int layer, int s, int head) {
  if (b.ll) {
    const int i = layer * b.n_seqs + s;
    return max(0, min(b.ll[b.ll_heads ? i * b.ll_heads + head : i], b.max_len));
  }
  return b.cu ? (b.cu[s + 1] - b.cu[s]) : b.max_len;
}
__device__ __forceinline__ int tok_base(const Batch& b, int s) { return b.cu ? b.cu[s] : s * b.max_len; }

// element offset of row 0 of (layer, seq, head)
__device__ __forceinline__ int64_t unit_offset(const View& v, const Batch& b, int layer, int s, int h) {
  int64_t off = (int64_t)layer * v.sl + (int64_t)h * v.sh;
  off += b.cu ? (int64_t)b.cu[s] * v.st : (int64_t)s * v.ss;
  return off;
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// 8 consecutive elements -> 8 floats (16-byte aligned source for bf16, 32-byte for fp32)
__device__ __forceinline__ void load8(const float* p, float* out) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float* out) {
  uint4 r = *reinterpret_cast<const uint4*>(p);
  uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
__host__ __device__ inline int row_words_for(int max_len) { return 4 * ((max_len + 127) / 128); }

// ---- candidate records of the similarity kernel ------------------------------------------------------
// A record is one non-zero word of the strict upper triangle of the adjacency: .x = row << kRecRowShift |
// word column (32 columns per word), .y = the word's bits.
constexpr int kRecRowShift = 11;   // word columns < 2048, i.e. sequences of fewer than 65536 tokens
// Record pool of a unit: the similarity kernel's row block `blk` of pair p = blk / 2 computes the tiles p .. T-1 (T tiles of 256
// columns for the call's longest sequence), so its region holds rec_per_tile * (T - p) records and
// starts after those of the blocks before it.
__host__ __device__ inline long long rec_region_offset(int blk, int T, int rec_per_tile) {
  const long long p = blk >> 1, r = blk & 1;
  return (long long)rec_per_tile * (2 * p * T - p * (p - 1) + r * (T - p));
}
__host__ __device__ inline long long rec_unit_capacity(int T, int rec_per_tile) { return (long long)rec_per_tile * T * (T + 1); }

struct SimRecordPool {   // device buffers of the candidate records of one CodeBook call
  uint2* rec;            // [units][rec_unit_capacity]
  int32_t* rec_cnt;      // [units][row blocks]
  int32_t* ovf;          // [units]
  int rec_per_tile;
  int32_t* work_list;    // [units] the units whose overflow flag is set, ascending (written before the bit-matrix pass)
  int32_t* n_work;       // [1] how many
};
constexpr int kFallbackSlots = 16;   // pairs of blocks per row span that the bit-matrix pass behind a record pool launches

// 32x32 bit transpose across a warp: in: lane r holds bits (r, c) at bit c; out: lane c holds bit r.
// Five butterfly stages (j = 16, 8, 4, 2, 1): a lane takes from its partner the half of every 2j-bit
// group that it does not keep, moved by j positions.  The move is a rotation (the bits that wrap
// around fall outside the kept mask), so a stage is one shuffle, one funnel shift and one logic op;
// rotation amounts and masks depend on the lane only and are set up once.
struct TransposeLane {
  uint32_t rot[5], keep[5];
  __device__ __forceinline__ void init(int lane) {
    uint32_t m = 0x0000FFFFu;
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      const int j = 16 >> k;
      const bool hi = (lane & j) != 0;
      keep[k] = hi ? ~m : m;
      rot[k] = hi ? 32 - j : j;
      m ^= m << (j >> 1);
    }
  }
  __device__ __forceinline__ uint32_t apply(uint32_t x) const {
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      const uint32_t y = __shfl_xor_sync(0xffffffffu, x, 16 >> k);
      const uint32_t r = __funnelshift_l(y, y, rot[k]);
      x = (x & keep[k]) | (r & ~keep[k]);
    }
    return x;
  }
};

// exclusive prefix sum of one int per thread over the block; returns the block total through `total`
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) warp_sums[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    int ws = lane < (int)((blockDim.x + 31) >> 5) ? warp_sums[lane] : 0;   // blocks of fewer than 32 warps
    int winc = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += n;
    }
    warp_sums[lane] = winc - ws;
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  int res = warp_sums[wid] + inc - v;
  total = warp_sums[32];
  __syncthreads();
  return res;
}

// Per-device "done once" flags for host-side set-up (function attributes, occupancy queries): the
// library may be used from several devices of one process.
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
  bool done[kMaxDevices] = {};
  // index of the current device, or -1
  static int current() {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices ? dev : -1;
  }
};

// ---- limits that tests may tighten (host) -----------------------------------------------------------
constexpr int kDefaultRecPerTile = 512;             // candidate records per 128 x 256 tile of a row block's region
constexpr long long kDefaultMbarWaitCycles = 4000000000ll;   // about two seconds of SM clock
struct Tuning {
  int rec_per_tile;          // 0: no candidate records, every unit goes through the bit matrix
  int round_cap;             // greedy rounds (never more than the sequence length)
  long long mbar_wait_cycles;
  int sim_block_pairs;       // pairs of blocks the candidate-record kernel runs on; 0: as many as the device holds
};
Tuning current_tuning();

// ---- launch bookkeeping (host) ---------------------------------------------------------------
void note_launch(int kclass, cudaStream_t st, bool before);
struct LaunchScope {
  int kc; cudaStream_t st;
  LaunchScope(int k, cudaStream_t s) : kc(k), st(s) { note_launch(kc, st, true); }
  ~LaunchScope() { note_launch(kc, st, false); }
};

}  // namespace skv

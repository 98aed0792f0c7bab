// C ABI of the SpindleKV reduction library: argument checks, the host-side budget planner,
// launch counting and optional per-kernel event timing.  Every device step lives in the kernels
// of evict.cu / codebook.cu / compact.cu.
#include <math.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "args.cuh"
#include "common.cuh"
#include "spindlekv_test_hooks.h"

namespace skv {
size_t evict_workspace_bytes(const spindlekv_config& cfg, const spindlekv_batch& b);
size_t codebook_workspace_bytes(const spindlekv_config& cfg, const spindlekv_batch& b);
spindlekv_status evict_deep_impl(const spindlekv_config& cfg, const spindlekv_batch& b, const spindlekv_tensor& K,
                                 const spindlekv_tensor& Q, const int32_t* k_ctx, int32_t* keep_idx,
                                 int32_t* keep_cnt, float* scores, void* ws, size_t ws_bytes, cudaStream_t st);
spindlekv_status codebook_shallow_impl(const spindlekv_config& cfg, const spindlekv_batch& b,
                                       const spindlekv_tensor& Gamma, float theta, float* mag, int32_t* ref,
                                       int32_t* centre_idx, int32_t* n_entries, uint32_t* adj_bits, void* ws,
                                       size_t ws_bytes, cudaStream_t st);
spindlekv_status compact_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& src,
                              const int32_t* idx, const int32_t* cnt, const float* divide_by,
                              const spindlekv_tensor& dst, const int32_t* dst_cu, cudaStream_t st);

spindlekv_status reconstruct_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& C,
                                  const int32_t* ref, const float* mag, const spindlekv_tensor& dst, cudaStream_t st);

spindlekv_status union_lists_impl(int n_layers, int n_seqs, int n_heads, int n_lists, int lists_inner, int t_in, int seq_in,
                                  const int32_t* idx_in, const int32_t* cnt_in, int t_out, int seq_out,
                                  int32_t* idx_out, int32_t* cnt_out, cudaStream_t st);

const void* noalloc_scratch_of_current_device();

spindlekv_status rope_table_impl(int head_dim, int n_pos, double base, void* table, cudaStream_t st);
size_t decode_workspace_bytes(const spindlekv_batch& b, int n_q_heads, int n_kv_heads, int head_dim);
spindlekv_status decode_attend_impl(const spindlekv_batch& b, int n_q_heads, int n_kv_heads, int head_dim,
                                    const spindlekv_tensor& q, const int32_t* pos_q, const spindlekv_tensor& CK,
                                    const int32_t* ref_k, const float* mag_k, const spindlekv_tensor& CV,
                                    const int32_t* ref_v, const float* mag_v, const int32_t* positions,
                                    const void* table, int table_positions, float* out, void* ws, size_t ws_bytes,
                                    cudaStream_t st);

size_t match_workspace_bytes(const spindlekv_batch& b, int n_heads);
spindlekv_status match_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& G,
                            const spindlekv_tensor& C, const int32_t* n_entries, int c_rows, float theta, float* mag,
                            int32_t* ref, int32_t* left_idx, int32_t* left_cnt, void* ws, size_t ws_bytes, cudaStream_t st);
spindlekv_status append_impl(const spindlekv_batch& b, int n_heads, int head_dim, const spindlekv_tensor& Lt,
                             const float* mag_left, const int32_t* ref_left, const int32_t* centre_left,
                             const int32_t* n_left_entries, const int32_t* left_idx, const int32_t* left_cnt,
                             const spindlekv_tensor& C, int c_rows, int32_t* n_entries, int32_t* ref_new, cudaStream_t st);

spindlekv_status selftest_mbarrier_impl(uint32_t* hdr, long long wait_cycles, cudaStream_t st);

// ---- limits that tests may tighten --------------------------------------------------------------
static std::mutex g_tune_mu;
static Tuning g_tuning{kDefaultRecPerTile, 0x7FFFFFFF, kDefaultMbarWaitCycles, 0};
Tuning current_tuning() {
  std::lock_guard<std::mutex> lk(g_tune_mu);
  return g_tuning;
}

// ---- launch counting and timing ---------------------------------------------------------------
static std::mutex g_mu;
static int64_t g_launches = 0;
static bool g_timing = false;
struct TimedLaunch { int kc; cudaEvent_t a, b; };
static std::vector<TimedLaunch> g_timed;
static std::vector<cudaEvent_t> g_pool;

static cudaEvent_t get_event() {
  if (!g_pool.empty()) { cudaEvent_t e = g_pool.back(); g_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

void note_launch(int kclass, cudaStream_t st, bool before) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (before) {
    ++g_launches;
    if (g_timing) {
      TimedLaunch t{kclass, get_event(), get_event()};
      cudaEventRecord(t.a, st);
      g_timed.push_back(t);
    }
  } else if (g_timing && !g_timed.empty()) {
    cudaEventRecord(g_timed.back().b, st);
  }
}
}  // namespace skv

using namespace skv;

extern "C" {

const char* spindlekv_status_string(spindlekv_status s) {
  switch (s) {
    case SPINDLEKV_OK: return "ok";
    case SPINDLEKV_INVALID_ARG: return "invalid argument";
    case SPINDLEKV_BUDGET: return "context reserve ratio outside (beta, 1]";
    case SPINDLEKV_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SPINDLEKV_CAPACITY: return "output capacity exceeded";
    case SPINDLEKV_UNSUPPORTED: return "unsupported shape, dtype or device";
    case SPINDLEKV_CUDA: return "CUDA runtime error";
    case SPINDLEKV_TIMEOUT: return "bounded device wait gave up";
    default: return "unknown status";
  }
}

spindlekv_status spindlekv_plan_layers(const spindlekv_config* cfg, int32_t n_seqs, const int32_t* seq_lens,
                                       int32_t* layer_mode, double* r_c_layer, int32_t* k_ctx) {
  if (!cfg_ok(cfg) || n_seqs <= 0 || !seq_lens || !layer_mode || !r_c_layer || !k_ctx) return SPINDLEKV_INVALID_ARG;
  const int m = cfg->n_layers;
  if (cfg->n_shallow < -1 || cfg->n_shallow > m) return SPINDLEKV_INVALID_ARG;
  const bool literal = cfg->n_shallow == -1;   // every layer evicts, then builds CodeBooks of what it kept
  const int n_shallow = literal ? 0 : cfg->n_shallow;
  const int m_deep = m - n_shallow;
  const double beta = cfg->beta;
  const double alpha = 0.5 * (1.0 + beta);
  for (int lam = 0; lam < m; ++lam)
    layer_mode[lam] = literal ? (SPINDLEKV_MODE_EVICT | SPINDLEKV_MODE_CODEBOOK)
                              : (lam < n_shallow ? SPINDLEKV_MODE_CODEBOOK : SPINDLEKV_MODE_EVICT);
  for (int s = 0; s < n_seqs; ++s) {
    const int l = seq_lens[s];
    const int l_c = l - cfg->window;
    if (l_c <= 0) return SPINDLEKV_INVALID_ARG;
    for (int lam = 0; lam < n_shallow; ++lam) {
      r_c_layer[(size_t)lam * n_seqs + s] = 1.0;
      k_ctx[(size_t)lam * n_seqs + s] = l_c;
    }
    if (m_deep == 0) continue;
    const double rl = cfg->budget_tokens >= 0.0 ? cfg->budget_tokens : cfg->reserve_ratio * (double)l;
    const double r_c = (rl - (double)cfg->window) / (double)l_c;
    double r_first, r_last;
    if (beta < r_c && r_c <= alpha) {
      r_first = 2.0 * r_c - beta;
      r_last = beta;
    } else if (alpha < r_c && r_c <= 1.0) {
      r_first = 1.0;
      r_last = 2.0 * r_c - 1.0;
    } else {
      return SPINDLEKV_BUDGET;
    }
    for (int lam = 0; lam < m_deep; ++lam) {
      const double r = m_deep == 1 ? r_c : r_first + (r_last - r_first) / (double)(m_deep - 1) * (double)lam;
      int k = (int)floor(r * (double)l_c);
      if (k > l_c) k = l_c;
      r_c_layer[(size_t)(n_shallow + lam) * n_seqs + s] = r;
      k_ctx[(size_t)(n_shallow + lam) * n_seqs + s] = k;
    }
  }
  return SPINDLEKV_OK;
}

spindlekv_status spindlekv_reserve_ratio(int32_t n_heads, int32_t seq_len, int32_t kept, const int32_t* entries_k,
                                         const int32_t* entries_v, double* r1, double* r2) {
  if (n_heads <= 0 || seq_len <= 0 || kept <= 0 || !entries_k || !entries_v || !r1 || !r2) return SPINDLEKV_INVALID_ARG;
  double sum_k = 0.0, sum_v = 0.0;
  for (int j = 0; j < n_heads; ++j) {
    sum_k += (double)entries_k[j];
    sum_v += (double)entries_v[j];
  }
  *r1 = (2.0 * (double)n_heads * (double)kept) / (2.0 * (double)n_heads * (double)seq_len);
  *r2 = (sum_k + sum_v) / (2.0 * (double)n_heads * (double)kept);
  return SPINDLEKV_OK;
}

size_t spindlekv_workspace_bytes(const spindlekv_config* cfg, const spindlekv_batch* batch, int32_t which) {
  if (!cfg_ok(cfg) || !batch_ok(batch, cfg->window)) return 0;
  if (which == SPINDLEKV_WS_EVICT) return evict_workspace_bytes(*cfg, *batch);
  if (which == SPINDLEKV_WS_CODEBOOK) return codebook_workspace_bytes(*cfg, *batch);
  return 0;
}

spindlekv_status spindlekv_evict_deep(const spindlekv_config* cfg, const spindlekv_batch* batch, spindlekv_tensor K,
                                      spindlekv_tensor Qwin, const int32_t* k_ctx, int32_t* keep_idx,
                                      int32_t* keep_cnt, float* scores, void* ws, size_t ws_bytes, void* stream) {
  const spindlekv_status as = evict_args_status(cfg, batch, K, Qwin, k_ctx, keep_idx, keep_cnt, scores);
  if (as != SPINDLEKV_OK) return as;
  if (!ws || reinterpret_cast<uintptr_t>(ws) % 256) return SPINDLEKV_INVALID_ARG;
  return evict_deep_impl(*cfg, *batch, K, Qwin, k_ctx, keep_idx, keep_cnt, scores, ws, ws_bytes, (cudaStream_t)stream);
}

spindlekv_status spindlekv_codebook_shallow(const spindlekv_config* cfg, const spindlekv_batch* batch,
                                            spindlekv_tensor Gamma, float theta, float* mag, int32_t* ref,
                                            int32_t* centre_idx, int32_t* n_entries, uint32_t* adj_bits, void* ws,
                                            size_t ws_bytes, void* stream) {
  if (!cfg_ok(cfg) || !batch) return SPINDLEKV_INVALID_ARG;
  if (batch->n_layers <= 0 || batch->n_seqs <= 0 || batch->max_len <= 0 || batch->total_len < batch->max_len) return SPINDLEKV_INVALID_ARG;
  if (!batch->cu_seqlens && (int64_t)batch->total_len != (int64_t)batch->n_seqs * batch->max_len) return SPINDLEKV_INVALID_ARG;
  if (batch->layer_lens && batch->cu_seqlens) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(Gamma) || !mag || !ref || !centre_idx || !n_entries || !ws) return SPINDLEKV_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) % 256) return SPINDLEKV_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(adj_bits) % 16) return SPINDLEKV_INVALID_ARG;   // rows are moved 16 bytes at a time
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  return codebook_shallow_impl(*cfg, *batch, Gamma, theta, mag, ref, centre_idx, n_entries, adj_bits, ws, ws_bytes,
                               (cudaStream_t)stream);
}

spindlekv_status spindlekv_compact(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                   spindlekv_tensor src, const int32_t* idx, const int32_t* cnt,
                                   const float* divide_by, spindlekv_tensor dst, const int32_t* dst_cu_seqlens,
                                   void* stream) {
  if (!batch || batch->n_layers <= 0 || batch->n_seqs <= 0 || batch->max_len <= 0 || n_heads <= 0) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(src) || !tensor_ok(dst) || !idx || !cnt) return SPINDLEKV_INVALID_ARG;
  if (src.dtype != dst.dtype) return SPINDLEKV_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  return compact_impl(*batch, n_heads, head_dim, src, idx, cnt, divide_by, dst, dst_cu_seqlens, (cudaStream_t)stream);
}

spindlekv_status spindlekv_union_lists(int32_t n_layers, int32_t n_seqs, int32_t n_heads, int32_t n_lists, int32_t lists_inner,
                                       int32_t t_in, int32_t seq_in, const int32_t* idx_in, const int32_t* cnt_in,
                                       int32_t t_out, int32_t seq_out, int32_t* idx_out, int32_t* cnt_out, void* stream) {
  if (n_layers <= 0 || n_seqs <= 0 || n_heads <= 0 || n_lists <= 0 || t_in <= 0 || t_out <= 0) return SPINDLEKV_INVALID_ARG;
  if (seq_in <= 0 || seq_out <= 0 || (int64_t)n_seqs * seq_in > t_in || (int64_t)n_seqs * seq_out > t_out) return SPINDLEKV_INVALID_ARG;
  if (!idx_in || !cnt_in || !idx_out || !cnt_out) return SPINDLEKV_INVALID_ARG;
  if ((int64_t)n_layers * n_seqs * n_heads > 0x7FFFFFFF) return SPINDLEKV_UNSUPPORTED;
  return union_lists_impl(n_layers, n_seqs, n_heads, n_lists, lists_inner, t_in, seq_in, idx_in, cnt_in, t_out, seq_out, idx_out,
                          cnt_out, (cudaStream_t)stream);
}

static bool new_batch_ok(const spindlekv_batch* b) {
  if (!b || b->n_layers <= 0 || b->n_seqs <= 0 || b->max_len <= 0 || b->cu_seqlens) return false;
  return (int64_t)b->total_len == (int64_t)b->n_seqs * b->max_len;
}

size_t spindlekv_match_workspace_bytes(const spindlekv_batch* batch, int32_t n_heads) {
  if (!new_batch_ok(batch) || n_heads <= 0) return 0;
  return match_workspace_bytes(*batch, n_heads);
}

spindlekv_status spindlekv_codebook_match(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                          spindlekv_tensor Gamma_new, spindlekv_tensor C, const int32_t* n_entries,
                                          int32_t c_rows, float theta, float* mag_new, int32_t* ref_new,
                                          int32_t* left_idx, int32_t* left_cnt, void* ws, size_t ws_bytes, void* stream) {
  if (!new_batch_ok(batch) || n_heads <= 0 || c_rows <= 0) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(Gamma_new) || !tensor_ok(C) || !n_entries || !mag_new || !ref_new || !left_idx || !left_cnt || !ws)
    return SPINDLEKV_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) % 256) return SPINDLEKV_INVALID_ARG;
  if (Gamma_new.dtype != C.dtype) return SPINDLEKV_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  return match_impl(*batch, n_heads, head_dim, Gamma_new, C, n_entries, c_rows, theta, mag_new, ref_new, left_idx,
                    left_cnt, ws, ws_bytes, (cudaStream_t)stream);
}

spindlekv_status spindlekv_codebook_append(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                           spindlekv_tensor Gamma_left, const float* mag_left, const int32_t* ref_left,
                                           const int32_t* centre_left, const int32_t* n_left_entries,
                                           const int32_t* left_idx, const int32_t* left_cnt, spindlekv_tensor C,
                                           int32_t c_rows, int32_t* n_entries, int32_t* ref_new, void* stream) {
  if (!new_batch_ok(batch) || n_heads <= 0 || c_rows <= 0) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(Gamma_left) || !tensor_ok(C) || !mag_left || !ref_left || !centre_left || !n_left_entries || !left_idx ||
      !left_cnt || !n_entries || !ref_new)
    return SPINDLEKV_INVALID_ARG;
  if (Gamma_left.dtype != C.dtype) return SPINDLEKV_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  if ((int64_t)batch->n_layers * batch->n_seqs * n_heads > 0x7FFFFFFF) return SPINDLEKV_UNSUPPORTED;
  return append_impl(*batch, n_heads, head_dim, Gamma_left, mag_left, ref_left, centre_left, n_left_entries, left_idx,
                     left_cnt, C, c_rows, n_entries, ref_new, (cudaStream_t)stream);
}

spindlekv_status spindlekv_reconstruct(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                       spindlekv_tensor C, const int32_t* ref, const float* mag, spindlekv_tensor dst,
                                       void* stream) {
  if (!batch || batch->n_layers <= 0 || batch->n_seqs <= 0 || batch->max_len <= 0 || n_heads <= 0) return SPINDLEKV_INVALID_ARG;
  if (batch->layer_lens && batch->cu_seqlens) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(C) || !tensor_ok(dst) || !ref || !mag) return SPINDLEKV_INVALID_ARG;
  if (C.dtype != dst.dtype) return SPINDLEKV_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  return reconstruct_impl(*batch, n_heads, head_dim, C, ref, mag, dst, (cudaStream_t)stream);
}

size_t spindlekv_rope_table_bytes(int32_t head_dim, int32_t n_positions) {
  if ((head_dim != 64 && head_dim != 128) || n_positions <= 0) return 0;
  return (size_t)n_positions * (head_dim / 2) * sizeof(float) * 2;
}

spindlekv_status spindlekv_rope_table(int32_t head_dim, int32_t n_positions, double base, void* table, void* stream) {
  if (!table || n_positions <= 0 || !(base > 1.0) || reinterpret_cast<uintptr_t>(table) % 16) return SPINDLEKV_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  return rope_table_impl(head_dim, n_positions, base, table, (cudaStream_t)stream);
}

static bool decode_batch_ok(const spindlekv_batch* b) {
  if (!b || b->n_layers <= 0 || b->n_seqs <= 0 || b->max_len <= 0 || b->cu_seqlens) return false;
  return (int64_t)b->total_len == (int64_t)b->n_seqs * b->max_len;
}

size_t spindlekv_decode_workspace_bytes(const spindlekv_batch* batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim) {
  if (!decode_batch_ok(batch) || n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads) return 0;
  if (head_dim != 64 && head_dim != 128) return 0;
  return decode_workspace_bytes(*batch, n_q_heads, n_kv_heads, head_dim);
}

spindlekv_status spindlekv_decode_attend(const spindlekv_batch* batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                         spindlekv_tensor q, const int32_t* pos_q,
                                         spindlekv_tensor C_K, const int32_t* ref_K, const float* mag_K,
                                         spindlekv_tensor C_V, const int32_t* ref_V, const float* mag_V,
                                         const int32_t* positions, const void* rope_table, int32_t table_positions,
                                         float* out, void* ws, size_t ws_bytes, void* stream) {
  if (!decode_batch_ok(batch) || n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(q) || !tensor_ok(C_K) || !tensor_ok(C_V) || !pos_q || !ref_K || !mag_K || !ref_V || !mag_V || !rope_table ||
      table_positions <= 0 || !out || !ws)
    return SPINDLEKV_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(ws) % 256 || reinterpret_cast<uintptr_t>(rope_table) % 16) return SPINDLEKV_INVALID_ARG;
  if (q.dtype != C_K.dtype || q.dtype != C_V.dtype) return SPINDLEKV_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  if (n_q_heads / n_kv_heads > 8) return SPINDLEKV_UNSUPPORTED;
  return decode_attend_impl(*batch, n_q_heads, n_kv_heads, head_dim, q, pos_q, C_K, ref_K, mag_K, C_V, ref_V, mag_V, positions,
                            rope_table, table_positions, out, ws, ws_bytes, (cudaStream_t)stream);
}

spindlekv_status spindlekv_poll_status(const void* ws, int32_t* device_status, int32_t* detail) {
  if (!device_status) return SPINDLEKV_INVALID_ARG;
  if (!ws) ws = noalloc_scratch_of_current_device();   // NULL: the built-in scratch of the allocation-free entry point
  if (!ws) return SPINDLEKV_INVALID_ARG;
  int32_t h[8];
  if (cudaMemcpy(h, ws, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return SPINDLEKV_CUDA;
  *device_status = h[kHdrStatus];
  if (detail) { detail[0] = h[kHdrRounds]; detail[1] = h[kHdrLive]; detail[2] = h[kHdrBitUnits]; detail[3] = h[kHdrListEntries]; }
  return SPINDLEKV_OK;
}

spindlekv_status spindlekv_set_tuning(int32_t key, int64_t value) {
  std::lock_guard<std::mutex> lk(g_tune_mu);
  switch (key) {
    case SPINDLEKV_TUNE_RECORDS_PER_TILE:
      g_tuning.rec_per_tile = value < 0 ? kDefaultRecPerTile : (int)std::min<int64_t>(value, kDefaultRecPerTile);
      return SPINDLEKV_OK;
    case SPINDLEKV_TUNE_GREEDY_ROUND_CAP:
      g_tuning.round_cap = value < 0 ? 0x7FFFFFFF : (int)std::min<int64_t>(value, 0x7FFFFFFF);
      return SPINDLEKV_OK;
    case SPINDLEKV_TUNE_MBAR_WAIT_CYCLES:
      g_tuning.mbar_wait_cycles = value < 0 ? kDefaultMbarWaitCycles : value;
      return SPINDLEKV_OK;
    case SPINDLEKV_TUNE_SIM_BLOCK_PAIRS:
      g_tuning.sim_block_pairs = value < 0 ? 0 : (int)std::min<int64_t>(value, 1 << 20);
      return SPINDLEKV_OK;
    default:
      return SPINDLEKV_INVALID_ARG;
  }
}

int64_t spindlekv_get_tuning(int32_t key) {
  const Tuning t = current_tuning();
  switch (key) {
    case SPINDLEKV_TUNE_RECORDS_PER_TILE: return t.rec_per_tile;
    case SPINDLEKV_TUNE_GREEDY_ROUND_CAP: return t.round_cap;
    case SPINDLEKV_TUNE_MBAR_WAIT_CYCLES: return t.mbar_wait_cycles;
    case SPINDLEKV_TUNE_SIM_BLOCK_PAIRS: return t.sim_block_pairs;
    default: return -1;
  }
}

spindlekv_status spindlekv_selftest_mbarrier_timeout(void* ws, int64_t limit, void* stream) {
  if (!ws || reinterpret_cast<uintptr_t>(ws) % 256 || limit < 1 || limit > kDefaultMbarWaitCycles) return SPINDLEKV_INVALID_ARG;
  return selftest_mbarrier_impl(reinterpret_cast<uint32_t*>(ws), (long long)limit, (cudaStream_t)stream);
}

int64_t spindlekv_launch_count(int32_t reset) {
  std::lock_guard<std::mutex> lk(g_mu);
  int64_t v = g_launches;
  if (reset) g_launches = 0;
  return v;
}

void spindlekv_timing_enable(int32_t on) {
  std::lock_guard<std::mutex> lk(g_mu);
  for (auto& t : g_timed) { g_pool.push_back(t.a); g_pool.push_back(t.b); }
  g_timed.clear();
  g_timing = on != 0;
}

spindlekv_status spindlekv_timing_read(int32_t which, double* ms_total, int64_t* launches) {
  if (!ms_total || !launches || which < 0 || which >= KC_COUNT) return SPINDLEKV_INVALID_ARG;
  std::lock_guard<std::mutex> lk(g_mu);
  double tot = 0.0;
  int64_t n = 0;
  for (auto& t : g_timed) {
    if (t.kc != which) continue;
    if (cudaEventSynchronize(t.b) != cudaSuccess) return SPINDLEKV_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, t.a, t.b) != cudaSuccess) return SPINDLEKV_CUDA;
    tot += ms;
    ++n;
  }
  *ms_total = tot;
  *launches = n;
  return SPINDLEKV_OK;
}

}  // extern "C"

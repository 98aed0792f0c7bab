// Argument checks shared by the entry points (host only).  Every check runs before anything is
// enqueued, so a rejected call leaves the device untouched.
#pragma once

#include <stdint.h>

#include "spindlekv.h"

namespace skv {

inline bool tensor_ok(const spindlekv_tensor& t) {
  if (!t.ptr) return false;
  if (t.dtype != SPINDLEKV_F32 && t.dtype != SPINDLEKV_BF16) return false;
  if (reinterpret_cast<uintptr_t>(t.ptr) % 16) return false;   // rows are read 16 bytes at a time
  if (t.stride_layer % 8 || t.stride_seq % 8 || t.stride_head % 8 || t.stride_tok % 8) return false;
  return true;
}

inline bool cfg_ok(const spindlekv_config* c) {
  if (!c) return false;
  if (c->n_layers <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->window <= 0) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  return true;
}

inline bool batch_ok(const spindlekv_batch* b, int window) {
  if (!b) return false;
  if (b->layer_lens && b->cu_seqlens) return false;
  if (b->n_layers <= 0 || b->n_seqs <= 0 || b->max_len <= window || b->total_len < b->max_len) return false;
  if (!b->cu_seqlens && (int64_t)b->total_len != (int64_t)b->n_seqs * b->max_len) return false;
  return true;
}

// Everything spindlekv_evict_deep and spindlekv_evict_deep_noalloc have in common (the workspace is
// checked by the caller).
inline spindlekv_status evict_args_status(const spindlekv_config* cfg, const spindlekv_batch* batch,
                                          const spindlekv_tensor& K, const spindlekv_tensor& Qwin, const int32_t* k_ctx,
                                          const int32_t* keep_idx, const int32_t* keep_cnt, const float* scores) {
  if (!cfg_ok(cfg) || !batch_ok(batch, cfg->window)) return SPINDLEKV_INVALID_ARG;
  if (!tensor_ok(K) || !tensor_ok(Qwin) || !k_ctx || !keep_idx || !keep_cnt || !scores) return SPINDLEKV_INVALID_ARG;
  if (K.dtype != Qwin.dtype) return SPINDLEKV_UNSUPPORTED;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return SPINDLEKV_UNSUPPORTED;
  const int64_t out_heads = cfg->per_query_head ? cfg->n_q_heads : cfg->n_kv_heads;   // heads that select on their own
  if ((int64_t)batch->n_layers * batch->n_seqs * out_heads > 65535) return SPINDLEKV_UNSUPPORTED;
  return SPINDLEKV_OK;
}

}  // namespace skv

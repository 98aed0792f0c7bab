/*
 * spindlekv.h -- C ABI of the B200 (sm_100a) SpindleKV prefill KV-cache reduction pass.
 *
 * The pass runs once per layer after prompt encoding (Section 3 of the paper):
 *   deep layers    : attention-weight based token eviction  (Section 3.3, Eq. (1)(2)(3)(7));
 *   shallow layers : similarity based token replacement by a CodeBook (Section 3.4, Eq. (4), (8)-(13),
 *                    Algorithm 1).
 * Layers do not interact, so every call takes a batch of layers.
 *
 * Conventions shared by all entry points
 *   - Plain C: pointers, sizes, two small structs.  No allocation inside the library: the caller
 *     owns every buffer, including the scratch workspace (size from spindlekv_workspace_bytes).
 *   - "device" pointers are CUDA global memory of the current device; "host" pointers are ordinary
 *     host memory.  `stream` is a cudaStream_t passed as void*.
 *   - Device work is only enqueued; the functions return as soon as the launches are issued.  The
 *     return value reports argument / launch errors.  Conditions detected on the device (a bounded
 *     wait that gave up) land in a status word at the start of the workspace, read back with
 *     spindlekv_poll_status after the caller has synchronised the stream.
 *   - Tensors are addressed as
 *         ptr + layer*stride_layer + seq*stride_seq + head*stride_head + row*stride_tok   (+ 0..head_dim-1)
 *     with strides in ELEMENTS and head_dim contiguous.  When `cu_seqlens` is given (packed,
 *     variable-length batch) token t of sequence s lives at row cu_seqlens[s] + t and stride_seq
 *     is ignored for that tensor; otherwise every sequence has max_len tokens.
 *   - Per-token outputs (scores, keep_idx, mag, ref, centre_idx) are laid out [n_layers][n_kv_heads][T]
 *     where T = cu_seqlens[B] (packed) or B*max_len, and sequence s starts at column
 *     tok_base(s) = cu_seqlens[s] (packed) or s*max_len.  Per-unit counts are [n_layers][B][n_kv_heads].
 *   - head_dim must be 64 or 128; dtype fp32 or bf16; base pointers 16-byte aligned and
 *     strides multiples of 8 elements.
 *   - Nothing is written out of bounds on any error; outputs are undefined after a non-OK status.
 */
#ifndef SPINDLEKV_H_
#define SPINDLEKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t spindlekv_status;
enum {
  SPINDLEKV_OK = 0,
  SPINDLEKV_INVALID_ARG = 1,         /* null pointer, non-positive size, bad stride or alignment */
  SPINDLEKV_BUDGET = 2,              /* context reserve ratio outside (beta, 1], where Eq. (5) is undefined */
  SPINDLEKV_WORKSPACE_TOO_SMALL = 3,
  SPINDLEKV_CAPACITY = 4,            /* an output row is too short for what must be written */
  SPINDLEKV_UNSUPPORTED = 5,         /* head_dim, dtype, sequence length or device not supported */
  SPINDLEKV_CUDA = 6,                /* a CUDA runtime call failed */
  SPINDLEKV_TIMEOUT = 7              /* a bounded device-side wait gave up (device status word only) */
};

enum { SPINDLEKV_F32 = 0, SPINDLEKV_BF16 = 1 };
enum { SPINDLEKV_MODE_EVICT = 1, SPINDLEKV_MODE_CODEBOOK = 2 };
enum { SPINDLEKV_WS_EVICT = 0, SPINDLEKV_WS_CODEBOOK = 1 };

typedef struct {
  void* ptr;            /* device */
  int32_t dtype;        /* SPINDLEKV_F32 or SPINDLEKV_BF16 */
  int64_t stride_layer; /* elements */
  int64_t stride_seq;
  int64_t stride_head;
  int64_t stride_tok;
} spindlekv_tensor;

/* Hyper-parameters of the method (Table 3: theta_K 0.98, theta_V 0.95, beta 0.05) and model shape. */
typedef struct {
  int32_t n_layers;
  int32_t n_q_heads;      /* h   */
  int32_t n_kv_heads;     /* h_g; query head h_n*j+g reads KV head j, h_n = h / h_g */
  int32_t head_dim;       /* d_h */
  int32_t window;         /* l_w: the last l_w tokens are the observation window and are always reserved */
  int32_t n_shallow;      /* layers [0, n_shallow) build CodeBooks; layers [n_shallow, n_layers) evict;
                             -1: the composition of Section 3 as written: every layer evicts under the pyramid
                             of Eq. (5)(6) laid over all layers and then builds CodeBooks of what it kept */
  double reserve_ratio;   /* r of Section 3.3 (used when budget_tokens < 0) */
  double budget_tokens;   /* r*l given directly: tokens kept per head, window included; < 0: use reserve_ratio */
  double beta;            /* minimal retain ratio of any layer */
  float theta_k;          /* similarity thresholds of Eq. (9) */
  float theta_v;
  int32_t score_norm;     /* 0: divide by (l - a) as Eq. (2) prints; 1: plain window sum (not in the paper) */
  int32_t per_query_head; /* 0: scores are the group mean of Eq. (3) and every KV head selects once;
                             1: the GQA "repeat" alternative of Section 3.3: the KV vectors count once per query head,
                             every query head i selects with its own ac_i of Eq. (2); the per-head outputs of
                             spindlekv_evict_deep (scores, keep_idx, keep_cnt) are then indexed by query head */
} spindlekv_config;

/* Which layers and sequences one device call covers. */
typedef struct {
  int32_t n_layers;            /* layers in this call (tensor strides step through them) */
  int32_t n_seqs;              /* B */
  int32_t max_len;             /* longest sequence, l */
  int32_t total_len;           /* cu_seqlens[B] when packed, else B*max_len */
  const int32_t* cu_seqlens;   /* device [B+1], or NULL when all sequences have max_len tokens */
  const int32_t* layer_lens;   /* device [n_layers][B], or NULL.  When given (only without cu_seqlens): sequence s
                                  has layer_lens[layer*B + s] <= max_len tokens in layer `layer` of the call, rows
                                  still max_len apart.  This is how the CodeBook call takes the tokens that
                                  eviction kept, whose number differs from layer to layer (Eq. (5)(6)). */
  int32_t layer_lens_heads;    /* 0: layer_lens is indexed [layer][seq].  H > 0: it is indexed [layer][seq][head]
                                  with H heads per sequence (lengths that differ from head to head, e.g. the new
                                  tokens that found no CodeBook entry); a length may be 0. */
} spindlekv_batch;

/*
 * Budget planner, host only (Section 3.3: r_c = (r*l - l_w)/l_c; Eq. (5) with alpha = (1+beta)/2, read
 * as r_c(0) = 2 r_c - beta | 1 and r_c(m-1) = beta | 2 r_c - 1; Eq. (6); k = floor(r_c(lambda) * l_c), Eq. (7)).
 * The pyramid is laid over the evicting layers [n_shallow, n_layers); all arithmetic in IEEE double
 * in the order the equations print.
 *   seq_lens   host [B]
 *   layer_mode host out [n_layers]      SPINDLEKV_MODE_*
 *   r_c_layer  host out [n_layers][B]   retain ratio of the context (1 for CodeBook layers)
 *   k_ctx      host out [n_layers][B]   context tokens kept per head (l_c for CodeBook layers)
 * Returns BUDGET when some sequence has r_c <= beta or r_c > 1, INVALID_ARG when l <= l_w.
 */
spindlekv_status spindlekv_plan_layers(const spindlekv_config* cfg, int32_t n_seqs, const int32_t* seq_lens,
                                       int32_t* layer_mode, double* r_c_layer, int32_t* k_ctx);

/*
 * Reserve ratios of one layer, host only (Eq. (15) without its storage-type factor r3):
 *   r1 = kept K and V tokens over all K and V tokens      = (2 h kept) / (2 h l)
 *   r2 = CodeBook entries of K and V over kept K and V tokens = (sum_j |C_K,j| + sum_j |C_V,j|) / (2 h kept)
 * with h = n_heads heads (the KV heads; the query heads when GQA was unfolded), l = seq_len tokens per head
 * before the pass and `kept` tokens per head after eviction.  The layer keeps r1 * r2 of its cache rows.
 *   entries_k, entries_v  host [n_heads]: CodeBook sizes per head
 * INVALID_ARG for null pointers or non-positive sizes.
 */
spindlekv_status spindlekv_reserve_ratio(int32_t n_heads, int32_t seq_len, int32_t kept, const int32_t* entries_k,
                                         const int32_t* entries_v, double* r1, double* r2);

/* Bytes of device scratch the given call kind (SPINDLEKV_WS_*) needs for `batch`.  0 on bad arguments. */
size_t spindlekv_workspace_bytes(const spindlekv_config* cfg, const spindlekv_batch* batch, int32_t which);

/*
 * Eviction of deep layers (Eq. (1): causal softmax of the window queries over keys 0..b, scale 1/sqrt(d_h);
 * Eq. (2): per-key sum over the l_w window queries divided by (l - a); Eq. (3): mean over the h_n query
 * heads of a group; Eq. (7): argTopK with k = k_ctx, ties to the lower index).
 *   K        device, [layer][seq][kv head][token][d]
 *   Qwin     device, [layer][seq][q head][window row][d] (rows are the queries at positions l-l_w .. l-1;
 *            never packed: stride_seq always applies)
 *   k_ctx    device [n_layers][B]
 *   keep_idx device out [n_layers][n_kv_heads][T]: per unit, from tok_base(s): the k selected context
 *            positions ascending, then the l_w window positions
 *   keep_cnt device out [n_layers][B][n_kv_heads] = k + l_w
 *   scores   device out [n_layers][n_kv_heads][T] fp32: ac' of Eq. (3) for context positions
 *            (window columns are left untouched); may not be NULL
 * With cfg->per_query_head = 1 the three outputs have n_q_heads in place of n_kv_heads (query head h_n*j + g reads
 * KV head j), scores hold ac_i of Eq. (2), and every query head keeps its own k_ctx positions.
 */
spindlekv_status spindlekv_evict_deep(const spindlekv_config* cfg, const spindlekv_batch* batch,
                                      spindlekv_tensor K, spindlekv_tensor Qwin, const int32_t* k_ctx,
                                      int32_t* keep_idx, int32_t* keep_cnt, float* scores,
                                      void* ws, size_t ws_bytes, void* stream);

/*
 * The same eviction as spindlekv_evict_deep for callers that cannot allocate device memory (the paper
 * has no counterpart: this is a deployment convenience).  Typical callers: an inference server whose
 * own pool has claimed the whole GPU, code running under another framework's allocator lock, or a
 * latency-critical thread that must not trigger the implicit synchronisation of an allocation.  The
 * scratch the kernels need is a fixed array of SPINDLEKV_NOALLOC_SCRATCH_BYTES inside the library
 * image (present on every GPU that loads the library, until the process exits), so no workspace is
 * passed and the function never calls cudaMalloc/cudaFree or any allocating routine.
 *   - Arguments as spindlekv_evict_deep, minus the workspace, and checked in the same way (same
 *     status codes for null pointers, misaligned bases, strides that are not multiples of 8, unknown
 *     dtypes, inconsistent batches) before anything is enqueued.
 *   - Returns WORKSPACE_TOO_SMALL when the scratch this call would really use exceeds
 *     SPINDLEKV_NOALLOC_SCRATCH_BYTES: split the layers over several calls.  bf16 inputs whose window
 *     is 16, 32, 64 or 128 with at most 256 query rows per KV head run on the tensor-core kernel,
 *     which needs the status block only, so any batch fits; other inputs need
 *     spindlekv_workspace_bytes(cfg, batch, SPINDLEKV_WS_EVICT), e.g. about four fp32 layers of
 *     8 x 16k tokens.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.  With lazy module loading the same first call
 *     is what makes the array resident on the device: let it happen before the host's own pool
 *     claims the rest of the memory.
 *   - All calls share the one array, which keeps the previous call's contents; what must start at
 *     zero is cleared by the call itself.  Two calls whose kernels overlap on the GPU (different
 *     streams, no ordering between them) race on it: order them.
 *   - The device status word of the last call (a bounded wait that gave up) is read with
 *     spindlekv_poll_status(NULL, ...) after synchronising the stream, with the same device current.
 */
#define SPINDLEKV_NOALLOC_SCRATCH_BYTES (8 * 1024 * 1024)
spindlekv_status spindlekv_evict_deep_noalloc(const spindlekv_config* cfg, const spindlekv_batch* batch,
                                              spindlekv_tensor K, spindlekv_tensor Qwin, const int32_t* k_ctx,
                                              int32_t* keep_idx, int32_t* keep_cnt, float* scores, void* stream);

/*
 * CodeBook construction for shallow layers, one call per Gamma in {K, V} (Algorithm 1):
 * magnitudes (Eq. (8)); cosine similarity of all token pairs of a head (Eq. (4)); adjacency
 * G = [S > theta] with unit diagonal (Eq. (9)); then repeatedly: degrees (Eq. (10)), centre = arg-max
 * degree with ties to the lower index (Eq. (11)), every live neighbour of the centre refers to the new
 * entry (Eq. (12)), centre and neighbours leave the graph (Eq. (13)), until the graph is empty.
 * The decision S > theta is taken in fp32 as  dot(a,b) > theta * (|a| * |b|).
 *   Gamma      device, [layer][seq][kv head][token][d]
 *   mag        device out [n_layers][n_kv_heads][T] fp32   |gamma_a|
 *   ref        device out [n_layers][n_kv_heads][T] int32  CodeBook entry of each token
 *   centre_idx device out [n_layers][n_kv_heads][T] int32  per unit, from tok_base(s): token position of
 *              entry 0, 1, ... (the CodeBook itself is these rows divided by their magnitude: see
 *              spindlekv_compact)
 *   n_entries  device out [n_layers][B][n_kv_heads]
 *   adj_bits   device out, optional (NULL: kept in the workspace): the adjacency as a bit matrix,
 *              [n_layers*B*n_kv_heads][max_len][row_words] uint32, row_words = 4*ceil(max_len/128);
 *              bit (b & 31) of word b >> 5 of row a is G[a][b]; rows and words beyond a sequence's own
 *              length are not written; 16-byte aligned, else INVALID_ARG.  With NULL the matrix in the
 *              workspace is sparse: 64-column chunks of a row without a set bit may be left unwritten
 * Limits: sequences of at most 32768 tokens and at most 65535 (layer, sequence, head) units per call, else
 * UNSUPPORTED; two calls may run at the same time on different streams when each has a workspace of its own.
 * A bounded device wait that gave up, or a greedy cover that exceeded its round limit, leaves TIMEOUT in the
 * workspace's status word (spindlekv_poll_status), never an endless wait.
 */
spindlekv_status spindlekv_codebook_shallow(const spindlekv_config* cfg, const spindlekv_batch* batch,
                                            spindlekv_tensor Gamma, float theta,
                                            float* mag, int32_t* ref, int32_t* centre_idx, int32_t* n_entries,
                                            uint32_t* adj_bits, void* ws, size_t ws_bytes, void* stream);

/*
 * Gather rows into the output cache (Eq. (7), Gamma_r = Gamma[eta]; Eq. (11), C <- C + [gamma_hat_iota]).
 * For every (layer, seq, head) copies rows idx[0..cnt) of `src` to rows 0..cnt of `dst`.
 *   idx        device [n_layers][n_heads][T] as written by the two calls above
 *   cnt        device [n_layers][B][n_heads]
 *   divide_by  device, optional [n_layers][n_heads][T] fp32: when given, source row a is divided by
 *              divide_by[a] (in fp32, as a product with the correctly rounded reciprocal, then rounded to the
 *              storage type; a zero divisor yields a zero row); pass `mag` to obtain unit CodeBook vectors
 *   dst        device, same addressing rules as src; when dst_cu_seqlens is given, unit s starts at row
 *              dst_cu_seqlens[s] of dst, else rows are addressed like src (batch->cu_seqlens or stride_seq)
 * src and dst must have the same dtype and may not overlap.
 */
spindlekv_status spindlekv_compact(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                   spindlekv_tensor src, const int32_t* idx, const int32_t* cnt,
                                   const float* divide_by, spindlekv_tensor dst, const int32_t* dst_cu_seqlens,
                                   void* stream);

/*
 * Joins the kept-token lists of several eviction passes over the same KV heads (Section 3.3, the GQA
 * "repeat" alternative: the KV vectors are repeated h_n times, every query head of a group selects on its
 * own, and the CodeBook of Section 3.4 is built from all selections of the group, where repeated
 * tokens have cosine similarity 1 and share an entry).  For every (layer, seq, head): out list = list of
 * pass 0, then of pass 1, ...; out count = sum of the counts (clipped to seq_out).  Equal-length batches only.
 *   idx_in  device [n_lists][n_layers][n_heads][t_in], sequence s starting at column s * seq_in
 *   cnt_in  device [n_lists][n_layers][n_seqs][n_heads]
 *           (lists_inner = 1: [n_layers][n_heads][n_lists][t_in] and [n_layers][n_seqs][n_heads][n_lists], i.e. the
 *           per-query-head outputs of one spindlekv_evict_deep call with per_query_head = 1, n_lists = h_n)
 *   idx_out device [n_layers][n_heads][t_out], sequence s starting at column s * seq_out
 *   cnt_out device [n_layers][n_seqs][n_heads]
 */
spindlekv_status spindlekv_union_lists(int32_t n_layers, int32_t n_seqs, int32_t n_heads, int32_t n_lists, int32_t lists_inner,
                                       int32_t t_in, int32_t seq_in, const int32_t* idx_in, const int32_t* cnt_in,
                                       int32_t t_out, int32_t seq_out, int32_t* idx_out, int32_t* cnt_out, void* stream);

/*
 * Decode-time merging of new tokens into existing CodeBooks (Section 3.4, last paragraph: new entries of the
 * cache first look for a suitable CodeBook entry, with theta as the threshold; those that find one are
 * merged into it, for the others the CodeBook construction is repeated).  Three steps:
 *
 * spindlekv_codebook_match: for every new token the entry with the largest cosine similarity, if that
 * exceeds theta (strictly; ties to the lower entry number), else -1; and the ascending list of the tokens
 * without an entry.
 *   batch      describes the NEW tokens: sequence s of every (layer, head) has max_len of them, or
 *              layer_lens of them; equal-length form only (no cu_seqlens)
 *   Gamma_new  device, [layer][seq][head][new token][d]
 *   C          device, CodeBook rows [layer][seq][head][entry][d] (as written by spindlekv_compact with
 *              divide_by = mag); n_entries device [n_layers][B][n_heads]; c_rows: row capacity per unit
 *   mag_new    device out [n_layers][n_heads][T] fp32, ref_new device out [n_layers][n_heads][T] int32
 *   left_idx   device out [n_layers][n_heads][T]: per unit the positions of its unmatched tokens, ascending
 *   left_cnt   device out [n_layers][B][n_heads]
 *   ws         device scratch of spindlekv_match_workspace_bytes(batch, n_heads) bytes, 256-byte aligned
 * Then the caller gathers the unmatched rows (spindlekv_compact with left_idx, left_cnt) and builds their
 * CodeBook (spindlekv_codebook_shallow with layer_lens = left_cnt, layer_lens_heads = n_heads).
 *
 * spindlekv_codebook_append: the entries of that CodeBook become entries n_entries, n_entries + 1, ... of C
 * (unit vectors of their centre rows), the unmatched tokens' ref_new become n_entries + ref_left, and
 * n_entries grows by n_left_entries.  Entries beyond c_rows are not written: compare n_entries with c_rows
 * afterwards.
 *   Gamma_left     device, the gathered unmatched rows; mag_left, ref_left, centre_left, n_left_entries: the
 *                  outputs of spindlekv_codebook_shallow on them
 */
size_t spindlekv_match_workspace_bytes(const spindlekv_batch* batch, int32_t n_heads);
spindlekv_status spindlekv_codebook_match(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                          spindlekv_tensor Gamma_new, spindlekv_tensor C, const int32_t* n_entries,
                                          int32_t c_rows, float theta, float* mag_new, int32_t* ref_new,
                                          int32_t* left_idx, int32_t* left_cnt, void* ws, size_t ws_bytes, void* stream);
spindlekv_status spindlekv_codebook_append(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                           spindlekv_tensor Gamma_left, const float* mag_left, const int32_t* ref_left,
                                           const int32_t* centre_left, const int32_t* n_left_entries,
                                           const int32_t* left_idx, const int32_t* left_cnt, spindlekv_tensor C,
                                           int32_t c_rows, int32_t* n_entries, int32_t* ref_new, void* stream);

/*
 * Reconstruction of the replaced cache from a CodeBook (Eq. (14): Gamma_r = C[r] (x) m): for every
 * (layer, seq, head) and token t of the sequence, dst row t = C row ref[t] times mag[t] (product in fp32,
 * rounded to the storage type).
 *   C    device, CodeBook rows as written by spindlekv_compact with divide_by = mag, addressed like a cache tensor
 *   ref  device [n_layers][n_heads][T], mag device [n_layers][n_heads][T]: outputs of spindlekv_codebook_shallow
 *   dst  device, same addressing rules and dtype as C; may not overlap C
 */
spindlekv_status spindlekv_reconstruct(const spindlekv_batch* batch, int32_t n_heads, int32_t head_dim,
                                       spindlekv_tensor C, const int32_t* ref, const float* mag, spindlekv_tensor dst,
                                       void* stream);

/*
 * Decode-time attention of one new token over the replaced cache (Section 3.4: Eq. (14) inside Eq. (1)).  The
 * CodeBooks hold pre-RoPE keys, so the rotary embedding is applied again after reconstruction: for every
 * (layer, seq, KV head) and each of its h_n query heads g,
 *     K_t = RoPE(C_K[ref_K[t]] * mag_K[t], position of t),   V_t = C_V[ref_V[t]] * mag_V[t],
 *     out_g = softmax_t( RoPE(q_g, pos_q) . K_t / sqrt(d_h) ) V
 * over all cached tokens t (all of them precede the new token).  Rotary embedding as in the LLaMA / Mistral
 * models: element i < d_h/2 is paired with element i + d_h/2, angle = position * base^(-2 i / d_h).  The rebuilt
 * rows are never written to memory: CodeBook rows are gathered, scaled and rotated on the fly.
 *
 * spindlekv_rope_table fills the table of cosines and sines the call reads: float2 (cos, sin)
 * [n_positions][head_dim/2], computed in double precision; spindlekv_rope_table_bytes is its size.
 *
 * spindlekv_decode_attend
 *   batch       describes the cached tokens (max_len, or layer_lens per layer or per head; no cu_seqlens)
 *   q           device, [layer][seq][q head][d] pre-RoPE queries of the new token (stride_tok unused)
 *   pos_q       device [B]: position of the new token of every sequence
 *   C_K, C_V    device, CodeBook rows [layer][seq][kv head][entry][d] (spindlekv_compact with divide_by = mag)
 *   ref_*, mag_* device [n_layers][n_kv_heads][T]: outputs of spindlekv_codebook_shallow for K and for V
 *   positions   device [n_layers][n_kv_heads][T] int32: original position of every cached token (the kept
 *               positions when the CodeBooks were built from an evicted cache), or NULL: token t is at position t
 *   rope_table, table_positions: the table and its number of positions; positions beyond it are clamped
 *   out         device [n_layers][B][n_q_heads][d] fp32
 *   ws          device scratch of spindlekv_decode_workspace_bytes bytes, 256-byte aligned
 * At most 8 query heads per KV head; q, C_K and C_V share one dtype.
 */
size_t spindlekv_rope_table_bytes(int32_t head_dim, int32_t n_positions);
spindlekv_status spindlekv_rope_table(int32_t head_dim, int32_t n_positions, double base, void* table, void* stream);
size_t spindlekv_decode_workspace_bytes(const spindlekv_batch* batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim);
spindlekv_status spindlekv_decode_attend(const spindlekv_batch* batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                         spindlekv_tensor q, const int32_t* pos_q,
                                         spindlekv_tensor C_K, const int32_t* ref_K, const float* mag_K,
                                         spindlekv_tensor C_V, const int32_t* ref_V, const float* mag_V,
                                         const int32_t* positions, const void* rope_table, int32_t table_positions,
                                         float* out, void* ws, size_t ws_bytes, void* stream);

/*
 * Reads the device status word of a workspace (blocking copy; synchronise the stream first).
 *   ws            the workspace of the call in question; NULL: the built-in scratch that
 *                 spindlekv_evict_deep_noalloc uses on the current device (INVALID_ARG before the first
 *                 such call on this device)
 *   device_status host out: SPINDLEKV_OK or SPINDLEKV_TIMEOUT
 *   detail        host out, optional [4]: {greedy rounds used, live tokens left, units of the call whose
 *                 adjacency was computed as a bit matrix (all of them for fp32 input; for bf16 input only
 *                 those whose candidate pairs did not fit the record pool), neighbour-list entries built
 *                 from candidate records (two per similar pair) over the other units}
 */
spindlekv_status spindlekv_poll_status(const void* ws, int32_t* device_status, int32_t* detail);

/* Number of kernels this library has launched since load (or since the last reset). */
int64_t spindlekv_launch_count(int32_t reset);

/*
 * Optional per-kernel timing with CUDA events recorded on the caller's stream around each launch.
 * spindlekv_timing_enable(1) starts collecting (costs two event records per launch);
 * spindlekv_timing_read synchronises the recorded events and returns, for kernel class `which`
 * (0 window-score, 1 top-k, 2 norms, 3 similarity, 4 neighbour lists, 5 greedy cover, 6 entry numbering, 7 gather,
 * 8 the bit-matrix pass of the similarity kernel over units that overflowed their record pool, 9 decode attention),
 * the summed milliseconds and the number of launches since the last spindlekv_timing_enable call.
 */
void spindlekv_timing_enable(int32_t on);
spindlekv_status spindlekv_timing_read(int32_t which, double* ms_total, int64_t* launches);

const char* spindlekv_status_string(spindlekv_status s);

#ifdef __cplusplus
}
#endif
#endif /* SPINDLEKV_H_ */

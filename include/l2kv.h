/* l2kv -- L2-norm KV-cache compression and decode attention for NVIDIA B200 (sm_100a).
 *
 * C ABI of the library.  The operations are those of "A Simple and Effective L2
 * Norm-Based Strategy for KV Cache Compression" (arXiv 2406.11430):
 *
 *   - keep, per layer and head, only the cached keys with the lowest L2 norm and
 *     the corresponding values (Section 1; Section 3, the dropped set D_{l,h} of Eq. 5),
 *     leaving a caller-given list of layers uncompressed (Section 3, last paragraph;
 *     Section 4: the first two layers by default);
 *   - decode attention of one query per head over the cached keys and values
 *     (Eq. 2 applied as in Eq. 4);
 *   - a cache that grows to a pre-defined length and then discards the token with
 *     the highest key norm at every step (Section 4, "Language Modelling Tasks").
 *
 * Conventions shared by every entry point
 *   - Pointers named *_dev, and all tensor pointers (K, V, q, outputs, workspace),
 *     are DEVICE pointers owned by the caller.  `const l2kv_layout*` and the
 *     `uncompressed_layers` list are HOST pointers read before the call returns.
 *     Any memory the device can address will do: l2kv_select_compact, for one, may be given a
 *     V cache that lies in mapped pinned host memory, and then reads only the rows it keeps
 *     over the link.
 *   - The library allocates nothing and keeps no state.  Calls enqueue work on
 *     `stream` (a cudaStream_t passed as void*; NULL = the default stream) and
 *     return at once; outputs are valid in stream order.
 *   - Return value: L2KV_OK (0) or a negative l2kv_status.  Arguments are checked on
 *     the host and nothing is launched when a check fails.  Conditions only the
 *     device can see (a cache row that does not fit t_cap) are recorded in the
 *     status word at the start of the workspace: see l2kv_read_device_status.
 *   - A cache tensor is described by l2kv_layout: logical shape
 *     [batch, layers, kv_heads, t_cap, head_dim], head_dim contiguous, the other
 *     strides in ELEMENTS.  Base pointers and every row must be 16-byte aligned
 *     (all strides * element size multiples of 16).  Supported: bf16 and fp32
 *     elements, head_dim 64 or 128; q_heads a multiple of kv_heads with
 *     q_heads / kv_heads in {1, 2, 4, 8}.  Query head j reads KV head
 *     j / (q_heads / kv_heads).
 *   - Packed caches, for ragged batches without padding (the serving case of Section 4's
 *     budget-maintained cache: sequences of very different lengths, and compressed layers
 *     that need far fewer rows than uncompressed ones).  With row_off_dev != NULL the tensor
 *     is [kv_heads, total_rows, head_dim] (strides stride_h, stride_t; stride_b and stride_l
 *     are ignored) and the rows of (b, l), for every head, are the row_cap_dev[b, l] rows
 *     starting at row row_off_dev[b, l] of that shared row axis: row t of (b, l, h) begins at
 *     element h * stride_h + (row_off_dev[b, l] + t) * stride_t.  Ranges must not overlap and
 *     must end at or before total_rows (not checked: the arrays live on the device).  t_cap
 *     is then a host upper bound of row_cap_dev.  Every per-row companion array of such a
 *     cache (idx, sumsq, the outputs of l2kv_key_norms) is dense [kv_heads, total_rows] with
 *     the same row axis.  Accepted by l2kv_key_norms, l2kv_select_compact (input, output or
 *     both), l2kv_decode_attention, l2kv_append_evict, their _per_head / _static forms, the
 *     prefix-attention calls and l2kv_attention_loss.
 *   - `len_dev[b]` is the number of valid tokens of sequence b; `max_len` is a host
 *     upper bound on every length the call will meet (it sizes grids and scratch;
 *     device lengths above it are clamped to it).
 *   - The ordering key of a cached key row is its fp32 sum of squares (monotone in
 *     the L2 norm), accumulated in a fixed order: the row is cut into 16-byte
 *     pieces; each piece is summed front to back with acc = fma(x, x, acc) from 0;
 *     the P piece sums are combined by a butterfly (for off = P/2 .. 1:
 *     p[i] += p[i ^ off]).  Tokens are ordered by (key, position): among equal keys
 *     the lower position counts as the smaller.
 */
#ifndef L2KV_H_
#define L2KV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  L2KV_OK = 0,
  L2KV_ERR_INVALID_ARG = -1,         /* null pointer, non-positive size, bad enum          */
  L2KV_ERR_UNSUPPORTED = -2,         /* dtype / head_dim / group size outside the list     */
  L2KV_ERR_MISALIGNED = -3,          /* a base pointer or stride breaks 16-byte alignment  */
  L2KV_ERR_WORKSPACE_TOO_SMALL = -4,
  L2KV_ERR_OUT_OF_RANGE = -5,        /* max_len > t_cap, layer index outside [0, layers)   */
  L2KV_ERR_CUDA = -6,                /* a CUDA runtime call failed                         */
  L2KV_ERR_DEVICE_OVERFLOW = -7,     /* device status: a row did not fit t_cap             */
  L2KV_ERR_TIMEOUT = -8,             /* device status: a bounded wait in a kernel gave up  */
  L2KV_ERR_DEBUG_BOUNDS = -9         /* device status, debug build only: an index check    */
} l2kv_status;

typedef enum { L2KV_F32 = 0, L2KV_BF16 = 1 } l2kv_dtype;

/* Which tokens survive compression.  LOWEST is the paper's method; HIGHEST and
 * RANDOM are its ablation baselines (Section 4: keeping the highest-norm tokens,
 * keeping random tokens).  RANDOM orders the tokens of unit u = (b * layers + l) *
 * kv_heads + h by a seeded counter-based key instead of the norm: the upper 32 bits
 * of the SplitMix64 output function (Steele, Lea, Flood 2014) applied to the state
 * seed + (u << 32 | t), i.e. z = state + 0x9E3779B97F4A7C15; z = (z ^ z >> 30) *
 * 0xBF58476D1CE4E5B9; z = (z ^ z >> 27) * 0x94D049BB133111EB; z ^= z >> 31 (mod 2^64);
 * the `keep` smallest keys are kept, equal keys going to the lower position. */
typedef enum {
  L2KV_KEEP_LOWEST_NORM = 0,
  L2KV_KEEP_HIGHEST_NORM = 1,
  L2KV_KEEP_RANDOM = 2
} l2kv_policy;

typedef struct {
  int32_t batch, layers, kv_heads, q_heads, head_dim, t_cap;
  int32_t dtype;                                     /* l2kv_dtype                          */
  int32_t reserved;
  int64_t stride_b, stride_l, stride_h, stride_t;    /* in elements; stride_t >= head_dim   */
  /* Packed caches; NULL, NULL, 0 for the dense form described above. */
  const int64_t* row_off_dev;                        /* DEVICE int64 [batch, layers]        */
  const int32_t* row_cap_dev;                        /* DEVICE int32 [batch, layers]        */
  int64_t total_rows;
} l2kv_layout;

/* Text for a status code (static storage, never NULL). */
const char* l2kv_status_string(int status);

/* keep = clamp(ceil(keep_ratio * len), 1, len) (0 when len == 0).  keep_ratio is the
 * fraction KEPT, i.e. 1 - the paper's compression ratio (Section 4 quotes ratios
 * of 0 % to 90 % dropped and gives no rounding rule; this one is the library's).
 * Host only. */
int l2kv_keep_count(int32_t len, double keep_ratio, int32_t* keep);

/* Bytes of device scratch that suffice for any call on caches of this layout with
 * lengths up to max_len.  The first 256 bytes hold the device status word; zero
 * the workspace once before first use.  Host only. */
int l2kv_workspace_bytes(const l2kv_layout* lay, int32_t max_len, size_t* bytes);

/* Reads (and waits for) the device status word of a workspace.  Synchronises `stream`.
 * *status becomes
 *   L2KV_OK                   nothing happened;
 *   L2KV_ERR_DEVICE_OVERFLOW  l2kv_append_evict had no row left for an append (the row was
 *                             dropped, everything else went ahead);
 *   L2KV_ERR_TIMEOUT          a kernel of l2kv_decode_attention or l2kv_prefix_attention gave up
 *                             waiting for a copy or a tensor-core operation (every such wait
 *                             is bounded so that a fault cannot hang the GPU).  The kernel
 *                             also sets a mark in the status block at which the rest of its
 *                             grid, and EVERY LATER decode / prefix call on this workspace,
 *                             leaves at once without writing its output;
 *   L2KV_ERR_DEBUG_BOUNDS     only from a library built with -DL2KV_DEBUG: an index check
 *                             failed (the access was skipped).
 * The word keeps the last anomaly until the workspace is cleared: after any non-zero status,
 * and after any call that returned L2KV_ERR_CUDA (a launch that died may leave the per-unit
 * completion counters of l2kv_select_compact / l2kv_append_evict non-zero, and the next call
 * would then skip a unit's selection), call l2kv_workspace_reset or zero the workspace. */
int l2kv_read_device_status(const void* workspace, void* stream, int32_t* status);

/* Puts a workspace back into its initial state in stream order: zeroes the status block
 * and the completion counters (the first l2kv_workspace_bytes(lay, 0) bytes; scratch beyond
 * them never needs clearing).  Allocates nothing. */
int l2kv_workspace_reset(void* workspace, size_t workspace_bytes, const l2kv_layout* lay,
                         void* stream);

/* Self-test of the give-up path, for test suites: one thread block waits, with a small poll
 * limit, on a barrier that nothing will ever complete (no copy is in flight, nothing faults),
 * gives up, and records L2KV_ERR_TIMEOUT and the abort mark in `workspace` exactly as the
 * decode and prefix kernels do.  The paper has no counterpart. */
int l2kv_selftest_wait_timeout(void* workspace, size_t workspace_bytes, void* stream);

/* Key norms (Abstract; Section 3): for every valid token t < len_dev[b] of every
 * (b, l, h), sumsq_out[b,l,h,t] = sum_d K[b,l,h,t,d]^2 in the fixed order above, and,
 * if norm_out is not NULL, norm_out = sqrt(sumsq).  Both outputs are dense fp32
 * [batch, layers, kv_heads, t_cap]; entries at t >= len are left untouched. */
int l2kv_key_norms(const void* K, const l2kv_layout* lay, const int32_t* len_dev, int32_t max_len,
                   float* sumsq_out, float* norm_out, void* stream);

/* Compression (Section 1; Section 3): for every (b, l, h) with l not in
 * uncompressed_layers, keep the keep_dev[b] tokens that come first in the order
 * (key, position) -- last, for L2KV_KEEP_HIGHEST_NORM, with ties still to the lower
 * position -- and write them, in increasing position, to the first rows of the
 * output cache:  K_out[b,l,h,j] = K[b,l,h,t_j], V_out likewise (bit copies),
 * idx_out[b,l,h,j] = t_j, sumsq_out[b,l,h,j] = key of t_j, kept_len_dev[b,l] =
 * keep_dev[b].  Layers in uncompressed_layers (host array, may be NULL when
 * n_uncompressed == 0) are copied whole: kept_len = len, idx = identity.
 * `seed` is used by L2KV_KEEP_RANDOM only.  `sumsq_in` may be NULL; if it is given it
 * must hold the keys of K as l2kv_key_norms writes them (dense fp32
 * [batch, layers, kv_heads, in->t_cap], e.g. produced when the rows were written to
 * the cache): the pass over K that computes the keys is then skipped.
 * Requires 0 <= keep_dev[b] <= len_dev[b] <= max_len <= in->t_cap and kept_len <=
 * out->t_cap (the host checks what it can see: max_len and the layouts; a device
 * value outside its range is clamped).  `in` and `out` must agree in batch, layers,
 * kv_heads, head_dim and dtype, and the output tensors must not overlap the
 * inputs.  idx_out / sumsq_out are dense [batch, layers, kv_heads, out->t_cap];
 * rows at and beyond kept_len are left untouched. */
int l2kv_select_compact(const void* K, const void* V, const l2kv_layout* in,
                        const int32_t* len_dev, const int32_t* keep_dev, int32_t max_len,
                        const int32_t* uncompressed_layers, int32_t n_uncompressed, int32_t policy,
                        uint64_t seed, const float* sumsq_in,
                        void* K_out, void* V_out, const l2kv_layout* out, int32_t* idx_out,
                        float* sumsq_out, int32_t* kept_len_dev, void* workspace,
                        size_t workspace_bytes, void* stream);

/* Decode attention (Eq. 2 over the cache, Eq. 4): for every (b, l, query head j)
 *   out[b,l,j,:] = sum_i softmax_i( scale * q[b,l,j,:] . K_c[b,l,j/G,i,:] ) * V_c[b,l,j/G,i,:]
 * over rows i < cur_len_dev[b,l], G = q_heads / kv_heads, no mask.  q is dense
 * [batch, layers, q_heads, head_dim] in the cache's dtype; out is dense fp32 of the
 * same shape.  scale <= 0 selects 1 / sqrt(head_dim).  Products and sums are fp32.
 * An empty cache (cur_len == 0) gives zeros.  cur_len <= max_len <= lay->t_cap. */
int l2kv_decode_attention(const void* q, const void* K_c, const void* V_c, const l2kv_layout* lay,
                          const int32_t* cur_len_dev, int32_t max_len, float scale, float* out,
                          void* workspace, size_t workspace_bytes, void* stream);

/* A keep count of its own for every head -- the per-head compression ratios that the paper
 * names as future work (Limitations section); the method itself uses one ratio for all
 * heads.  l2kv_select_compact_per_head is l2kv_select_compact with keep_unit_dev dense
 * int32 [batch, layers, kv_heads] in place of keep_dev (0 <= keep_unit_dev[b,l,h] <=
 * len_dev[b]; layers in uncompressed_layers ignore it) and kept_len_unit_dev of the same
 * shape in place of kept_len_dev.  l2kv_decode_attention_per_head is l2kv_decode_attention
 * over rows i < cur_len_unit_dev[b,l,j/G] (dense int32 [batch, layers, kv_heads]).
 * l2kv_append_evict_per_head is l2kv_append_evict with cur_len_unit_dev (in/out) and
 * budget_unit_dev dense int32 [batch, layers, kv_heads]: every head appends until it holds its
 * own budget and evicts from then on.  l2kv_prefix_attention_per_head is
 * l2kv_prefix_attention over rows i < cur_len_unit_dev[b,l,j/G].  All other arguments,
 * layouts, ownership and errors are those of the per-sequence calls. */
int l2kv_select_compact_per_head(const void* K, const void* V, const l2kv_layout* in,
                                 const int32_t* len_dev, const int32_t* keep_unit_dev,
                                 int32_t max_len, const int32_t* uncompressed_layers,
                                 int32_t n_uncompressed, int32_t policy, uint64_t seed,
                                 const float* sumsq_in, void* K_out, void* V_out,
                                 const l2kv_layout* out, int32_t* idx_out, float* sumsq_out,
                                 int32_t* kept_len_unit_dev, void* workspace,
                                 size_t workspace_bytes, void* stream);
int l2kv_decode_attention_per_head(const void* q, const void* K_c, const void* V_c,
                                   const l2kv_layout* lay, const int32_t* cur_len_unit_dev,
                                   int32_t max_len, float scale, float* out, void* workspace,
                                   size_t workspace_bytes, void* stream);
int l2kv_append_evict_per_head(void* K_c, void* V_c, int32_t* idx, float* sumsq_c,
                               const l2kv_layout* lay, int32_t* cur_len_unit_dev,
                               const int32_t* budget_unit_dev, const int32_t* uncompressed_layers,
                               int32_t n_uncompressed, const void* k_new, const void* v_new,
                               const int32_t* pos_new_dev, void* workspace, size_t workspace_bytes,
                               void* stream);
int l2kv_prefix_attention_per_head(const void* q, const void* K_c, const void* V_c,
                                   const l2kv_layout* lay, const int32_t* cur_len_unit_dev,
                                   int32_t max_len, int32_t n_queries, float scale, float* out,
                                   float* lse_out, void* workspace, size_t workspace_bytes,
                                   void* stream);

/* Budget-maintained cache (Section 4, "Language Modelling Tasks"): append one new
 * token per (b, l, h).  If l is uncompressed or cur_len_dev[b,l] < budget_dev[b] the
 * row is appended at slot cur_len and cur_len grows by one.  Otherwise the entry
 * that comes last in the order (key, position) among the stored ones and the new
 * one is discarded: if that is the new token nothing changes, else the new row
 * overwrites the discarded slot (the cache stays dense, no longer position-
 * ordered; idx keeps original positions).  k_new, v_new are dense
 * [batch, layers, kv_heads, head_dim]; pos_new_dev[b] is the new token's position.
 * K_c, V_c, idx, sumsq_c and cur_len_dev are updated in place (idx and sumsq_c dense
 * [batch, layers, kv_heads, lay->t_cap]).  A row that would land at slot >= t_cap is
 * not written and sets the device status word to L2KV_ERR_DEVICE_OVERFLOW.  The
 * workspace may be the one of the other calls or a small one of its own: any zeroed
 * buffer of at least l2kv_workspace_bytes(lay, 0) bytes. */
int l2kv_append_evict(void* K_c, void* V_c, int32_t* idx, float* sumsq_c, const l2kv_layout* lay,
                      int32_t* cur_len_dev, const int32_t* budget_dev,
                      const int32_t* uncompressed_layers, int32_t n_uncompressed,
                      const void* k_new, const void* v_new, const int32_t* pos_new_dev,
                      void* workspace, size_t workspace_bytes, void* stream);

/* Prefix attention: n_queries new queries per (b, l) -- a prefill chunk, or several draft
 * tokens -- over the compressed cache, with the fused online-softmax formulation that the
 * method stays compatible with because it never needs the attention scores (Abstract;
 * Section 1).  Eq. 2 per query, over the cached rows i < cur_len_dev[b,l], no mask (every
 * cached token precedes the new ones; attention among the new tokens themselves is the
 * caller's, to be merged with this result through lse_out):
 *   out[b,l,s,j,:] = sum_i softmax_i( scale * q[b,l,s,j,:] . K_c[b,l,j/G,i,:] ) * V_c[b,l,j/G,i,:]
 * q is dense bf16 [batch, layers, n_queries, q_heads, head_dim]; out dense fp32 of the same
 * shape; lse_out (may be NULL) dense fp32 [batch, layers, n_queries, q_heads] receives the
 * natural-log sum of exponentials of the scaled scores.  bf16 caches with head_dim 128 only
 * (L2KV_ERR_UNSUPPORTED otherwise, also for strides a tensor map cannot express).  Products
 * are exact, sums fp32; the softmax weights are rounded to bf16 before they multiply V, as
 * in FlashAttention.  An empty cache gives zeros and lse = -inf.  workspace may be NULL; if
 * given (>= 256 bytes, its first 256 zeroed) its status word reports a copy or MMA wait that
 * gave up.  With a workspace of l2kv_prefix_attention_workspace_bytes(lay, max_len, n_queries)
 * bytes the call may also split the cache into pieces handled by different thread blocks and
 * merge their results (the same rows up to the bf16 rounding of the weights): that keeps the
 * GPU busy when there are few KV heads and queries per call (one layer at a time), and for
 * very long caches (max_len >= 65536), whose (b, l) pairs may differ widely in length, the
 * work is dealt out in equal shares to a fixed grid of resident thread blocks.  With less
 * room it runs unsplit.  Beyond its first 256 bytes the workspace needs no initial contents. */
int l2kv_prefix_attention_workspace_bytes(const l2kv_layout* lay, int32_t max_len,
                                          int32_t n_queries, size_t* bytes);
/* The same for a prefill chunk whose own keys and values are already in the cache: the last
 * n_queries cached rows of every (b, l) are the new tokens', in order, and query s attends to
 * rows i < cur_len_dev[b,l] - n_queries + s + 1 (everything before the chunk, and the chunk up
 * to itself) -- the causal mask of Eq. 2 as a model applies it during prefill.  Meant for
 * caches whose tail is in position order (appended rows; not after an eviction has reused a
 * slot).  A query with no row to see gives zeros and lse = -inf.  Everything else as above. */
int l2kv_prefix_attention_causal(const void* q, const void* K_c, const void* V_c,
                                 const l2kv_layout* lay, const int32_t* cur_len_dev,
                                 int32_t max_len, int32_t n_queries, float scale, float* out,
                                 float* lse_out, void* workspace, size_t workspace_bytes,
                                 void* stream);
int l2kv_prefix_attention(const void* q, const void* K_c, const void* V_c, const l2kv_layout* lay,
                          const int32_t* cur_len_dev, int32_t max_len, int32_t n_queries, float scale,
                          float* out, float* lse_out, void* workspace, size_t workspace_bytes,
                          void* stream);
/* The general form of the three calls above (Eq. 2 per query over the cache, as they state it):
 * `flags` is any combination of
 *   L2KV_PREFIX_CAUSAL         the chunk's own rows are the cache's last n_queries rows
 *                              (l2kv_prefix_attention_causal);
 *   L2KV_PREFIX_LEN_PER_HEAD   cur_len_dev is [batch, layers, kv_heads]
 *                              (l2kv_prefix_attention_per_head);
 *   L2KV_PREFIX_SPLIT_WEIGHTS  every softmax weight multiplies V as the sum of two bf16 terms
 *                              (16 significant bits) instead of one rounded bf16 (8 bits).  The
 *                              result then has the accuracy of l2kv_decode_attention (fp32
 *                              accumulation of exact products; |error| <= 2e-3 + 1e-2 |exact|
 *                              with a wide margin), at the price of a second P.V contraction.
 *                              Without the flag single rounded weights are used, as fused
 *                              attention kernels commonly do; measured |error| then stays below
 *                              4e-3 + 1e-2 |exact| (it is largest for short caches, where few
 *                              weights carry the sum).
 * Any other bit gives L2KV_ERR_INVALID_ARG. */
#define L2KV_PREFIX_CAUSAL 1u
#define L2KV_PREFIX_LEN_PER_HEAD 2u
#define L2KV_PREFIX_SPLIT_WEIGHTS 4u
int l2kv_prefix_attention_flags(const void* q, const void* K_c, const void* V_c,
                                const l2kv_layout* lay, const int32_t* cur_len_dev, int32_t max_len,
                                int32_t n_queries, float scale, uint32_t flags, float* out,
                                float* lse_out, void* workspace, size_t workspace_bytes,
                                void* stream);

/* Attention loss of the norm-based compression against the ideal one (Section 3,
 * Eqs. 5-7), for one query per query head over the cached keys i < cur_len_dev[b,l]:
 *   a_p       = softmax_p(scale * q . K_p)                       (attention scores, Eq. 2)
 *   L^m       = sum of a_p over the m tokens the method drops first, i.e. the m last
 *               in the order (key, position)                      (Eq. 5)
 *   L^{m,ref} = sum of the m smallest a_p (the ideal compression)
 *   Y         = sum_{m=1..n} (L^m - L^{m,ref})                     (Eqs. 6, 7)
 * sumsq holds the keys of K as l2kv_key_norms writes them (dense fp32
 * [batch, layers, kv_heads, t_cap]; [kv_heads, total_rows] for a packed cache).  alr_out is dense fp32 [batch, layers, q_heads].
 * loss_out / loss_ref_out may be NULL; otherwise dense fp32
 * [batch, layers, q_heads, t_cap] receiving L^m / L^{m,ref} at index m - 1 (entries at
 * and beyond n untouched).  Sums are fp64 internally.  An empty cache gives Y = 0.
 * The workspace needs l2kv_attention_loss_workspace_bytes(lay, max_len) bytes (it is
 * separate from, and much larger than, the one of the other calls: about 8 bytes per cached
 * token and query head; no zeroing needed).  The query heads of a KV head are scored from one
 * read of its keys; every head's scores are then sorted (radix sort), so this is an analysis
 * tool with the cost of a sort per head, not a step of the decode path. */
int l2kv_attention_loss_workspace_bytes(const l2kv_layout* lay, int32_t max_len, size_t* bytes);
int l2kv_attention_loss(const void* q, const void* K, const l2kv_layout* lay,
                        const int32_t* cur_len_dev, int32_t max_len, float scale,
                        const float* sumsq, float* alr_out, float* loss_out, float* loss_ref_out,
                        void* workspace, size_t workspace_bytes, void* stream);
/* The same with a cache length per (b, l, kv head): cur_len_unit_dev dense int32
 * [batch, layers, kv_heads], as l2kv_select_compact_per_head leaves it. */
int l2kv_attention_loss_per_head(const void* q, const void* K, const l2kv_layout* lay,
                                 const int32_t* cur_len_unit_dev, int32_t max_len, float scale,
                                 const float* sumsq, float* alr_out, float* loss_out,
                                 float* loss_ref_out, void* workspace, size_t workspace_bytes,
                                 void* stream);

/* Decode attention without a workspace -- the paper has no counterpart to this entry
 * point; it exists for the callers of this library that cannot allocate device memory.
 *
 * Same operation, arguments, result and errors as l2kv_decode_attention, but the scratch
 * for the per-split partial results is a fixed array of L2KV_STATIC_SCRATCH_BYTES that
 * is part of the library image: every GPU that loads the library holds that much memory
 * until the process exits, and no call here ever runs cudaMalloc, cudaFree or any other
 * allocating routine.  Meant for code that runs where allocation is forbidden or would
 * stall (a thread that may not take the allocator's lock, a callback, a serving loop whose
 * pool is already handed out) and that has no spare buffer to pass as a workspace.
 *
 *   - Limit: batch * layers * q_heads * ceil(max_len / 1024) * (head_dim + 2) * 4 bytes must
 *     not exceed L2KV_STATIC_SCRATCH_BYTES - 256 (16 MiB less the status block: e.g. one layer of 32 query heads at
 *     batch 4 up to a cache of about 250k tokens, or a whole 32-layer model at batch 4 up to 7k
 *     tokens).  Beyond it the call returns L2KV_ERR_WORKSPACE_TOO_SMALL and launches
 *     nothing: call per layer, or use l2kv_decode_attention with your own workspace.
 *   - The first call on each device looks up the array's device address, with the current
 *     device taken as the one `stream` belongs to.  The library calls no allocator, but that
 *     first call is where the CUDA runtime loads this part of the library onto the device, and
 *     the 16 MiB of the array are reserved then: make the call once at start-up, outside any
 *     stream capture, and expect L2KV_ERR_CUDA from it if the device has no memory left.
 *   - The first 256 bytes of the array are its status block, the rest holds the partial
 *     results.  l2kv_decode_attention_static_status reads the status word as
 *     l2kv_read_device_status does for a workspace (L2KV_OK or L2KV_ERR_TIMEOUT) and, with
 *     reset != 0, then zeroes the status block in stream order, which a call needs after a
 *     L2KV_ERR_TIMEOUT before it will write results again.
 *   - All calls on a device share the one array, which simply keeps what the last call
 *     left in it (nothing in it needs clearing between calls).  Two calls whose kernels can
 *     overlap on the GPU -- different streams, no dependency -- race on it and give wrong
 *     results: order them, or use the workspace variant for concurrent streams. */
#define L2KV_STATIC_SCRATCH_BYTES (16u << 20)
int l2kv_decode_attention_static(const void* q, const void* K_c, const void* V_c,
                                 const l2kv_layout* lay, const int32_t* cur_len_dev,
                                 int32_t max_len, float scale, float* out, void* stream);
int l2kv_decode_attention_static_status(void* stream, int32_t* status, int32_t reset);

#ifdef __cplusplus
}
#endif
#endif /* L2KV_H_ */

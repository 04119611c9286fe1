// The C entry points: argument checks on the host, then the kernel launchers.
#include <cmath>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace {

using namespace l2kv;

// One NVTX range per entry point (no cost unless a profiler is attached).
struct Range {
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int elem_bytes(int dtype) { return dtype == L2KV_BF16 ? 2 : 4; }

// Checks everything about a layout that does not depend on a particular call.
int check_layout(const l2kv_layout* a) {
  if (!a) return L2KV_ERR_INVALID_ARG;
  if (a->batch < 0 || a->layers < 0 || a->kv_heads < 0 || a->q_heads < 0 || a->t_cap < 0)
    return L2KV_ERR_INVALID_ARG;
  if (a->dtype != L2KV_F32 && a->dtype != L2KV_BF16) return L2KV_ERR_UNSUPPORTED;
  if (a->head_dim != 64 && a->head_dim != 128) return L2KV_ERR_UNSUPPORTED;
  if (a->layers > kMaxLayers) return L2KV_ERR_OUT_OF_RANGE;
  const int64_t per16 = 16 / elem_bytes(a->dtype);
  if (a->row_off_dev) {
    // packed cache [kv_heads, total_rows, head_dim]: stride_b and stride_l are not used
    if (!a->row_cap_dev || a->total_rows < 0) return L2KV_ERR_INVALID_ARG;
    if (a->stride_t < a->head_dim || a->stride_h < 0) return L2KV_ERR_INVALID_ARG;
    if (a->stride_h % per16 || a->stride_t % per16) return L2KV_ERR_MISALIGNED;
    if ((reinterpret_cast<uintptr_t>(a->row_off_dev) & 7u) || (reinterpret_cast<uintptr_t>(a->row_cap_dev) & 3u))
      return L2KV_ERR_MISALIGNED;
    return L2KV_OK;
  }
  if (a->row_cap_dev) return L2KV_ERR_INVALID_ARG;
  if (a->stride_t < a->head_dim || a->stride_b < 0 || a->stride_l < 0 || a->stride_h < 0)
    return L2KV_ERR_INVALID_ARG;
  if (a->stride_b % per16 || a->stride_l % per16 || a->stride_h % per16 || a->stride_t % per16)
    return L2KV_ERR_MISALIGNED;
  return L2KV_OK;
}

int check_groups(const l2kv_layout* a) {
  if (a->kv_heads == 0) return a->q_heads == 0 ? L2KV_OK : L2KV_ERR_INVALID_ARG;
  if (a->q_heads % a->kv_heads) return L2KV_ERR_INVALID_ARG;
  const int G = a->q_heads / a->kv_heads;
  if (G != 1 && G != 2 && G != 4 && G != 8) return L2KV_ERR_UNSUPPORTED;
  return L2KV_OK;
}

int make_mask(const int32_t* layers, int n, int n_layers, LayerMask* m) {
  *m = LayerMask{};
  if (n < 0 || (n > 0 && !layers)) return L2KV_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    if (layers[i] < 0 || layers[i] >= n_layers) return L2KV_ERR_OUT_OF_RANGE;
    m->w[layers[i] >> 5] |= 1u << (layers[i] & 31);
  }
  return L2KV_OK;
}

bool empty(const l2kv_layout* a) { return a->batch == 0 || a->layers == 0 || a->kv_heads == 0; }

}  // namespace

extern "C" {

const char* l2kv_status_string(int status) {
  switch (status) {
    case L2KV_OK: return "ok";
    case L2KV_ERR_INVALID_ARG: return "invalid argument";
    case L2KV_ERR_UNSUPPORTED: return "unsupported dtype, head_dim or query-group size";
    case L2KV_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
    case L2KV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case L2KV_ERR_OUT_OF_RANGE: return "length, capacity or layer index out of range";
    case L2KV_ERR_CUDA: return "CUDA runtime error";
    case L2KV_ERR_DEVICE_OVERFLOW: return "a cache row did not fit t_cap (device status)";
    case L2KV_ERR_TIMEOUT: return "a bounded wait inside a kernel gave up (device status)";
    case L2KV_ERR_DEBUG_BOUNDS: return "an index check of the debug build failed (device status)";
  }
  return "unknown status";
}

int l2kv_keep_count(int32_t len, double keep_ratio, int32_t* keep) {
  if (!keep || len < 0 || !(keep_ratio == keep_ratio)) return L2KV_ERR_INVALID_ARG;
  if (len == 0) { *keep = 0; return L2KV_OK; }
  double k = std::ceil(keep_ratio * (double)len);
  if (k < 1.0) k = 1.0;
  if (k > (double)len) k = (double)len;
  *keep = (int32_t)k;
  return L2KV_OK;
}

int l2kv_workspace_bytes(const l2kv_layout* lay, int32_t max_len, size_t* bytes) {
  if (!bytes || max_len < 0) return L2KV_ERR_INVALID_ARG;
  const int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  *bytes = plan_workspace(*lay, max_len).total;
  return L2KV_OK;
}

int l2kv_read_device_status(const void* workspace, void* stream, int32_t* status) {
  if (!workspace || !status) return L2KV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t word = 0;
  if (cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return L2KV_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return L2KV_ERR_CUDA;
  *status = word;
  return L2KV_OK;
}

int l2kv_workspace_reset(void* workspace, size_t workspace_bytes, const l2kv_layout* lay,
                         void* stream) {
  const int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  if (!workspace) return L2KV_ERR_INVALID_ARG;
  const size_t head = plan_workspace(*lay, 0).sumsq_off;   // status block + completion counters
  if (workspace_bytes < head) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  return cudaMemsetAsync(workspace, 0, head, static_cast<cudaStream_t>(stream)) == cudaSuccess
             ? L2KV_OK : L2KV_ERR_CUDA;
}

int l2kv_key_norms(const void* K, const l2kv_layout* lay, const int32_t* len_dev, int32_t max_len,
                   float* sumsq_out, float* norm_out, void* stream) {
  const Range nvtx_range("l2kv_key_norms");
  int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  if (max_len < 0) return L2KV_ERR_INVALID_ARG;
  if (max_len > lay->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if (empty(lay) || max_len == 0) return L2KV_OK;
  if (!K || !len_dev || !sumsq_out) return L2KV_ERR_INVALID_ARG;
  if (!aligned16(K)) return L2KV_ERR_MISALIGNED;
  // leading dimension -1: the outputs are laid out like the cache's rows
  return launch_key_norms(K, make_geom(*lay), lay->dtype, len_dev, max_len, sumsq_out, -1,
                          norm_out, kKeysOnly, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

// Both forms of the compression call: keep counts and result lengths per sequence
// (per_head false: keep [B], kept_len [B, L]) or per head (keep and kept_len [B, L, H]).
static int select_compact_impl(bool per_head, const void* K, const void* V, const l2kv_layout* in,
                               const int32_t* len_dev, const int32_t* keep_dev, int32_t max_len,
                               const int32_t* uncompressed_layers, int32_t n_uncompressed,
                               int32_t policy, uint64_t seed, const float* sumsq_in, void* K_out,
                               void* V_out, const l2kv_layout* out, int32_t* idx_out,
                               float* sumsq_out, int32_t* kept_len_dev, void* workspace,
                               size_t workspace_bytes, void* stream) {
  const Range nvtx_range("l2kv_select_compact");
  int rc = check_layout(in);
  if (rc != L2KV_OK) return rc;
  rc = check_layout(out);
  if (rc != L2KV_OK) return rc;
  if (in->batch != out->batch || in->layers != out->layers || in->kv_heads != out->kv_heads ||
      in->head_dim != out->head_dim || in->dtype != out->dtype)
    return L2KV_ERR_INVALID_ARG;
  if (policy != L2KV_KEEP_LOWEST_NORM && policy != L2KV_KEEP_HIGHEST_NORM &&
      policy != L2KV_KEEP_RANDOM)
    return L2KV_ERR_INVALID_ARG;
  if (max_len < 0) return L2KV_ERR_INVALID_ARG;
  if (max_len > in->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if ((long long)max_len > (long long)kGatherChunk * kMaxChunks) return L2KV_ERR_OUT_OF_RANGE;
  LayerMask unc;
  rc = make_mask(uncompressed_layers, n_uncompressed, in->layers, &unc);
  if (rc != L2KV_OK) return rc;
  if (n_uncompressed > 0 && max_len > out->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if (empty(in)) return L2KV_OK;
  if (!K || !V || !len_dev || !keep_dev || !K_out || !V_out || !idx_out || !sumsq_out ||
      !kept_len_dev || !workspace)
    return L2KV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out) ||
      !aligned16(workspace))
    return L2KV_ERR_MISALIGNED;
  const WorkspacePlan plan = plan_workspace(*in, max_len);
  if (workspace_bytes < plan.total) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  return launch_select_compact(K, V, make_geom(*in), in->dtype, len_dev,
                               per_head ? nullptr : keep_dev, per_head ? keep_dev : nullptr,
                               max_len, unc, policy, seed, sumsq_in, K_out, V_out,
                               make_geom(*out), idx_out, sumsq_out,
                               per_head ? nullptr : kept_len_dev, per_head ? kept_len_dev : nullptr,
                               static_cast<char*>(workspace), plan,
                               static_cast<cudaStream_t>(stream));
}

int l2kv_select_compact(const void* K, const void* V, const l2kv_layout* in,
                        const int32_t* len_dev, const int32_t* keep_dev, int32_t max_len,
                        const int32_t* uncompressed_layers, int32_t n_uncompressed, int32_t policy,
                        uint64_t seed, const float* sumsq_in,
                        void* K_out, void* V_out, const l2kv_layout* out, int32_t* idx_out,
                        float* sumsq_out, int32_t* kept_len_dev, void* workspace,
                        size_t workspace_bytes, void* stream) {
  return select_compact_impl(false, K, V, in, len_dev, keep_dev, max_len, uncompressed_layers,
                             n_uncompressed, policy, seed, sumsq_in, K_out, V_out, out, idx_out,
                             sumsq_out, kept_len_dev, workspace, workspace_bytes, stream);
}

int l2kv_select_compact_per_head(const void* K, const void* V, const l2kv_layout* in,
                                 const int32_t* len_dev, const int32_t* keep_unit_dev,
                                 int32_t max_len, const int32_t* uncompressed_layers,
                                 int32_t n_uncompressed, int32_t policy, uint64_t seed,
                                 const float* sumsq_in, void* K_out, void* V_out,
                                 const l2kv_layout* out, int32_t* idx_out, float* sumsq_out,
                                 int32_t* kept_len_unit_dev, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  return select_compact_impl(true, K, V, in, len_dev, keep_unit_dev, max_len,
                             uncompressed_layers, n_uncompressed, policy, seed, sumsq_in, K_out,
                             V_out, out, idx_out, sumsq_out, kept_len_unit_dev, workspace,
                             workspace_bytes, stream);
}

static int decode_attention_impl(bool per_head, const void* q, const void* K_c, const void* V_c,
                                 const l2kv_layout* lay, const int32_t* cur_len_dev,
                                 int32_t max_len, float scale, float* out, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  const Range nvtx_range("l2kv_decode_attention");
  int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  rc = check_groups(lay);
  if (rc != L2KV_OK) return rc;
  if (max_len < 0 || !(scale == scale)) return L2KV_ERR_INVALID_ARG;
  if (max_len > lay->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if (empty(lay)) return L2KV_OK;
  if (!q || !K_c || !V_c || !cur_len_dev || !out || !workspace) return L2KV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(K_c) || !aligned16(V_c) || !aligned16(workspace))
    return L2KV_ERR_MISALIGNED;
  const WorkspacePlan plan = plan_workspace(*lay, max_len);
  if (workspace_bytes < plan.total) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  const float sc = scale > 0.f ? scale : 1.0f / std::sqrt((float)lay->head_dim);
  const LenView lens{cur_len_dev, per_head ? 1 : 0};
  return launch_decode_attention(q, K_c, V_c, make_geom(*lay), lay->dtype, lens, max_len, sc,
                                 out, static_cast<char*>(workspace), plan,
                                 static_cast<cudaStream_t>(stream));
}

int l2kv_decode_attention(const void* q, const void* K_c, const void* V_c, const l2kv_layout* lay,
                          const int32_t* cur_len_dev, int32_t max_len, float scale, float* out,
                          void* workspace, size_t workspace_bytes, void* stream) {
  return decode_attention_impl(false, q, K_c, V_c, lay, cur_len_dev, max_len, scale, out,
                               workspace, workspace_bytes, stream);
}

int l2kv_decode_attention_per_head(const void* q, const void* K_c, const void* V_c,
                                   const l2kv_layout* lay, const int32_t* cur_len_unit_dev,
                                   int32_t max_len, float scale, float* out, void* workspace,
                                   size_t workspace_bytes, void* stream) {
  return decode_attention_impl(true, q, K_c, V_c, lay, cur_len_unit_dev, max_len, scale, out,
                               workspace, workspace_bytes, stream);
}

static int append_evict_impl(bool per_head, void* K_c, void* V_c, int32_t* idx, float* sumsq_c,
                             const l2kv_layout* lay, int32_t* cur_len_dev,
                             const int32_t* budget_dev, const int32_t* uncompressed_layers,
                             int32_t n_uncompressed, const void* k_new, const void* v_new,
                             const int32_t* pos_new_dev, void* workspace, size_t workspace_bytes,
                             void* stream) {
  const Range nvtx_range("l2kv_append_evict");
  int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  LayerMask unc;
  rc = make_mask(uncompressed_layers, n_uncompressed, lay->layers, &unc);
  if (rc != L2KV_OK) return rc;
  if (empty(lay)) return L2KV_OK;
  if (!K_c || !V_c || !idx || !sumsq_c || !cur_len_dev || !budget_dev || !k_new || !v_new ||
      !pos_new_dev || !workspace)
    return L2KV_ERR_INVALID_ARG;
  if (!aligned16(K_c) || !aligned16(V_c) || !aligned16(k_new) || !aligned16(v_new) ||
      !aligned16(workspace))
    return L2KV_ERR_MISALIGNED;
  const WorkspacePlan plan = plan_workspace(*lay, 0);    // status word and tickets only
  if (workspace_bytes < plan.sumsq_off) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  char* ws = static_cast<char*>(workspace);
  return launch_append_evict(K_c, V_c, idx, sumsq_c, make_geom(*lay), lay->dtype, cur_len_dev,
                             budget_dev, unc, k_new, v_new, pos_new_dev,
                             reinterpret_cast<int32_t*>(ws),
                             reinterpret_cast<int32_t*>(ws + plan.ticket_off), per_head ? 1 : 0,
                             static_cast<cudaStream_t>(stream));
}

int l2kv_append_evict(void* K_c, void* V_c, int32_t* idx, float* sumsq_c, const l2kv_layout* lay,
                      int32_t* cur_len_dev, const int32_t* budget_dev,
                      const int32_t* uncompressed_layers, int32_t n_uncompressed,
                      const void* k_new, const void* v_new, const int32_t* pos_new_dev,
                      void* workspace, size_t workspace_bytes, void* stream) {
  return append_evict_impl(false, K_c, V_c, idx, sumsq_c, lay, cur_len_dev, budget_dev,
                           uncompressed_layers, n_uncompressed, k_new, v_new, pos_new_dev,
                           workspace, workspace_bytes, stream);
}

int l2kv_append_evict_per_head(void* K_c, void* V_c, int32_t* idx, float* sumsq_c,
                               const l2kv_layout* lay, int32_t* cur_len_unit_dev,
                               const int32_t* budget_unit_dev, const int32_t* uncompressed_layers,
                               int32_t n_uncompressed, const void* k_new, const void* v_new,
                               const int32_t* pos_new_dev, void* workspace, size_t workspace_bytes,
                               void* stream) {
  return append_evict_impl(true, K_c, V_c, idx, sumsq_c, lay, cur_len_unit_dev, budget_unit_dev,
                           uncompressed_layers, n_uncompressed, k_new, v_new, pos_new_dev,
                           workspace, workspace_bytes, stream);
}

static int prefix_attention_impl(bool per_head, bool causal, bool split_weights, const void* q, const void* K_c, const void* V_c,
                                 const l2kv_layout* lay, const int32_t* cur_len_dev,
                                 int32_t max_len, int32_t n_queries, float scale, float* out,
                                 float* lse_out, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  const Range nvtx_range("l2kv_prefix_attention");
  int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  rc = check_groups(lay);
  if (rc != L2KV_OK) return rc;
  if (lay->dtype != L2KV_BF16 || lay->head_dim != 128) return L2KV_ERR_UNSUPPORTED;
  if (max_len < 0 || n_queries < 0 || !(scale == scale)) return L2KV_ERR_INVALID_ARG;
  if (max_len > lay->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if (empty(lay) || n_queries == 0) return L2KV_OK;
  if (!q || !K_c || !V_c || !cur_len_dev || !out) return L2KV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(K_c) || !aligned16(V_c) || !aligned16(out))
    return L2KV_ERR_MISALIGNED;
  if (workspace && workspace_bytes < (size_t)kStatusBytes) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  const float sc = scale > 0.f ? scale : 1.0f / std::sqrt((float)lay->head_dim);
  const LenView lens{cur_len_dev, per_head ? 1 : 0};
  // beyond its status block the workspace is scratch for the per-chunk results of a split launch
  float* scratch = nullptr;
  size_t scratch_bytes = 0;
  if (workspace && workspace_bytes > (size_t)kStatusBytes) {
    scratch = reinterpret_cast<float*>(static_cast<char*>(workspace) + kStatusBytes);
    scratch_bytes = workspace_bytes - kStatusBytes;
  }
  return launch_prefix_attention(q, K_c, V_c, make_geom(*lay), lay->dtype, n_queries, lens,
                                 max_len, sc, out, lse_out, static_cast<int32_t*>(workspace),
                                 scratch, scratch_bytes, causal ? 1 : 0, split_weights ? 1 : 0,
                                 static_cast<cudaStream_t>(stream));
}

int l2kv_prefix_attention_causal(const void* q, const void* K_c, const void* V_c,
                                 const l2kv_layout* lay, const int32_t* cur_len_dev,
                                 int32_t max_len, int32_t n_queries, float scale, float* out,
                                 float* lse_out, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  return prefix_attention_impl(false, true, false, q, K_c, V_c, lay, cur_len_dev, max_len, n_queries, scale,
                               out, lse_out, workspace, workspace_bytes, stream);
}

int l2kv_prefix_attention_workspace_bytes(const l2kv_layout* lay, int32_t max_len,
                                          int32_t n_queries, size_t* bytes) {
  if (!bytes) return L2KV_ERR_INVALID_ARG;
  int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  rc = check_groups(lay);
  if (rc != L2KV_OK) return rc;
  if (max_len < 0 || n_queries < 0) return L2KV_ERR_INVALID_ARG;
  if (max_len > lay->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  *bytes = (size_t)kStatusBytes;
  if (empty(lay) || n_queries == 0 || lay->dtype != L2KV_BF16 || lay->head_dim != 128)
    return L2KV_OK;
  *bytes += prefix_attention_scratch(make_geom(*lay), n_queries, max_len);
  return L2KV_OK;
}

int l2kv_prefix_attention(const void* q, const void* K_c, const void* V_c, const l2kv_layout* lay,
                          const int32_t* cur_len_dev, int32_t max_len, int32_t n_queries, float scale,
                          float* out, float* lse_out, void* workspace, size_t workspace_bytes,
                          void* stream) {
  return prefix_attention_impl(false, false, false, q, K_c, V_c, lay, cur_len_dev, max_len, n_queries, scale, out,
                               lse_out, workspace, workspace_bytes, stream);
}

int l2kv_prefix_attention_per_head(const void* q, const void* K_c, const void* V_c,
                                   const l2kv_layout* lay, const int32_t* cur_len_unit_dev,
                                   int32_t max_len, int32_t n_queries, float scale, float* out,
                                   float* lse_out, void* workspace, size_t workspace_bytes,
                                   void* stream) {
  return prefix_attention_impl(true, false, false, q, K_c, V_c, lay, cur_len_unit_dev, max_len, n_queries, scale,
                               out, lse_out, workspace, workspace_bytes, stream);
}

int l2kv_prefix_attention_flags(const void* q, const void* K_c, const void* V_c,
                                const l2kv_layout* lay, const int32_t* cur_len_dev, int32_t max_len,
                                int32_t n_queries, float scale, uint32_t flags, float* out,
                                float* lse_out, void* workspace, size_t workspace_bytes,
                                void* stream) {
  if (flags & ~(uint32_t)(L2KV_PREFIX_CAUSAL | L2KV_PREFIX_LEN_PER_HEAD | L2KV_PREFIX_SPLIT_WEIGHTS))
    return L2KV_ERR_INVALID_ARG;
  return prefix_attention_impl((flags & L2KV_PREFIX_LEN_PER_HEAD) != 0, (flags & L2KV_PREFIX_CAUSAL) != 0,
                               (flags & L2KV_PREFIX_SPLIT_WEIGHTS) != 0, q, K_c, V_c, lay, cur_len_dev,
                               max_len, n_queries, scale, out, lse_out, workspace, workspace_bytes,
                               stream);
}

int l2kv_attention_loss_workspace_bytes(const l2kv_layout* lay, int32_t max_len, size_t* bytes) {
  if (!bytes || max_len < 0) return L2KV_ERR_INVALID_ARG;
  const int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  *bytes = attention_loss_workspace(*lay, max_len);
  return L2KV_OK;
}

static int attention_loss_impl(bool per_head, const void* q, const void* K, const l2kv_layout* lay,
                               const int32_t* cur_len_dev, int32_t max_len, float scale,
                               const float* sumsq, float* alr_out, float* loss_out,
                               float* loss_ref_out, void* workspace, size_t workspace_bytes,
                               void* stream) {
  const Range nvtx_range("l2kv_attention_loss");
  int rc = check_layout(lay);
  if (rc != L2KV_OK) return rc;
  if (lay->kv_heads > 0 && lay->q_heads % lay->kv_heads) return L2KV_ERR_INVALID_ARG;
  if (max_len < 0 || !(scale == scale)) return L2KV_ERR_INVALID_ARG;
  if (max_len > lay->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if ((long long)max_len > (1ll << 24)) return L2KV_ERR_OUT_OF_RANGE;
  if (empty(lay) || lay->q_heads == 0) return L2KV_OK;
  if (!q || !K || !cur_len_dev || !sumsq || !alr_out || !workspace) return L2KV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(K) || !aligned16(workspace)) return L2KV_ERR_MISALIGNED;
  if (workspace_bytes < attention_loss_workspace(*lay, max_len)) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  const float sc = scale > 0.f ? scale : 1.0f / std::sqrt((float)lay->head_dim);
  const LenView lens{cur_len_dev, per_head ? 1 : 0};
  return launch_attention_loss(q, K, make_geom(*lay), lay->dtype, lens, max_len, sc, sumsq,
                               alr_out, loss_out, loss_ref_out, static_cast<char*>(workspace),
                               static_cast<cudaStream_t>(stream));
}

int l2kv_attention_loss(const void* q, const void* K, const l2kv_layout* lay,
                        const int32_t* cur_len_dev, int32_t max_len, float scale,
                        const float* sumsq, float* alr_out, float* loss_out, float* loss_ref_out,
                        void* workspace, size_t workspace_bytes, void* stream) {
  return attention_loss_impl(false, q, K, lay, cur_len_dev, max_len, scale, sumsq, alr_out, loss_out,
                             loss_ref_out, workspace, workspace_bytes, stream);
}

int l2kv_attention_loss_per_head(const void* q, const void* K, const l2kv_layout* lay,
                                 const int32_t* cur_len_unit_dev, int32_t max_len, float scale,
                                 const float* sumsq, float* alr_out, float* loss_out,
                                 float* loss_ref_out, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  return attention_loss_impl(true, q, K, lay, cur_len_unit_dev, max_len, scale, sumsq, alr_out, loss_out,
                             loss_ref_out, workspace, workspace_bytes, stream);
}

}  // extern "C"

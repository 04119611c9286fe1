// Decode attention for callers that must not allocate device memory.
//
// l2kv_decode_attention needs scratch for the per-split partial results, and the ordinary
// entry point takes it from a caller-provided workspace.  Some callers cannot provide one:
// code that runs inside a region where cudaMalloc is forbidden or would deadlock (for
// instance while another thread holds the allocator, inside a library callback, or in a
// serving loop whose memory pool is already fully handed out) and that has no buffer of
// its own to spare.  For them the scratch lives here, in a file-scope device array that every
// GPU which loads this library carries from load to exit.
#include <mutex>

#include "common.cuh"

namespace {

// The whole built-in scratch.  Modest on purpose: it is paid for on every GPU, used or not.
static __device__ __align__(256) unsigned char g_decode_scratch[L2KV_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_decode_scratch on the current device.  In host code the array's name
// is only a handle for the runtime, not an address a kernel could use, so the address is
// asked for once per device (with that device current) and remembered.
int scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return L2KV_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || !p) return L2KV_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return L2KV_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int l2kv_decode_attention_static(const void* q, const void* K_c, const void* V_c,
                                            const l2kv_layout* lay, const int32_t* cur_len_dev,
                                            int32_t max_len, float scale, float* out,
                                            void* stream) {
  using namespace l2kv;
  // Layout checks are those of the workspace query (same rules as every other entry point).
  size_t unused = 0;
  if (max_len < 0 || !(scale == scale)) return L2KV_ERR_INVALID_ARG;
  int rc = l2kv_workspace_bytes(lay, max_len, &unused);
  if (rc != L2KV_OK) return rc;
  if (lay->kv_heads > 0) {
    if (lay->q_heads % lay->kv_heads) return L2KV_ERR_INVALID_ARG;
    const int G = lay->q_heads / lay->kv_heads;
    if (G != 1 && G != 2 && G != 4 && G != 8) return L2KV_ERR_UNSUPPORTED;
  }
  if (max_len > lay->t_cap) return L2KV_ERR_OUT_OF_RANGE;
  if (lay->batch == 0 || lay->layers == 0 || lay->kv_heads == 0) return L2KV_OK;
  if (!q || !K_c || !V_c || !cur_len_dev || !out) return L2KV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(K_c) || !aligned16(V_c)) return L2KV_ERR_MISALIGNED;

  // Only the partial results need scratch: [B * L * Hq][splits][D + 2] floats, placed after
  // the status block that starts the array as it starts every workspace.
  WorkspacePlan plan = plan_workspace(*lay, max_len);
  const size_t need = plan.total - plan.partial_off;
  if (need > (size_t)L2KV_STATIC_SCRATCH_BYTES - kStatusBytes) return L2KV_ERR_WORKSPACE_TOO_SMALL;
  plan.partial_off = kStatusBytes;
  plan.ticket_off = plan.partial_off;         // no completion counters here: the merge is a kernel

  void* scratch = nullptr;
  rc = scratch_address(&scratch);
  if (rc != L2KV_OK) return rc;
  const float sc = scale > 0.f ? scale : 1.0f / sqrtf((float)lay->head_dim);
  // The status block starts at zero (the array is zero-initialised when it is loaded) and
  // changes only if a wait gives up; nothing else in the scratch has to start at zero: every
  // partial that the merge step reads is written by the split step of the same call.
  const LenView lens{cur_len_dev, 0};
  return launch_decode_attention(q, K_c, V_c, make_geom(*lay), lay->dtype, lens, max_len, sc,
                                 out, static_cast<char*>(scratch), plan,
                                 static_cast<cudaStream_t>(stream));
}

extern "C" int l2kv_decode_attention_static_status(void* stream, int32_t* status, int32_t reset) {
  if (!status) return L2KV_ERR_INVALID_ARG;
  void* scratch = nullptr;
  int rc = scratch_address(&scratch);
  if (rc != L2KV_OK) return rc;
  rc = l2kv_read_device_status(scratch, stream, status);
  if (rc != L2KV_OK || !reset) return rc;
  return cudaMemsetAsync(scratch, 0, l2kv::kStatusBytes, static_cast<cudaStream_t>(stream)) ==
                 cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

// Selection and compaction.
//
//   selection       runs inside the norm pass (key_norms.cu, select_unit.cuh): exact k-th
//                   smallest of the ordering keys by a most-significant-digit radix select
//                   (4 passes of 8 bits), then per-chunk slot bases by a scan.
//   gather_kernel   one CTA per (unit, chunk of input tokens; two chunks where little is kept): rebuilds the keep flags
//                   from the threshold, ranks the kept tokens with a block scan and copies
//                   their K and V rows (16-byte pieces, LPR lanes per row) to the dense,
//                   position-ordered output together with the index map and the keys.
//
// The kept set is exactly { t : (key_t, t) among the `keep` smallest }: every key below
// the threshold, plus the first `admit` tokens (in position order) whose key equals it.
#include "common.cuh"

namespace l2kv {

constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;
// Chunks of kGatherChunk input tokens that one CTA may take.  The grid has one CTA per chunk.  In
// a unit that keeps at most a quarter of its tokens a CTA would move few rows between three
// dependent round trips to memory (keys, rows in, rows out) and the kernel would idle on latency
// (keep 0.1: 4.4 TB/s), so there the CTAs of even chunks take the next chunk as well and the odd
// ones leave at once; elsewhere one chunk per CTA measured fastest.
#ifndef L2KV_GATHER_GROUP
#define L2KV_GATHER_GROUP 2
#endif
constexpr int kGatherGroup = L2KV_GATHER_GROUP;
constexpr int kGatherSpan = kGatherGroup * kGatherChunk;   // input tokens per CTA

template <typename T, int D>
__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(const T* __restrict__ K, const T* __restrict__ V, Geom gi, T* __restrict__ K_out,
              T* __restrict__ V_out, Geom go, const int32_t* __restrict__ len_dev, int max_len,
              const float* __restrict__ sumsq, long long ld, int policy,
              const UnitRec* __restrict__ unit_rec, const int2* __restrict__ chunk_rec,
              int n_chunks, int32_t* __restrict__ idx_out, float* __restrict__ sumsq_out,
              [[maybe_unused]] int32_t* __restrict__ status_word) {
  constexpr int LPR = D / Elem<T>::kPerVec;
  constexpr int RPS = kGatherThreads / LPR;              // rows per copy step of the CTA
  constexpr int TPT = kGatherSpan / kGatherThreads;      // tokens ranked per thread
  static_assert(kGatherSpan < 65536, "the packed (below, equal) counts hold 16 bits each");
  __shared__ int s_src[kGatherSpan];                     // kept tokens of this CTA's span, in order
  __shared__ int s_warp[kGatherThreads / 32];
  __shared__ int s_total;

  const long long unit = blockIdx.x / n_chunks;
  const int chunk = blockIdx.x % n_chunks;               // first (or only) chunk of this CTA
  const int h = (int)(unit % gi.H);
  const int l = (int)((unit / gi.H) % gi.L);
  const int b = (int)(unit / ((long long)gi.H * gi.L));
  const long long bl = (long long)b * gi.L + l;
  const int len = max(0, min(len_dev[b], min(max_len, gi.cap(bl))));
  const int t0 = chunk * kGatherChunk;
  if (t0 >= len) return;
  const UnitRec ur = unit_rec[unit];
  if (ur.n_keep == 0 || (ur.flags & kFlagCopied)) return;   // nothing kept, or copied by the norm pass
  const int my_chunks = (long long)ur.n_keep * 4 <= len ? kGatherGroup : 1;
  if (chunk % my_chunks) return;                         // a neighbour takes this chunk
  const int t_end = min(len, t0 + my_chunks * kGatherChunk);
  const int2 cr = chunk_rec[unit * n_chunks + chunk];
  const int tid = threadIdx.x;
  const float* key = sumsq + (ld >= 0 ? unit * ld : gi.meta(unit));
  const bool identity = ur.flags & kFlagIdentity;

  int n_kept;
  if (identity) {
    n_kept = t_end - t0;
  } else {
    // Rank this chunk's tokens: packed (below, equal) counts, one exclusive block scan.
    uint32_t kb[TPT];
    int cnt = 0;                                         // low 16 bits: equal, high: below
    // a thread's TPT tokens are consecutive: 16-byte key loads where the array allows them
    [[maybe_unused]] const bool vec = (reinterpret_cast<uintptr_t>(key + t0) & 15u) == 0;
#pragma unroll
    for (int i = 0; i < TPT; ++i) kb[i] = 0xffffffffu;
    if constexpr (TPT % 4 == 0) {
#pragma unroll
      for (int i = 0; i < TPT; i += 4) {
        const int t = t0 + tid * TPT + i;
        if (vec && t + 3 < t_end) {
          const float4 v = *reinterpret_cast<const float4*>(key + t);
          kb[i] = order_bits(v.x, policy);     kb[i + 1] = order_bits(v.y, policy);
          kb[i + 2] = order_bits(v.z, policy); kb[i + 3] = order_bits(v.w, policy);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (t + j < t_end) kb[i + j] = order_bits(key[t + j], policy);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < TPT; ++i) {
        const int t = t0 + tid * TPT + i;
        if (t < t_end) kb[i] = order_bits(key[t], policy);
      }
    }
#pragma unroll
    for (int i = 0; i < TPT; ++i) {
      const int t = t0 + tid * TPT + i;
      if (t < t_end) cnt += (kb[i] < ur.thr ? 0x10000 : 0) + (kb[i] == ur.thr ? 1 : 0);
    }
    int inc = cnt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, inc, off);
      if ((tid & 31) >= off) inc += n;
    }
    if ((tid & 31) == 31) s_warp[tid >> 5] = inc;
    __syncthreads();
    int wbase = 0;
    for (int w = 0; w < (tid >> 5); ++w) wbase += s_warp[w];
    int before = wbase + inc - cnt;
    const int adm0 = min(cr.y, ur.admit);                // admitted ties in earlier chunks
#pragma unroll
    for (int i = 0; i < TPT; ++i) {
      const int t = t0 + tid * TPT + i;
      if (t < t_end) {
        const int less_b = before >> 16, eq_b = before & 0xffff;
        const bool is_less = kb[i] < ur.thr;
        const bool is_eq = kb[i] == ur.thr;
        if (is_less || (is_eq && cr.y + eq_b < ur.admit))
          s_src[less_b + min(cr.y + eq_b, ur.admit) - adm0] = t;
        before += (is_less ? 0x10000 : 0) + (is_eq ? 1 : 0);
      }
    }
    if (tid == kGatherThreads - 1)
      s_total = (before >> 16) + min(cr.y + (before & 0xffff), ur.admit) - adm0;
    __syncthreads();
    n_kept = s_total;
  }

  // Copy the kept rows: LPR adjacent lanes move one row as 16-byte pieces.
  const int piece = tid % LPR, sub = tid / LPR;
  const long long in_base = gi.base(b, l, h) + (long long)piece * Elem<T>::kPerVec;
  const long long out_base = go.base(b, l, h) + (long long)piece * Elem<T>::kPerVec;
  const long long meta_base = go.meta(unit);
  const int out_cap = go.cap(bl);
  const bool no_keys = ur.flags & kFlagNoKeys;
  const int slot0 = cr.x;
  for (int jb = 0; jb < n_kept; jb += RPS * kGatherUnroll) {
    uint4 vk[kGatherUnroll], vv[kGatherUnroll];
    int src[kGatherUnroll];
#pragma unroll
    for (int i = 0; i < kGatherUnroll; ++i) {
      const int j = jb + i * RPS + sub;
      src[i] = j < n_kept ? (identity ? t0 + j : s_src[j]) : -1;
      vk[i] = make_uint4(0, 0, 0, 0);
      vv[i] = make_uint4(0, 0, 0, 0);
      if (src[i] >= 0 && !L2KV_BOUNDS(src[i] >= t0 && src[i] < t_end, status_word)) src[i] = -1;
      if (src[i] >= 0) {
        vk[i] = ld_stream(K + in_base + (long long)src[i] * gi.st);
        vv[i] = ld_stream(V + in_base + (long long)src[i] * gi.st);
      }
    }
#pragma unroll
    for (int i = 0; i < kGatherUnroll; ++i) {
      const int j = jb + i * RPS + sub;
      float s = 0.f;
      if (no_keys) s = piece_sumsq_reduce<T, LPR>(vk[i]);      // CTA-uniform branch
      if (src[i] >= 0) {
        const long long slot = slot0 + j;
        if (slot < out_cap && L2KV_BOUNDS(slot >= 0 && slot < ur.n_keep, status_word)) {
          st_stream(K_out + out_base + slot * go.st, vk[i]);
          st_stream(V_out + out_base + slot * go.st, vv[i]);
          if (piece == 0) {
            idx_out[meta_base + slot] = src[i];
            sumsq_out[meta_base + slot] = no_keys ? s : key[src[i]];
          }
        }
      }
    }
  }
}

template <typename T, int D>
static int launch_sc_t(const void* K, const void* V, const Geom& gi, const int32_t* len_dev,
                       const int32_t* keep_dev, const int32_t* keep_unit_dev, int max_len,
                       const LayerMask& unc, int policy, unsigned long long seed,
                       const float* sumsq_in, void* K_out, void* V_out, const Geom& go,
                       int32_t* idx_out, float* sumsq_out, int32_t* kept_len_dev,
                       int32_t* kept_len_unit_dev, char* ws, const WorkspacePlan& plan,
                       cudaStream_t s) {
  const long long units = (long long)gi.B * gi.L * gi.H;
  if (units == 0) return L2KV_OK;
  if (plan.n_chunks > kMaxChunks) return L2KV_ERR_OUT_OF_RANGE;
  if (units * plan.n_chunks > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  UnitRec* urec = reinterpret_cast<UnitRec*>(ws + plan.unit_off);
  int2* crec = reinterpret_cast<int2*>(ws + plan.chunk_off);
  // Where the ordering keys come from: a pass over K (the default), the caller (keys kept
  // from the time the rows were written: no pass over K at all), or a seeded hash.
  int key_mode = kKeysFromK;
  float* keys = reinterpret_cast<float*>(ws + plan.sumsq_off);
  long long ld = plan.ld_sumsq;
  if (policy == L2KV_KEEP_RANDOM) {
    key_mode = kKeysRandom;
  } else if (sumsq_in) {
    key_mode = kKeysGiven;
    keys = const_cast<float*>(sumsq_in);                 // read-only in this mode
    ld = -1;                                             // laid out like the input cache
  }
  SelectArgs sel;
  sel.keep_dev = keep_dev; sel.keep_unit_dev = keep_unit_dev; sel.out_t_cap = go.t_cap;
  sel.out_row_cap = go.row_cap;
  sel.kept_len_unit_dev = kept_len_unit_dev;
  sel.policy = policy == L2KV_KEEP_HIGHEST_NORM ? L2KV_KEEP_HIGHEST_NORM : L2KV_KEEP_LOWEST_NORM;
  sel.seed = seed;
  sel.n_chunks = plan.n_chunks; sel.unc = unc; sel.unit_rec = urec; sel.chunk_rec = crec;
  sel.tickets = reinterpret_cast<int32_t*>(ws + plan.ticket_off);
  sel.kept_len_dev = kept_len_dev;
  sel.status_word = reinterpret_cast<int32_t*>(ws);
  // Keys of the layers that are compressed (the others are copied whole), and, as each
  // unit's last chunk of keys lands, its selection.
  CopyArgs cp{};
  int n_unc = 0;
  for (int l = 0; l < gi.L; ++l) n_unc += unc.test(l) ? 1 : 0;
  const long long copy_blocks = (long long)gi.B * n_unc * gi.H * plan.n_chunks;
  if (key_mode == kKeysFromK && max_len > 0 && copy_blocks > 0 && copy_blocks < 0x3fffffffLL) {
    cp.V = V; cp.K_out = K_out; cp.V_out = V_out; cp.idx_out = idx_out; cp.sumsq_out = sumsq_out;
    cp.go = go; cp.n_blocks = (int)copy_blocks; cp.n_unc = n_unc; cp.chunks = plan.n_chunks;
  }
  const int rc = launch_key_norms(K, gi, Elem<T>::kDtype, len_dev, max_len, keys, ld, nullptr,
                                  key_mode, &sel, &cp, s);
  if (rc != L2KV_OK) return rc;
  if (max_len > 0) {
    gather_kernel<T, D><<<(unsigned)(units * plan.n_chunks), kGatherThreads, 0, s>>>(
        static_cast<const T*>(K), static_cast<const T*>(V), gi, static_cast<T*>(K_out),
        static_cast<T*>(V_out), go, len_dev, max_len, keys, ld, sel.policy, urec, crec,
        plan.n_chunks, idx_out, sumsq_out, reinterpret_cast<int32_t*>(ws));
    if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  }
  return L2KV_OK;
}

int launch_select_compact(const void* K, const void* V, const Geom& gi, int dtype,
                          const int32_t* len_dev, const int32_t* keep_dev,
                          const int32_t* keep_unit_dev, int max_len,
                          const LayerMask& unc, int policy, unsigned long long seed,
                          const float* sumsq_in, void* K_out, void* V_out, const Geom& go,
                          int32_t* idx_out, float* sumsq_out, int32_t* kept_len_dev,
                          int32_t* kept_len_unit_dev, char* ws,
                          const WorkspacePlan& plan, cudaStream_t s) {
#define L2KV_SC(T, D)                                                                           \
  return launch_sc_t<T, D>(K, V, gi, len_dev, keep_dev, keep_unit_dev, max_len, unc, policy,    \
                           seed, sumsq_in, K_out, V_out, go, idx_out, sumsq_out, kept_len_dev,  \
                           kept_len_unit_dev, ws, plan, s)
  if (dtype == L2KV_BF16) {
    if (gi.D == 128) L2KV_SC(__nv_bfloat16, 128);
    if (gi.D == 64) L2KV_SC(__nv_bfloat16, 64);
  } else if (dtype == L2KV_F32) {
    if (gi.D == 128) L2KV_SC(float, 128);
    if (gi.D == 64) L2KV_SC(float, 64);
  }
#undef L2KV_SC
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

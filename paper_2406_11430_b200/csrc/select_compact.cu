// Selection and compaction.
//
//   select_kernel   one CTA per (b, l, h): exact k-th smallest of the ordering keys by a
//                   most-significant-digit radix select (4 passes of 8 bits) over the
//                   L2-resident key array, then per-chunk slot bases by a scan.
//   gather_kernel   one CTA per (unit, chunk of input tokens): rebuilds the keep flags
//                   from the threshold, ranks the kept tokens with a block scan and copies
//                   their K and V rows (16-byte pieces, LPR lanes per row) to the dense,
//                   position-ordered output together with the index map and the keys.
//
// The kept set is exactly { t : (key_t, t) among the `keep` smallest }: every key below
// the threshold, plus the first `admit` tokens (in position order) whose key equals it.
#include "common.cuh"

namespace l2kv {

constexpr int kSelectThreads = 1024;
constexpr int kGatherThreads = 256;
constexpr int kGatherUnroll = 4;
constexpr uint32_t kFlagIdentity = 1u;           // every valid token is kept
constexpr uint32_t kFlagNoKeys = 2u;             // keys were not precomputed for this unit

struct UnitRec { uint32_t thr; int32_t admit; int32_t n_keep; uint32_t flags; };

__global__ void __launch_bounds__(kSelectThreads)
select_kernel(const float* __restrict__ sumsq, long long ld, Geom g,
              const int32_t* __restrict__ len_dev, const int32_t* __restrict__ keep_dev,
              int max_len, int out_t_cap, LayerMask unc, int policy,
              UnitRec* __restrict__ unit_rec, int2* __restrict__ chunk_rec, int n_chunks,
              int32_t* __restrict__ kept_len_dev) {
  __shared__ int hist[256];
  __shared__ int s_bucket, s_before;
  __shared__ int c_less[kMaxChunks];
  __shared__ int c_eq[kMaxChunks];

  const long long unit = blockIdx.x;
  const int h = (int)(unit % g.H);
  const int l = (int)((unit / g.H) % g.L);
  const int b = (int)(unit / ((long long)g.H * g.L));
  const int tid = threadIdx.x;
  const int len = max(0, min(len_dev[b], min(max_len, g.t_cap)));
  const bool whole = unc.test(l);
  const int keep_req = whole ? len : max(0, min(keep_dev[b], len));
  const bool identity = whole || keep_req == len;
  const int keep = min(keep_req, out_t_cap);      // rows that fit the output; the rest is cut
  if (h == 0 && tid == 0) kept_len_dev[b * g.L + l] = keep;

  const int my_chunks = (len + kGatherChunk - 1) / kGatherChunk;
  int2* crec = chunk_rec + unit * n_chunks;

  if (identity) {
    if (tid == 0) {
      UnitRec r; r.thr = 0xffffffffu; r.admit = 0; r.n_keep = keep;
      r.flags = kFlagIdentity | (whole ? kFlagNoKeys : 0u);
      unit_rec[unit] = r;
    }
    for (int c = tid; c < my_chunks; c += kSelectThreads) crec[c] = make_int2(c * kGatherChunk, 0);
    return;
  }
  if (keep == 0) {
    if (tid == 0) {
      UnitRec r; r.thr = 0u; r.admit = 0; r.n_keep = 0; r.flags = 0u;
      unit_rec[unit] = r;
    }
    for (int c = tid; c < my_chunks; c += kSelectThreads) crec[c] = make_int2(0, 0);
    return;
  }

  const float* key = sumsq + unit * ld;
  uint32_t prefix = 0, mask = 0;
  int k_rem = keep;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    // Run-length accumulation: neighbouring tokens mostly share the high digits.
    int cur = -1, cnt = 0;
    for (int t = tid; t < len; t += kSelectThreads) {
      const uint32_t kb = order_bits(key[t], policy);
      if ((kb & mask) == prefix) {
        const int d = (kb >> shift) & 255;
        if (d == cur) {
          ++cnt;
        } else {
          if (cnt) atomicAdd(&hist[cur], cnt);
          cur = d; cnt = 1;
        }
      }
    }
    if (cnt) atomicAdd(&hist[cur], cnt);
    __syncthreads();
    if (tid < 32) {
      // 8 bins per lane: lane totals -> warp scan -> locate the bin holding rank k_rem.
      int v[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { v[i] = hist[tid * 8 + i]; tot += v[i]; }
      int inc = tot;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, off);
        if (tid >= off) inc += n;
      }
      int before = inc - tot;
      if (before < k_rem && k_rem <= inc) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (before < k_rem && k_rem <= before + v[i]) { s_bucket = tid * 8 + i; s_before = before; }
          before += v[i];
        }
      }
    }
    __syncthreads();
    prefix |= (uint32_t)s_bucket << shift;
    mask |= 255u << shift;
    k_rem -= s_before;
    __syncthreads();
  }
  const uint32_t thr = prefix;      // the keep-th smallest key; k_rem of its copies are admitted
  if (tid == 0) {
    UnitRec r; r.thr = thr; r.admit = k_rem; r.n_keep = keep; r.flags = 0u;
    unit_rec[unit] = r;
  }

  // Per-chunk counts of keys below / equal to the threshold, one warp per chunk.
  const int warp = tid >> 5, lane = tid & 31;
  for (int c = warp; c < my_chunks; c += kSelectThreads / 32) {
    const int t0 = c * kGatherChunk;
    int nl = 0, ne = 0;
    for (int t = t0 + lane; t < min(len, t0 + kGatherChunk); t += 32) {
      const uint32_t kb = order_bits(key[t], policy);
      nl += kb < thr;
      ne += kb == thr;
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      nl += __shfl_xor_sync(0xffffffffu, nl, off);
      ne += __shfl_xor_sync(0xffffffffu, ne, off);
    }
    if (lane == 0) { c_less[c] = nl; c_eq[c] = ne; }
  }
  __syncthreads();
  if (tid == 0) {
    int slot = 0, eq_before = 0;
    for (int c = 0; c < my_chunks; ++c) {
      crec[c] = make_int2(slot, eq_before);
      const int adm = max(0, min(c_eq[c], k_rem - eq_before));
      slot += c_less[c] + adm;
      eq_before += c_eq[c];
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(const T* __restrict__ K, const T* __restrict__ V, Geom gi, T* __restrict__ K_out,
              T* __restrict__ V_out, Geom go, const int32_t* __restrict__ len_dev, int max_len,
              const float* __restrict__ sumsq, long long ld, int policy,
              const UnitRec* __restrict__ unit_rec, const int2* __restrict__ chunk_rec,
              int n_chunks, int32_t* __restrict__ idx_out, float* __restrict__ sumsq_out) {
  constexpr int LPR = D / Elem<T>::kPerVec;
  constexpr int RPS = kGatherThreads / LPR;              // rows per copy step of the CTA
  constexpr int TPT = kGatherChunk / kGatherThreads;     // tokens ranked per thread
  __shared__ int s_src[kGatherChunk];                    // kept tokens of this chunk, in order
  __shared__ int s_warp[kGatherThreads / 32];
  __shared__ int s_total;

  const long long unit = blockIdx.x / n_chunks;
  const int chunk = blockIdx.x % n_chunks;
  const int h = (int)(unit % gi.H);
  const int l = (int)((unit / gi.H) % gi.L);
  const int b = (int)(unit / ((long long)gi.H * gi.L));
  const int len = max(0, min(len_dev[b], min(max_len, gi.t_cap)));
  const int t0 = chunk * kGatherChunk;
  if (t0 >= len) return;
  const int t_end = min(len, t0 + kGatherChunk);
  const UnitRec ur = unit_rec[unit];
  if (ur.n_keep == 0) return;
  const int2 cr = chunk_rec[unit * n_chunks + chunk];
  const int tid = threadIdx.x;
  const float* key = sumsq + unit * ld;
  const bool identity = ur.flags & kFlagIdentity;

  int n_kept;
  if (identity) {
    n_kept = t_end - t0;
  } else {
    // Rank this chunk's tokens: packed (below, equal) counts, one exclusive block scan.
    uint32_t kb[TPT];
    int cnt = 0;                                         // low 16 bits: equal, high: below
#pragma unroll
    for (int i = 0; i < TPT; ++i) {
      const int t = t0 + tid * TPT + i;
      kb[i] = t < t_end ? order_bits(key[t], policy) : 0xffffffffu;
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
  const long long in_base = b * gi.sb + l * gi.sl + h * gi.sh + (long long)piece * Elem<T>::kPerVec;
  const long long out_base = b * go.sb + l * go.sl + h * go.sh + (long long)piece * Elem<T>::kPerVec;
  const long long meta_base = unit * (long long)go.t_cap;
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
        if (slot < go.t_cap) {
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
                       const int32_t* keep_dev, int max_len, const LayerMask& unc, int policy,
                       void* K_out, void* V_out, const Geom& go, int32_t* idx_out, float* sumsq_out,
                       int32_t* kept_len_dev, char* ws, const WorkspacePlan& plan, cudaStream_t s) {
  const long long units = (long long)gi.B * gi.L * gi.H;
  if (units == 0) return L2KV_OK;
  if (plan.n_chunks > kMaxChunks) return L2KV_ERR_OUT_OF_RANGE;
  if (units * plan.n_chunks > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  float* sumsq = reinterpret_cast<float*>(ws + plan.sumsq_off);
  UnitRec* urec = reinterpret_cast<UnitRec*>(ws + plan.unit_off);
  int2* crec = reinterpret_cast<int2*>(ws + plan.chunk_off);
  // Keys of the layers that are compressed (the others are copied whole).
  const int rc = launch_key_norms(K, gi, Elem<T>::kDtype, len_dev, max_len, sumsq, plan.ld_sumsq,
                                  nullptr, &unc, s);
  if (rc != L2KV_OK) return rc;
  select_kernel<<<(unsigned)units, kSelectThreads, 0, s>>>(
      sumsq, plan.ld_sumsq, gi, len_dev, keep_dev, max_len, go.t_cap, unc, policy, urec, crec,
      plan.n_chunks, kept_len_dev);
  if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  if (max_len > 0) {
    gather_kernel<T, D><<<(unsigned)(units * plan.n_chunks), kGatherThreads, 0, s>>>(
        static_cast<const T*>(K), static_cast<const T*>(V), gi, static_cast<T*>(K_out),
        static_cast<T*>(V_out), go, len_dev, max_len, sumsq, plan.ld_sumsq, policy, urec, crec,
        plan.n_chunks, idx_out, sumsq_out);
    if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  }
  return L2KV_OK;
}

int launch_select_compact(const void* K, const void* V, const Geom& gi, int dtype,
                          const int32_t* len_dev, const int32_t* keep_dev, int max_len,
                          const LayerMask& unc, int policy, void* K_out, void* V_out,
                          const Geom& go, int32_t* idx_out, float* sumsq_out, int32_t* kept_len_dev,
                          char* ws, const WorkspacePlan& plan, cudaStream_t s) {
#define L2KV_SC(T, D)                                                                             \
  return launch_sc_t<T, D>(K, V, gi, len_dev, keep_dev, max_len, unc, policy, K_out, V_out, go,   \
                           idx_out, sumsq_out, kept_len_dev, ws, plan, s)
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

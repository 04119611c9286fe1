// Shared device/host helpers of the l2kv kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "l2kv.h"

namespace l2kv {

constexpr int kStatusBytes = 256;      // device status word lives at the start of a workspace
constexpr int kMaxLayers = 1024;       // size of the uncompressed-layer bit mask
constexpr int kGatherChunk = 512;      // input tokens per gather CTA / per scan chunk
constexpr int kMaxChunks = 4096;       // kGatherChunk * kMaxChunks tokens per unit at most
#ifndef L2KV_DECODE_CHUNK
#define L2KV_DECODE_CHUNK 1024
#endif
constexpr int kDecodeChunk = L2KV_DECODE_CHUNK;   // cached tokens per split of decode attention

// Cache geometry handed to kernels by value (strides in elements).  Dense caches are
// [B, L, H, t_cap, D]; packed caches (row_off != null) are [H, total_rows, D] with the rows of
// (b, l) at [row_off[b * L + l], + row_cap[b * L + l]) of the shared row axis, for every head.
// The per-row index map and keys follow the cache: [B, L, H, t_cap] or [H, total_rows].
struct Geom {
  int B, L, H, Hq, D, t_cap;
  long long sb, sl, sh, st;
  const long long* row_off;
  const int32_t* row_cap;
  long long total_rows;
  // element offset of row 0 of unit (b, l, h)
  __device__ __forceinline__ long long base(int b, int l, int h) const {
    return row_off ? h * sh + row_off[(long long)b * L + l] * st : b * sb + l * sl + h * sh;
  }
  // rows that (b, l) may hold
  __device__ __forceinline__ int cap(long long bl) const { return row_off ? row_cap[bl] : t_cap; }
  // first entry of unit = (b * L + l) * H + h in the index map / key arrays
  __device__ __forceinline__ long long meta(long long unit) const {
    return row_off ? (unit % H) * total_rows + row_off[unit / H] : unit * (long long)t_cap;
  }
  // first row of (b, l) on the row axis of a packed cache (0 for dense ones)
  __device__ __forceinline__ long long row0(long long bl) const { return row_off ? row_off[bl] : 0; }
};

// Result of the selection for one (b, l, h) unit, consumed by the gather kernel.
struct UnitRec { uint32_t thr; int32_t admit; int32_t n_keep; uint32_t flags; };
constexpr uint32_t kFlagIdentity = 1u;           // every valid token is kept
constexpr uint32_t kFlagNoKeys = 2u;             // keys were not precomputed for this unit
constexpr uint32_t kFlagCopied = 4u;             // the norm pass copies this unit itself (see CopyArgs)

struct LayerMask {
  uint32_t w[kMaxLayers / 32];
  __host__ __device__ bool test(int l) const { return (w[l >> 5] >> (l & 31)) & 1u; }
};

// Valid lengths, one per (b, l) or, for caches compressed with a keep count per head, one
// per (b, l, h).
struct LenView {
  const int32_t* p;
  int per_head;
  __device__ __forceinline__ int at(long long bl, int h, int H) const {
    return p[per_head ? bl * H + h : bl];
  }
};

inline Geom make_geom(const l2kv_layout& a) {
  Geom g;
  g.B = a.batch; g.L = a.layers; g.H = a.kv_heads; g.Hq = a.q_heads; g.D = a.head_dim;
  g.t_cap = a.t_cap;
  g.sb = a.stride_b; g.sl = a.stride_l; g.sh = a.stride_h; g.st = a.stride_t;
  g.row_off = reinterpret_cast<const long long*>(a.row_off_dev);
  g.row_cap = a.row_cap_dev;
  g.total_rows = a.total_rows;
  return g;
}

__host__ __device__ inline long long round_up_ll(long long x, long long m) {
  return (x + m - 1) / m * m;
}

// Workspace carve-up (offsets in bytes), identical for every entry point.
struct WorkspacePlan {
  size_t sumsq_off;      // float  [units][ld_sumsq]         ordering keys of the input cache
  size_t unit_off;       // uint32 [units][4]                threshold, admitted ties, kept, flags
  size_t chunk_off;      // int32  [units][n_chunks][2]      slot base / equal-keys-before per chunk
  size_t ticket_off;     // int32  [units]                   norm CTAs finished per unit (rests at 0)
  size_t partial_off;    // float  [B*L*Hq][n_splits][D + 2] decode partials
  size_t total;
  long long ld_sumsq;
  int n_chunks, n_splits;
};

inline WorkspacePlan plan_workspace(const l2kv_layout& a, int max_len) {
  WorkspacePlan p;
  const long long units = (long long)a.batch * a.layers * a.kv_heads;
  p.ld_sumsq = round_up_ll(max_len > 0 ? max_len : 1, 64);
  p.n_chunks = (int)((max_len + kGatherChunk - 1) / kGatherChunk);
  if (p.n_chunks < 1) p.n_chunks = 1;
  p.n_splits = (int)((max_len + kDecodeChunk - 1) / kDecodeChunk);
  if (p.n_splits < 1) p.n_splits = 1;
  size_t off = kStatusBytes;
  // Tickets come first so that their place does not depend on max_len (append/evict, which
  // has no max_len, uses one ticket per (b, l); the norm pass one per unit).
  p.ticket_off = off;  off += (size_t)round_up_ll(units * 4, 256);
  p.sumsq_off = off;   off += (size_t)round_up_ll(units * p.ld_sumsq * 4, 256);
  p.unit_off = off;    off += (size_t)round_up_ll(units * 16, 256);
  p.chunk_off = off;   off += (size_t)round_up_ll(units * p.n_chunks * 8, 256);
  p.partial_off = off;
  off += (size_t)round_up_ll((long long)a.batch * a.layers * a.q_heads * p.n_splits *
                                 (a.head_dim + 2) * 4, 256);
  p.total = off;
  return p;
}

// ---- device status -------------------------------------------------------------------
// Word 0 of a workspace: the first anomaly a kernel saw (an l2kv_status); word 2: abort mark,
// set together with L2KV_ERR_TIMEOUT so that the remaining CTAs of a grid leave at once.
__device__ __forceinline__ void record_timeout(int32_t* status_word) {
  if (!status_word) return;
  atomicExch(status_word, (int)L2KV_ERR_TIMEOUT);
  atomicExch(status_word + 2, 1);
}

// Index checks of the debug build (-DL2KV_DEBUG): L2KV_BOUNDS(ok, status_word) is true when the
// access may go ahead; when it may not, the debug build records L2KV_ERR_DEBUG_BOUNDS and the
// caller skips the access (nothing traps).  The release build compiles the check away.
#ifdef L2KV_DEBUG
__device__ __forceinline__ bool debug_bounds(bool ok, int32_t* status_word) {
  if (!ok && status_word) atomicExch(status_word, (int)L2KV_ERR_DEBUG_BOUNDS);
  return ok;
}
#define L2KV_BOUNDS(ok, status_word) (::l2kv::debug_bounds((ok), (status_word)))
#else
#define L2KV_BOUNDS(ok, status_word) (true)
#endif

// ---- element access ------------------------------------------------------------------

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPerVec = 4;                      // elements in a 16-byte piece
  static constexpr int kDtype = L2KV_F32;
  __device__ static void unpack(const uint4& v, float (&x)[4]) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
    x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  static constexpr int kDtype = L2KV_BF16;
  // bf16 is the upper half of an fp32: widening is a shift / mask, exact.
  __device__ static void unpack(const uint4& v, float (&x)[8]) {
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
    x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
  }
};

// 16-byte streaming load: read-only path, no L1 allocation.
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void st_stream(void* p, const uint4& v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
               :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// The ordering key of a row: every lane of the LPR-lane group that owns the row passes
// its 16-byte piece; all lanes return the same sum.  Fixed order: piece front to back
// by fma, then a butterfly over the pieces (off = LPR/2 .. 1).  Must be reached by
// whole warps.
template <typename T, int LPR>
__device__ __forceinline__ float piece_sumsq_reduce(const uint4& v) {
  float x[Elem<T>::kPerVec];
  Elem<T>::unpack(v, x);
  float acc = 0.f;
#pragma unroll
  for (int e = 0; e < Elem<T>::kPerVec; ++e) acc = __fmaf_rn(x[e], x[e], acc);
#pragma unroll
  for (int off = LPR / 2; off >= 1; off >>= 1) acc = acc + __shfl_xor_sync(0xffffffffu, acc, off);
  return acc;
}

// Sums N per-lane values over the LPR adjacent lanes that share a row, N <= LPR.  Halving
// exchange: at each step a lane keeps half of its values and hands the other half to its
// partner (lane ^ off), so N values cost N - 1 + log2(LPR / N) shuffles instead of
// N * log2(LPR).  Every value is still summed over the lanes by the butterfly off = LPR/2 .. 1
// (x[i] + x[i ^ off] at each level), so the result has the bits of the plain butterfly.  On
// return d[0] is complete for value number  piece / (LPR / N).  Must be reached by whole warps.
template <int N, int LPR>
__device__ __forceinline__ float halving_reduce(float (&d)[N], int piece) {
  int cnt = N;
#pragma unroll
  for (int off = LPR / 2; off >= 1; off >>= 1) {
    if (cnt > 1) {
      const int half = cnt / 2;
      const bool upper = piece & off;
#pragma unroll
      for (int i = 0; i < (N > 1 ? N / 2 : 1); ++i) {
        if (i < half) {
          const float send = upper ? d[i] : d[i + half];
          const float keep = upper ? d[i + half] : d[i];
          d[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
      }
      cnt = half;
    } else {
      d[0] += __shfl_xor_sync(0xffffffffu, d[0], off);
    }
  }
  return d[0];
}

// Ordering key of the keep-random policy: upper half of the SplitMix64 output function
// (Steele, Lea, Flood 2014) applied to the state seed + (unit << 32 | t).
__host__ __device__ inline uint32_t random_key_bits(unsigned long long seed, unsigned long long unit,
                                                    uint32_t t) {
  unsigned long long z = seed + ((unit << 32) | t) + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  z ^= z >> 31;
  return (uint32_t)(z >> 32);
}

// Total order on (key bits, position) used everywhere: non-negative floats order as
// their bit patterns.  For the keep-highest policy the bits are complemented.
__device__ __forceinline__ uint32_t order_bits(float sumsq, int policy) {
  const uint32_t b = __float_as_uint(sumsq);
  return policy == L2KV_KEEP_HIGHEST_NORM ? ~b : b;
}

// Launchers, one per source file (arguments already validated by the C entry points).
// Arguments of the selection that the norm pass runs for each unit as its last chunk finishes.
enum KeyMode { kKeysOnly = 0, kKeysFromK = 1, kKeysRandom = 2, kKeysGiven = 3 };
struct SelectArgs {
  const int32_t* keep_dev;                    // [B], or null when keep_unit_dev is given
  const int32_t* keep_unit_dev;               // [B, L, H] or null
  int32_t* kept_len_unit_dev;                 // [B, L, H] or null
  int out_t_cap, policy, n_chunks;            // policy: how key bits order (lowest / highest)
  const int32_t* out_row_cap;                 // packed output: rows per (b, l), else null
  unsigned long long seed;                    // kKeysRandom
  LayerMask unc;
  UnitRec* unit_rec;
  int2* chunk_rec;
  int32_t* tickets;
  int32_t* kept_len_dev;                      // [B, L] (head 0's length) or null
  int32_t* status_word;                       // workspace status word, or null
};
// Uncompressed layers inside l2kv_select_compact: their whole-unit copies run as the LAST blocks
// of the norm pass's grid, so that they fill the GPU while the selections of the last compressed
// units (one block each, after the stream of K has ended) are still running.
struct CopyArgs {
  const void* V;
  void* K_out;
  void* V_out;
  int32_t* idx_out;
  float* sumsq_out;
  Geom go;
  int n_blocks;                               // trailing copy blocks of the grid (0 = none)
  int n_unc;                                  // uncompressed layers
  int chunks;                                 // kGatherChunk-row chunks per unit
};
int launch_key_norms(const void* K, const Geom& g, int dtype, const int32_t* len_dev, int max_len,
                     float* sumsq, long long ld_sumsq, float* norm_out, int key_mode,
                     const SelectArgs* select, const CopyArgs* copy, cudaStream_t s);
int launch_select_compact(const void* K, const void* V, const Geom& gi, int dtype,
                          const int32_t* len_dev, const int32_t* keep_dev,
                          const int32_t* keep_unit_dev, int max_len,
                          const LayerMask& unc, int policy, unsigned long long seed,
                          const float* sumsq_in, void* K_out, void* V_out, const Geom& go,
                          int32_t* idx_out, float* sumsq_out, int32_t* kept_len_dev,
                          int32_t* kept_len_unit_dev, char* ws,
                          const WorkspacePlan& plan, cudaStream_t s);
int launch_decode_attention(const void* q, const void* K, const void* V, const Geom& g, int dtype,
                            const LenView& cur_len_dev, int max_len, float scale, float* out,
                            char* ws, const WorkspacePlan& plan, cudaStream_t s);
int launch_append_evict(void* K, void* V, int32_t* idx, float* sumsq, const Geom& g, int dtype,
                        int32_t* cur_len_dev, const int32_t* budget_dev, const LayerMask& unc,
                        const void* k_new, const void* v_new, const int32_t* pos_new_dev,
                        int32_t* status_word, int32_t* tickets, int per_head, cudaStream_t s);

int launch_prefix_attention(const void* q, const void* K, const void* V, const Geom& g, int dtype,
                            int n_queries, const LenView& cur_len_dev, int max_len, float scale,
                            float* out, float* lse_out, int32_t* status_word, float* scratch,
                            size_t scratch_bytes, int causal, int split_weights, cudaStream_t s);
size_t prefix_attention_scratch(const Geom& g, int n_queries, int max_len);
size_t attention_loss_workspace(const l2kv_layout& a, int max_len);
int launch_attention_loss(const void* q, const void* K, const Geom& g, int dtype,
                          const LenView& cur_len_dev, int max_len, float scale, const float* sumsq,
                          float* alr_out, float* loss_out, float* loss_ref_out, char* ws,
                          cudaStream_t s);

}  // namespace l2kv

// Decode attention over the (compressed) cache: one query per query head, all G = Hq / Hkv
// query heads of a KV head served by a single read of its K and V rows.
//
//   decode_split_kernel    one CTA per (b, l, kv head, split of kDecodeChunk cached tokens).
//                          Phase 1 streams the split's K rows and leaves the G scores of every
//                          token in shared memory (log2 domain); phase 2 takes the exact
//                          maximum of the split and turns scores into weights 2^(s - m);
//                          phase 3 streams the V rows and accumulates sum_t w_t V_t.  Because
//                          the maximum is known before any weight is used, nothing is ever
//                          rescaled.  The partial (m, sum w, acc[D]) goes to scratch.
//   decode_combine_kernel  merges the partials of all splits of a query head.
//
// All arithmetic is fp32 on values widened exactly from the stored bf16 / fp32.
#include <cstdlib>
#include <cstring>

#include "async_copy.cuh"

namespace l2kv {

constexpr int kDecThreads = 256;
constexpr int kDecUnroll = 4;
constexpr float kLog2e = 1.4426950408889634f;

template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecThreads)
decode_split_kernel(const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                    Geom g, LenView cur_len_dev, int max_len,
                    float scale_log2e, float* __restrict__ partial, int n_splits) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  constexpr int RPS = kDecThreads / LPR;
  constexpr int NW = kDecThreads / 32;
  constexpr int kSmemFloats = (kDecodeChunk * G > NW * G * D) ? kDecodeChunk * G : NW * G * D;
  __shared__ __align__(16) float s_buf[kSmemFloats];     // weights [token][G]; later warp sums
  __shared__ float s_red[NW][G];
  __shared__ float s_m[G], s_l[G];

  const int split = blockIdx.x % n_splits;
  const long long unit = blockIdx.x / n_splits;          // (b * L + l) * H + h
  const int h = (int)(unit % g.H);
  const long long bl = unit / g.H;
  const int l = (int)(bl % g.L);
  const int b = (int)(bl / g.L);
  const int n = max(0, min(cur_len_dev.at(bl, h, g.H), min(max_len, g.cap(bl))));
  const int t0 = split * kDecodeChunk;
  if (t0 >= n) return;
  const int t_end = min(n, t0 + kDecodeChunk);
  const int nt = t_end - t0;

  const int tid = threadIdx.x, piece = tid % LPR, sub = tid / LPR;
  const int warp = tid >> 5, lane = tid & 31;
  const long long kv_base = g.base(b, l, h) + (long long)piece * EPV;

  // ---- phase 1: scores ------------------------------------------------------------
  float qf[G][EPV];
#pragma unroll
  for (int gi = 0; gi < G; ++gi) {
    const uint4 v =
        *reinterpret_cast<const uint4*>(q + ((bl * g.Hq + h * G + gi) * D + piece * EPV));
    Elem<T>::unpack(v, qf[gi]);
#pragma unroll
    for (int e = 0; e < EPV; ++e) qf[gi][e] *= scale_log2e;
  }
  const int my_head = piece / (LPR / G);
  const bool writer = (piece % (LPR / G)) == 0;
  for (int rb = 0; rb < nt; rb += RPS * kDecUnroll) {
    uint4 v[kDecUnroll];
#pragma unroll
    for (int i = 0; i < kDecUnroll; ++i) {
      const int tl = rb + i * RPS + sub;
      v[i] = tl < nt ? ld_stream(K + kv_base + (long long)(t0 + tl) * g.st)
                     : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < kDecUnroll; ++i) {
      const int tl = rb + i * RPS + sub;
      float x[EPV], d[G];
      Elem<T>::unpack(v[i], x);
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) a = fmaf(qf[gi][e], x[e], a);
        d[gi] = a;
      }
      const float s = halving_reduce<G, LPR>(d, piece);
      if (writer && tl < nt) s_buf[tl * G + my_head] = s;
    }
  }
  __syncthreads();

  // ---- phase 2: exact maximum of the split, weights, their sum -----------------------
  float mx[G];
#pragma unroll
  for (int gi = 0; gi < G; ++gi) mx[gi] = -INFINITY;
  for (int tl = tid; tl < nt; tl += kDecThreads) {
#pragma unroll
    for (int gi = 0; gi < G; ++gi) mx[gi] = fmaxf(mx[gi], s_buf[tl * G + gi]);
  }
#pragma unroll
  for (int gi = 0; gi < G; ++gi) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1)
      mx[gi] = fmaxf(mx[gi], __shfl_xor_sync(0xffffffffu, mx[gi], off));
    if (lane == 0) s_red[warp][gi] = mx[gi];
  }
  __syncthreads();
  if (tid < G) {
    float m = s_red[0][tid];
    for (int w = 1; w < NW; ++w) m = fmaxf(m, s_red[w][tid]);
    s_m[tid] = m;
  }
  __syncthreads();
  float sum[G];
#pragma unroll
  for (int gi = 0; gi < G; ++gi) { mx[gi] = s_m[gi]; sum[gi] = 0.f; }
  for (int tl = tid; tl < nt; tl += kDecThreads) {
#pragma unroll
    for (int gi = 0; gi < G; ++gi) {
      const float w = exp2f(s_buf[tl * G + gi] - mx[gi]);
      s_buf[tl * G + gi] = w;
      sum[gi] += w;
    }
  }
#pragma unroll
  for (int gi = 0; gi < G; ++gi) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) sum[gi] += __shfl_xor_sync(0xffffffffu, sum[gi], off);
    if (lane == 0) s_red[warp][gi] = sum[gi];          // s_red's maxima were consumed above
  }
  __syncthreads();
  if (tid < G) {
    float acc = 0.f;
    for (int w = 0; w < NW; ++w) acc += s_red[w][tid];
    s_l[tid] = acc;
  }

  // ---- phase 3: weighted sum of the V rows ------------------------------------------
  float acc[G][EPV];
#pragma unroll
  for (int gi = 0; gi < G; ++gi)
#pragma unroll
    for (int e = 0; e < EPV; ++e) acc[gi][e] = 0.f;
  for (int rb = 0; rb < nt; rb += RPS * kDecUnroll) {
    uint4 v[kDecUnroll];
#pragma unroll
    for (int i = 0; i < kDecUnroll; ++i) {
      const int tl = rb + i * RPS + sub;
      v[i] = tl < nt ? ld_stream(V + kv_base + (long long)(t0 + tl) * g.st)
                     : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < kDecUnroll; ++i) {
      const int tl = rb + i * RPS + sub;
      if (tl < nt) {
        float x[EPV], w[G];
        Elem<T>::unpack(v[i], x);
        if constexpr (G == 4) {
          const float4 w4 = *reinterpret_cast<const float4*>(&s_buf[tl * G]);
          w[0] = w4.x; w[1] = w4.y; w[2] = w4.z; w[3] = w4.w;
        } else {
#pragma unroll
          for (int gi = 0; gi < G; ++gi) w[gi] = s_buf[tl * G + gi];
        }
#pragma unroll
        for (int gi = 0; gi < G; ++gi)
#pragma unroll
          for (int e = 0; e < EPV; ++e) acc[gi][e] = fmaf(w[gi], x[e], acc[gi][e]);
      }
    }
  }
  // Row groups of one warp first (lanes that own the same piece), then across warps.
#pragma unroll
  for (int off = 16; off >= LPR; off >>= 1)
#pragma unroll
    for (int gi = 0; gi < G; ++gi)
#pragma unroll
      for (int e = 0; e < EPV; ++e) acc[gi][e] += __shfl_xor_sync(0xffffffffu, acc[gi][e], off);
  __syncthreads();                                       // every read of the weights is done
  if (lane < LPR) {
#pragma unroll
    for (int gi = 0; gi < G; ++gi)
#pragma unroll
      for (int e = 0; e < EPV; ++e) s_buf[(warp * G + gi) * D + lane * EPV + e] = acc[gi][e];
  }
  __syncthreads();
  for (int o = tid; o < G * D; o += kDecThreads) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) a += s_buf[w * G * D + o];
    const int gi = o / D, dd = o % D;
    float* p = partial + ((bl * g.Hq + h * G + gi) * n_splits + split) * (long long)(D + 2);
    p[2 + dd] = a;
    if (dd == 0) { p[0] = s_m[gi]; p[1] = s_l[gi]; }
  }
}

template <int D>
__global__ void __launch_bounds__(D)
decode_combine_kernel(const float* __restrict__ partial, LenView cur_len_dev,
                      int max_len, Geom g, int n_splits, float* __restrict__ out,
                      const int32_t* __restrict__ status_word) {
  // a split kernel that gave up left partial results behind that mean nothing: write no output
  if (status_word && status_word[2] != 0) return;
  const int H = g.H, Hq = g.Hq;
  const long long row = blockIdx.x;                      // (b * L + l) * Hq + hq
  const long long bl = row / Hq;
  const int h = (int)(row % Hq) / (Hq / H);
  const int n = max(0, min(cur_len_dev.at(bl, h, H), min(max_len, g.cap(bl))));
  const int ns = (n + kDecodeChunk - 1) / kDecodeChunk;
  const int d = threadIdx.x;
  const float* p = partial + row * n_splits * (long long)(D + 2);
  __shared__ float s_w[D], s_l[D], s_red[D / 32];
  // the splits' maxima: strided over the threads, then reduced (exact in any order)
  float m = -INFINITY;
  for (int s = d; s < ns; s += D) m = fmaxf(m, p[s * (D + 2)]);
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
  if ((d & 31) == 0) s_red[d >> 5] = m;
  __syncthreads();
#pragma unroll
  for (int w = 0; w < D / 32; ++w) m = fmaxf(m, s_red[w]);
  // D splits at a time: their weights and sums go to shared memory once, then every thread adds
  // its output element over the splits in order (independent loads, same sums as a plain loop)
  float den = 0.f, num = 0.f;
  for (int s0 = 0; s0 < ns; s0 += D) {
    const int tile = min(D, ns - s0);
    __syncthreads();
    if (d < tile) {
      s_w[d] = exp2f(p[(s0 + d) * (D + 2)] - m);
      s_l[d] = p[(s0 + d) * (D + 2) + 1];
    }
    __syncthreads();
    const float* acc = p + (long long)s0 * (D + 2) + 2 + d;
#pragma unroll 8
    for (int t = 0; t < tile; ++t) {
      den = fmaf(s_w[t], s_l[t], den);
      num = fmaf(s_w[t], acc[t * (D + 2)], num);
    }
  }
  out[row * D + d] = ns > 0 ? num / den : 0.f;
}

// ---------------------------------------------------------------------------------------
// bf16, head_dim 128: the same three phases with the two contractions on tensor cores.
//
// The CUDA-core kernel above spends ~70 warp instructions per cached token (unpack, FMA,
// shuffles), which at G = 4 fills two thirds of the issue slots and leaves the kernel
// latency-bound well below the HBM rate.  Here the work per token is a handful of
// instructions, so the kernel is a pure stream:
//   * K and V rows travel global -> shared memory with 16-byte cp.async copies through a
//     ring of kStages stages of kStageTok tokens (16-byte pieces XOR-swizzled by row so that
//     ldmatrix reads are conflict-free); nothing is staged in registers.
//   * scores: S^T[token, head] = K[token, :] . Q^T -- mma.m16n8k16, A = 16 tokens x 16 dims of
//     K (ldmatrix), B = Q^T with the G heads padded to N = 8, fp32 accumulators.
//   * output: O^T[dim, head] = V^T[dim, token] . P^T -- A = V^T via ldmatrix.trans, B = the
//     weights split into two bf16 terms (hi + lo carries 16 mantissa bits), fp32 accumulators.
//     Warp w owns output dims [16w, 16w + 16) for the whole split, so no cross-warp sum.
// bf16 x bf16 products are exact in fp32, so the arithmetic is the same as above up to the
// summation order inside the tensor core and the 2^-17 relative split of the weights.
#ifndef L2KV_MMA_WARPS
#define L2KV_MMA_WARPS 8
#endif
#ifndef L2KV_MMA_STAGES
#define L2KV_MMA_STAGES 3
#endif
#ifndef L2KV_MMA_MIN_CTAS
#define L2KV_MMA_MIN_CTAS 2
#endif
constexpr int kMmaWarps = L2KV_MMA_WARPS;              // 8, 4 or 2: each warp scores 16 tokens a stage
constexpr int kMmaThreads = 32 * kMmaWarps;
constexpr int kStageTok = 16 * kMmaWarps;              // tokens per ring stage
constexpr int kStages = L2KV_MMA_STAGES;
constexpr int kDbw = 8 / kMmaWarps;                    // 16-dim output blocks per warp
constexpr int kRowBytes = 256;                         // 128 bf16
constexpr int kScLd = kDecodeChunk + 4;                // floats per head row of the score buffer

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst), "l"(src), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Shared-memory address of the 16-byte piece `ch` of row `row` of a stage.  cp.async path:
// rows of 256 bytes, piece index XORed with row & 7.  TMA path: the two halves of the head
// dimension are separate [kStageTok][128 B] tiles, and the tensor map's 128-byte swizzle XORs
// address bits 4..6 with address bits 7..9 (the 128-byte line number; sb is 128-byte aligned
// and the tiles are whole multiples of 1024 bytes apart).
template <bool TMA>
__device__ __forceinline__ uint32_t tile_addr(uint32_t sb, int row, int ch) {
  if constexpr (TMA) {
    const int line = (int)(sb >> 7) + row;
    return sb + (ch >> 3) * (kStageTok * 128) + row * 128 + (((ch & 7) ^ (line & 7)) << 4);
  } else {
    return sb + row * kRowBytes + ((ch ^ (row & 7)) << 4);
  }
}

template <int G, bool TMA>
__global__ void __launch_bounds__(kMmaThreads, L2KV_MMA_MIN_CTAS)
decode_split_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ K,
                        const __nv_bfloat16* __restrict__ V, Geom g,
                        LenView cur_len_dev, int max_len, float scale_log2e,
                        float* __restrict__ partial, int n_splits,
                        const __grid_constant__ CUtensorMap map_k,
                        const __grid_constant__ CUtensorMap map_v, int32_t* __restrict__ status_word,
                        int32_t* __restrict__ tickets, float* __restrict__ out) {
  constexpr int D = 128;
  constexpr int NW = kMmaWarps;
  constexpr int TPT = kDecodeChunk / kMmaThreads;        // tokens per thread in phase 2
  constexpr int kStageBytes = kStageTok * kRowBytes;
  extern __shared__ unsigned char smem_raw[];
  // Stages start on a 128-byte boundary (required of a tensor-copy destination).
  unsigned char* smem = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  unsigned char* s_stage = smem;                         // [kStages][kStageTok rows of 256 B]
  float* s_sc = reinterpret_cast<float*>(smem + kStages * kStageBytes);           // [G][kScLd]
  __shared__ __align__(8) unsigned long long s_bar[kStages];
  __shared__ float s_red[NW][G];
  __shared__ float s_m[G], s_l[G];

  const int split = blockIdx.x % n_splits;
  const long long unit = blockIdx.x / n_splits;          // (b * L + l) * H + h
  const int h = (int)(unit % g.H);
  const long long bl = unit / g.H;
  const int l = (int)(bl % g.L);
  const int b = (int)(bl / g.L);
  const int n = max(0, min(cur_len_dev.at(bl, h, g.H), min(max_len, g.cap(bl))));
  const int t0 = split * kDecodeChunk;
  if (t0 >= n) {
    // an empty cache has no split to merge: with the merge inside this kernel, split 0 writes the zeros
    if (tickets && split == 0 && n == 0)
      for (int o = threadIdx.x; o < G * D; o += kMmaThreads) out[(bl * g.Hq + h * G) * D + o] = 0.f;
    return;
  }
  if constexpr (TMA) {
    // A copy that timed out in an earlier CTA marks the workspace; the rest of the grid
    // then leaves at once instead of timing out CTA by CTA.
    if (status_word && *reinterpret_cast<volatile int32_t*>(status_word + 2) != 0) return;
  }
  const int nt = min(n, t0 + kDecodeChunk) - t0;
  const int n_st = (nt + kStageTok - 1) / kStageTok;     // stages of K, and again of V
  const int total = 2 * n_st;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int fr = lane >> 2, fc = lane & 3;               // fragment row / column-pair indices
  const __nv_bfloat16* Kb = K + g.base(b, l, h) + (long long)t0 * g.st;
  const __nv_bfloat16* Vb = V + g.base(b, l, h) + (long long)t0 * g.st;
  // Tensor-map coordinates of this unit: (token, head, layer, batch) for a dense cache; a packed
  // cache is one [H, total_rows] plane, so the unit's first row joins the token coordinate.
  [[maybe_unused]] const int tm_row = (int)g.row0(bl) + t0;
  [[maybe_unused]] const int tm_l = g.row_off ? 0 : l, tm_b = g.row_off ? 0 : b;
  const uint32_t stage0 = smem_u32(s_stage);

  // Copy plan of this thread, fixed for the whole kernel: it moves the 16-byte piece c_ch of
  // rows c_row, c_row + kRowStep, ... of every stage.  kRowStep is a multiple of 8, so the
  // swizzled piece index is the same for all of them and only pointers advance.
  static_assert(kMmaWarps == 4 || kMmaWarps == 8, "copy plan needs a row step that is a multiple of 8");
  constexpr int kRowStep = kMmaThreads / 16;
  constexpr int kCopies = kStageTok / kRowStep;            // 8 pieces per thread per stage
  const int c_row = tid >> 4, c_ch = tid & 15;
  const uint32_t c_dst = stage0 + c_row * kRowBytes + ((c_ch ^ (c_row & 7)) << 4);
  const long long row_bytes = g.st * 2;                    // global bytes between cached rows
  const char* c_k = reinterpret_cast<const char*>(Kb) + c_row * row_bytes + c_ch * 16;
  const char* c_v = reinterpret_cast<const char*>(Vb) + c_row * row_bytes + c_ch * 16;
  auto issue = [&](int s) {
    const int st = s < n_st ? s : s - n_st;
    if constexpr (TMA) {
      // One thread hands the whole stage to the copy engine: two boxes of kStageTok rows x
      // 64 elements.  Rows past the tensor's t_cap arrive as zeros; rows between the valid
      // length and t_cap arrive as stored and are masked where they could matter.
      if (tid == 0) {
        const uint32_t bar = smem_u32(&s_bar[s % kStages]);
        const uint32_t dst = stage0 + (s % kStages) * kStageBytes;
        const CUtensorMap* map = s < n_st ? &map_k : &map_v;
        mbar_expect_tx(bar, kStageBytes);
        tma_load_5d(dst, map, bar, 0, tm_row + st * kStageTok, h, tm_l, tm_b);
        tma_load_5d(dst + kStageTok * 128, map, bar, 64, tm_row + st * kStageTok, h, tm_l, tm_b);
      }
    } else {
      const char* src = (s < n_st ? c_k : c_v) + (long long)st * kStageTok * row_bytes;
      const uint32_t dst = c_dst + (s % kStages) * kStageBytes;
      const int rows = nt - st * kStageTok;                // valid rows of this stage (>= 1)
      if (rows >= kStageTok) {
#pragma unroll
        for (int i = 0; i < kCopies; ++i)
          cp_async16(dst + i * kRowStep * kRowBytes, src + i * kRowStep * row_bytes, 16);
      } else {
#pragma unroll
        for (int i = 0; i < kCopies; ++i) {
          const bool ok = c_row + i * kRowStep < rows;     // rows past the end are zero-filled
          cp_async16(dst + i * kRowStep * kRowBytes,
                     ok ? src + i * kRowStep * row_bytes : src - c_row * row_bytes, ok ? 16 : 0);
        }
      }
    }
  };

  if constexpr (TMA) {
    if (tid == 0) {
      for (int i = 0; i < kStages; ++i) mbar_init(smem_u32(&s_bar[i]), 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
  }
  for (int s = 0; s < kStages - 1; ++s) {
    if (s < total) issue(s);
    if constexpr (!TMA) cp_async_commit();
  }

  // Q^T fragments: lane (fr, fc) holds head fr's dims 16j + 2fc (+1) and 16j + 2fc + 8 (+9).
  uint32_t qb[8][2];
#pragma unroll
  for (int j = 0; j < 8; ++j) { qb[j][0] = 0u; qb[j][1] = 0u; }
  if (fr < G) {
    const __nv_bfloat16* qrow = q + (bl * g.Hq + h * G + fr) * D;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      qb[j][0] = *reinterpret_cast<const uint32_t*>(qrow + 16 * j + 2 * fc);
      qb[j][1] = *reinterpret_cast<const uint32_t*>(qrow + 16 * j + 2 * fc + 8);
    }
  }

  float oacc[kDbw][4];                                     // O^T[16 (kDbw warp + db) + fr (+8)][2 fc (+1)]
#pragma unroll
  for (int db = 0; db < kDbw; ++db) { oacc[db][0] = oacc[db][1] = oacc[db][2] = oacc[db][3] = 0.f; }
  bool copy_ok = true;
  for (int s = 0; s < total; ++s) {
    if constexpr (TMA) {
      copy_ok = mbar_wait(smem_u32(&s_bar[s % kStages]), (s / kStages) & 1) && copy_ok;
    } else {
      cp_async_wait<kStages - 2>();
    }
    __syncthreads();                                       // stage s landed; stage s-1 is free
    if (s + kStages - 1 < total) issue(s + kStages - 1);
    if constexpr (!TMA) cp_async_commit();
    const uint32_t sb = stage0 + (s % kStages) * kStageBytes;

    if (s < n_st) {
      // ---- phase 1: scores of tokens [16 warp, 16 warp + 16) of this stage ------------
      const int tl0 = s * kStageTok + warp * 16;
      if (tl0 < nt) {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint32_t a[4];
          ldmatrix_x4(a, tile_addr<TMA>(sb, row, 2 * j + (lane >> 4)));
          mma_bf16(c, a, qb[j][0], qb[j][1]);
        }
        if (2 * fc < G) {
          s_sc[(2 * fc) * kScLd + tl0 + fr] = c[0] * scale_log2e;
          s_sc[(2 * fc) * kScLd + tl0 + fr + 8] = c[2] * scale_log2e;
        }
        if (2 * fc + 1 < G) {
          s_sc[(2 * fc + 1) * kScLd + tl0 + fr] = c[1] * scale_log2e;
          s_sc[(2 * fc + 1) * kScLd + tl0 + fr + 8] = c[3] * scale_log2e;
        }
      }
      if (s == n_st - 1) {
        // ---- phase 2: exact maximum, weights as bf16 hi + lo, their sum -----------------
        __syncthreads();
        float sc[TPT][G], mx[G], sum[G];
#pragma unroll
        for (int gi = 0; gi < G; ++gi) mx[gi] = -INFINITY;
#pragma unroll
        for (int i = 0; i < TPT; ++i) {
          const int tl = tid + i * kMmaThreads;
#pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            sc[i][gi] = tl < nt ? s_sc[gi * kScLd + tl] : -INFINITY;
            mx[gi] = fmaxf(mx[gi], sc[i][gi]);
          }
        }
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1)
            mx[gi] = fmaxf(mx[gi], __shfl_xor_sync(0xffffffffu, mx[gi], off));
          if (lane == 0) s_red[warp][gi] = mx[gi];
        }
        __syncthreads();                                   // also: every score is in registers
        if (tid < G) {
          float m = s_red[0][tid];
          for (int w = 1; w < NW; ++w) m = fmaxf(m, s_red[w][tid]);
          s_m[tid] = m;
        }
        __syncthreads();
#pragma unroll
        for (int gi = 0; gi < G; ++gi) { mx[gi] = s_m[gi]; sum[gi] = 0.f; }
#pragma unroll
        for (int i = 0; i < TPT; ++i) {
          const int tl = tid + i * kMmaThreads;
#pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            const float w = exp2f(sc[i][gi] - mx[gi]);     // 0 for tokens past the end
            sum[gi] += w;
            const __nv_bfloat16 hi = __float2bfloat16_rn(w);
            const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
            __nv_bfloat16* prow = reinterpret_cast<__nv_bfloat16*>(s_sc + gi * kScLd);
            prow[tl] = hi;                                 // hi terms: first half of the row
            prow[kScLd + tl] = lo;                         // lo terms: second half
          }
        }
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) sum[gi] += __shfl_xor_sync(0xffffffffu, sum[gi], off);
          if (lane == 0) s_red[warp][gi] = sum[gi];
        }
        __syncthreads();                                   // weights and partial sums visible
        if (tid < G) {
          float acc = 0.f;
          for (int w = 0; w < NW; ++w) acc += s_red[w][tid];
          s_l[tid] = acc;
        }
      }
    } else {
      // ---- phase 3: O^T[16 warp .. +16, head] += V^T . P^T over this stage's tokens ------
      const int st = s - n_st;
      const int ksteps = min(kStageTok / 16, (nt - st * kStageTok + 15) / 16);
      // Per-lane constants: weights of head fr as packed token pairs; V^T tile addresses.
      const uint32_t* pw = reinterpret_cast<const uint32_t*>(s_sc + fr * kScLd) +
                           st * (kStageTok / 2) + fc;
      const int vrow = (lane & 7) + (lane >> 4) * 8;
      constexpr int kPitch = TMA ? 128 : kRowBytes;        // bytes between rows of a tile
      uint32_t voff[kDbw];
#pragma unroll
      for (int db = 0; db < kDbw; ++db)
        voff[db] = tile_addr<TMA>(sb, vrow, 2 * (warp * kDbw + db) + ((lane >> 3) & 1));
      // TMA path only: tokens of the last, partial 16-token step that lie past the valid
      // length hold whatever the cache holds there; their V^T entries are cleared in
      // registers so that 0 * (Inf or NaN) cannot reach the accumulators.
      const int valid = nt - st * kStageTok;               // valid tokens of this stage
      auto kstep = [&](int ks) {
        uint32_t h0 = 0u, h1 = 0u, l0 = 0u, l1 = 0u;
        if (fr < G) {
          h0 = pw[ks * 8];              h1 = pw[ks * 8 + 4];
          l0 = pw[kScLd / 2 + ks * 8];  l1 = pw[kScLd / 2 + ks * 8 + 4];
        }
#pragma unroll
        for (int db = 0; db < kDbw; ++db) {
          uint32_t a[4];
          ldmatrix_x4_trans(a, voff[db] + ks * 16 * kPitch);
          if constexpr (TMA) {
            if (ks * 16 + 16 > valid) {
              const int t = ks * 16 + 2 * fc;              // a[0], a[1]: tokens t, t+1; a[2], a[3]: +8
              const uint32_t m0 = (t < valid ? 0x0000ffffu : 0u) | (t + 1 < valid ? 0xffff0000u : 0u);
              const uint32_t m1 = (t + 8 < valid ? 0x0000ffffu : 0u) | (t + 9 < valid ? 0xffff0000u : 0u);
              a[0] &= m0; a[1] &= m0; a[2] &= m1; a[3] &= m1;
            }
          }
          mma_bf16(oacc[db], a, h0, h1);
          mma_bf16(oacc[db], a, l0, l1);
        }
      };
      if (ksteps == kStageTok / 16) {
#pragma unroll
        for (int ks = 0; ks < kStageTok / 16; ++ks) kstep(ks);
      } else {
        for (int ks = 0; ks < ksteps; ++ks) kstep(ks);
      }
    }
  }
  if constexpr (TMA) {
    if (!copy_ok && tid == 0) record_timeout(status_word);   // also marks the grid for leaving
  } else {
    cp_async_wait<0>();
  }

  // O^T fragments: rows = dims 16 (kDbw warp + db) + fr (+8), columns = heads 2 fc (+1).
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int head = 2 * fc + e;
    if (head < G) {
      float* p = partial + ((bl * g.Hq + h * G + head) * n_splits + split) * (long long)(D + 2);
      if (!L2KV_BOUNDS(split < n_splits && t0 + nt <= g.cap(bl), status_word)) continue;
#pragma unroll
      for (int db = 0; db < kDbw; ++db) {
        p[2 + 16 * (warp * kDbw + db) + fr] = oacc[db][e];
        p[2 + 16 * (warp * kDbw + db) + fr + 8] = oacc[db][2 + e];
      }
    }
  }
  if (tid < G) {
    float* p = partial + ((bl * g.Hq + h * G + tid) * n_splits + split) * (long long)(D + 2);
    p[0] = s_m[tid];
    p[1] = s_l[tid];
  }
  if (!tickets) return;                                    // the caller merges with a kernel of its own

  // ---- merge, by the split that finishes last (a ticket per unit; nobody waits) ----------------
  // out = sum_s 2^(m_s - m) acc_s / sum_s 2^(m_s - m) l_s over the unit's splits, in split order:
  // the same sums as decode_combine_kernel, whichever block happens to form them.
  __shared__ int s_last;
  __threadfence();                                         // this split's partial is visible device-wide
  __syncthreads();
  const int ns = (n + kDecodeChunk - 1) / kDecodeChunk;    // splits of this unit that hold tokens
  if (tid == 0) s_last = (ns == 1) || (atomicAdd(tickets + unit, 1) == ns - 1);
  __syncthreads();
  if (!s_last) return;
  if constexpr (TMA) {
    // a split of this grid gave up: its partial means nothing, so no output (the status is set)
    if (!copy_ok || (status_word && *reinterpret_cast<volatile int32_t*>(status_word + 2) != 0)) return;
  }
  __threadfence();                                         // see the other splits' partials
  float* s_w = s_sc;                                       // [G][ns] weights, then [G] denominators
  for (int i = tid; i < G * ns; i += kMmaThreads) {
    const int head = i / ns, sp = i % ns;
    s_w[i] = __ldcg(partial + ((bl * g.Hq + h * G + head) * n_splits + sp) * (long long)(D + 2));
  }
  __syncthreads();
  if (tid < G) {
    float m = -INFINITY;
    for (int sp = 0; sp < ns; ++sp) m = fmaxf(m, s_w[tid * ns + sp]);
    s_m[tid] = m;
  }
  __syncthreads();
  for (int i = tid; i < G * ns; i += kMmaThreads) s_w[i] = exp2f(s_w[i] - s_m[i / ns]);
  __syncthreads();
  for (int o = tid; o < G * D; o += kMmaThreads) {
    const int head = o / D, d = o % D;
    const float* p = partial + (bl * g.Hq + h * G + head) * n_splits * (long long)(D + 2);
    float den = 0.f, num = 0.f;
    for (int sp = 0; sp < ns; ++sp) {
      const float wgt = s_w[head * ns + sp];
      den = fmaf(wgt, __ldcg(p + sp * (D + 2) + 1), den);
      num = fmaf(wgt, __ldcg(p + sp * (D + 2) + 2 + d), num);
    }
    out[(bl * g.Hq + h * G + head) * D + d] = num / den;
  }
  if (tid == 0 && ns > 1) tickets[unit] = 0;               // counters rest at zero between calls
}

template <int G>
static int launch_dec_mma(const void* q, const void* K, const void* V, const Geom& g,
                          const LenView& cur_len_dev, int max_len, float scale, float* out,
                          char* ws, const WorkspacePlan& plan, cudaStream_t s) {
  const long long units = (long long)g.B * g.L * g.H;
  if (units == 0) return L2KV_OK;
  if (units * plan.n_splits > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  float* partial = reinterpret_cast<float*>(ws + plan.partial_off);
  // The per-unit completion counters of the workspace let the last split of a unit merge its
  // partials inside the split kernel; a scratch without them (the built-in one) gets the merge
  // kernel instead.  The weights of the merge reuse the score buffer: G * splits floats.
  int32_t* tickets = plan.ticket_off + (size_t)units * 4 <= plan.partial_off && plan.n_splits <= kDecodeChunk
                         ? reinterpret_cast<int32_t*>(ws + plan.ticket_off) : nullptr;
  if (std::getenv("L2KV_DECODE_MERGE_KERNEL")) tickets = nullptr;   // the two-kernel form, for comparison
  constexpr int smem_bytes = 128 + kStages * kStageTok * kRowBytes + G * kScLd * 4;
  if (max_len > 0) {
    // K and V rows reach shared memory through TMA tensor maps; L2KV_DECODE_COPY=cpasync (or a
    // geometry the encoder rejects) selects the per-thread cp.async copies instead.
    alignas(64) CUtensorMap map_k, map_v;
    std::memset(&map_k, 0, sizeof map_k);
    std::memset(&map_v, 0, sizeof map_v);
    const char* mode = std::getenv("L2KV_DECODE_COPY");
    const bool want_tma = !(mode && std::strcmp(mode, "cpasync") == 0);
    const bool tma = want_tma && make_cache_map(&map_k, K, g, kStageTok) && make_cache_map(&map_v, V, g, kStageTok);
    auto kern = tma ? decode_split_mma_kernel<G, true> : decode_split_mma_kernel<G, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) !=
        cudaSuccess)
      return L2KV_ERR_CUDA;
    kern<<<(unsigned)(units * plan.n_splits), kMmaThreads, smem_bytes, s>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(K),
        static_cast<const __nv_bfloat16*>(V), g, cur_len_dev, max_len, scale * kLog2e, partial,
        plan.n_splits, map_k, map_v,
        plan.partial_off >= (size_t)kStatusBytes ? reinterpret_cast<int32_t*>(ws) : nullptr,
        tickets, out);
    if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
    if (tickets) return L2KV_OK;                           // merged by the last split of every unit
  }
  decode_combine_kernel<128><<<(unsigned)((long long)g.B * g.L * g.Hq), 128, 0, s>>>(
      partial, cur_len_dev, max_len, g, plan.n_splits, out,
      plan.partial_off >= (size_t)kStatusBytes ? reinterpret_cast<const int32_t*>(ws) : nullptr);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

template <typename T, int D, int G>
static int launch_dec_t(const void* q, const void* K, const void* V, const Geom& g,
                        const LenView& cur_len_dev, int max_len, float scale, float* out, char* ws,
                        const WorkspacePlan& plan, cudaStream_t s) {
  const long long units = (long long)g.B * g.L * g.H;
  if (units == 0) return L2KV_OK;
  if (units * plan.n_splits > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  float* partial = reinterpret_cast<float*>(ws + plan.partial_off);
  if (max_len > 0) {
    decode_split_kernel<T, D, G><<<(unsigned)(units * plan.n_splits), kDecThreads, 0, s>>>(
        static_cast<const T*>(q), static_cast<const T*>(K), static_cast<const T*>(V), g,
        cur_len_dev, max_len, scale * kLog2e, partial, plan.n_splits);
    if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  }
  decode_combine_kernel<D><<<(unsigned)((long long)g.B * g.L * g.Hq), D, 0, s>>>(
      partial, cur_len_dev, max_len, g, plan.n_splits, out, nullptr);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

template <typename T, int D>
static int launch_dec_g(const void* q, const void* K, const void* V, const Geom& g,
                        const LenView& cur_len_dev, int max_len, float scale, float* out, char* ws,
                        const WorkspacePlan& plan, cudaStream_t s) {
  switch (g.Hq / g.H) {
    case 1: return launch_dec_t<T, D, 1>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
    case 2: return launch_dec_t<T, D, 2>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
    case 4: return launch_dec_t<T, D, 4>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
#if L2KV_DECODE_CHUNK <= 1024   /* the score buffer of 8 heads x a longer split exceeds static shared memory */
    case 8: return launch_dec_t<T, D, 8>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
#endif
  }
  return L2KV_ERR_UNSUPPORTED;
}

int launch_decode_attention(const void* q, const void* K, const void* V, const Geom& g, int dtype,
                            const LenView& cur_len_dev, int max_len, float scale, float* out,
                            char* ws, const WorkspacePlan& plan, cudaStream_t s) {
#define L2KV_DA(T, D) \
  return launch_dec_g<T, D>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s)
  if (dtype == L2KV_BF16) {
    if (g.D == 128) {
      switch (g.Hq / g.H) {
        case 1: return launch_dec_mma<1>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
        case 2: return launch_dec_mma<2>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
        case 4: return launch_dec_mma<4>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
        case 8: return launch_dec_mma<8>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
      }
      return L2KV_ERR_UNSUPPORTED;
    }
    if (g.D == 64) L2KV_DA(__nv_bfloat16, 64);
  } else if (dtype == L2KV_F32) {
    if (g.D == 128) L2KV_DA(float, 128);
    if (g.D == 64) L2KV_DA(float, 64);
  }
#undef L2KV_DA
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

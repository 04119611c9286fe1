// Attention loss of the norm-based compression against the ideal one (Section 3, Eqs. 5-7).
//
// For one query per query head over the cached keys: a_p = softmax_p(scale q . k_p);
// L^m = attention mass of the m tokens the method drops first (largest (key, position));
// L^{m,ref} = mass of the m smallest a_p; Y = sum_m (L^m - L^{m,ref}).
//
// One CTA of 1024 threads per (b, l, kv head) does everything for the G query heads of that KV head:
//   1. the method's drop order: a stable radix sort (4 passes of 8 bits) of the positions by
//      their key bits -- stable, so equal keys stay in position order;
//   2. the scores of all G heads from ONE read of the unit's K rows (bf16, head_dim 128: tensor
//      cores, mma.m16n8k16 with the K fragments loaded straight from global memory; other types:
//      CUDA cores, one head at a time);
//   3. per head: weights 2^(s - max), their fp64 running sum in drop order, a radix sort of the
//      weights (3 passes of 10 bits: a weight is a float in [0, 1], 30 significant bits) and the
//      fp64 running sum of the sorted values; the sums are divided by the weights' total last.
// A stable radix pass cuts the array into 32 contiguous segments, one per warp, and ranks 32
// consecutive elements at a time (equal digits found by ballots): destination = (elements with
// a smaller digit) + (same digit in earlier warps) + (same digit earlier in this warp).  Up to
// 32768 tokens the arrays bounce between global scratch and a 128 KB shared-memory buffer;
// longer caches use global scratch (L2) for both sides.
//
// Every index that is computed from data (a scatter slot, a position read back from a sorted
// array) is checked before it is used; one that is out of range is skipped and the unit's
// results become NaN, so a fault in the arithmetic shows as a wrong answer, never as a stray
// memory access.
#include "common.cuh"

namespace l2kv {

constexpr int kLossThreads = 1024;
constexpr int kLossWarps = kLossThreads / 32;
constexpr int kLossSmallMax = 32768;          // tokens whose arrays fit the shared buffer
constexpr int kProbBits = 10;                 // digit of the weight sort
constexpr int kOrderBits = 8;                 // digit of the drop-order sort

__device__ __forceinline__ uint32_t digit_of(uint32_t e, int shift, int bits) {
  return (e >> shift) & ((1u << bits) - 1u);
}

// Where element i of an array lives in the shared-memory buffer when the array is read by
// running_sums: rotating every group of 32 by its group number spreads the lanes' contiguous
// runs over the banks.
__device__ __forceinline__ int rotated(int i) { return (i & ~31) | ((i + (i >> 5)) & 31); }

// Lanes of the warp whose digit equals this lane's, among the lanes set in `valid`: one ballot
// per digit bit (match.any measured some 80 cycles a call here and made the sort many times
// slower).
template <int BITS>
__device__ __forceinline__ uint32_t same_digit(uint32_t d, uint32_t valid) {
  uint32_t peers = valid;
#pragma unroll
  for (int k = 0; k < BITS; ++k) {
    const bool bit = (d >> k) & 1u;
    const uint32_t b = __ballot_sync(0xffffffffu, bit);
    peers &= bit ? b : ~b;
  }
  return peers;
}

// Counter tables of the radix passes hold 16-bit entries when n <= 32768 (two per word) and
// 32-bit entries otherwise.
__device__ __forceinline__ void table_add_one(unsigned short* row, uint32_t d) {
  atomicAdd(reinterpret_cast<uint32_t*>(row) + (d >> 1), 1u << (16 * (d & 1u)));
}
__device__ __forceinline__ void table_add_one(uint32_t* row, uint32_t d) { atomicAdd(row + d, 1u); }

struct KeyIsElement {
  __device__ __forceinline__ uint32_t operator()(uint32_t e) const { return e; }
};
// Key of a position: the bits of its stored ordering key (a position out of range reads key 0
// and raises the flag).
struct KeyOfPosition {
  const float* key;
  int n;
  int* bad;
  __device__ __forceinline__ uint32_t operator()(uint32_t pos) const {
    if (pos >= (uint32_t)n) { *bad = 1; pos = 0; }
    return __float_as_uint(key[pos]);
  }
};

// One stable pass of a least-significant-digit radix sort of src[0, n) into dst[0, n) on the digit
// (key_of(element) >> shift) & (2^BITS - 1), by the whole CTA (IOTA: the source is 0, 1, 2, ...
// and src is not read).  table: shared [kLossWarps][2^BITS] of C (C must hold n); s_scan: shared
// [kLossWarps] ints; bad: shared flag raised when a slot falls outside [0, n).  src and dst may
// be global or shared memory and must not overlap (they are deliberately not __restrict__: a
// buffer is read again after the pass before wrote it, and loads through the read-only path
// could return lines cached two passes ago); ROT: element i of the result goes to
// dst[rotated(i)].  Ends with a barrier: dst is complete and table is free again.
template <typename C, int BITS, bool ROT, bool IOTA, typename KeyFn>
__device__ void radix_pass(const uint32_t* src, uint32_t* dst, int n, int shift, C* table, int* s_scan,
                           int* bad, KeyFn key_of) {
  constexpr int BINS = 1 << BITS;
  constexpr int R = 8;                                   // rounds whose loads are in flight together
  static_assert(BINS <= kLossThreads, "one digit per thread in the scan");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg = ((n + kLossWarps - 1) / kLossWarps + 31) & ~31;      // elements per warp, whole rounds
  const int lo = min(n, warp * seg), hi = min(n, lo + seg);
  C* mine = table + warp * BINS;
  for (int i = tid; i < kLossWarps * BINS; i += kLossThreads) table[i] = 0;
  __syncthreads();
  // counts per (warp, digit): shared-memory atomics on this warp's row
  for (int i0 = lo; i0 < hi; i0 += 32 * R) {
    uint32_t e[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int i = i0 + r * 32 + lane;
      e[r] = i < hi ? (IOTA ? (uint32_t)i : src[i]) : 0u;
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
      if (i0 + r * 32 + lane < hi) table_add_one(mine, digit_of(key_of(e[r]), shift, BITS));
  }
  __syncthreads();
  // exclusive offsets in the order (digit, warp)
  int total = 0;
  if (tid < BINS) {
    int run = 0;
#pragma unroll 8
    for (int w = 0; w < kLossWarps; ++w) {
      const int c = table[w * BINS + tid];
      table[w * BINS + tid] = (C)run;
      run += c;
    }
    total = run;
  }
  int inc = total;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += o;
  }
  if (lane == 31) s_scan[warp] = inc;
  __syncthreads();
  int base = inc - total;
  for (int w = 0; w < warp; ++w) base += s_scan[w];
  if (tid < BINS) {
#pragma unroll 8
    for (int w = 0; w < kLossWarps; ++w) table[w * BINS + tid] = (C)(table[w * BINS + tid] + base);
  }
  __syncthreads();
  // scatter: lanes of a round that share a digit take consecutive slots in lane order
  const uint32_t lt = (1u << lane) - 1u;
  for (int i0 = lo; i0 < hi; i0 += 32 * R) {
    uint32_t e[R], kd[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int i = i0 + r * 32 + lane;
      e[r] = i < hi ? (IOTA ? (uint32_t)i : src[i]) : 0u;
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
      kd[r] = i0 + r * 32 + lane < hi ? digit_of(key_of(e[r]), shift, BITS) : 0u;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (i0 + r * 32 < hi) {                            // uniform over the warp
        const bool ok = i0 + r * 32 + lane < hi;
        const uint32_t d = kd[r];
        const uint32_t peers = same_digit<BITS>(d, __ballot_sync(0xffffffffu, ok));
        int off = 0;
        if (ok) {
          off = mine[d];
          const int to = off + __popc(peers & lt);
          if (to >= 0 && to < n) dst[ROT ? rotated(to) : to] = e[r];
          else *bad = 1;
        }
        __syncwarp();
        if (ok && lane == __ffs(peers) - 1) mine[d] = (C)(off + __popc(peers));
        __syncwarp();
      }
    }
  }
  __syncthreads();
}

// The first pass of a sort of plain keys may put equal digits in any order: one table for the
// whole CTA (shared, uint32 [2^BITS]), slots handed out by atomics.
template <int BITS>
__device__ void radix_pass_unordered(const uint32_t* src, uint32_t* dst, int n, int shift,
                                     uint32_t* table, int* s_scan, int* bad) {
  constexpr int BINS = 1 << BITS;
  constexpr int R = 8;
  static_assert(BINS <= kLossThreads, "one digit per thread in the scan");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < BINS) table[tid] = 0;
  __syncthreads();
  for (int i0 = 0; i0 < n; i0 += kLossThreads * R) {
    uint32_t e[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int i = i0 + r * kLossThreads + tid;
      e[r] = i < n ? src[i] : 0u;
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
      if (i0 + r * kLossThreads + tid < n) atomicAdd(table + digit_of(e[r], shift, BITS), 1u);
  }
  __syncthreads();
  const int total = tid < BINS ? (int)table[tid] : 0;
  int inc = total;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += o;
  }
  if (lane == 31) s_scan[warp] = inc;
  __syncthreads();
  int base = inc - total;
  for (int w = 0; w < warp; ++w) base += s_scan[w];
  if (tid < BINS) table[tid] = (uint32_t)base;
  __syncthreads();
  for (int i0 = 0; i0 < n; i0 += kLossThreads * R) {
    uint32_t e[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int i = i0 + r * kLossThreads + tid;
      e[r] = i < n ? src[i] : 0u;
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (i0 + r * kLossThreads + tid < n) {
        const uint32_t to = atomicAdd(table + digit_of(e[r], shift, BITS), 1u);
        if (to < (uint32_t)n) dst[to] = e[r];
        else *bad = 1;
      }
    }
  }
  __syncthreads();
}

// Inclusive running sum, in index order, of f(i) for i in [0, n); emit(i, sum_i) is called when
// want_emit; returns the sum of all the running sums (every thread gets it).  fp64 throughout.
// A warp owns a contiguous range and each of its lanes a contiguous run of it, so that an element
// costs two additions (the running sum, and the sum of running sums); the runs' and ranges'
// starting values come from one warp scan and one pass over the warps' totals.
template <typename F, typename Emit>
__device__ double running_sums(int n, F f, Emit emit, bool want_emit, double* s_warp) {
  constexpr int R = 8;                                   // loads in flight together
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg = ((n + kLossWarps - 1) / kLossWarps + 31) & ~31;      // elements per warp
  const int run = seg >> 5;                                            // elements per lane
  const int lo = min(n, warp * seg + lane * run), hi = min(n, lo + run);
  // this lane's run from a start of 0: its sum, and the sum of its running sums
  double acc = 0.0, accs = 0.0;
  for (int i0 = lo; i0 < hi; i0 += R) {
    float x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) x[r] = i0 + r < hi ? f(i0 + r) : 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      if (i0 + r < hi) { acc += (double)x[r]; accs += acc; }
    }
  }
  // start of this lane's run inside the warp's range, then of the range inside the array
  double incl = acc;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const double o = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += o;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  double start = incl - acc;
  for (int w = 0; w < warp; ++w) start += s_warp[w];
  __syncthreads();
  double runs = accs + start * (double)(hi - lo);
  if (want_emit) {
    double v = start;
    for (int i0 = lo; i0 < hi; i0 += R) {
      float x[R];
#pragma unroll
      for (int r = 0; r < R; ++r) x[r] = i0 + r < hi ? f(i0 + r) : 0.f;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (i0 + r < hi) { v += (double)x[r]; emit(i0 + r, v); }
      }
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) runs += __shfl_xor_sync(0xffffffffu, runs, off);
  if (lane == 0) s_warp[warp] = runs;
  __syncthreads();
  double sum = 0.0;
  for (int w = 0; w < kLossWarps; ++w) sum += s_warp[w];
  __syncthreads();
  return sum;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Scores (log2 domain) of G <= 8 query heads of one KV head for all n cached keys, written to
// probs[g * ld + t]; the heads' maxima to s_max[g].  bf16 / head_dim 128: a warp takes 16 tokens
// at a time.  The contraction index of an mma step may be any fixed arrangement of the head
// dimension as long as both operands use the same one, so a lane loads whole 16-byte pieces of
// its two key rows (pieces 4 jj + (lane & 3), jj = 0..3) and feeds each piece to two steps; the
// query fragments are the same pieces of head (lane >> 2)'s query.
__device__ void scores_mma(const __nv_bfloat16* __restrict__ q_unit, const __nv_bfloat16* __restrict__ Kb,
                           long long st, int n, int G /* <= 8 */, float scale_log2e, float* probs,
                           long long ld, float* s_max, float* s_red /*[kLossWarps][8]*/) {
  constexpr int D = 128;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int fr = lane >> 2, fc = lane & 3;
  uint4 qv[4];
#pragma unroll
  for (int jj = 0; jj < 4; ++jj)
    qv[jj] = fr < G ? *reinterpret_cast<const uint4*>(q_unit + fr * D + 8 * (4 * jj + fc))
                    : make_uint4(0, 0, 0, 0);
  float mx0 = -INFINITY, mx1 = -INFINITY;                // heads 2 fc and 2 fc + 1
  const int tiles = (n + 15) / 16;
  for (int tile = warp; tile < tiles; tile += kLossWarps) {
    const int r0 = tile * 16 + fr, r1 = r0 + 8;
    uint4 ka[4], kb[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      ka[jj] = r0 < n ? ld_stream(Kb + (long long)r0 * st + 8 * (4 * jj + fc)) : make_uint4(0, 0, 0, 0);
      kb[jj] = r1 < n ? ld_stream(Kb + (long long)r1 * st + 8 * (4 * jj + fc)) : make_uint4(0, 0, 0, 0);
    }
    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      mma_bf16_16816(c, ka[jj].x, kb[jj].x, ka[jj].y, kb[jj].y, qv[jj].x, qv[jj].y);
      mma_bf16_16816(c, ka[jj].z, kb[jj].z, ka[jj].w, kb[jj].w, qv[jj].z, qv[jj].w);
    }
    if (2 * fc < G) {
      const float s0 = c[0] * scale_log2e, s2 = c[2] * scale_log2e;
      if (r0 < n) { probs[(2 * fc) * ld + r0] = s0; mx0 = fmaxf(mx0, s0); }
      if (r1 < n) { probs[(2 * fc) * ld + r1] = s2; mx0 = fmaxf(mx0, s2); }
    }
    if (2 * fc + 1 < G) {
      const float s1 = c[1] * scale_log2e, s3 = c[3] * scale_log2e;
      if (r0 < n) { probs[(2 * fc + 1) * ld + r0] = s1; mx1 = fmaxf(mx1, s1); }
      if (r1 < n) { probs[(2 * fc + 1) * ld + r1] = s3; mx1 = fmaxf(mx1, s3); }
    }
  }
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {               // lanes with the same fc
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
  }
  if (lane < 4) { s_red[warp * 8 + 2 * lane] = mx0; s_red[warp * 8 + 2 * lane + 1] = mx1; }
  __syncthreads();
  if (tid < G) {
    float m = -INFINITY;
    for (int w = 0; w < kLossWarps; ++w) m = fmaxf(m, s_red[w * 8 + tid]);
    s_max[tid] = m;
  }
  __syncthreads();
}

// The same on CUDA cores for the other element types: one head at a time, LPR adjacent lanes
// own one key row.
template <typename T, int D>
__device__ void scores_plain(const T* __restrict__ q_unit, const T* __restrict__ Kb, long long st,
                             int n, int G, float scale_log2e, float* probs, long long ld,
                             float* s_max, float* s_red) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  constexpr int RPS = kLossThreads / LPR;
  constexpr int U = 4;                                   // key rows in flight per thread
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int piece = tid % LPR, sub = tid / LPR;
  for (int g = 0; g < G; ++g) {
    float qf[EPV];
    {
      const uint4 v = *reinterpret_cast<const uint4*>(q_unit + g * D + piece * EPV);
      Elem<T>::unpack(v, qf);
#pragma unroll
      for (int e = 0; e < EPV; ++e) qf[e] *= scale_log2e;
    }
    float mx = -INFINITY;
    for (int rb = 0; rb < n; rb += RPS * U) {
      uint4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int t = rb + u * RPS + sub;
        v[u] = t < n ? ld_stream(Kb + (long long)t * st + piece * EPV) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int t = rb + u * RPS + sub;
        float x[EPV], d[1];
        Elem<T>::unpack(v[u], x);
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < EPV; ++e) acc = fmaf(qf[e], x[e], acc);
        d[0] = acc;
        const float s = halving_reduce<1, LPR>(d, piece);
        if (piece == 0 && t < n) { probs[g * ld + t] = s; mx = fmaxf(mx, s); }
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    if (tid == 0) {
      float m = s_red[0];
      for (int w = 1; w < kLossWarps; ++w) m = fmaxf(m, s_red[w]);
      s_max[g] = m;
    }
    __syncthreads();
  }
}

// SMALL: max_len <= kLossSmallMax; the dynamic shared memory then holds a buffer of max_len
// words after the tables, and the tables are 16 bits wide.
template <typename T, int D, bool SMALL>
__global__ void __launch_bounds__(kLossThreads)
attention_loss_kernel(const T* __restrict__ q, const T* __restrict__ K, Geom g,
                      LenView cur_len_dev, int max_len, float scale_log2e,
                      const float* __restrict__ sumsq, uint32_t* order, uint32_t* order_tmp,
                      long long ld, float* probs, float* sorted, float* alr_out, float* loss_out,
                      float* loss_ref_out) {
  using C = typename std::conditional<SMALL, unsigned short, uint32_t>::type;
  extern __shared__ __align__(16) unsigned char loss_smem[];
  C* table = reinterpret_cast<C*>(loss_smem);            // [kLossWarps][2^kProbBits]
  [[maybe_unused]] uint32_t* s_buf =
      reinterpret_cast<uint32_t*>(loss_smem + sizeof(C) * kLossWarps * (1 << kProbBits));
  __shared__ double s_warp[kLossWarps];
  __shared__ float s_red[kLossWarps * 8];
  __shared__ float s_max[8];
  __shared__ int s_scan[kLossWarps];
  __shared__ int s_bad;

  const long long unit = blockIdx.x;                     // (b * L + l) * H + h
  const int h = (int)(unit % g.H);
  const long long bl = unit / g.H;
  const int l = (int)(bl % g.L), b = (int)(bl / g.L);
  const int G = g.Hq / g.H;
  const int n = max(0, min(cur_len_dev.at(bl, h, g.H), min(max_len, g.cap(bl))));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long row0 = bl * g.Hq + (long long)h * G;   // first query head of this KV head
  if (n == 0) {
    for (int gi = tid; gi < G; gi += kLossThreads) alr_out[row0 + gi] = 0.f;
    return;
  }
  if (tid == 0) s_bad = 0;
  __syncthreads();

  // Drop order of the unit: the positions in ascending (key, position) order; read backwards it
  // is the order in which the method drops tokens.  Four stable passes over the 32 key bits move
  // positions only (the key of a position is looked up); the start is position order, so equal
  // keys end up in position order.
  uint32_t* ord = order + unit * ld;
  uint32_t* ord_tmp = SMALL ? s_buf : order_tmp + unit * ld;
  const KeyOfPosition key_of{sumsq + g.meta(unit), n, &s_bad};
  const T* Kb = K + g.base(b, l, h);
  // The blocks of a wave start together and do the same work, so they would all stream K at the
  // same time and all sort at the same time.  Every other block therefore takes the two steps
  // in the other order: half of the GPU reads K while the other half sorts.
  const bool scores_first = (blockIdx.x & 1) == 0;

  for (int g0 = 0; g0 < G; g0 += 8) {
    const int ng = min(8, G - g0);
    float* P = probs + (row0 + g0) * ld;
    const T* q_part = q + (row0 + g0) * D;
#pragma unroll 1
    for (int step = 0; step < 2; ++step) {
      const bool do_scores = (step == 0) == (scores_first || g0 > 0);
      if (do_scores) {
        // scores of up to 8 heads at a time from one read of K
        if constexpr (std::is_same<T, __nv_bfloat16>::value && D == 128) {
          scores_mma(q_part, Kb, g.st, n, ng, scale_log2e, P, ld, s_max, s_red);
        } else {
          scores_plain<T, D>(q_part, Kb, g.st, n, ng, scale_log2e, P, ld, s_max, s_red);
        }
        __syncthreads();
      } else if (g0 == 0) {
        radix_pass<C, kOrderBits, false, true>(nullptr, ord_tmp, n, 0, table, s_scan, &s_bad, key_of);
        radix_pass<C, kOrderBits, false, false>(ord_tmp, ord, n, kOrderBits, table, s_scan, &s_bad, key_of);
        radix_pass<C, kOrderBits, false, false>(ord, ord_tmp, n, 2 * kOrderBits, table, s_scan, &s_bad, key_of);
        radix_pass<C, kOrderBits, false, false>(ord_tmp, ord, n, 3 * kOrderBits, table, s_scan, &s_bad, key_of);
      }
    }

    for (int gi = 0; gi < ng; ++gi) {
      // weights 2^(s - max), kept unnormalised: the sums are divided by their total at the end
      float* a = P + gi * ld;
      const long long row = row0 + g0 + gi;
      const float m = s_max[gi];
      double part = 0.0;
      for (int t = tid; t < n; t += kLossThreads) {
        const float w = exp2f(a[t] - m);
        a[t] = w;
        part += (double)w;
      }
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
      if (lane == 0) s_warp[warp] = part;
      __syncthreads();
      double denom = 0.0;
      for (int w = 0; w < kLossWarps; ++w) denom += s_warp[w];
      __syncthreads();
      const double inv = 1.0 / denom;

      // L^m: running sum of the weights in the method's drop order (largest key first).  The
      // weights are first gathered into that order (coalesced reads of the order, scattered reads
      // of the weights) in the buffer the sort below will use, then summed from there.
      uint32_t* other = SMALL ? s_buf : reinterpret_cast<uint32_t*>(sorted + row * ld);
      {
        float* stage = reinterpret_cast<float*>(other);
        constexpr int R = 8;
        for (int r0 = 0; r0 < n; r0 += kLossThreads * R) {
          uint32_t pos[R];
#pragma unroll
          for (int j = 0; j < R; ++j) {
            const int r = r0 + j * kLossThreads + tid;
            pos[j] = r < n ? ord[n - 1 - r] : 0u;
            if (pos[j] >= (uint32_t)n) { s_bad = 1; pos[j] = 0u; }
          }
          float x[R];
#pragma unroll
          for (int j = 0; j < R; ++j) x[j] = a[pos[j]];
#pragma unroll
          for (int j = 0; j < R; ++j) {
            const int r = r0 + j * kLossThreads + tid;
            if (r < n) stage[SMALL ? rotated(r) : r] = x[j];
          }
        }
        __syncthreads();
      }
      float* lo = loss_out ? loss_out + row * g.t_cap : nullptr;
      const float* staged = reinterpret_cast<const float*>(other);
      const double sum_l = running_sums(
          n, [=](int r) { return staged[SMALL ? rotated(r) : r]; },
          [=](int r, double v) { lo[r] = (float)(v * inv); }, lo != nullptr, s_warp);

      // L^{m,ref}: running sum of the weights sorted ascending (non-negative floats order as their
      // bit patterns; a weight is at most 1.0 = 0x3f800000, below 2^30)
      uint32_t* src = reinterpret_cast<uint32_t*>(a);
      radix_pass_unordered<kProbBits>(src, other, n, 0, reinterpret_cast<uint32_t*>(table), s_scan, &s_bad);
      radix_pass<C, kProbBits, false, false>(other, src, n, kProbBits, table, s_scan, &s_bad, KeyIsElement());
      radix_pass<C, kProbBits, SMALL, false>(src, other, n, 2 * kProbBits, table, s_scan, &s_bad, KeyIsElement());
      const float* srt = reinterpret_cast<const float*>(other);
      float* lr = loss_ref_out ? loss_ref_out + row * g.t_cap : nullptr;
      const double sum_ref = running_sums(
          n, [=](int r) { return srt[SMALL ? rotated(r) : r]; },
          [=](int r, double v) { lr[r] = (float)(v * inv); }, lr != nullptr, s_warp);
      if (tid == 0) alr_out[row] = s_bad ? __int_as_float(0x7fc00000) : (float)((sum_l - sum_ref) * inv);
      __syncthreads();
    }
  }
}

static long long loss_ld(int max_len) { return round_up_ll(max_len > 0 ? max_len : 1, 64); }

size_t attention_loss_workspace(const l2kv_layout& a, int max_len) {
  const long long ld = loss_ld(max_len);
  const long long units = (long long)a.batch * a.layers * a.kv_heads;
  const long long heads = (long long)a.batch * a.layers * a.q_heads;
  return (size_t)(2 * round_up_ll(units * ld * 4, 256) + 2 * round_up_ll(heads * ld * 4, 256));
}

template <typename T, int D>
static int launch_al_t(const void* q, const void* K, const Geom& g, const LenView& cur_len_dev,
                       int max_len, float scale, const float* sumsq, float* alr_out, float* loss_out,
                       float* loss_ref_out, char* ws, cudaStream_t s) {
  const long long units = (long long)g.B * g.L * g.H;
  const long long heads = (long long)g.B * g.L * g.Hq;
  if (units == 0 || heads == 0) return L2KV_OK;
  if (units > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  const long long ld = loss_ld(max_len);
  uint32_t* order = reinterpret_cast<uint32_t*>(ws);
  uint32_t* order_tmp = order + round_up_ll(units * ld * 4, 256) / 4;
  float* probs = reinterpret_cast<float*>(ws + 2 * round_up_ll(units * ld * 4, 256));
  float* sorted = probs + round_up_ll(heads * ld * 4, 256) / 4;
  const bool small = max_len <= kLossSmallMax;
  const size_t smem = small ? sizeof(unsigned short) * kLossWarps * (1 << kProbBits) + (size_t)ld * 4
                            : sizeof(uint32_t) * kLossWarps * (1 << kProbBits);
  auto kern = small ? attention_loss_kernel<T, D, true> : attention_loss_kernel<T, D, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return L2KV_ERR_CUDA;
  kern<<<(unsigned)units, kLossThreads, smem, s>>>(
      static_cast<const T*>(q), static_cast<const T*>(K), g, cur_len_dev, max_len,
      scale * 1.4426950408889634f, sumsq, order, order_tmp, ld, probs, sorted, alr_out, loss_out,
      loss_ref_out);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

int launch_attention_loss(const void* q, const void* K, const Geom& g, int dtype,
                          const LenView& cur_len_dev, int max_len, float scale, const float* sumsq,
                          float* alr_out, float* loss_out, float* loss_ref_out, char* ws,
                          cudaStream_t s) {
#define L2KV_AL(T, D) \
  return launch_al_t<T, D>(q, K, g, cur_len_dev, max_len, scale, sumsq, alr_out, loss_out, loss_ref_out, ws, s)
  if (dtype == L2KV_BF16) {
    if (g.D == 128) L2KV_AL(__nv_bfloat16, 128);
    if (g.D == 64) L2KV_AL(__nv_bfloat16, 64);
  } else if (dtype == L2KV_F32) {
    if (g.D == 128) L2KV_AL(float, 128);
    if (g.D == 64) L2KV_AL(float, 64);
  }
#undef L2KV_AL
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

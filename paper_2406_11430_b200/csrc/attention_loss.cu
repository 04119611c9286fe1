// Attention loss of the norm-based compression against the ideal one (Section 3, Eqs. 5-7).
//
// For one query per query head over the cached keys: a_p = softmax_p(scale q . k_p);
// L^m = attention mass of the m tokens the method drops first (largest (key, position));
// L^{m,ref} = mass of the m smallest a_p; Y = sum_m (L^m - L^{m,ref}).
//
//   drop_order_kernel      one CTA per (b, l, kv head): sorts (key bits << 32 | position)
//                          ascending; read backwards this is the method's drop order,
//                          shared by the G query heads of the KV head.
//   attention_loss_kernel  one CTA per (b, l, query head): scores -> probabilities, their
//                          running sum in drop order, a sort of the probabilities and its
//                          running sum, and the sum over m of the difference (fp64 sums).
//
// Sorting is a bitonic network on power-of-two padded arrays in global scratch, with every
// run of steps whose distance fits a 64 KB tile done in shared memory (arrays up to the tile
// size never leave it between load and store).  This is an
// analysis tool, not part of the decode hot path.
#include "common.cuh"

namespace l2kv {

constexpr int kLossThreads = 1024;
constexpr int kSortTileBytes = 64 * 1024;   // dynamic shared memory of both kernels: 2-3 CTAs per SM

__host__ __device__ inline int next_pow2(int n) {
  int p = 1;
  while (p < n) p <<= 1;
  return p;
}

// One compare-exchange of the ascending bitonic network (k = size of the sorted runs being
// merged, j = distance), i = global index of the lower partner.
template <typename K>
__device__ __forceinline__ void cmp_swap(K& x, K& y, int i, int k) {
  const bool asc = (i & k) == 0;
  if ((x > y) == asc) { const K t = x; x = y; y = t; }
}

// A full tile (kSortTileBytes) is held E elements per thread in registers, element e of the tile
// = thread * E + r.  Steps of distance j < E are compare-exchanges inside a thread, E <= j < 32 E
// exchanges between lanes of a warp (shuffles), and only j >= 32 E goes through shared memory
// (element (thread, r) at tile[r * threads + thread]: conflict-free for any partner thread).
template <typename K>
__device__ __forceinline__ K keep_of(K mine, K other, int i, int j, int k) {
  const bool lower = (i & j) == 0, asc = (i & k) == 0;
  const bool keep_min = lower == asc;
  const K lo = mine < other ? mine : other, hi = mine < other ? other : mine;
  return keep_min ? lo : hi;
}
// Steps j = j_hi .. 1 of the network for runs of size k, on the tile whose first element has
// global index base.
template <typename K, int E>
__device__ __forceinline__ void tile_steps_regs(K (&x)[E], int base, int k, int j_hi,
                                                K* __restrict__ tile) {
  const int tid = threadIdx.x;
  const int i0 = base + tid * E;
  int j = j_hi;
  for (; j >= 32 * E; j >>= 1) {                         // partner thread in another warp
    const int pt = tid ^ (j / E);
    __syncthreads();                                     // earlier readers of the tile are done
#pragma unroll
    for (int r = 0; r < E; ++r) tile[r * kLossThreads + tid] = x[r];
    __syncthreads();
#pragma unroll
    for (int r = 0; r < E; ++r) x[r] = keep_of(x[r], tile[r * kLossThreads + pt], i0 + r, j, k);
  }
  for (; j >= E; j >>= 1) {                              // partner thread in this warp
    const int lm = j / E;
#pragma unroll
    for (int r = 0; r < E; ++r) x[r] = keep_of(x[r], __shfl_xor_sync(0xffffffffu, x[r], lm), i0 + r, j, k);
  }
#pragma unroll
  for (int jj = E / 2; jj > 0; jj >>= 1) {               // both elements in this thread
    if (jj <= j) {
#pragma unroll
      for (int r = 0; r < E; ++r)
        if ((r & jj) == 0) cmp_swap(x[r], x[r | jj], i0 + r, k);
    }
  }
}

// Sorts a[0, n2) ascending (n2 a power of two) with the whole CTA; tile = shared scratch of
// kSortTileBytes.
template <typename K>
__device__ void bitonic_sort(K* __restrict__ a, int n2, K* __restrict__ tile) {
  const int tid = threadIdx.x;
  constexpr int kFull = kSortTileBytes / (int)sizeof(K);
  constexpr int E = kFull / kLossThreads;
  const int tile_n = min(n2, kFull);
  if (tile_n == kFull) {
    // Full tiles: the register formulation above; global memory only for distances >= a tile.
    auto load = [&](K (&x)[E], int base) {
      const uint4* src = reinterpret_cast<const uint4*>(a + base + tid * E);
      uint4* dst = reinterpret_cast<uint4*>(x);
#pragma unroll
      for (int v = 0; v < (int)(E * sizeof(K) / 16); ++v) dst[v] = src[v];
    };
    auto store = [&](const K (&x)[E], int base) {
      uint4* dst = reinterpret_cast<uint4*>(a + base + tid * E);
      const uint4* src = reinterpret_cast<const uint4*>(x);
#pragma unroll
      for (int v = 0; v < (int)(E * sizeof(K) / 16); ++v) dst[v] = src[v];
    };
    for (int base = 0; base < n2; base += kFull) {       // every tile sorted (direction by position)
      K x[E];
      load(x, base);
      for (int k = 2; k <= kFull; k <<= 1) tile_steps_regs<K, E>(x, base, k, k >> 1, tile);
      store(x, base);
    }
    __syncthreads();
    for (int k = kFull << 1; k <= n2; k <<= 1) {         // merges of runs larger than a tile
      for (int j = k >> 1; j >= kFull; j >>= 1) {
        for (int t = tid; t < n2 / 2; t += kLossThreads) {
          const int lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));
          K x = a[lo], y = a[lo | j];
          cmp_swap(x, y, lo, k);
          a[lo] = x; a[lo | j] = y;
        }
        __syncthreads();
      }
      for (int base = 0; base < n2; base += kFull) {
        K x[E];
        load(x, base);
        tile_steps_regs<K, E>(x, base, k, kFull >> 1, tile);
        store(x, base);
      }
      __syncthreads();
    }
    return;
  }
  // Phase I: each tile sorted (in alternating directions given by its global position).
  for (int base = 0; base < n2; base += tile_n) {
    for (int i = tid; i < tile_n; i += kLossThreads) tile[i] = a[base + i];
    __syncthreads();
    for (int k = 2; k <= tile_n; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int t = tid; t < tile_n / 2; t += kLossThreads) {
          const int lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));      // index with bit j clear
          cmp_swap(tile[lo], tile[lo | j], base + lo, k);
        }
        __syncthreads();
      }
    }
    for (int i = tid; i < tile_n; i += kLossThreads) a[base + i] = tile[i];
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kLossThreads)
drop_order_kernel(const float* __restrict__ sumsq, Geom g, const int32_t* __restrict__ cur_len_dev,
                  int max_len, unsigned long long* __restrict__ order, int ld_order) {
  extern __shared__ __align__(16) unsigned char sort_smem[];
  unsigned long long* tile = reinterpret_cast<unsigned long long*>(sort_smem);
  const long long unit = blockIdx.x;
  const long long bl = unit / g.H;
  const int n = max(0, min(cur_len_dev[bl], min(max_len, g.t_cap)));
  if (n == 0) return;
  const int n2 = next_pow2(n);
  unsigned long long* a = order + unit * ld_order;
  const float* key = sumsq + unit * g.t_cap;
  for (int t = threadIdx.x; t < n2; t += kLossThreads)
    a[t] = t < n ? ((unsigned long long)__float_as_uint(key[t]) << 32) | (uint32_t)t
                 : 0xffffffffffffffffull;                     // padding sorts to the end
  __syncthreads();
  bitonic_sort(a, n2, tile);
}

// Inclusive running sum, in position order, of f(i) for i in [0, n); calls emit(i, sum_i) and
// returns the sum of all the running sums (every thread gets it).  fp64 throughout.
template <typename F, typename E>
__device__ double running_sums(int n, F f, E emit, double* s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  double carry = 0.0, total = 0.0;
  for (int base = 0; base < n; base += kLossThreads) {
    const int i = base + tid;
    double v = i < n ? (double)f(i) : 0.0;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const double o = __shfl_up_sync(0xffffffffu, v, off);
      if (lane >= off) v += o;
    }
    if (lane == 31) s_warp[warp] = v;
    __syncthreads();
    double before = carry;
    for (int w = 0; w < warp; ++w) before += s_warp[w];
    double all = 0.0;
    for (int w = 0; w < kLossThreads / 32; ++w) all += s_warp[w];
    const double run = before + v;
    if (i < n) { emit(i, run); total += run; }
    carry += all;
    __syncthreads();
  }
  // block sum of the per-thread totals
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) total += __shfl_xor_sync(0xffffffffu, total, off);
  if (lane == 0) s_warp[warp] = total;
  __syncthreads();
  double sum = 0.0;
  for (int w = 0; w < kLossThreads / 32; ++w) sum += s_warp[w];
  __syncthreads();
  return sum;
}

template <typename T, int D>
__global__ void __launch_bounds__(kLossThreads)
attention_loss_kernel(const T* __restrict__ q, const T* __restrict__ K, Geom g,
                      const int32_t* __restrict__ cur_len_dev, int max_len, float scale_log2e,
                      const unsigned long long* __restrict__ order, int ld_order,
                      float* __restrict__ probs, float* __restrict__ sorted, float* __restrict__ alr_out,
                      float* __restrict__ loss_out, float* __restrict__ loss_ref_out) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  constexpr int RPS = kLossThreads / LPR;
  extern __shared__ __align__(16) unsigned char sort_smem[];
  float* tile = reinterpret_cast<float*>(sort_smem);
  __shared__ double s_warp[kLossThreads / 32];
  __shared__ float s_redf[kLossThreads / 32];
  __shared__ float s_max;

  const long long row = blockIdx.x;                      // (b * L + l) * Hq + hq
  const int hq = (int)(row % g.Hq);
  const long long bl = row / g.Hq;
  const int l = (int)(bl % g.L), b = (int)(bl / g.L);
  const int G = g.Hq / g.H;
  const int h = hq / G;
  const int n = max(0, min(cur_len_dev[bl], min(max_len, g.t_cap)));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (n == 0) { if (tid == 0) alr_out[row] = 0.f; return; }
  const int n2 = next_pow2(n);
  float* a = probs + row * ld_order;
  float* srt = sorted + row * ld_order;
  const unsigned long long* ord = order + (bl * g.H + h) * ld_order;

  // scores (log2 domain): LPR adjacent lanes own one key row
  const int piece = tid % LPR, sub = tid / LPR;
  float qf[EPV];
  {
    const uint4 v = *reinterpret_cast<const uint4*>(q + row * D + piece * EPV);
    Elem<T>::unpack(v, qf);
#pragma unroll
    for (int e = 0; e < EPV; ++e) qf[e] *= scale_log2e;
  }
  const T* kbase = K + b * g.sb + l * g.sl + h * g.sh + (long long)piece * EPV;
  float mx = -INFINITY;
  constexpr int U = 4;                                   // key rows in flight per thread
  for (int rb = 0; rb < n; rb += RPS * U) {
    uint4 v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = rb + u * RPS + sub;
      v[u] = t < n ? ld_stream(kbase + (long long)t * g.st) : make_uint4(0, 0, 0, 0);
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
      if (piece == 0 && t < n) { a[t] = s; mx = fmaxf(mx, s); }
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  if (lane == 0) s_redf[warp] = mx;
  __syncthreads();
  if (tid == 0) {
    float m = s_redf[0];
    for (int w = 1; w < kLossThreads / 32; ++w) m = fmaxf(m, s_redf[w]);
    s_max = m;
  }
  __syncthreads();
  const float m = s_max;
  // weights and their sum
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
  for (int w = 0; w < kLossThreads / 32; ++w) denom += s_warp[w];
  __syncthreads();
  const float inv = (float)(1.0 / denom);
  for (int t = tid; t < n2; t += kLossThreads) {
    const float p = t < n ? a[t] * inv : __uint_as_float(0x7f800000u);   // +inf pads the sort
    if (t < n) a[t] = p;
    srt[t] = p;
  }
  __syncthreads();

  // L^m: running sum of the probabilities in the method's drop order (largest key first)
  float* lo = loss_out ? loss_out + row * g.t_cap : nullptr;
  const double sum_l = running_sums(
      n, [&](int r) { return a[(uint32_t)(ord[n - 1 - r] & 0xffffffffull)]; },
      [&](int r, double v) { if (lo) lo[r] = (float)v; }, s_warp);

  // L^{m,ref}: running sum of the probabilities sorted ascending (non-negative floats order
  // as their bit patterns)
  bitonic_sort(reinterpret_cast<uint32_t*>(srt), n2, reinterpret_cast<uint32_t*>(tile));
  float* lr = loss_ref_out ? loss_ref_out + row * g.t_cap : nullptr;
  const double sum_ref = running_sums(
      n, [&](int r) { return srt[r]; }, [&](int r, double v) { if (lr) lr[r] = (float)v; }, s_warp);
  if (tid == 0) alr_out[row] = (float)(sum_l - sum_ref);
}

size_t attention_loss_workspace(const l2kv_layout& a, int max_len) {
  const long long ld = next_pow2(max_len > 0 ? max_len : 1);
  const long long units = (long long)a.batch * a.layers * a.kv_heads;
  const long long heads = (long long)a.batch * a.layers * a.q_heads;
  return (size_t)(round_up_ll(units * ld * 8, 256) + 2 * round_up_ll(heads * ld * 4, 256));
}

template <typename T, int D>
static int launch_al_t(const void* q, const void* K, const Geom& g, const int32_t* cur_len_dev,
                       int max_len, float scale, const float* sumsq, float* alr_out, float* loss_out,
                       float* loss_ref_out, char* ws, cudaStream_t s) {
  const long long units = (long long)g.B * g.L * g.H;
  const long long heads = (long long)g.B * g.L * g.Hq;
  if (units == 0 || heads == 0) return L2KV_OK;
  if (heads > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  const int ld = next_pow2(max_len > 0 ? max_len : 1);
  unsigned long long* order = reinterpret_cast<unsigned long long*>(ws);
  float* probs = reinterpret_cast<float*>(ws + round_up_ll(units * (long long)ld * 8, 256));
  float* sorted = probs + round_up_ll(heads * (long long)ld * 4, 256) / 4;
  if (cudaFuncSetAttribute(drop_order_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSortTileBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attention_loss_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSortTileBytes) != cudaSuccess)
    return L2KV_ERR_CUDA;
  drop_order_kernel<<<(unsigned)units, kLossThreads, kSortTileBytes, s>>>(sumsq, g, cur_len_dev, max_len,
                                                                          order, ld);
  if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  attention_loss_kernel<T, D><<<(unsigned)heads, kLossThreads, kSortTileBytes, s>>>(
      static_cast<const T*>(q), static_cast<const T*>(K), g, cur_len_dev, max_len,
      scale * 1.4426950408889634f, order, ld, probs, sorted, alr_out, loss_out, loss_ref_out);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

int launch_attention_loss(const void* q, const void* K, const Geom& g, int dtype,
                          const int32_t* cur_len_dev, int max_len, float scale, const float* sumsq,
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

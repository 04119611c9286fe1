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
#include "common.cuh"

namespace l2kv {

constexpr int kDecThreads = 256;
constexpr int kDecUnroll = 4;
constexpr float kLog2e = 1.4426950408889634f;

// Sums G per-lane partial dot products over the LPR lanes that share a row.  Halving
// exchange: at each step a lane keeps half of its values and hands the other half to its
// partner, so G values cost G - 1 + log2(LPR / G) shuffles instead of G * log2(LPR).
// On return d[0] is complete for head  piece / (LPR / G).
template <int G, int LPR>
__device__ __forceinline__ float reduce_heads(float (&d)[G], int piece) {
  int cnt = G;
#pragma unroll
  for (int off = LPR / 2; off >= 1; off >>= 1) {
    if (cnt > 1) {
      const int half = cnt / 2;
      const bool upper = piece & off;
#pragma unroll
      for (int i = 0; i < G / 2; ++i) {
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

template <typename T, int D, int G>
__global__ void __launch_bounds__(kDecThreads)
decode_split_kernel(const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                    Geom g, const int32_t* __restrict__ cur_len_dev, int max_len,
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
  const int n = max(0, min(cur_len_dev[bl], min(max_len, g.t_cap)));
  const int t0 = split * kDecodeChunk;
  if (t0 >= n) return;
  const int t_end = min(n, t0 + kDecodeChunk);
  const int nt = t_end - t0;

  const int tid = threadIdx.x, piece = tid % LPR, sub = tid / LPR;
  const int warp = tid >> 5, lane = tid & 31;
  const long long kv_base = b * g.sb + l * g.sl + h * g.sh + (long long)piece * EPV;

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
      const float s = reduce_heads<G, LPR>(d, piece);
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
decode_combine_kernel(const float* __restrict__ partial, const int32_t* __restrict__ cur_len_dev,
                      int max_len, int t_cap, int Hq, int n_splits, float* __restrict__ out) {
  const long long row = blockIdx.x;                      // (b * L + l) * Hq + hq
  const long long bl = row / Hq;
  const int n = max(0, min(cur_len_dev[bl], min(max_len, t_cap)));
  const int ns = (n + kDecodeChunk - 1) / kDecodeChunk;
  const int d = threadIdx.x;
  const float* p = partial + row * n_splits * (long long)(D + 2);
  float m = -INFINITY;
  for (int s = 0; s < ns; ++s) m = fmaxf(m, p[s * (D + 2)]);
  float den = 0.f, num = 0.f;
  for (int s = 0; s < ns; ++s) {
    const float w = exp2f(p[s * (D + 2)] - m);
    den = fmaf(w, p[s * (D + 2) + 1], den);
    num = fmaf(w, p[s * (D + 2) + 2 + d], num);
  }
  out[row * D + d] = ns > 0 ? num / den : 0.f;
}

template <typename T, int D, int G>
static int launch_dec_t(const void* q, const void* K, const void* V, const Geom& g,
                        const int32_t* cur_len_dev, int max_len, float scale, float* out, char* ws,
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
      partial, cur_len_dev, max_len, g.t_cap, g.Hq, plan.n_splits, out);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

template <typename T, int D>
static int launch_dec_g(const void* q, const void* K, const void* V, const Geom& g,
                        const int32_t* cur_len_dev, int max_len, float scale, float* out, char* ws,
                        const WorkspacePlan& plan, cudaStream_t s) {
  switch (g.Hq / g.H) {
    case 1: return launch_dec_t<T, D, 1>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
    case 2: return launch_dec_t<T, D, 2>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
    case 4: return launch_dec_t<T, D, 4>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
    case 8: return launch_dec_t<T, D, 8>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s);
  }
  return L2KV_ERR_UNSUPPORTED;
}

int launch_decode_attention(const void* q, const void* K, const void* V, const Geom& g, int dtype,
                            const int32_t* cur_len_dev, int max_len, float scale, float* out,
                            char* ws, const WorkspacePlan& plan, cudaStream_t s) {
#define L2KV_DA(T, D) \
  return launch_dec_g<T, D>(q, K, V, g, cur_len_dev, max_len, scale, out, ws, plan, s)
  if (dtype == L2KV_BF16) {
    if (g.D == 128) L2KV_DA(__nv_bfloat16, 128);
    if (g.D == 64) L2KV_DA(__nv_bfloat16, 64);
  } else if (dtype == L2KV_F32) {
    if (g.D == 128) L2KV_DA(float, 128);
    if (g.D == 64) L2KV_DA(float, 64);
  }
#undef L2KV_DA
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

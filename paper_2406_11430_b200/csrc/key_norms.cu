// Key norms: one streaming pass over K that writes the fp32 sum of squares of every
// cached key row (the ordering key of the compression) and, optionally, its square
// root (the L2 norm itself).  HBM-bound: each byte of K is read exactly once with
// 16-byte coalesced loads; LPR = row bytes / 16 adjacent lanes own one row.
#include "common.cuh"

namespace l2kv {

constexpr int kNormThreads = 256;
constexpr int kNormUnroll = 8;
constexpr int kNormRowsPerCta = 1024;

template <typename T, int D>
__global__ void __launch_bounds__(kNormThreads)
key_norms_kernel(const T* __restrict__ K, Geom g, const int32_t* __restrict__ len_dev,
                 float* __restrict__ sumsq, long long ld, float* __restrict__ norm_out,
                 LayerMask skip, int use_skip, int chunks_per_unit, int max_len) {
  constexpr int LPR = D / Elem<T>::kPerVec;            // lanes per row
  constexpr int RPS = kNormThreads / LPR;              // rows per load step of the CTA
  const long long unit = blockIdx.x / chunks_per_unit;
  const int chunk = blockIdx.x % chunks_per_unit;
  const int h = (int)(unit % g.H);
  const int l = (int)((unit / g.H) % g.L);
  const int b = (int)(unit / ((long long)g.H * g.L));
  if (use_skip && skip.test(l)) return;
  const int len = min(len_dev[b], min(max_len, g.t_cap));
  const int row0 = chunk * kNormRowsPerCta;
  if (row0 >= len) return;
  const int row_end = min(len, row0 + kNormRowsPerCta);

  const int piece = threadIdx.x % LPR;
  const int sub = threadIdx.x / LPR;
  const T* base = K + b * g.sb + l * g.sl + h * g.sh + (long long)piece * Elem<T>::kPerVec;
  float* out = sumsq + unit * ld;
  float* nout = norm_out ? norm_out + unit * ld : nullptr;

  // Loop bounds are uniform over the CTA so that the shuffles below always see full warps.
  for (int rb = row0; rb < row_end; rb += RPS * kNormUnroll) {
    uint4 v[kNormUnroll];
#pragma unroll
    for (int i = 0; i < kNormUnroll; ++i) {
      const int t = rb + i * RPS + sub;
      v[i] = (t < row_end) ? ld_stream(base + (long long)t * g.st) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < kNormUnroll; ++i) {
      const int t = rb + i * RPS + sub;
      const float s = piece_sumsq_reduce<T, LPR>(v[i]);
      if (piece == 0 && t < row_end) {
        out[t] = s;
        if (nout) nout[t] = sqrtf(s);
      }
    }
  }
}

template <typename T, int D>
static int launch_norms_t(const void* K, const Geom& g, const int32_t* len_dev, int max_len,
                          float* sumsq, long long ld, float* norm_out, const LayerMask* skip,
                          cudaStream_t s) {
  const long long units = (long long)g.B * g.L * g.H;
  const int chunks = (max_len + kNormRowsPerCta - 1) / kNormRowsPerCta;
  if (units == 0 || chunks == 0) return L2KV_OK;
  const long long blocks = units * chunks;
  if (blocks > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  LayerMask m = {};
  if (skip) m = *skip;
  key_norms_kernel<T, D><<<(unsigned)blocks, kNormThreads, 0, s>>>(
      static_cast<const T*>(K), g, len_dev, sumsq, ld, norm_out, m, skip ? 1 : 0, chunks, max_len);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

int launch_key_norms(const void* K, const Geom& g, int dtype, const int32_t* len_dev, int max_len,
                     float* sumsq, long long ld_sumsq, float* norm_out, const LayerMask* skip,
                     cudaStream_t s) {
#define L2KV_KN(T, D) \
  return launch_norms_t<T, D>(K, g, len_dev, max_len, sumsq, ld_sumsq, norm_out, skip, s)
  if (dtype == L2KV_BF16) {
    if (g.D == 128) L2KV_KN(__nv_bfloat16, 128);
    if (g.D == 64) L2KV_KN(__nv_bfloat16, 64);
  } else if (dtype == L2KV_F32) {
    if (g.D == 128) L2KV_KN(float, 128);
    if (g.D == 64) L2KV_KN(float, 64);
  }
#undef L2KV_KN
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

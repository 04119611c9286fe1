// Key norms: one streaming pass over K that writes the fp32 sum of squares of every
// cached key row (the ordering key of the compression) and, optionally, its square
// root (the L2 norm itself).  HBM-bound: each byte of K is read exactly once with
// 16-byte coalesced loads; LPR = row bytes / 16 adjacent lanes own one row.
//
// Inside l2kv_select_compact the same pass also runs the selection: the CTA that finishes
// the last chunk of a unit (an atomic ticket per unit, nobody waits) selects that unit's
// threshold while the other CTAs keep streaming, so selection costs no time of its own
// except after the very last units.
#include "select_unit.cuh"

namespace l2kv {

#ifndef L2KV_NORM_THREADS
#define L2KV_NORM_THREADS 256
#endif
#ifndef L2KV_NORM_ROWS
#define L2KV_NORM_ROWS 1024
#endif
constexpr int kNormThreads = L2KV_NORM_THREADS;
constexpr int kNormUnroll = 8;                 // rows per thread per step, all loads in flight
constexpr int kNormRowsPerCta = L2KV_NORM_ROWS;

// Length of a unit's compressed rows: per unit where the caller asked for that, and head 0's
// per (b, l).
__device__ __forceinline__ void publish_kept_len(const SelectArgs& sel, long long unit, int bl,
                                                 int h, int keep) {
  if (sel.kept_len_unit_dev) sel.kept_len_unit_dev[unit] = keep;
  if (h == 0 && sel.kept_len_dev) sel.kept_len_dev[bl] = keep;
}

// One kGatherChunk-row chunk of an uncompressed unit, copied whole: K and V rows to the same
// slots of the output cache, idx = the row's own position, key computed from the row on the way.
template <typename T, int D>
__device__ __forceinline__ void copy_whole_chunk(const T* __restrict__ K, const T* __restrict__ V,
                                                 const Geom& gi, const CopyArgs& cp,
                                                 const int32_t* __restrict__ len_dev, int max_len,
                                                 const LayerMask& unc, int c) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  constexpr int RPS = kNormThreads / LPR;
  constexpr int U = 4;
  __shared__ long long s_cin, s_cout, s_cmeta;
  __shared__ int s_c[3];
  const int tid = threadIdx.x;
  if (tid == 0) {
    const int chunk = c % cp.chunks;
    const long long uu = c / cp.chunks;
    const int h = (int)(uu % gi.H);
    const int li = (int)((uu / gi.H) % cp.n_unc);
    const int b = (int)(uu / ((long long)gi.H * cp.n_unc));
    int l = 0, seen = -1;                               // the li-th layer of the list
    for (int x = 0; x < gi.L; ++x)
      if (unc.test(x) && ++seen == li) { l = x; break; }
    const long long bl = (long long)b * gi.L + l;
    const int len = max(0, min(len_dev[b], min(max_len, gi.cap(bl))));
    s_c[0] = chunk * kGatherChunk;
    s_c[1] = min(len, s_c[0] + kGatherChunk);
    s_c[2] = cp.go.cap(bl);
    s_cin = gi.base(b, l, h);
    s_cout = cp.go.base(b, l, h);
    s_cmeta = cp.go.meta(bl * gi.H + h);
  }
  __syncthreads();
  const int t0 = s_c[0], t_end = s_c[1], out_cap = s_c[2];
  if (t0 >= t_end) return;
  const int piece = tid % LPR, sub = tid / LPR;
  const T* kin = K + s_cin + (long long)piece * EPV;
  const T* vin = V + s_cin + (long long)piece * EPV;
  T* kout = static_cast<T*>(cp.K_out) + s_cout + (long long)piece * EPV;
  T* vout = static_cast<T*>(cp.V_out) + s_cout + (long long)piece * EPV;
  const long long meta = s_cmeta;
  for (int jb = t0; jb < t_end; jb += RPS * U) {         // bounds uniform over the block
    uint4 vk[U], vv[U];
#pragma unroll
    for (int i = 0; i < U; ++i) {
      const int t = jb + i * RPS + sub;
      vk[i] = make_uint4(0, 0, 0, 0);
      vv[i] = make_uint4(0, 0, 0, 0);
      if (t < t_end) {
        vk[i] = ld_stream(kin + (long long)t * gi.st);
        vv[i] = ld_stream(vin + (long long)t * gi.st);
      }
    }
#pragma unroll
    for (int i = 0; i < U; ++i) {
      const int t = jb + i * RPS + sub;
      const float s = piece_sumsq_reduce<T, LPR>(vk[i]);
      if (t < t_end && t < out_cap) {
        st_stream(kout + (long long)t * cp.go.st, vk[i]);
        st_stream(vout + (long long)t * cp.go.st, vv[i]);
        if (piece == 0) {
          cp.idx_out[meta + t] = t;
          cp.sumsq_out[meta + t] = s;
        }
      }
    }
  }
}

template <typename T, int D, int MODE>
__global__ void __launch_bounds__(kNormThreads)
key_norms_kernel(const T* __restrict__ K, Geom g, const int32_t* __restrict__ len_dev,
                 float* __restrict__ sumsq, long long ld, float* __restrict__ norm_out,
                 int chunks_per_unit, int max_len, SelectArgs sel, CopyArgs cp) {
  constexpr int LPR = D / Elem<T>::kPerVec;            // lanes per row
  constexpr int RPS = kNormThreads / LPR;              // row groups of the CTA
  constexpr int U = kNormUnroll;
  constexpr bool SEL = MODE != kKeysOnly;
  static_assert(U <= LPR, "the halving reduction needs at least as many lanes as rows");
  if constexpr (MODE == kKeysFromK) {
    const int norm_blocks = (int)gridDim.x - cp.n_blocks;
    if ((int)blockIdx.x >= norm_blocks) {                // trailing blocks: uncompressed layers
      copy_whole_chunk<T, D>(K, static_cast<const T*>(cp.V), g, cp, len_dev, max_len, sel.unc,
                             (int)blockIdx.x - norm_blocks);
      return;
    }
  }
  const long long unit = blockIdx.x / chunks_per_unit;
  const int chunk = blockIdx.x % chunks_per_unit;
  const int tid = threadIdx.x;
  // Where this unit lives: worked out by one thread and handed round through shared memory, so
  // that the streaming loop below is compiled free of the addressing arithmetic (dense or packed).
  __shared__ long long s_kbase, s_keyoff;
  __shared__ int s_ctx[6];
  if (tid == 0) {
    const int h0 = (int)(unit % g.H);
    const int l0 = (int)((unit / g.H) % g.L);
    const int b0 = (int)(unit / ((long long)g.H * g.L));
    const long long bl0 = (long long)b0 * g.L + l0;
    s_ctx[0] = h0; s_ctx[1] = l0; s_ctx[2] = b0;
    s_ctx[3] = max(0, min(len_dev[b0], min(max_len, g.cap(bl0))));
    s_ctx[4] = SEL ? (sel.out_row_cap ? sel.out_row_cap[bl0] : sel.out_t_cap) : 0;
    s_kbase = g.base(b0, l0, h0);
    s_keyoff = ld >= 0 ? unit * ld : g.meta(unit);         // ld < 0: keys laid out like the cache
  }
  __syncthreads();
  const int h = s_ctx[0], l = s_ctx[1], b = s_ctx[2], len = s_ctx[3];
  [[maybe_unused]] const int out_cap = s_ctx[4];
  [[maybe_unused]] const long long bl = (long long)b * g.L + l;

  if constexpr (SEL) {
    // Units that need no keys: copied layers and empty sequences get their record here.
    const bool whole = sel.unc.test(l);
    if (whole || len == 0) {
      if (chunk == 0) {
        const int keep = min(len, out_cap);
        identity_unit<kNormThreads>(len, keep, true, sel.unit_rec + unit,
                                    sel.chunk_rec + unit * sel.n_chunks,
                                    MODE == kKeysFromK && whole && cp.n_blocks > 0);
        if (tid == 0) publish_kept_len(sel, unit, b * g.L + l, h, keep);
      }
      return;
    }
  }
  float* out = sumsq + s_keyoff;
  if constexpr (MODE != kKeysGiven) {
    const int row0 = chunk * kNormRowsPerCta;
    if (row0 >= len) return;
    const int row_end = min(len, row0 + kNormRowsPerCta);
    if constexpr (MODE == kKeysRandom) {
      // Keys that do not depend on K: seeded counter-based bits, stored as raw 32-bit patterns.
      for (int t = row0 + tid; t < row_end; t += kNormThreads)
        out[t] = __uint_as_float(random_key_bits(sel.seed, (unsigned long long)unit, (uint32_t)t));
    } else {
      const int piece = tid % LPR;
      const int sub = tid / LPR;
      const T* base = K + s_kbase + (long long)piece * Elem<T>::kPerVec;
      float* nout = norm_out ? norm_out + s_keyoff : nullptr;
      const int my_row = piece / (LPR / U);              // which of its U rows this lane reports
      const bool writer = (piece % (LPR / U)) == 0;

      // Thread (sub, piece) owns piece `piece` of rows rb + sub * U + [0, U).  Loop bounds are
      // uniform over the CTA so that the shuffles always see full warps.
      for (int rb = row0; rb < row_end; rb += RPS * U) {
        uint4 v[U];
        const int t0 = rb + sub * U;
#pragma unroll
        for (int i = 0; i < U; ++i)
          v[i] = (t0 + i < row_end) ? ld_stream(base + (long long)(t0 + i) * g.st)
                                    : make_uint4(0, 0, 0, 0);
        float p[U];
#pragma unroll
        for (int i = 0; i < U; ++i) {
          float x[Elem<T>::kPerVec];
          Elem<T>::unpack(v[i], x);
          float acc = 0.f;
#pragma unroll
          for (int e = 0; e < Elem<T>::kPerVec; ++e) acc = __fmaf_rn(x[e], x[e], acc);
          p[i] = acc;
        }
        const float s = halving_reduce<U, LPR>(p, piece);
        const int t = t0 + my_row;
        if (writer && t < row_end && L2KV_BOUNDS(t >= 0 && t < g.cap(bl), sel.status_word)) {
          out[t] = s;
          if (nout) nout[t] = sqrtf(s);
        }
      }
    }
  }

  if constexpr (SEL) {
    __shared__ SelectSmem sm;
    __shared__ int s_last;
    if constexpr (MODE != kKeysGiven) {
      __threadfence();                                   // this CTA's keys are visible device-wide
      __syncthreads();
      if (tid == 0) {
        const int n_ctas = (len + kNormRowsPerCta - 1) / kNormRowsPerCta;
        s_last = atomicAdd(sel.tickets + unit, 1) == n_ctas - 1;
      }
      __syncthreads();
      if (!s_last) return;
      __threadfence();                                   // see the other CTAs' keys
    }
    const int keep_arg = sel.keep_unit_dev ? sel.keep_unit_dev[unit] : sel.keep_dev[b];
    const int keep_req = max(0, min(keep_arg, len));
    const int keep = min(keep_req, out_cap);             // rows that fit the output; the rest is cut
    if (tid == 0) publish_kept_len(sel, unit, b * g.L + l, h, keep);
    if (keep_req == len) {
      identity_unit<kNormThreads>(len, keep, MODE == kKeysRandom, sel.unit_rec + unit,
                                  sel.chunk_rec + unit * sel.n_chunks);
    } else if (keep == 0) {
      if (tid == 0) {
        UnitRec r; r.thr = 0u; r.admit = 0; r.n_keep = 0; r.flags = 0u;
        sel.unit_rec[unit] = r;
      }
    } else {
      select_unit<kNormThreads>(sm, out, len, keep, sel.policy,
                                MODE == kKeysRandom ? kFlagNoKeys : 0u, sel.unit_rec + unit,
                                sel.chunk_rec + unit * sel.n_chunks);
    }
    if (MODE != kKeysGiven && tid == 0) sel.tickets[unit] = 0;   // tickets rest at zero between calls
  }
}

template <typename T, int D>
static int launch_norms_t(const void* K, const Geom& g, const int32_t* len_dev, int max_len,
                          float* sumsq, long long ld, float* norm_out, int key_mode,
                          const SelectArgs* select, const CopyArgs* copy, cudaStream_t s) {
  const long long units = (long long)g.B * g.L * g.H;
  int chunks = (max_len + kNormRowsPerCta - 1) / kNormRowsPerCta;
  if (key_mode != kKeysOnly && chunks < 1) chunks = 1;   // records are written even for max_len 0
  if (key_mode == kKeysGiven) chunks = 1;                // one CTA per unit: selection only
  if (units == 0 || chunks == 0) return L2KV_OK;
  CopyArgs cp = copy ? *copy : CopyArgs{};
  if (key_mode != kKeysFromK) cp.n_blocks = 0;
  const long long blocks = units * chunks + cp.n_blocks;
  if (blocks > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  const T* Kt = static_cast<const T*>(K);
  const SelectArgs sa = select ? *select : SelectArgs{};
  const unsigned nb = (unsigned)blocks;
  switch (key_mode) {
    case kKeysOnly:
      key_norms_kernel<T, D, kKeysOnly><<<nb, kNormThreads, 0, s>>>(Kt, g, len_dev, sumsq, ld, norm_out, chunks, max_len, sa, cp);
      break;
    case kKeysFromK:
      key_norms_kernel<T, D, kKeysFromK><<<nb, kNormThreads, 0, s>>>(Kt, g, len_dev, sumsq, ld, norm_out, chunks, max_len, sa, cp);
      break;
    case kKeysRandom:
      key_norms_kernel<T, D, kKeysRandom><<<nb, kNormThreads, 0, s>>>(Kt, g, len_dev, sumsq, ld, norm_out, chunks, max_len, sa, cp);
      break;
    case kKeysGiven:
      key_norms_kernel<T, D, kKeysGiven><<<nb, kNormThreads, 0, s>>>(Kt, g, len_dev, sumsq, ld, norm_out, chunks, max_len, sa, cp);
      break;
    default:
      return L2KV_ERR_INVALID_ARG;
  }
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

int launch_key_norms(const void* K, const Geom& g, int dtype, const int32_t* len_dev, int max_len,
                     float* sumsq, long long ld_sumsq, float* norm_out, int key_mode,
                     const SelectArgs* select, const CopyArgs* copy, cudaStream_t s) {
#define L2KV_KN(T, D) \
  return launch_norms_t<T, D>(K, g, len_dev, max_len, sumsq, ld_sumsq, norm_out, key_mode, select, copy, s)
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

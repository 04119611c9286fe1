// Budget-maintained cache: append one token per (b, l, h); once a sequence holds `budget`
// tokens, discard the entry that comes last in the order (key, position).
//
// One CTA per (b, l, h).  Per unit: the new key's ordering key (same fixed summation order
// as the norm pass), a block-wide arg-max over the stored keys packed as
// (key bits << 32 | position), then two 16-byte-piece row copies.  The length cur_len[b, l]
// is shared by the KV heads of a layer: every CTA reads it first and takes a ticket of its
// (b, l) when done; the CTA that takes the last ticket -- by then all heads have read the
// old value -- stores the new length and resets the ticket.  Nobody waits.
#include "common.cuh"

namespace l2kv {

// Small blocks: a unit's work is a chain of dependent round trips (lengths, keys, reduction,
// rows, ticket), and what hides them is the number of units in flight per SM.  Measured on 16384
// units of 1k-8k entries: 256 threads x 4 loads 287 us, 128 x 2 133 us, 64 x 2 125 us; on 1024
// units of 16384 entries 45 / 39 / 47 us.
constexpr int kAppendThreads = 128;
constexpr int kAppendUnroll = 2;

template <typename T, int D>
__global__ void __launch_bounds__(kAppendThreads)
append_evict_kernel(T* __restrict__ K, T* __restrict__ V, int32_t* __restrict__ idx,
                    float* __restrict__ sumsq, Geom g, int32_t* __restrict__ cur_len_dev,
                    const int32_t* __restrict__ budget_dev, LayerMask unc,
                    const T* __restrict__ k_new, const T* __restrict__ v_new,
                    const int32_t* __restrict__ pos_new_dev, int32_t* __restrict__ status_word,
                    int32_t* __restrict__ tickets, int per_head) {
  constexpr int EPV = Elem<T>::kPerVec;
  constexpr int LPR = D / EPV;
  constexpr int NW = kAppendThreads / 32;
  __shared__ unsigned long long s_best[NW];
  __shared__ int s_slot;

  const long long unit = blockIdx.x;                     // (b * L + l) * H + h
  const int h = (int)(unit % g.H);
  const long long bl = unit / g.H;
  const int l = (int)(bl % g.L);
  const int b = (int)(bl / g.L);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // per_head: a length and a budget of its own for every (b, l, h)
  const int cap = g.cap(bl);
  const long long meta0 = g.meta(unit);
  const int n = max(0, min(cur_len_dev[per_head ? unit : bl], cap));
  const bool grow = unc.test(l) || n < budget_dev[per_head ? unit : (long long)b];
  const bool overflow = grow && n >= cap;
  const int pos_new = pos_new_dev[b];

  if (!overflow) {
    // Warp 0 holds the new rows: lanes < LPR own one 16-byte piece each.
    uint4 vk = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
    float s_new = 0.f;
    if (warp == 0) {
      if (lane < LPR) {
        vk = *reinterpret_cast<const uint4*>(k_new + unit * D + lane * EPV);
        vv = *reinterpret_cast<const uint4*>(v_new + unit * D + lane * EPV);
      }
      s_new = piece_sumsq_reduce<T, LPR>(vk);            // lanes < LPR end with the row's key
      s_new = __shfl_sync(0xffffffffu, s_new, 0);
    }
    int slot = n;
    if (!grow) {
      const float* key = sumsq + meta0;
      const int32_t* pos = idx + meta0;
      unsigned long long best = 0ull;
      int best_j = -1;
      auto consider = [&](uint32_t kb, uint32_t pb, int j) {
        const unsigned long long c = ((unsigned long long)kb << 32) | pb;
        if (best_j < 0 || c > best) { best = c; best_j = j; }
      };
      int j_done = 0;
      if (((reinterpret_cast<uintptr_t>(key) | reinterpret_cast<uintptr_t>(pos)) & 15u) == 0) {
        // 16-byte loads of four (key, position) pairs, kAppendUnroll of them in flight per thread
        const int n4 = n >> 2;
        const uint4* key4 = reinterpret_cast<const uint4*>(key);
        const uint4* pos4 = reinterpret_cast<const uint4*>(pos);
        for (int i0 = 0; i0 < n4; i0 += kAppendThreads * kAppendUnroll) {
          uint4 kv[kAppendUnroll], pv[kAppendUnroll];
#pragma unroll
          for (int u = 0; u < kAppendUnroll; ++u) {
            const int i = i0 + u * kAppendThreads + tid;
            kv[u] = i < n4 ? key4[i] : make_uint4(0, 0, 0, 0);
            pv[u] = i < n4 ? pos4[i] : make_uint4(0, 0, 0, 0);
          }
#pragma unroll
          for (int u = 0; u < kAppendUnroll; ++u) {
            const int i = i0 + u * kAppendThreads + tid;
            if (i < n4) {
              consider(kv[u].x, pv[u].x, 4 * i); consider(kv[u].y, pv[u].y, 4 * i + 1);
              consider(kv[u].z, pv[u].z, 4 * i + 2); consider(kv[u].w, pv[u].w, 4 * i + 3);
            }
          }
        }
        j_done = n4 << 2;
      }
      for (int j0 = j_done; j0 < n; j0 += kAppendThreads * kAppendUnroll) {
        uint32_t kb[kAppendUnroll], pb[kAppendUnroll];
#pragma unroll
        for (int u = 0; u < kAppendUnroll; ++u) {
          const int j = j0 + u * kAppendThreads + tid;
          kb[u] = j < n ? __float_as_uint(key[j]) : 0u;
          pb[u] = j < n ? (uint32_t)pos[j] : 0u;
        }
#pragma unroll
        for (int u = 0; u < kAppendUnroll; ++u) {
          const int j = j0 + u * kAppendThreads + tid;
          if (j < n) consider(kb[u], pb[u], j);
        }
      }
      unsigned long long wbest = best;
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, wbest, off);
        wbest = o > wbest ? o : wbest;
      }
      if (lane == 0) s_best[warp] = wbest;
      if (tid == 0) s_slot = -1;
      __syncthreads();
      unsigned long long top = s_best[0];
#pragma unroll
      for (int w = 1; w < NW; ++w) top = s_best[w] > top ? s_best[w] : top;
      // (key, position) pairs are distinct, so at most one thread owns the maximum.
      if (best_j >= 0 && best == top) s_slot = best_j;
      __syncthreads();
      slot = s_slot;
      if (warp == 0) {
        const unsigned long long c_new =
            ((unsigned long long)__float_as_uint(s_new) << 32) | (uint32_t)pos_new;
        if (slot < 0 || c_new > top) slot = -1;          // the newcomer is the one discarded
      }
    }
    if (warp == 0 && slot >= 0 && lane < LPR && L2KV_BOUNDS(slot < cap && slot <= n, status_word)) {
      const long long row = g.base(b, l, h) + (long long)slot * g.st + lane * EPV;
      *reinterpret_cast<uint4*>(K + row) = vk;
      *reinterpret_cast<uint4*>(V + row) = vv;
      if (lane == 0) {
        idx[meta0 + slot] = pos_new;
        sumsq[meta0 + slot] = s_new;
      }
    }
  }

  // Ticket of (b, l): the last of the layer's heads to finish publishes the new length.  With
  // a length per head every CTA publishes its own.
  __syncthreads();
  if (tid == 0 && per_head) {
    if (overflow) atomicExch(status_word, (int)L2KV_ERR_DEVICE_OVERFLOW);
    else if (grow) cur_len_dev[unit] = n + 1;
  } else if (tid == 0) {
    __threadfence();
    if (atomicAdd(tickets + bl, 1) == g.H - 1) {
      if (overflow) atomicExch(status_word, (int)L2KV_ERR_DEVICE_OVERFLOW);
      else if (grow) cur_len_dev[bl] = n + 1;
      tickets[bl] = 0;
    }
  }
}

template <typename T, int D>
static int launch_ae_t(void* K, void* V, int32_t* idx, float* sumsq, const Geom& g,
                       int32_t* cur_len_dev, const int32_t* budget_dev, const LayerMask& unc,
                       const void* k_new, const void* v_new, const int32_t* pos_new_dev,
                       int32_t* status_word, int32_t* tickets, int per_head, cudaStream_t s) {
  const long long blocks = (long long)g.B * g.L * g.H;
  if (blocks == 0) return L2KV_OK;
  if (blocks > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  append_evict_kernel<T, D><<<(unsigned)blocks, kAppendThreads, 0, s>>>(
      static_cast<T*>(K), static_cast<T*>(V), idx, sumsq, g, cur_len_dev, budget_dev, unc,
      static_cast<const T*>(k_new), static_cast<const T*>(v_new), pos_new_dev, status_word,
      tickets, per_head);
  return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
}

int launch_append_evict(void* K, void* V, int32_t* idx, float* sumsq, const Geom& g, int dtype,
                        int32_t* cur_len_dev, const int32_t* budget_dev, const LayerMask& unc,
                        const void* k_new, const void* v_new, const int32_t* pos_new_dev,
                        int32_t* status_word, int32_t* tickets, int per_head, cudaStream_t s) {
#define L2KV_AE(T, D)                                                                            \
  return launch_ae_t<T, D>(K, V, idx, sumsq, g, cur_len_dev, budget_dev, unc, k_new, v_new,      \
                           pos_new_dev, status_word, tickets, per_head, s)
  if (dtype == L2KV_BF16) {
    if (g.D == 128) L2KV_AE(__nv_bfloat16, 128);
    if (g.D == 64) L2KV_AE(__nv_bfloat16, 64);
  } else if (dtype == L2KV_F32) {
    if (g.D == 128) L2KV_AE(float, 128);
    if (g.D == 64) L2KV_AE(float, 64);
  }
#undef L2KV_AE
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

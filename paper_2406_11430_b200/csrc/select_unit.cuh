// Exact k-selection for one (b, l, h) unit, run by one CTA of NT threads.
//
// Finds the keep-th smallest ordering key by a most-significant-digit radix select (4
// passes of 8 bits) over the unit's key array in global memory (L2-resident: it was
// written moments before), then counts, per gather chunk, the keys below and equal to the
// threshold and scans those counts into slot bases.  No waiting on other CTAs anywhere.
#pragma once

#include "common.cuh"

namespace l2kv {

constexpr int kCandCap = 2 * kMaxChunks;        // candidate keys that fit the shared list

struct SelectSmem {
  int hist[256];
  int bucket, before, in_bucket, n_cand;
  union {
    struct { int c_less[kMaxChunks]; int c_eq[kMaxChunks]; };   // after the passes
    uint32_t cand[kCandCap];                                    // during the passes
  };
};

// Keys may have been written by other CTAs of the same grid: read them through L2.
__device__ __forceinline__ uint32_t load_key_bits(const float* p, int policy) {
  return order_bits(__ldcg(p), policy);
}

template <int NT>
__device__ void select_unit(SelectSmem& sm, const float* __restrict__ key, int len, int keep,
                            int policy, uint32_t flags, UnitRec* __restrict__ rec,
                            int2* __restrict__ crec) {
  constexpr int kBatch = 8;                      // independent key loads in flight per thread
  const bool vec = (reinterpret_cast<uintptr_t>(key) & 15u) == 0;   // caller-provided keys may not be
  const int tid = threadIdx.x;
  const int my_chunks = (len + kGatherChunk - 1) / kGatherChunk;
  uint32_t prefix = 0, mask = 0;
  int k_rem = keep;
  // Passes scan every key until the keys that still match the prefix fit the shared list;
  // the next pass then also collects them, and the passes after that only look at the list.
  bool collect = false, listed = false;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += NT) sm.hist[i] = 0;
    if (tid == 0 && collect) sm.n_cand = 0;
    __syncthreads();
    // Run-length accumulation: neighbouring tokens mostly share the high digits, so the
    // shared-memory atomics of the first passes collapse to a few per thread.
    int cur = -1, cnt = 0;
    auto tally = [&](uint32_t kb) {
      if ((kb & mask) != prefix) return false;
      const int d = (kb >> shift) & 255;
      if (d == cur) {
        ++cnt;
      } else {
        if (cnt) atomicAdd(&sm.hist[cur], cnt);
        cur = d; cnt = 1;
      }
      return true;
    };
    if (listed) {
      const int n_cand = sm.n_cand;
      for (int i = tid; i < n_cand; i += NT) tally(sm.cand[i]);
    } else {
      auto visit = [&](uint32_t kb) {
        if (tally(kb) && collect) sm.cand[atomicAdd(&sm.n_cand, 1)] = kb;
      };
      if (vec) {
        // 16-byte loads, kBatch of them in flight per thread: the pass is bound by how many
        // bytes one CTA keeps outstanding towards L2.
        const int n4 = len >> 2;
        const float4* key4 = reinterpret_cast<const float4*>(key);
        for (int base = 0; base < n4; base += NT * kBatch) {
          float4 v[kBatch];
#pragma unroll
          for (int j = 0; j < kBatch; ++j) {
            const int i = base + j * NT + tid;
            v[j] = i < n4 ? __ldcg(key4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int j = 0; j < kBatch; ++j) {
            if (base + j * NT + tid < n4) {
              visit(order_bits(v[j].x, policy)); visit(order_bits(v[j].y, policy));
              visit(order_bits(v[j].z, policy)); visit(order_bits(v[j].w, policy));
            }
          }
        }
        if (tid < (len & 3)) visit(load_key_bits(key + (n4 << 2) + tid, policy));
      } else {
        for (int base = 0; base < len; base += NT * kBatch) {
          uint32_t kb[kBatch];
#pragma unroll
          for (int j = 0; j < kBatch; ++j) {
            const int t = base + j * NT + tid;
            kb[j] = t < len ? load_key_bits(key + t, policy) : 0u;
          }
#pragma unroll
          for (int j = 0; j < kBatch; ++j)
            if (base + j * NT + tid < len) visit(kb[j]);
        }
      }
    }
    if (cnt) atomicAdd(&sm.hist[cur], cnt);
    __syncthreads();
    if (tid < 32) {
      // 8 bins per lane: lane totals -> warp scan -> locate the bin holding rank k_rem.
      int v[8], tot = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { v[i] = sm.hist[tid * 8 + i]; tot += v[i]; }
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
          if (before < k_rem && k_rem <= before + v[i]) {
            sm.bucket = tid * 8 + i; sm.before = before; sm.in_bucket = v[i];
          }
          before += v[i];
        }
      }
    }
    __syncthreads();
    prefix |= (uint32_t)sm.bucket << shift;
    mask |= 255u << shift;
    k_rem -= sm.before;
    if (collect) { listed = true; collect = false; }
    else if (!listed && sm.in_bucket <= kCandCap) collect = true;
    __syncthreads();
  }
  const uint32_t thr = prefix;      // the keep-th smallest key; k_rem of its copies are admitted
  if (tid == 0) {
    UnitRec r; r.thr = thr; r.admit = k_rem; r.n_keep = keep; r.flags = flags;
    *rec = r;
  }
  // Per-chunk counts of keys below / equal to the threshold, one warp per chunk (the
  // candidate list is dead by now: its storage becomes the count arrays).
  const int warp = tid >> 5, lane = tid & 31;
  for (int c = warp; c < my_chunks; c += NT / 32) {
    const int t0 = c * kGatherChunk;
    const int t1 = min(len, t0 + kGatherChunk);
    int nl = 0, ne = 0;
    auto count = [&](uint32_t kb) { nl += kb < thr; ne += kb == thr; };
    if (vec && t1 == t0 + kGatherChunk) {
      const float4* key4 = reinterpret_cast<const float4*>(key + t0);
      float4 v[kGatherChunk / 128];
#pragma unroll
      for (int j = 0; j < kGatherChunk / 128; ++j) v[j] = __ldcg(key4 + j * 32 + lane);
#pragma unroll
      for (int j = 0; j < kGatherChunk / 128; ++j) {
        count(order_bits(v[j].x, policy)); count(order_bits(v[j].y, policy));
        count(order_bits(v[j].z, policy)); count(order_bits(v[j].w, policy));
      }
    } else {
#pragma unroll 4
      for (int t = t0 + lane; t < t1; t += 32) count(load_key_bits(key + t, policy));
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
      nl += __shfl_xor_sync(0xffffffffu, nl, off);
      ne += __shfl_xor_sync(0xffffffffu, ne, off);
    }
    if (lane == 0) { sm.c_less[c] = nl; sm.c_eq[c] = ne; }
  }
  __syncthreads();
  if (tid == 0) {
    int slot = 0, eq_before = 0;
    for (int c = 0; c < my_chunks; ++c) {
      crec[c] = make_int2(slot, eq_before);
      const int adm = max(0, min(sm.c_eq[c], k_rem - eq_before));
      slot += sm.c_less[c] + adm;
      eq_before += sm.c_eq[c];
    }
  }
}

// Record of a unit whose valid tokens are all kept (uncompressed layer, or keep == len).
template <int NT>
__device__ void identity_unit(int len, int keep, bool keys_missing, UnitRec* __restrict__ rec,
                              int2* __restrict__ crec, bool copied = false) {
  const int my_chunks = (len + kGatherChunk - 1) / kGatherChunk;
  if (threadIdx.x == 0) {
    UnitRec r; r.thr = 0xffffffffu; r.admit = 0; r.n_keep = keep;
    r.flags = kFlagIdentity | (keys_missing ? kFlagNoKeys : 0u) | (copied ? kFlagCopied : 0u);
    *rec = r;
  }
  for (int c = threadIdx.x; c < my_chunks; c += NT) crec[c] = make_int2(c * kGatherChunk, 0);
}

}  // namespace l2kv

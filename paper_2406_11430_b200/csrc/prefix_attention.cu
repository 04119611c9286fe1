// Prefix attention: a block of new queries (a prefill chunk, or several draft tokens) attends
// to the whole compressed cache.  Unlike single-query decode this is a dense contraction --
// 4 * Sq * Hq * D flop per cached token per (b, l) -- so it runs on the Blackwell tensor cores
// (tcgen05.mma, operands in shared memory, accumulators in tensor memory).
//
// A query tile is 128 rows: the (query, head-of-the-group) pairs of 128 / G queries that share
// one KV head.  For every block of cached tokens
//   K block  -- TMA --> shared memory (128-byte swizzle)
//   S = Q . K^T             tcgen05.mma (M 128, K 16 per instruction), fp32 in tensor memory
//   softmax threads read their rows of S (tcgen05.ld): running maximum, weights 2^(s - m) as
//   bf16 pairs written back over the score columns (tcgen05.st), running sum
//   V block  -- TMA --> shared memory;  O += P . V   tcgen05.mma with A in tensor memory and V as
//   an N-major operand; O stays in tensor memory and is rescaled only when a maximum has drifted.
// Two kernels share these pieces: the pipelined one (default) and a basic single-role one.
// Every wait on an mbarrier is bounded (a wait that gives up ends the CTA's loop and marks
// the status word); tensor memory is released on every path.
#include <climits>
#include <cmath>
#include <cstdlib>
#include <cstring>

#include "async_copy.cuh"

namespace l2kv {

constexpr int kPfThreads = 256;                // basic kernel: two threads per query row
constexpr int kPfRows = 128;                    // query rows per CTA, cached tokens per block
constexpr int kPfHalf = kPfRows * 128;          // one [128 rows][64 bf16] swizzled tile: 16 KB
constexpr int kPfTileBytes = 2 * kPfHalf;       // both halves of the head dimension: 32 KB
constexpr int kPfTmemCols = 256;                // basic kernel: S in columns 0..127, O in 128..255
constexpr int kPfPolls = 18;                    // log2 of the polls a wait may take
constexpr float kPfLog2e = 1.4426950408889634f;

// Instruction descriptor of tcgen05.mma kind::f16: fp32 accumulate (bits 4-5 = 1), bf16 A and B
// (bits 7-9 and 10-12 = 1), A/B major-ness (bits 15, 16; 0 = K-major), N / 8 (bits 17-22),
// M / 16 (bits 24-28).
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescQK | (1u << 16);       // V is N-major (head_dim contiguous)

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all / 16),
// descriptor version 1 (bit 46), 128-byte swizzle (layout type 2 in bits 61-63).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
               :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
               : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               :: "r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's tensor-memory lane.  Whole warps only.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                 "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]),
                 "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
                 "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                 "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
                 "=r"(r[31])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// 64 consecutive fp32 columns of this thread's tensor-memory lane: both loads are issued before
// the one wait, so their latencies overlap.  Whole warps only.
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t (&a)[32], uint32_t (&b)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%64];\n\t"
               "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
               "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%65];\n\t"
               "tcgen05.wait::ld.sync.aligned;"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]),
                 "=r"(a[6]), "=r"(a[7]), "=r"(a[8]), "=r"(a[9]), "=r"(a[10]), "=r"(a[11]),
                 "=r"(a[12]), "=r"(a[13]), "=r"(a[14]), "=r"(a[15]), "=r"(a[16]), "=r"(a[17]),
                 "=r"(a[18]), "=r"(a[19]), "=r"(a[20]), "=r"(a[21]), "=r"(a[22]), "=r"(a[23]),
                 "=r"(a[24]), "=r"(a[25]), "=r"(a[26]), "=r"(a[27]), "=r"(a[28]), "=r"(a[29]),
                 "=r"(a[30]), "=r"(a[31]),
                 "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]), "=r"(b[4]), "=r"(b[5]),
                 "=r"(b[6]), "=r"(b[7]), "=r"(b[8]), "=r"(b[9]), "=r"(b[10]), "=r"(b[11]),
                 "=r"(b[12]), "=r"(b[13]), "=r"(b[14]), "=r"(b[15]), "=r"(b[16]), "=r"(b[17]),
                 "=r"(b[18]), "=r"(b[19]), "=r"(b[20]), "=r"(b[21]), "=r"(b[22]), "=r"(b[23]),
                 "=r"(b[24]), "=r"(b[25]), "=r"(b[26]), "=r"(b[27]), "=r"(b[28]), "=r"(b[29]),
                 "=r"(b[30]), "=r"(b[31])
               : "r"(taddr), "r"(taddr + 32)
               : "memory");
}
// A operand taken from tensor memory (bf16 pairs packed two per 32-bit column, row = lane).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc,
                                             uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
               :: "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
               : "memory");
}
// Stores 32 consecutive 32-bit columns of this thread's tensor-memory lane.  Whole warps only.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
               "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
               "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
               :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),
                  "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]),
                  "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
                  "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
                  "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
               : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void st_shared16(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" :: "r"(addr), "r"(a), "r"(b), "r"(c), "r"(d)
               : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// The part of a weight pair that its bf16 rounding `packed` left out, again as a bf16 pair:
// hi + lo carries 16 significant bits of each weight.
__device__ __forceinline__ uint32_t pack_bf16_rest(float lo, float hi, uint32_t packed) {
  return pack_bf16(lo - __uint_as_float(packed << 16), hi - __uint_as_float(packed & 0xffff0000u));
}

// 2^x by the hardware approximation (one MUFU instruction; x <= 0 here, -inf gives 0).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Eight columns at a time: the rarely taken rescaling of O, kept small in registers.
__device__ __forceinline__ void tmem_scale8(uint32_t taddr, float factor) {
  uint32_t r0, r1, r2, r3, r4, r5, r6, r7;
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3), "=r"(r4), "=r"(r5), "=r"(r6), "=r"(r7)
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  r0 = __float_as_uint(__uint_as_float(r0) * factor); r1 = __float_as_uint(__uint_as_float(r1) * factor);
  r2 = __float_as_uint(__uint_as_float(r2) * factor); r3 = __float_as_uint(__uint_as_float(r3) * factor);
  r4 = __float_as_uint(__uint_as_float(r4) * factor); r5 = __float_as_uint(__uint_as_float(r5) * factor);
  r6 = __float_as_uint(__uint_as_float(r6) * factor); r7 = __float_as_uint(__uint_as_float(r7) * factor);
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               :: "r"(taddr), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(r4), "r"(r5), "r"(r6), "r"(r7)
               : "memory");
}

// Query rows of one tile into shared memory (K-major, 128-byte swizzle), by one warp: rows
// row0 .. row0 + 31 of the tile, pieces [16 first, 16 first + 16 count) of the 32 instruction
// slots (slot i: rows row0 + 2i and row0 + 2i + 1).  Lanes 0-15 and 16-31 each read one whole
// 256-byte row per instruction, so a request touches 4 lines instead of 32.  Row r of tile
// number `tile_no` of the unit is query tile_no * (128 / G) + r / G, head h * G + r % G.
template <int G>
__device__ __forceinline__ void load_query_rows(const __nv_bfloat16* __restrict__ q, long long bl,
                                                int n_queries, int Hq, int h, int tile_no, int row0,
                                                uint32_t sQ, int first, int count) {
  constexpr int QT = kPfRows / G;
  const int lane = threadIdx.x & 31, c = lane & 15;
#pragma unroll 8
  for (int i = first; i < first + count; ++i) {
    const int r = row0 + 2 * i + (lane >> 4);
    const int s_idx = tile_no * QT + r / G;
    const long long off = ((bl * n_queries + s_idx) * Hq + h * G + r % G) * 128 + c * 8;
    const uint4 v = s_idx < n_queries ? *reinterpret_cast<const uint4*>(q + off) : make_uint4(0, 0, 0, 0);
    st_shared16(sQ + (c >> 3) * kPfHalf + r * 128 + (((c & 7) ^ (r & 7)) << 4), v.x, v.y, v.z, v.w);
  }
}

// The basic kernel (L2KV_PREFIX_KERNEL=basic): one role, two CTAs per SM that fill each other's
// gaps.  The weights never go to shared memory: they are written as bf16 pairs into the
// tensor-memory columns that held the scores and feed the second contraction from there
// (tcgen05.mma with A in tensor memory); the output accumulates in tensor memory across
// blocks and is rescaled only when a row's maximum has grown by more than 2^8 since the last
// rescale (weights stay <= 2^8, well inside bf16 / fp32 range); K and V each have their own
// shared-memory tile, so the next K block is fetched while the softmax and the second
// contraction of the current one run.
constexpr float kPfRescaleGap = 8.f;            // log2 units a maximum may drift before O is rescaled

template <int G, bool SW>
__global__ void __launch_bounds__(kPfThreads, 2)
prefix_attention_basic_kernel(const __nv_bfloat16* __restrict__ q, Geom g, int n_queries,
                           LenView cur_len_dev, int max_len, float scale_log2e,
                           float* __restrict__ out, float* __restrict__ lse_out,
                           const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_v,
                           int32_t* __restrict__ status_word, int split_len, long long rows_total,
                           int causal) {
  constexpr int D = 128;
  constexpr int QT = kPfRows / G;                       // queries per CTA
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long s_bar[4];  // K landed, V landed, QK done, PV done
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;
  __shared__ float s_x[2][kPfRows];                     // row maxima / sums of the two column halves

  const int q_tiles = (n_queries + QT - 1) / QT;
  const int qt = blockIdx.x % q_tiles;
  const long long unit = blockIdx.x / q_tiles;          // (b * L + l) * H + h
  const int h = (int)(unit % g.H);
  const long long bl = unit / g.H;
  const int l = (int)(bl % g.L), b = (int)(bl / g.L);
  const int n_all = max(0, min(cur_len_dev.at(bl, h, g.H), min(max_len, g.cap(bl))));
  // blockIdx.y: the chunk of split_len cached tokens this CTA covers (one chunk = the whole cache
  // unless the launcher split it; then out / lse_out are the per-chunk partial results)
  const int t_base = (int)blockIdx.y * split_len;
  // tensor-map coordinates: (token, head, layer, batch) of a dense cache; a packed cache is one
  // [H, total_rows] plane, so the first row of (b, l) joins the token coordinate
  const int tm_row = (int)g.row0(bl) + t_base;
  const int tm_l = g.row_off ? 0 : l, tm_b = g.row_off ? 0 : b;
  const int n = gridDim.y > 1 ? min(n_all, t_base + split_len) - t_base : n_all;
  if (gridDim.y > 1) {
    if (n <= 0) return;                                 // nothing cached in this chunk
    out += (long long)blockIdx.y * rows_total * 128;
    lse_out += (long long)blockIdx.y * rows_total;
  }
  // Two threads per query row: thread (row, hf) owns score columns and output dims
  // [64 hf, 64 hf + 64).  Warps w and w + 4 share a tensor-memory lane quarter.
  const int tid = threadIdx.x, warp = tid >> 5;
  const int row = tid & (kPfRows - 1), hf = tid >> 7;
  const int s_idx = qt * QT + row / G;                  // this row's query and head
  const int head = h * G + row % G;
  const bool row_valid = s_idx < n_queries;
  const long long row_off = ((bl * n_queries + s_idx) * g.Hq + head);
  // causal: the last n_queries cached rows are the new tokens' own; query s stops at its own
  const int n_row = causal && row_valid ? min(n, max(0, n_all - n_queries + s_idx + 1) - t_base) : n;
  if (n == 0) {                                         // empty cache: zeros, log-sum-exp = -inf
    if (row_valid) {
      for (int d = 0; d < 64; ++d) out[row_off * D + hf * 64 + d] = 0.f;
      if (lse_out && hf == 0) lse_out[row_off] = -INFINITY;
    }
    return;
  }
  // A wait that gave up in an earlier CTA marks the workspace; the rest of the grid leaves.
  if (status_word && *reinterpret_cast<volatile int32_t*>(status_word + 2) != 0) return;
  const int n_blocks = (n + kPfRows - 1) / kPfRows;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 1024-byte aligned tiles
  const uint32_t sQ = base, sK = base + kPfTileBytes, sV = base + 2 * kPfTileBytes;
  const uint32_t bar_k = smem_u32(&s_bar[0]), bar_v = smem_u32(&s_bar[1]);
  const uint32_t bar_s = smem_u32(&s_bar[2]), bar_o = smem_u32(&s_bar[3]);

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 :: "r"(smem_u32(&s_tmem)), "r"(kPfTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    mbar_init(bar_k, 1); mbar_init(bar_v, 1); mbar_init(bar_s, 1); mbar_init(bar_o, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_fail = 0;
  }
  __syncwarp();
  // Q rows: warps w and w + 4 share rows 32 (w & 3) .. + 31 and load half of them each
  load_query_rows<G>(q, bl, n_queries, g.Hq, h, qt, (warp & 3) * 32, sQ, hf * 8, 8);
  proxy_fence();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);   // this warp's lane quarter
  const uint32_t t_s = t_lane + hf * 64;                // scores of this thread's 64 tokens
  const uint32_t t_p = t_lane + hf * 32;                // their weights, two per column
  const uint32_t t_o = t_lane + 128 + hf * 64;          // this thread's 64 output dims

  auto load_k = [&](int kb) {                           // thread 0 only
    mbar_expect_tx(bar_k, kPfTileBytes);
    tma_load_5d(sK, &map_k, bar_k, 0, tm_row + kb * kPfRows, h, tm_l, tm_b);
    tma_load_5d(sK + kPfHalf, &map_k, bar_k, 64, tm_row + kb * kPfRows, h, tm_l, tm_b);
  };
  auto load_v = [&](int kb) {
    mbar_expect_tx(bar_v, kPfTileBytes);
    tma_load_5d(sV, &map_v, bar_v, 0, tm_row + kb * kPfRows, h, tm_l, tm_b);
    tma_load_5d(sV + kPfHalf, &map_v, bar_v, 64, tm_row + kb * kPfRows, h, tm_l, tm_b);
  };
  if (tid == 0) { load_k(0); load_v(0); }
  __syncwarp();

  float m_ref = -INFINITY, l_run = 0.f;                 // reference maximum; sum of this half's weights

  for (int kb = 0; kb < n_blocks; ++kb) {
    const int valid_all = min(kPfRows, n - kb * kPfRows);   // valid tokens of this block
    const int valid = min(valid_all, n_row - kb * kPfRows) - hf * 64;   // ... among this thread's 64
    // ---- S = Q K^T; fetch V for this block and K for the next as their tiles come free ---
    if (tid == 0) {
      if (!mbar_wait<kPfPolls>(bar_k, kb & 1)) s_fail = 1;
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint32_t off = (k >> 2) * kPfHalf + (k & 3) * 32;
        umma_bf16(tmem, umma_desc(sQ + off, 16, 1024), umma_desc(sK + off, 16, 1024), kIdescQK, k > 0);
      }
      umma_commit(bar_s);
      if (kb > 0) {                                      // P.V of the previous block is done:
        if (!mbar_wait<kPfPolls>(bar_o, (kb - 1) & 1)) s_fail = 1;   // O is quiet, the V tile is free
        else load_v(kb);
      }
      if (!mbar_wait<kPfPolls>(bar_s, kb & 1)) s_fail = 1;
      else if (kb + 1 < n_blocks) load_k(kb + 1);        // the K tile is free again
    }
    __syncthreads();                                     // S is complete (thread 0 saw the commit)
    if (s_fail) break;
    tc_fence_after();
    // ---- this thread's 64 scores (log2 domain), kept in registers ---------------------------
    // (raw products; the scale is folded into the exponent's multiply-add below)
    float sv[64];
    float bmax = -INFINITY;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      uint32_t r[32];
      tmem_ld32(t_s + c * 32, r);
      if (valid >= 64) {                                 // only the last (or a causal row's own) block masks
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          sv[c * 32 + i] = __uint_as_float(r[i]);
          bmax = fmaxf(bmax, sv[c * 32 + i]);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          sv[c * 32 + i] = c * 32 + i < valid ? __uint_as_float(r[i]) : -INFINITY;
          bmax = fmaxf(bmax, sv[c * 32 + i]);
        }
      }
    }
    s_x[hf][row] = bmax * scale_log2e;                   // scale > 0: the maximum commutes with it
    tc_fence_before();
    __syncthreads();                                     // maxima exchanged; every score has been read
    tc_fence_after();
    const float m_new = fmaxf(m_ref, fmaxf(s_x[0][row], s_x[1][row]));
    if (kb == 0) m_ref = m_new;
    // ---- rescale O only when this row's maximum has drifted far from the reference ----------
    const bool need = m_new > m_ref + kPfRescaleGap;
    if (__any_sync(0xffffffffu, need)) {
      const float factor = need ? fast_exp2(m_ref - m_new) : 1.f;
#pragma unroll 1
      for (int c = 0; c < 64; c += 8) tmem_scale8(t_o + c, factor);
      tmem_wait_st();
      if (need) { l_run *= factor; m_ref = m_new; }
    }
    // ---- weights 2^(s - m_ref) as bf16 pairs over the score columns -------------------------
    {
      uint32_t pk[32];
      [[maybe_unused]] uint32_t pr[SW ? 32 : 1];
      float rowsum0 = 0.f, rowsum1 = 0.f;
      const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;   // a row with nothing to see yet
#pragma unroll
      for (int i = 0; i < 64; i += 2) {
        const float p0 = fast_exp2(__fmaf_rn(sv[i], scale_log2e, neg_m));     // -inf -> 0
        const float p1 = fast_exp2(__fmaf_rn(sv[i + 1], scale_log2e, neg_m));
        rowsum0 += p0;
        rowsum1 += p1;
        pk[i >> 1] = pack_bf16(p0, p1);
        if constexpr (SW) pr[i >> 1] = pack_bf16_rest(p0, p1, pk[i >> 1]);
      }
      tmem_st32(t_p, pk);
      if constexpr (SW) tmem_st32(t_p + 64, pr);          // second terms: columns 64..127
      tmem_wait_st();
      l_run += rowsum0 + rowsum1;
    }
    if (valid_all < kPfRows) {
      // Last, partial block: rows of the V tile past the valid length hold whatever the cache
      // holds there; clear them so that a zero weight times Inf/NaN cannot reach O.
      if (tid == 0 && !mbar_wait<kPfPolls>(bar_v, kb & 1)) s_fail = 1;
      __syncthreads();
      if (row >= valid_all) {
#pragma unroll
        for (int c = 0; c < 8; ++c) st_shared16(sV + hf * kPfHalf + row * 128 + (c << 4), 0, 0, 0, 0);
      }
      proxy_fence();
    }
    tc_fence_before();
    __syncthreads();                                     // all weights are in tensor memory
    // ---- O += P V ----------------------------------------------------------------------------
    if (tid == 0) {
      if (valid_all == kPfRows && !mbar_wait<kPfPolls>(bar_v, kb & 1)) s_fail = 1;
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        umma_bf16_ts(tmem + 128, tmem + k * 8, umma_desc(sV + k * 2048, kPfHalf, 1024), kIdescPV,
                     (kb > 0 || k > 0) ? 1u : 0u);
        if constexpr (SW)
          umma_bf16_ts(tmem + 128, tmem + 64 + k * 8, umma_desc(sV + k * 2048, kPfHalf, 1024), kIdescPV, 1u);
      }
      umma_commit(bar_o);
    }
  }

  if (tid == 0 && !s_fail && !mbar_wait<kPfPolls>(bar_o, (n_blocks - 1) & 1)) s_fail = 1;
  __syncthreads();                                       // O is complete
  tc_fence_after();
  const bool failed = s_fail != 0;
  // the two halves of a row share the reference maximum; their weight sums add up
  s_x[hf][row] = l_run;
  __syncthreads();
  const float l_tot = s_x[0][row] + s_x[1][row];
  if (!failed) {
    const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;   // nothing seen: zeros, log-sum-exp -inf
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      uint32_t r[32];
      tmem_ld32(t_o + c * 32, r);
      if (row_valid) {
        float4* dst = reinterpret_cast<float4*>(out + row_off * D + hf * 64 + c * 32);
#pragma unroll
        for (int i = 0; i < 32; i += 4)
          dst[i >> 2] = make_float4(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv,
                                    __uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
      }
    }
    if (row_valid && lse_out && hf == 0)
      lse_out[row_off] = (m_ref + log2f(l_tot)) * 0.6931471805599453f;
  }
  if (failed && tid == 0) record_timeout(status_word);
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "r"(kPfTmemCols)
                 : "memory");
}

// Epilogue of the kernels with one softmax thread per query row: this warp's 32 rows of O (128
// fp32 each, in tensor memory at t_o, one row per lane) times the lane's `inv`, written to the
// rows at `dst` (the lane's own destination row; nullptr: the row does not exist).  A thread
// that stored its own row would put 16 bytes into each of 32 different 128-byte lines per
// instruction; instead the rows go through 4 KB of shared memory (`stage`, this warp's own), 32
// columns at a time, and leave as 128-byte pieces, four rows per instruction.
constexpr int kPfStageBytes = 4096;
__device__ __forceinline__ void store_rows_via_stage(uint32_t t_o, float inv, float* dst, float4* stage) {
  const int lane = threadIdx.x & 31;
  float* dst_k[8];                                      // destination rows 4k + (lane >> 3)
#pragma unroll
  for (int k = 0; k < 8; ++k)
    dst_k[k] = reinterpret_cast<float*>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(dst),
                                                    4 * k + (lane >> 3)));
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    uint32_t r[32];
    tmem_ld32(t_o + c * 32, r);
#pragma unroll
    for (int i = 0; i < 8; ++i)                         // piece i of row `lane`, swizzled by the row
      stage[lane * 8 + (i ^ (lane & 7))] =
          make_float4(__uint_as_float(r[4 * i]) * inv, __uint_as_float(r[4 * i + 1]) * inv,
                      __uint_as_float(r[4 * i + 2]) * inv, __uint_as_float(r[4 * i + 3]) * inv);
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int rr = 4 * k + (lane >> 3);
      const float4 v = stage[rr * 8 + ((lane & 7) ^ (rr & 7))];
      if (dst_k[k]) reinterpret_cast<float4*>(dst_k[k] + c * 32)[lane & 7] = v;
    }
    __syncwarp();
  }
}

// The pipelined kernel walks the cache in sub-blocks of 64 tokens.
constexpr int kPfSub = 64;                      // cached tokens per sub-block
constexpr int kPfSubHalf = kPfSub * 128;        // one [64 tokens][64 bf16] swizzled tile: 8 KB
constexpr int kPfSubTile = 2 * kPfSubHalf;      // both halves of the head dimension: 16 KB
constexpr uint32_t kIdescQK64 =
    (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr int kPfStages = 4;                    // K tiles (and V tiles) in flight
// 1 (default): Q K(j+2)^T is issued right behind P(j) V(j) although it overwrites the columns that
// P(j) V(j) reads its weights from -- see the issuing thread.  0: wait for P(j) V(j) to be
// committed first (8-12 % slower; the form to fall back to if the assumption is ever in doubt).
#ifndef L2KV_PREFIX_MMA_IN_ORDER
#define L2KV_PREFIX_MMA_IN_ORDER 1
#endif
constexpr int kPfPipeTmemCols = 512;            // two query tiles x (2 x 64 score + 128 output columns)

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile("{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; "
               "selp.u32 %0, 1, 0, p; }" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  return done != 0;
}
// A wait that is usually over already: one non-blocking test first.
__device__ __forceinline__ bool mbar_wait_likely(uint32_t bar, uint32_t parity) {
  return mbar_test(bar, parity) || mbar_wait<kPfPolls>(bar, parity);
}

// The pipelined kernel, the launcher's choice unless the query tiles per KV head are few and
// odd.  The two contractions and the softmax
// run concurrently, each in warps of its own, and one CTA per SM works on two query tiles
// (256 rows) that share every K and V tile:
//   - the cache is walked in sub-blocks of 64 tokens; per query tile two score buffers of 64
//     columns and the 128 output columns live in tensor memory (2 x 256 = all 512 columns), so
//     S(j+1) = Q K(j+1)^T is computed while the softmax works on S(j), and O += P(j) V(j) runs
//     while it works on S(j+1);
//   - one softmax thread per query row (four warps per query tile): a row's maximum and sum
//     are thread-local, the softmax warps never synchronise with one another; they wait for
//     scores and hand over weights (bf16 pairs written over the score columns);
//   - one issuing thread per query tile, one thread that fetches K tiles and one that fetches
//     V tiles by TMA into rings of four tiles each, freed by tcgen05.commit.
// Hand-offs are mbarriers (scores ready / tile free / output quiet: tcgen05.commit; weights
// ready: one arrival per softmax warp); every wait on them is bounded.
constexpr int kPfPipeThreads = 2 * kPfRows + 4 * 32;      // softmax A, softmax B, issuer A, issuer B, K, V

template <int G, bool SW>
__global__ void __launch_bounds__(kPfPipeThreads, 1)
prefix_attention_pipelined_kernel(const __nv_bfloat16* __restrict__ q, Geom g, int n_queries,
                           LenView cur_len_dev, int max_len, float scale_log2e,
                           float* __restrict__ out, float* __restrict__ lse_out,
                           const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_v,
                           int32_t* __restrict__ status_word, int split_len, long long rows_total,
                           int causal) {
  constexpr int D = 128;
  constexpr int QT = kPfRows / G;                       // queries per query tile
  constexpr int NS = kPfStages;
  extern __shared__ unsigned char smem_raw[];
  // mbarriers: K landed [NS], V landed [NS], K tile free [NS], V tile free [NS], then per query
  // tile: scores ready [2], weights ready [2], output quiet [1], output complete [1]
  __shared__ __align__(8) unsigned long long s_bar[4 * NS + 12];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;

  const int q_tiles = (n_queries + QT - 1) / QT;
  const int q_pairs = (q_tiles + 1) / 2;
  const int qp = blockIdx.x % q_pairs;
  const long long unit = blockIdx.x / q_pairs;          // (b * L + l) * H + h
  const int h = (int)(unit % g.H);
  const long long bl = unit / g.H;
  const int l = (int)(bl % g.L), b = (int)(bl / g.L);
  const int n_all = max(0, min(cur_len_dev.at(bl, h, g.H), min(max_len, g.cap(bl))));
  // blockIdx.y: the chunk of split_len cached tokens this CTA covers (one chunk = the whole cache
  // unless the launcher split it; then out / lse_out are the per-chunk partial results)
  const int t_base = (int)blockIdx.y * split_len;
  // tensor-map coordinates: (token, head, layer, batch) of a dense cache; a packed cache is one
  // [H, total_rows] plane, so the first row of (b, l) joins the token coordinate
  const int tm_row = (int)g.row0(bl) + t_base;
  const int tm_l = g.row_off ? 0 : l, tm_b = g.row_off ? 0 : b;
  const int n = gridDim.y > 1 ? min(n_all, t_base + split_len) - t_base : n_all;
  if (gridDim.y > 1) {
    if (n <= 0) return;                                 // nothing cached in this chunk
    out += (long long)blockIdx.y * rows_total * 128;
    lse_out += (long long)blockIdx.y * rows_total;
  }
  const int tid = threadIdx.x, warp = tid >> 5;
  const bool softmax_thread = tid < 2 * kPfRows;
  const int n_tiles = (2 * qp + 1 < q_tiles) ? 2 : 1;   // query tiles of this CTA that exist
  // Softmax threads: one per query row of query tile `tile`.
  const int tile = softmax_thread ? tid >> 7 : warp & 1;
  const int row = tid & (kPfRows - 1);
  const int wq = warp & 3;                              // tensor-memory lane quarter of this warp
  const int s_idx = (2 * qp + tile) * QT + row / G;     // this row's query and head
  const int head = h * G + row % G;
  const bool row_valid = softmax_thread && s_idx < n_queries;
  const long long row_off = ((bl * n_queries + s_idx) * g.Hq + head);
  // causal: the last n_queries cached rows are the new tokens' own; query s stops at its own
  const int n_row = causal && row_valid ? min(n, max(0, n_all - n_queries + s_idx + 1) - t_base) : n;
  if (n == 0) {                                         // empty cache: zeros, log-sum-exp = -inf
    if (row_valid) {
      for (int d = 0; d < D; ++d) out[row_off * D + d] = 0.f;
      if (lse_out) lse_out[row_off] = -INFINITY;
    }
    return;
  }
  // A wait that gave up in an earlier CTA marks the workspace; the rest of the grid leaves.
  if (status_word && *reinterpret_cast<volatile int32_t*>(status_word + 2) != 0) return;
  const int nb = (n + kPfSub - 1) / kPfSub;

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 1024-byte aligned tiles
  const uint32_t sQ = base + (uint32_t)tile * kPfTileBytes;      // this query tile's rows
  const uint32_t sK = base + 2 * kPfTileBytes, sV = sK + NS * kPfSubTile;
  // behind the tiles: 4 KB per softmax warp for the epilogue's way out
  unsigned char* const stage_base = smem_raw + (base - smem_u32(smem_raw)) + 2 * kPfTileBytes + 2 * NS * kPfSubTile;
  const uint32_t bar0 = smem_u32(&s_bar[0]);
  auto bar_k = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  auto bar_v = [&](int i) { return bar0 + 8u * (uint32_t)(NS + i); };
  auto bar_kfree = [&](int i) { return bar0 + 8u * (uint32_t)(2 * NS + i); };
  auto bar_vfree = [&](int i) { return bar0 + 8u * (uint32_t)(3 * NS + i); };
  const uint32_t bar_t = bar0 + 8u * (uint32_t)(4 * NS + 6 * tile);   // this query tile's six
  auto bar_s = [&](int i) { return bar_t + 8u * (uint32_t)i; };
  auto bar_p = [&](int i) { return bar_t + 8u * (uint32_t)(2 + i); };
  // bar_o completes a phase per P V (a waiter that is two phases behind would read its parity
  // wrongly, so only the rescaling path, which is at most one behind, waits on it); bar_done
  // completes once, behind the last P V
  const uint32_t bar_o = bar_t + 32u, bar_done = bar_t + 40u;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 :: "r"(smem_u32(&s_tmem)), "r"(kPfPipeTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < 2 * NS; ++i) mbar_init(bar0 + 8u * i, 1);
    for (int i = 2 * NS; i < 4 * NS; ++i) mbar_init(bar0 + 8u * i, n_tiles);   // one commit per query tile
    for (int t = 0; t < 2; ++t) {
      const uint32_t bt = bar0 + 8u * (uint32_t)(4 * NS + 6 * t);
      mbar_init(bt, 1); mbar_init(bt + 8, 1);
      mbar_init(bt + 16, kPfRows / 32); mbar_init(bt + 24, kPfRows / 32);   // one arrival per softmax warp
      mbar_init(bt + 32, 1); mbar_init(bt + 40, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_fail = 0;
  }
  __syncwarp();
  if (softmax_thread)                                   // every softmax warp loads its own 32 rows
    load_query_rows<G>(q, bl, n_queries, g.Hq, h, 2 * qp + tile, wq * 32, sQ, 0, 16);
  proxy_fence();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem + (uint32_t)tile * 256;  // this query tile's 256 columns
  bool gave_up = false;
  float m_ref = -INFINITY, l_run = 0.f;                 // reference maximum; sum of this row's weights
  const uint32_t t_lane = tmem + ((uint32_t)(wq * 32) << 16);
  const uint32_t t_o = t_lane + 128;                    // this row's 128 output dims
  const bool tile_active = tile < n_tiles;

  if (!softmax_thread) {
    if ((tid & 31) == 0 && warp >= 10) {
      // ---- the two fetching threads: K tiles (warp 10), V tiles (warp 11) ---------------------
      const bool is_k = warp == 10;
      const CUtensorMap* map = is_k ? &map_k : &map_v;
      bool ok = true;
      for (int j = 0; ok && j < nb; ++j) {
        const int st = j % NS, use = j / NS;
        const uint32_t full = is_k ? bar_k(st) : bar_v(st);
        if (use > 0) ok = mbar_wait<kPfPolls>(is_k ? bar_kfree(st) : bar_vfree(st), (uint32_t)(use - 1) & 1u);
        if (!ok) break;
        const uint32_t dst = (is_k ? sK : sV) + st * kPfSubTile;
        mbar_expect_tx(full, kPfSubTile);
        tma_load_5d(dst, map, full, 0, tm_row + j * kPfSub, h, tm_l, tm_b);
        tma_load_5d(dst + kPfSubHalf, map, full, 64, tm_row + j * kPfSub, h, tm_l, tm_b);
      }
      if (!ok) s_fail = 1;
    } else if ((tid & 31) == 0 && tile_active) {
      // ---- the issuing thread of query tile `tile` ---------------------------------------------
      auto issue_qk = [&](int j) {                      // S[j & 1] = Q K(j)^T; then the K tile is free
        const uint32_t kt = sK + (j % NS) * kPfSubTile;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_bf16(tmem + (j & 1) * 64,
                    umma_desc(sQ + (k >> 2) * kPfHalf + (k & 3) * 32, 16, 1024),
                    umma_desc(kt + (k >> 2) * kPfSubHalf + (k & 3) * 32, 16, 1024), kIdescQK64, k > 0);
        umma_commit(bar_s(j & 1));
        umma_commit(bar_kfree(j % NS));
      };
      bool ok = mbar_wait<kPfPolls>(bar_k(0), 0);
      if (ok) { tc_fence_after(); issue_qk(0); }
      if (ok && nb > 1) {
        ok = mbar_wait<kPfPolls>(bar_k(1 % NS), 0);
        if (ok) { tc_fence_after(); issue_qk(1); }
      }
      for (int j = 0; ok && j < nb; ++j) {
        const int s = j & 1;
        // The tiles this iteration needs were fetched well ahead; checking them here, while the
        // softmax still works on S(j), keeps the checks off the path from weights to scores.
        ok = mbar_wait_likely(bar_v(j % NS), (uint32_t)(j / NS) & 1u);
        if (ok && j + 2 < nb) ok = mbar_wait_likely(bar_k((j + 2) % NS), (uint32_t)((j + 2) / NS) & 1u);
        ok = ok && mbar_wait<kPfPolls>(bar_p(s), (uint32_t)(j >> 1) & 1u);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vt = sV + (j % NS) * kPfSubTile;
#pragma unroll
        for (int k = 0; k < 4; ++k) {                   // O += P(j) V(j); slice k = tokens 16k .. 16k + 15
          umma_bf16_ts(tmem + 128, tmem + s * 64 + k * 8,
                       umma_desc(vt + k * 2048, kPfSubHalf, 1024), kIdescPV, (j > 0 || k > 0) ? 1u : 0u);
          if constexpr (SW)                             // the weights' second terms: columns 32..63
            umma_bf16_ts(tmem + 128, tmem + s * 64 + 32 + k * 8,
                         umma_desc(vt + k * 2048, kPfSubHalf, 1024), kIdescPV, 1u);
        }
        umma_commit(bar_o);
        umma_commit(bar_vfree(j % NS));
#if L2KV_PREFIX_MMA_IN_ORDER
        // The score buffer that P(j) V(j) reads its weights from takes sub-block j + 2.  The two
        // operations are issued by this one thread to this CTA's tensor core, which executes
        // what it is given in issue order: Q K(j+2)^T is queued right behind P(j) V(j) and
        // cannot overwrite the weights before they have been read.
        if (j + 2 < nb) issue_qk(j + 2);
#else
        // P(j) V(j) done: the score buffer it read its weights from takes sub-block j + 2
        ok = mbar_wait<kPfPolls>(bar_o, (uint32_t)j & 1u);
        if (!ok) break;
        if (j + 2 < nb) { tc_fence_after(); issue_qk(j + 2); }
#endif
      }
      if (ok) umma_commit(bar_done);                    // behind every P V of this query tile
      if (!ok) s_fail = 1;
    }
  } else if (tile_active) {
    // ---- the softmax warps of query tile `tile`: one thread per row ----------------------------
    for (int j = 0; j < nb; ++j) {
      const int s = j & 1;
      const int valid = min(kPfSub, n - j * kPfSub);       // valid tokens of this sub-block
      const uint32_t t_s = t_lane + s * 64;                   // this row's scores, later its weights
      if (!mbar_wait_likely(bar_s(s), (uint32_t)(j >> 1) & 1u)) gave_up = true;
      tc_fence_after();
      if (__any_sync(0xffffffffu, gave_up)) { gave_up = true; break; }
      float sv[64];                                       // raw products; the scale is folded in below
      float bmax = -INFINITY;
      {
        uint32_t r0[32], r1[32];
        tmem_ld64(t_s, r0, r1);
        const int valid_row = min(valid, n_row - j * kPfSub);
        if (valid_row >= kPfSub) {                        // only the last (or a causal row's own) sub-block masks
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            sv[i] = __uint_as_float(r0[i]);
            sv[32 + i] = __uint_as_float(r1[i]);
            bmax = fmaxf(bmax, fmaxf(sv[i], sv[32 + i]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            sv[i] = i < valid_row ? __uint_as_float(r0[i]) : -INFINITY;
            sv[32 + i] = 32 + i < valid_row ? __uint_as_float(r1[i]) : -INFINITY;
            bmax = fmaxf(bmax, fmaxf(sv[i], sv[32 + i]));
          }
        }
      }
      const float m_new = fmaxf(m_ref, bmax * scale_log2e);   // scale > 0: the maximum commutes with it
      if (j == 0) m_ref = m_new;
      // ---- rescale O only when this row's maximum has drifted far from the reference --------
      const bool need = m_new > m_ref + kPfRescaleGap;
      if (__any_sync(0xffffffffu, need)) {
        // O must be quiet: P(j-1) V(j-1) has to be complete (P(j) V(j) waits for this thread)
        if (!mbar_wait<kPfPolls>(bar_o, (uint32_t)(j - 1) & 1u)) gave_up = true;
        tc_fence_after();
        const float factor = need ? fast_exp2(m_ref - m_new) : 1.f;
#pragma unroll 1
        for (int c = 0; c < D; c += 8) tmem_scale8(t_o + c, factor);
        if (need) { l_run *= factor; m_ref = m_new; }
      }
      // ---- weights 2^(s - m_ref) as bf16 pairs over the first half of the score columns -----
      {
        uint32_t pk[32];
        [[maybe_unused]] uint32_t pr[SW ? 32 : 1];
        float rowsum0 = 0.f, rowsum1 = 0.f;
        const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;   // a row with nothing to see yet
#pragma unroll
        for (int i = 0; i < 64; i += 2) {
          const float p0 = fast_exp2(__fmaf_rn(sv[i], scale_log2e, neg_m));     // -inf -> 0
          const float p1 = fast_exp2(__fmaf_rn(sv[i + 1], scale_log2e, neg_m));
          rowsum0 += p0;
          rowsum1 += p1;
          pk[i >> 1] = pack_bf16(p0, p1);
          if constexpr (SW) pr[i >> 1] = pack_bf16_rest(p0, p1, pk[i >> 1]);
        }
        tmem_st32(t_s, pk);
        if constexpr (SW) tmem_st32(t_s + 32, pr);        // second terms: the other half of the buffer
        tmem_wait_st();
        l_run += rowsum0 + rowsum1;
      }
      if (valid < kPfSub) {
        // Last, partial sub-block: rows of the V tile past the valid length hold whatever the
        // cache holds there; clear them so that a zero weight times Inf/NaN cannot reach O
        // (both query tiles write the same zeros).
        if (!mbar_wait<kPfPolls>(bar_v(j % NS), (uint32_t)(j / NS) & 1u)) gave_up = true;
        if (row >= valid && row < kPfSub) {
#pragma unroll
          for (int c = 0; c < 16; ++c)
            st_shared16(sV + (j % NS) * kPfSubTile + (c >> 3) * kPfSubHalf + row * 128 + ((c & 7) << 4), 0, 0, 0, 0);
        }
        proxy_fence();
      }
      tc_fence_before();
      __syncwarp();                                       // the warp's 32 rows are in place:
      if ((tid & 31) == 0) mbar_arrive(bar_p(s));         // one arrival per warp
    }
    // O is complete when the commit behind the last P V has arrived
    if (!gave_up && !mbar_wait<kPfPolls>(bar_done, 0)) gave_up = true;
    if (gave_up) s_fail = 1;
  }
  __syncthreads();                                       // every role is done with the loop
  tc_fence_after();
  const bool failed = s_fail != 0;
  const float l_tot = l_run;
  if (!failed && softmax_thread && tile_active) {
    const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;   // nothing seen: zeros, log-sum-exp -inf
    store_rows_via_stage(t_o, inv, row_valid ? out + row_off * D : nullptr,
                         reinterpret_cast<float4*>(stage_base + warp * kPfStageBytes));
    if (row_valid && lse_out)
      lse_out[row_off] = (m_ref + log2f(l_tot)) * 0.6931471805599453f;
  }
  if (failed && tid == 0) record_timeout(status_word);
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(s_tmem), "r"(kPfPipeTmemCols)
                 : "memory");
}

// The persistent, work-balanced kernel (L2KV_PREFIX_KERNEL=persistent; needs a workspace with
// room for its partial results).  The pipelined kernel's roles and hand-offs, but a fixed grid of
// kPfPersistCtas CTAs, each of which stays on its SM and walks an equal share of the call's work:
//   - a work item is (pair of query tiles, unit); its cost is its number of 64-token sub-blocks
//     plus kPfItemOverhead (what starting and finishing an item costs, in sub-blocks' time).
//     Every CTA adds up the costs of all items (the lengths live in device memory) and takes the
//     range [c P, (c + 1) P) of the running total, P = ceil(total / CTAs): whole items, plus at
//     most one item cut at its start and one cut at its end;
//   - an item that lies in one CTA's range is written straight to out / lse_out; the pieces of a
//     cut item go, normalised and with their log-sum-exp, to two slots per CTA in the workspace
//     (slot 2c: the piece that is CTA c's first segment; 2c + 1: a piece that begins inside its
//     range); the CTA that hands in an item's last piece (a counter per cut item) adds them up;
//   - tensor memory, the mbarriers and the K / V rings are set up once; the fetching threads run
//     ahead across item boundaries; between two segments the softmax threads write the next
//     query rows into shared memory and tell the issuing thread (one more mbarrier per tile).
constexpr int kPfPersistCtas = 148;
constexpr int kPfSlotRows = 2 * kPfRows;         // rows of one partial result: both query tiles
constexpr int kPfMinShare = 16;                  // sub-blocks: no share below 1024 tokens
constexpr int kPfAutoShare = 48;                 // sub-blocks per CTA from which a small grid is dealt out this way
constexpr int kPfTicketWord = 16;                // first word of the ticket bytes in the status block
static_assert(kPfTicketWord * 4 + kPfPersistCtas <= kStatusBytes && kPfPersistCtas < 256,
              "a ticket byte per CTA inside the status block; a count fits its byte");
constexpr int kPfItemOverhead = 8;               // measured: about 15 k cycles against 1.9 k per sub-block

template <int G, bool SW>
__global__ void __launch_bounds__(kPfPipeThreads, 1)
prefix_attention_persistent_kernel(const __nv_bfloat16* __restrict__ q, Geom g, int n_queries,
                           LenView cur_len_dev, int max_len, float scale_log2e,
                           float* __restrict__ out, float* __restrict__ lse_out,
                           const __grid_constant__ CUtensorMap map_k,
                           const __grid_constant__ CUtensorMap map_v,
                           int32_t* __restrict__ status_word, float* __restrict__ part_out,
                           float* __restrict__ part_lse, int causal) {
  constexpr int D = 128;
  constexpr int QT = kPfRows / G;                       // queries per query tile
  constexpr int NS = kPfStages;
  constexpr int NT = kPfPipeThreads;
  extern __shared__ unsigned char smem_raw[];
  // mbarriers: K landed [NS], V landed [NS], K tile free [NS], V tile free [NS], then per query
  // tile: scores ready [2], weights ready [2], output quiet [1], query rows ready [1], the
  // segment's output complete [1]; then: a piece's rows written [1], its turn known [1]
  __shared__ __align__(8) unsigned long long s_bar[4 * NS + 16];
  __shared__ int s_merge;                               // this CTA handed in the item's last piece
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail;
  __shared__ int s_sum[NT / 32];
  __shared__ unsigned long long s_first;                // first item of this CTA's walk
  __shared__ int s_first_at;                            // running total before that item

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = (int)blockIdx.x, n_cta = (int)gridDim.x;
  const int q_tiles = (n_queries + QT - 1) / QT;
  const int q_pairs = (q_tiles + 1) / 2;
  // items are numbered pair-major (item = pair * units + unit): CTAs a whole number of units apart
  // then walk the same K and V rows at about the same time, and the second read hits the L2
  const long long units = (long long)g.B * g.L * g.H;
  const long long items = units * q_pairs;
  // A wait that gave up in an earlier call marks the workspace; nothing runs until it is cleared.
  if (status_word && *reinterpret_cast<volatile int32_t*>(status_word + 2) != 0) return;

  // cached rows of item `it`, and its cost in sub-blocks
  auto item_rows = [&](long long it) {
    const long long unit = it % units, bl = unit / g.H;
    return max(0, min(cur_len_dev.at(bl, (int)(unit % g.H), g.H), min(max_len, g.cap(bl))));
  };
  // (the overhead comes first in an item's range of the running total, its sub-blocks after it)
  auto item_cost = [&](long long it) {
    const int nb_it = (item_rows(it) + kPfSub - 1) / kPfSub;
    return nb_it > 0 ? nb_it + kPfItemOverhead : 0;
  };

  // ---- every CTA adds up all costs: thread t takes the items [t chunk, (t + 1) chunk) -----------
  const long long chunk = (items + NT - 1) / NT;
  const long long c_lo = min(items, (long long)tid * chunk), c_hi = min(items, c_lo + chunk);
  int mine = 0;
  for (long long it = c_lo; it < c_hi; ++it) mine += item_cost(it);
  int incl = mine;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += o;
  }
  if (lane == 31) s_sum[warp] = incl;
  if (tid == 0) { s_first = ~0ull; s_first_at = 0; s_fail = 0; }
  __syncthreads();
  int before = incl - mine, total = 0;
  for (int w = 0; w < NT / 32; ++w) {
    if (w < warp) before += s_sum[w];
    total += s_sum[w];
  }
  // The CTAs are dealt out in equal groups, one per pair of query tiles (every pair's items cost
  // the same: the costs depend on the unit alone), when the grid divides that way: CTA c of one
  // group and CTA c of the next then walk the same K and V rows at the same time, and one of the
  // two reads hits the L2.  Otherwise one group takes everything.
  const int groups = (total > 0 && n_cta % q_pairs == 0) ? q_pairs : 1;
  const int per_group = n_cta / groups, group_total = total / groups;
  const int share = max(kPfMinShare, (group_total + per_group - 1) / per_group);
  // first position of CTA c's range, and the CTA whose range holds position x (x < total)
  auto lo_of = [&](int c) {                              // (a group's surplus CTAs get its end: nothing)
    const long long g0 = (long long)(c / per_group) * group_total;
    return (int)min(g0 + (long long)(c % per_group) * share, g0 + group_total);
  };
  auto cta_of = [&](int x) {
    const int grp = min(groups - 1, x / max(group_total, 1));
    return grp * per_group + min(per_group - 1, (x - grp * group_total) / share);
  };
  // this CTA's range of the running total; the last CTA's is open-ended (trailing empty items)
  const int lo = lo_of(cta);
  const int hi = cta == n_cta - 1 ? INT_MAX
               : (cta % per_group == per_group - 1 ? (cta / per_group + 1) * group_total
                                                  : min(lo_of(cta) + share, (cta / per_group + 1) * group_total));
  // the walk starts at the first item that reaches past lo, or begins at or after it
  {
    int at = before;
    for (long long it = c_lo; it < c_hi; ++it) {
      const int c = item_cost(it);
      if (at + c > lo || at >= lo) { atomicMin(&s_first, (unsigned long long)it); break; }
      at += c;
    }
  }
  __syncthreads();
  {
    int at = before;
    for (long long it = c_lo; it < c_hi; ++it) {
      if ((unsigned long long)it == s_first) { s_first_at = at; break; }
      at += item_cost(it);
    }
  }

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 1024-byte aligned tiles
  const bool softmax_thread = tid < 2 * kPfRows;
  const int tile = softmax_thread ? tid >> 7 : warp & 1;
  const int row = tid & (kPfRows - 1);
  const int wq = warp & 3;                              // tensor-memory lane quarter of this warp
  const uint32_t sQ = base + (uint32_t)tile * kPfTileBytes;
  const uint32_t sK = base + 2 * kPfTileBytes, sV = sK + NS * kPfSubTile;
  // behind the tiles: 4 KB per softmax warp for the epilogue's way out
  unsigned char* const stage_base = smem_raw + (base - smem_u32(smem_raw)) + 2 * kPfTileBytes + 2 * NS * kPfSubTile;
  const uint32_t bar0 = smem_u32(&s_bar[0]);
  auto bar_k = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  auto bar_v = [&](int i) { return bar0 + 8u * (uint32_t)(NS + i); };
  auto bar_kfree = [&](int i) { return bar0 + 8u * (uint32_t)(2 * NS + i); };
  auto bar_vfree = [&](int i) { return bar0 + 8u * (uint32_t)(3 * NS + i); };
  const uint32_t bar_t = bar0 + 8u * (uint32_t)(4 * NS + 7 * tile);   // this query tile's seven
  auto bar_s = [&](int i) { return bar_t + 8u * (uint32_t)i; };
  auto bar_p = [&](int i) { return bar_t + 8u * (uint32_t)(2 + i); };
  const uint32_t bar_o = bar_t + 32u, bar_q = bar_t + 40u, bar_done = bar_t + 48u;
  const uint32_t bar_piece = bar0 + 8u * (uint32_t)(4 * NS + 14), bar_turn = bar_piece + 8u;

  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 :: "r"(smem_u32(&s_tmem)), "r"(kPfPipeTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    for (int i = 0; i < 2 * NS; ++i) mbar_init(bar0 + 8u * i, 1);
    for (int i = 2 * NS; i < 4 * NS; ++i) mbar_init(bar0 + 8u * i, 2);     // one arrival per query tile
    for (int t = 0; t < 2; ++t) {
      const uint32_t bt = bar0 + 8u * (uint32_t)(4 * NS + 7 * t);
      mbar_init(bt, 1); mbar_init(bt + 8, 1);
      mbar_init(bt + 16, kPfRows / 32); mbar_init(bt + 24, kPfRows / 32);   // one arrival per softmax warp
      mbar_init(bt + 32, 1);
      mbar_init(bt + 40, kPfRows / 32);
      mbar_init(bt + 48, 1);
    }
    mbar_init(bar_piece, 2 * kPfRows / 32);               // one arrival per softmax warp, both tiles
    mbar_init(bar_turn, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem + (uint32_t)tile * 256;  // this query tile's 256 columns
  const uint32_t t_lane = tmem + ((uint32_t)(wq * 32) << 16);
  const uint32_t t_o = t_lane + 128;                    // this row's 128 output dims

  // Every thread that has a role walks the same segments: (item, sub-blocks [j0, j1) of it).
  long long w_it = (long long)s_first;
  int w_at = s_first_at;
  long long it = 0;                                     // the segment's item
  int at = 0, cost = 0, nb_it = 0, j0 = 0, j1 = 0;      // its place in the total, cost, sub-blocks, range
  auto next_segment = [&]() {
    if (w_it < 0 || w_it >= items || w_at >= hi) return false;
    it = w_it; at = w_at; cost = item_cost(it);
    nb_it = max(0, cost - kPfItemOverhead);
    j0 = max(0, lo - at - kPfItemOverhead); j1 = min(nb_it, hi - at - kPfItemOverhead);
    ++w_it; w_at += cost;
    return true;
  };
  int jj = 0;                                           // sub-blocks this CTA has been through
  bool gave_up = false;

  if (!softmax_thread) {
    if (lane == 0 && warp >= 10) {
      // ---- the two fetching threads: K tiles (warp 10), V tiles (warp 11) ---------------------
      const bool is_k = warp == 10;
      const CUtensorMap* map = is_k ? &map_k : &map_v;
      bool ok = true;
      while (ok && next_segment()) {
        const long long unit = it % units, bl = unit / g.H;
        const int h = (int)(unit % g.H);
        const int tm_row = (int)g.row0(bl);
        const int tm_l = g.row_off ? 0 : (int)(bl % g.L), tm_b = g.row_off ? 0 : (int)(bl / g.L);
        for (int j = j0; ok && j < j1; ++j, ++jj) {
          const int st = jj % NS, use = jj / NS;
          const uint32_t full = is_k ? bar_k(st) : bar_v(st);
          if (use > 0) ok = mbar_wait<kPfPolls>(is_k ? bar_kfree(st) : bar_vfree(st), (uint32_t)(use - 1) & 1u);
          if (!ok) break;
          const uint32_t dst = (is_k ? sK : sV) + st * kPfSubTile;
          mbar_expect_tx(full, kPfSubTile);
          tma_load_5d(dst, map, full, 0, tm_row + j * kPfSub, h, tm_l, tm_b);
          tma_load_5d(dst + kPfSubHalf, map, full, 64, tm_row + j * kPfSub, h, tm_l, tm_b);
        }
      }
      if (!ok) s_fail = 1;
    } else if (lane == 0) {
      // ---- the issuing thread of query tile `tile` ---------------------------------------------
      // S[a & 1] = Q K^T for the K tile at ring position x; a counts this query tile's sub-blocks
      auto issue_qk = [&](int x, int a) {
        const uint32_t kt = sK + (x % NS) * kPfSubTile;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_bf16(tmem + (a & 1) * 64,
                    umma_desc(sQ + (k >> 2) * kPfHalf + (k & 3) * 32, 16, 1024),
                    umma_desc(kt + (k >> 2) * kPfSubHalf + (k & 3) * 32, 16, 1024), kIdescQK64, k > 0);
        umma_commit(bar_s(a & 1));
        umma_commit(bar_kfree(x % NS));
      };
      bool ok = true;
      int seg = 0, ja = 0;                              // segments / sub-blocks this tile took part in
      while (ok && next_segment()) {
        const int nbs = j1 - j0;
        if (nbs <= 0) continue;
        const int qp = (int)(it / units);
        if (2 * qp + tile >= q_tiles) {
          // this query tile does not exist in the item: hand every K and V tile back as it lands
          for (int x = jj; ok && x < jj + nbs; ++x) {
            ok = mbar_wait<kPfPolls>(bar_k(x % NS), (uint32_t)(x / NS) & 1u);
            if (ok) mbar_arrive(bar_kfree(x % NS));
            ok = ok && mbar_wait<kPfPolls>(bar_v(x % NS), (uint32_t)(x / NS) & 1u);
            if (ok) mbar_arrive(bar_vfree(x % NS));
          }
          jj += nbs;
          continue;
        }
        ok = mbar_wait<kPfPolls>(bar_q, (uint32_t)seg & 1u);          // the segment's query rows
        ++seg;
        if (ok) ok = mbar_wait<kPfPolls>(bar_k(jj % NS), (uint32_t)(jj / NS) & 1u);
        if (ok) { tc_fence_after(); issue_qk(jj, ja); }
        if (ok && nbs > 1) {
          ok = mbar_wait<kPfPolls>(bar_k((jj + 1) % NS), (uint32_t)((jj + 1) / NS) & 1u);
          if (ok) { tc_fence_after(); issue_qk(jj + 1, ja + 1); }
        }
        const int end = jj + nbs;
        for (int x = jj; ok && x < end; ++x) {
          const int a = ja + (x - jj), s = a & 1;
          ok = mbar_wait_likely(bar_v(x % NS), (uint32_t)(x / NS) & 1u);
          if (ok && x + 2 < end) ok = mbar_wait_likely(bar_k((x + 2) % NS), (uint32_t)((x + 2) / NS) & 1u);
          ok = ok && mbar_wait<kPfPolls>(bar_p(s), (uint32_t)(a >> 1) & 1u);
          if (!ok) break;
          tc_fence_after();
          const uint32_t vt = sV + (x % NS) * kPfSubTile;
#pragma unroll
          for (int k = 0; k < 4; ++k) {                 // O += P V; slice k = tokens 16k .. 16k + 15
            umma_bf16_ts(tmem + 128, tmem + s * 64 + k * 8,
                         umma_desc(vt + k * 2048, kPfSubHalf, 1024), kIdescPV, (x > jj || k > 0) ? 1u : 0u);
            if constexpr (SW)
              umma_bf16_ts(tmem + 128, tmem + s * 64 + 32 + k * 8,
                           umma_desc(vt + k * 2048, kPfSubHalf, 1024), kIdescPV, 1u);
          }
          umma_commit(bar_o);
          umma_commit(bar_vfree(x % NS));
          // queued right behind P V, whose weights it overwrites: the tensor core executes this
          // thread's operations in issue order (see the pipelined kernel)
          if (x + 2 < end) issue_qk(x + 2, a + 2);
        }
        if (ok) umma_commit(bar_done);                  // behind every P V of the segment
        jj = end;
        ja += nbs;
      }
      if (!ok) s_fail = 1;
    }
  } else {
    // ---- the softmax warps of query tile `tile`: one thread per row ------------------------------
    int seg = 0, ja = 0;                                // segments / sub-blocks this tile took part in
    int pieces = 0;                                     // partial results this CTA has written
    while (!gave_up && next_segment()) {
      const long long unit = it % units, bl = unit / g.H;
      const int qp = (int)(it / units), h = (int)(unit % g.H);
      const int s_idx = (2 * qp + tile) * QT + row / G;     // this row's query and head
      const int head = h * G + row % G;
      const bool row_valid = s_idx < n_queries;
      const long long row_off = ((bl * n_queries + s_idx) * g.Hq + head);
      if (cost == 0) {                                    // empty cache: zeros, log-sum-exp = -inf
        if (row_valid) {
          for (int d = 0; d < D; ++d) out[row_off * D + d] = 0.f;
          if (lse_out) lse_out[row_off] = -INFINITY;
        }
        continue;
      }
      const int nbs = j1 - j0;
      if (nbs <= 0) continue;
      const bool partial = j0 > 0 || j1 < nb_it;
      // a piece that is this CTA's first segment (the item begins at or before the range) takes
      // slot 2c, one that begins inside the range slot 2c + 1
      const int slot = at <= lo ? 2 * cta : 2 * cta + 1;
      const bool active = 2 * qp + tile < q_tiles;
      if (!active) jj += nbs;
      if (active) {
        const int n_all = item_rows(it);
        // causal: the last n_queries cached rows are the new tokens' own; query s stops at its own
        const int n_row = causal && row_valid ? min(n_all, max(0, n_all - n_queries + s_idx + 1)) : n_all;
        {                                                   // this warp's 32 query rows
          load_query_rows<G>(q, bl, n_queries, g.Hq, h, 2 * qp + tile, wq * 32, sQ, 0, 16);
          proxy_fence();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_q);
        }
        float m_ref = -INFINITY, l_run = 0.f;               // reference maximum; sum of this row's weights
        const int end = jj + nbs;
        for (int x = jj; x < end; ++x) {
          const int j = j0 + (x - jj);                      // sub-block of the item
          const int a = ja + (x - jj), s = a & 1;
          const int valid = min(kPfSub, n_all - j * kPfSub);   // valid tokens of this sub-block
          const uint32_t t_s = t_lane + s * 64;               // this row's scores, later its weights
          if (!mbar_wait_likely(bar_s(s), (uint32_t)(a >> 1) & 1u)) gave_up = true;
          tc_fence_after();
          if (__any_sync(0xffffffffu, gave_up)) { gave_up = true; break; }
          float sv[64];                                     // raw products; the scale is folded in below
          float bmax = -INFINITY;
          {
            uint32_t r0[32], r1[32];
            tmem_ld64(t_s, r0, r1);
            const int valid_row = min(valid, n_row - j * kPfSub);
            if (valid_row >= kPfSub) {
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                sv[i] = __uint_as_float(r0[i]);
                sv[32 + i] = __uint_as_float(r1[i]);
                bmax = fmaxf(bmax, fmaxf(sv[i], sv[32 + i]));
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                sv[i] = i < valid_row ? __uint_as_float(r0[i]) : -INFINITY;
                sv[32 + i] = 32 + i < valid_row ? __uint_as_float(r1[i]) : -INFINITY;
                bmax = fmaxf(bmax, fmaxf(sv[i], sv[32 + i]));
              }
            }
          }
          const float m_new = fmaxf(m_ref, bmax * scale_log2e);
          if (x == jj) m_ref = m_new;
          const bool need = m_new > m_ref + kPfRescaleGap;
          if (__any_sync(0xffffffffu, need)) {
            // O must be quiet: the previous P V has to be complete (this one waits for this thread)
            if (!mbar_wait<kPfPolls>(bar_o, (uint32_t)(a - 1) & 1u)) gave_up = true;
            tc_fence_after();
            const float factor = need ? fast_exp2(m_ref - m_new) : 1.f;
#pragma unroll 1
            for (int c = 0; c < D; c += 8) tmem_scale8(t_o + c, factor);
            if (need) { l_run *= factor; m_ref = m_new; }
          }
          {
            uint32_t pk[32];
            [[maybe_unused]] uint32_t pr[SW ? 32 : 1];
            float rowsum0 = 0.f, rowsum1 = 0.f;
            const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;   // a row with nothing to see yet
#pragma unroll
            for (int i = 0; i < 64; i += 2) {
              const float p0 = fast_exp2(__fmaf_rn(sv[i], scale_log2e, neg_m));     // -inf -> 0
              const float p1 = fast_exp2(__fmaf_rn(sv[i + 1], scale_log2e, neg_m));
              rowsum0 += p0;
              rowsum1 += p1;
              pk[i >> 1] = pack_bf16(p0, p1);
              if constexpr (SW) pr[i >> 1] = pack_bf16_rest(p0, p1, pk[i >> 1]);
            }
            tmem_st32(t_s, pk);
            if constexpr (SW) tmem_st32(t_s + 32, pr);
            tmem_wait_st();
            l_run += rowsum0 + rowsum1;
          }
          if (valid < kPfSub) {
            // partial sub-block: clear the V rows past the valid length (both query tiles write
            // the same zeros) so that a zero weight times Inf/NaN cannot reach O
            if (!mbar_wait<kPfPolls>(bar_v(x % NS), (uint32_t)(x / NS) & 1u)) gave_up = true;
            if (row >= valid && row < kPfSub) {
#pragma unroll
              for (int c = 0; c < 16; ++c)
                st_shared16(sV + (x % NS) * kPfSubTile + (c >> 3) * kPfSubHalf + row * 128 + ((c & 7) << 4), 0, 0, 0, 0);
            }
            proxy_fence();
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p(s));             // one arrival per warp
        }
        if (gave_up) break;
        // the segment's O is complete when the commit behind its last P V has arrived
        if (!mbar_wait<kPfPolls>(bar_done, (uint32_t)seg & 1u)) { gave_up = true; break; }
        ++seg;
        tc_fence_after();
        jj = end;
        ja += nbs;
        {
          const float inv = l_run > 0.f ? 1.f / l_run : 0.f;   // nothing seen: zeros, log-sum-exp -inf
          const long long p_row = (long long)slot * kPfSlotRows + tile * kPfRows + row;
          float* dst_row = partial ? part_out + p_row * D : out + row_off * D;
          store_rows_via_stage(t_o, inv, row_valid ? dst_row : nullptr,
                               reinterpret_cast<float4*>(stage_base + warp * kPfStageBytes));
          const float lse = (m_ref + log2f(l_run)) * 0.6931471805599453f;
          if (row_valid) {
            if (partial) part_lse[p_row] = lse;
            else if (lse_out) lse_out[row_off] = lse;
          }
          tc_fence_before();                                // O has been read before the next segment's P V
        }
      }
      if (gave_up) break;
      if (partial) {
        // A piece of a cut item: once both tiles' rows are in the workspace, this CTA takes a
        // ticket of the item (counter of the CTA the item starts in); whoever takes the last one
        // adds the pieces up.  Nobody waits for another CTA; the counter goes back to zero.
        const int c_first = cta_of(at + kPfItemOverhead), c_last = cta_of(at + cost - 1);   // CTAs with sub-blocks
        __threadfence();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_piece);
        if (!mbar_wait<kPfPolls>(bar_piece, (uint32_t)pieces & 1u)) { gave_up = true; break; }
        if (tid == 0) {
          // the counters: one byte per CTA, four to a word, in the workspace's status block (zero
          // before the call like the rest of the block, and zero again after the last ticket)
          unsigned int* const word = reinterpret_cast<unsigned int*>(status_word) + kPfTicketWord + (c_first >> 2);
          const int shift = (c_first & 3) * 8;
          const int turn = (int)((atomicAdd(word, 1u << shift) >> shift) & 0xffu);
          s_merge = turn == c_last - c_first;
          if (s_merge) atomicSub(word, (unsigned int)(c_last - c_first + 1) << shift);
          __threadfence();
          mbar_arrive(bar_turn);
        }
        if (!mbar_wait<kPfPolls>(bar_turn, (uint32_t)pieces & 1u)) { gave_up = true; break; }
        ++pieces;
        if (s_merge && active) {
          // A warp adds up its 32 rows together: every lane works out the weights of its own
          // row's pieces, then the lanes go through the rows side by side (a row is 32 float4),
          // 8 rows' loads in flight at a time.
          __threadfence();
          const int r = tile * kPfRows + row;
          auto slot_of = [&](int p) { return p == c_first && at > lo_of(c_first) ? 2 * p + 1 : 2 * p; };
          float m = -INFINITY;
          if (row_valid)
            for (int p = c_first; p <= c_last; ++p)
              m = fmaxf(m, __ldcg(part_lse + (long long)slot_of(p) * kPfSlotRows + r));
          float den = 0.f;
          if (row_valid)
            for (int p = c_first; p <= c_last; ++p) {
              const float lp = __ldcg(part_lse + (long long)slot_of(p) * kPfSlotRows + r);
              den += lp > -INFINITY ? __expf(lp - m) : 0.f;
            }
          const bool any = m > -INFINITY;                 // some piece had rows this query may see
          const float inv = any ? 1.f / den : 0.f;
          const uint32_t valid_rows = __ballot_sync(0xffffffffu, row_valid);
          const int r_warp = r - lane;                    // first row of this warp
#pragma unroll 1
          for (int part = 0; part < 4; ++part) {
            float4 acc[8] = {};
            for (int p = c_first; p <= c_last; ++p) {
              const long long pr = (long long)slot_of(p) * kPfSlotRows + r;
              const float lp = row_valid ? __ldcg(part_lse + pr) : -INFINITY;
              const float w = lp > -INFINITY ? __expf(lp - m) * inv : 0.f;
              const float4* src = reinterpret_cast<const float4*>(
                  part_out + ((long long)slot_of(p) * kPfSlotRows + r_warp + part * 8) * D) + lane;
              float4 v[8];
#pragma unroll
              for (int rr = 0; rr < 8; ++rr)
                v[rr] = (valid_rows >> (part * 8 + rr)) & 1u ? __ldcg(src + rr * (D / 4))
                                                              : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int rr = 0; rr < 8; ++rr) {
                const float wr = __shfl_sync(0xffffffffu, w, part * 8 + rr);
                acc[rr].x = fmaf(wr, v[rr].x, acc[rr].x); acc[rr].y = fmaf(wr, v[rr].y, acc[rr].y);
                acc[rr].z = fmaf(wr, v[rr].z, acc[rr].z); acc[rr].w = fmaf(wr, v[rr].w, acc[rr].w);
              }
            }
#pragma unroll
            for (int rr = 0; rr < 8; ++rr) {
              const long long ro = __shfl_sync(0xffffffffu, row_off, part * 8 + rr);
              if ((valid_rows >> (part * 8 + rr)) & 1u)
                reinterpret_cast<float4*>(out + ro * D)[lane] = acc[rr];
            }
          }
          if (row_valid && lse_out) lse_out[row_off] = any ? m + logf(den) : -INFINITY;
        }
      }
    }
    if (gave_up) s_fail = 1;
  }
  __syncthreads();                                       // every role is done
  if (s_fail != 0 && tid == 0) record_timeout(status_word);
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(s_tmem), "r"(kPfPipeTmemCols)
                 : "memory");
}

// Merge of the per-chunk results of a split launch: out = sum_c w_c O_c / sum_c w_c with
// w_c = exp(lse_c - max lse), lse = max + log(sum_c w_c), over the chunks that hold cached rows.
__global__ void __launch_bounds__(128)
prefix_merge_kernel(const float* __restrict__ part_out, const float* __restrict__ part_lse,
                    LenView cur_len_dev, int max_len, Geom g, int H, int Hq, int n_queries,
                    int split_len, long long rows_total, float* __restrict__ out,
                    float* __restrict__ lse_out, const int32_t* __restrict__ status_word) {
  if (status_word && status_word[2] != 0) return;       // a chunk gave up: no output
  const long long row = blockIdx.x;                      // ((b * L + l) * n_queries + s) * Hq + head
  const long long bl = row / ((long long)n_queries * Hq);
  const int h = (int)(row % Hq) / (Hq / H);
  const int n = max(0, min(cur_len_dev.at(bl, h, H), min(max_len, g.cap(bl))));
  const int nc = (n + split_len - 1) / split_len;        // chunks with cached rows
  const int d = threadIdx.x;
  float m = -INFINITY;
  for (int c = 0; c < nc; ++c) m = fmaxf(m, part_lse[c * rows_total + row]);
  float den = 0.f, num = 0.f;
  for (int c = 0; c < nc; ++c) {
    const float lc = part_lse[c * rows_total + row];
    const float w = lc > -INFINITY ? __expf(lc - m) : 0.f;
    den += w;
    num = fmaf(w, part_out[(c * rows_total + row) * 128 + d], num);
  }
  const bool any = nc > 0 && m > -INFINITY;             // some chunk had rows this query may see
  out[row * 128 + d] = any ? num / den : 0.f;
  if (lse_out && d == 0) lse_out[row] = any ? m + logf(den) : -INFINITY;
}

// How a launch is laid out.  Kernel: the pipelined one works on pairs of query tiles; with an odd,
// small number of tiles per KV head (one tile: up to 128 / G queries) too many of its CTAs would
// run half empty, and the single-role kernel with two CTAs per SM is the faster one
// (L2KV_PREFIX_KERNEL=basic / =pipelined overrides the choice).  Chunks: the cache is split over
// blockIdx.y, with a merge pass after, when the unsplit grid would leave SMs idle (few KV heads
// and query tiles, as in a call for one layer); chunks are multiples of 128 tokens and at least
// 1024 long.  A cache so long that (b, l) pairs of different lengths would leave a few CTAs
// running alone at the end goes to the work-balanced persistent kernel instead
// (L2KV_PREFIX_KERNEL=persistent asks for it anywhere), or, without the workspace it needs, is
// split into chunks of 16k tokens if there is room for that.
struct PrefixPlan {
  bool basic;
  bool persistent;         // the work-balanced kernel was asked for and its totals fit 32 bits
  long long ctas;          // per chunk
  int chunks, split_len;
  long long rows;          // B * L * n_queries * Hq
  size_t scratch_bytes;    // partial results of a split launch (0 when chunks == 1)
};
static PrefixPlan plan_prefix(const Geom& g, int n_queries, int max_len) {
  PrefixPlan p;
  const int G = g.Hq / g.H;
  const int QT = kPfRows / G;
  const int q_tiles = (n_queries + QT - 1) / QT;
  const char* which = std::getenv("L2KV_PREFIX_KERNEL");
  p.basic = (q_tiles & 1) && q_tiles < 9;
  if (which && std::strcmp(which, "basic") == 0) p.basic = true;
  if (which && std::strcmp(which, "pipelined") == 0) p.basic = false;
  const long long pairs_all = (long long)g.B * g.L * g.H * ((q_tiles + 1) / 2);
  // the work-balanced kernel: on request, and by itself (a) for very long caches, where (b, l)
  // pairs of different lengths would otherwise leave a few CTAs running alone at the end, and
  // (b) for grids of less than two waves whose work still gives each of its CTAs a share of at
  // least kPfAutoShare sub-blocks (measured: below that its set-up and the merging of many short
  // pieces cost more than the even shares gain)
  const bool fits = pairs_all * ((long long)max_len / kPfSub + 1 + kPfItemOverhead) < (long long)INT_MAX / 2;
  if (which && std::strcmp(which, "persistent") == 0) p.basic = false;
  const bool small_grid = pairs_all < 2 * 148 &&
                          pairs_all * (((long long)max_len + kPfSub - 1) / kPfSub) >= (long long)kPfAutoShare * kPfPersistCtas;
  p.persistent = fits && !p.basic &&
                 ((which && std::strcmp(which, "persistent") == 0) || (!which && (max_len >= 65536 || small_grid)));
  const long long units = (long long)g.B * g.L * g.H;
  p.ctas = units * (p.basic ? q_tiles : (q_tiles + 1) / 2);
  p.rows = (long long)g.B * g.L * n_queries * g.Hq;
  const long long slots = 148LL * (p.basic ? 2 : 1);     // CTAs the GPU holds at once
  const long long by_len = max_len / 1024 > 1 ? max_len / 1024 : 1;
  long long chunks = 1;
  if (p.ctas > 0 && p.ctas < 2 * slots) {
    // few CTAs: the chunk count that fills whole waves best, a CTA's fixed cost (set-up, the
    // first fetches, the epilogue) counted as 256 tokens' worth of work
    double best = 0.0;
    for (long long c = 1; c <= by_len && c <= 64; ++c) {
      const double waves = (double)(p.ctas * c) / (double)slots;
      const double len = (double)max_len / (double)c;
      const double eff = waves / std::ceil(waves) * len / (len + 256.0);
      if (eff > best * 1.02) { best = eff; chunks = c; }   // more chunks only for a real gain
    }
  }
  if (max_len >= 65536 && chunks < (max_len + 16383) / 16384) chunks = (max_len + 16383) / 16384;
  p.split_len = (int)round_up_ll((max_len + chunks - 1) / chunks, 128);
  if (p.split_len < 128) p.split_len = 128;
  p.chunks = max_len > 0 ? (max_len + p.split_len - 1) / p.split_len : 1;
  p.scratch_bytes = p.chunks > 1 ? (size_t)p.chunks * p.rows * 129 * sizeof(float) : 0;
  return p;
}

// Scratch of the persistent kernel: the log-sum-exps and the rows of the two partial results a
// CTA may write (its ticket counters live in the status block).
constexpr size_t kPfPartLseBytes = (size_t)2 * kPfPersistCtas * kPfSlotRows * sizeof(float);
constexpr size_t kPfPersistBytes = kPfPartLseBytes * (1 + 128);

size_t prefix_attention_scratch(const Geom& g, int n_queries, int max_len) {
  const PrefixPlan p = plan_prefix(g, n_queries, max_len);
  return p.persistent ? kPfPersistBytes : p.scratch_bytes;
}

template <int G, bool SW>
static int launch_pf(const void* q, const void* K, const void* V, const Geom& g, int n_queries,
                     const LenView& cur_len_dev, int max_len, float scale, float* out,
                     float* lse_out, int32_t* status_word, float* scratch, size_t scratch_bytes,
                     int causal, cudaStream_t s) {
  PrefixPlan p = plan_prefix(g, n_queries, max_len);
  if (p.ctas == 0) return L2KV_OK;
  if (p.chunks > 1 && (!scratch || scratch_bytes < p.scratch_bytes)) {   // no room: one chunk
    p.chunks = 1;
    p.split_len = max_len > 128 ? (int)round_up_ll(max_len, 128) : 128;
  }
  if (p.ctas > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
  alignas(64) CUtensorMap map_k, map_v;
  std::memset(&map_k, 0, sizeof map_k);
  std::memset(&map_v, 0, sizeof map_v);
  const int sub_rows = p.basic ? kPfRows : kPfSub;
  if (!make_cache_map(&map_k, K, g, sub_rows) || !make_cache_map(&map_v, V, g, sub_rows))
    return L2KV_ERR_UNSUPPORTED;
  // A split launch writes per-chunk results (normalised rows, then their log-sum-exps) to the
  // scratch; the merge pass below turns them into out / lse_out.
  float* k_out = p.chunks > 1 ? scratch : out;
  float* k_lse = p.chunks > 1 ? scratch + (size_t)p.chunks * p.rows * 128 : lse_out;
  const dim3 grid((unsigned)p.ctas, (unsigned)p.chunks);
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  if (p.persistent && status_word && scratch && scratch_bytes >= kPfPersistBytes) {
    constexpr int smem_pipe = 1024 + 2 * kPfTileBytes + 2 * kPfStages * kPfSubTile + (2 * kPfRows / 32) * kPfStageBytes;
    auto kern = prefix_attention_persistent_kernel<G, SW>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_pipe) != cudaSuccess)
      return L2KV_ERR_CUDA;
    char* sc = reinterpret_cast<char*>(scratch);
    float* part_lse = reinterpret_cast<float*>(sc);
    float* part_out = reinterpret_cast<float*>(sc + kPfPartLseBytes);
    kern<<<kPfPersistCtas, kPfPipeThreads, smem_pipe, s>>>(qb, g, n_queries, cur_len_dev, max_len,
                                                          scale * kPfLog2e, out, lse_out, map_k, map_v,
                                                          status_word, part_out, part_lse, causal);
    return cudaGetLastError() == cudaSuccess ? L2KV_OK : L2KV_ERR_CUDA;
  }
  if (!p.basic) {
    constexpr int smem_pipe = 1024 + 2 * kPfTileBytes + 2 * kPfStages * kPfSubTile + (2 * kPfRows / 32) * kPfStageBytes;
    auto kern_pipe = prefix_attention_pipelined_kernel<G, SW>;
    if (cudaFuncSetAttribute(kern_pipe, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_pipe) != cudaSuccess)
      return L2KV_ERR_CUDA;
    kern_pipe<<<grid, kPfPipeThreads, smem_pipe, s>>>(qb, g, n_queries, cur_len_dev, max_len,
                                                      scale * kPfLog2e, k_out, k_lse, map_k, map_v,
                                                      status_word, p.split_len, p.rows, causal);
  } else {
    constexpr int smem_bytes = 1024 + 3 * kPfTileBytes;
    auto kern = prefix_attention_basic_kernel<G, SW>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess)
      return L2KV_ERR_CUDA;
    kern<<<grid, kPfThreads, smem_bytes, s>>>(qb, g, n_queries, cur_len_dev, max_len, scale * kPfLog2e,
                                              k_out, k_lse, map_k, map_v, status_word, p.split_len,
                                              p.rows, causal);
  }
  if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  if (p.chunks > 1) {
    if (p.rows > 0x7fffffffLL) return L2KV_ERR_OUT_OF_RANGE;
    prefix_merge_kernel<<<(unsigned)p.rows, 128, 0, s>>>(k_out, k_lse, cur_len_dev, max_len, g,
                                                         g.H, g.Hq, n_queries, p.split_len, p.rows,
                                                         out, lse_out, status_word);
    if (cudaGetLastError() != cudaSuccess) return L2KV_ERR_CUDA;
  }
  return L2KV_OK;
}

int launch_prefix_attention(const void* q, const void* K, const void* V, const Geom& g, int dtype,
                            int n_queries, const LenView& cur_len_dev, int max_len, float scale,
                            float* out, float* lse_out, int32_t* status_word, float* scratch,
                            size_t scratch_bytes, int causal, int split_weights, cudaStream_t s) {
  if (dtype != L2KV_BF16 || g.D != 128) return L2KV_ERR_UNSUPPORTED;
#define L2KV_PF(G)                                                                              \
  return split_weights                                                                          \
      ? launch_pf<G, true>(q, K, V, g, n_queries, cur_len_dev, max_len, scale, out, lse_out,    \
                           status_word, scratch, scratch_bytes, causal, s)                      \
      : launch_pf<G, false>(q, K, V, g, n_queries, cur_len_dev, max_len, scale, out, lse_out,   \
                            status_word, scratch, scratch_bytes, causal, s)
  switch (g.Hq / g.H) {
    case 1: L2KV_PF(1);
    case 2: L2KV_PF(2);
    case 4: L2KV_PF(4);
    case 8: L2KV_PF(8);
  }
#undef L2KV_PF
  return L2KV_ERR_UNSUPPORTED;
}

}  // namespace l2kv

// CPU oracle for L2-norm KV-cache compression and single-query decode attention.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
// GPU library must compute.  It shares no code with the CUDA path, is never
// called by it, and may be used only by the tests, the smoke check and the
// CPU-baseline leg of the benchmark.
//
// Every routine is the definition written out:
//   * key norm        -- the paper's compression criterion, the L2 norm of each
//                        cached key embedding (Abstract; Section 1; Section 3).
//                        The ordering key is the sum of squares, which orders
//                        tokens exactly as the norm does.
//   * selection       -- "keep only the keys with the lowest L2 norm, and the
//                        corresponding values" (Section 1), per layer and head
//                        as the dropped set D_{l,h} of Eq. 5 is indexed
//                        (Section 3): a full stable sort.
//   * compaction      -- byte copies of the kept rows, in position order.
//   * skipped layers  -- the listed layers are left uncompressed (Section 3,
//                        last paragraph; Section 4, default = first two).
//   * attention       -- Eq. 2 applied to the cached keys and values as in
//                        Eq. 4, one query per head: softmax(q K^T / sqrt(d_k)) V,
//                        two passes, fp64.
//   * append / evict  -- "let the KV cache grow until a pre-defined length and
//                        subsequently discard the tokens with the highest L2
//                        norm" (Section 4, Language Modelling).
//
// Readings of points the paper leaves open (ties, rounding of keep counts,
// slot reuse after eviction, ...) are listed beside each routine.
//
// Parity pins (tests, CPU only): brute-force enumeration on tiny inputs, closed
// forms for norms, selection invariants, keep-all == plain attention, one-token
// cache, equal keys -> mean of V, shift invariance, and streaming top-k ==
// one-shot selection.  The *quality* of the heuristic on real models (the
// paper's accuracy figures) needs weights and datasets: parity unpinned, and
// out of scope.
//
// Layout: a cache tensor is dense [B, L, H, T_cap, D] with D contiguous, or, in the
// *_packed routines, packed [H, total_rows, D]: the rows of (b, l) are the range
// [row_off[b, l], row_off[b, l] + row_cap[b, l]) of a row axis that all sequences and
// layers share, the same range for every head (ragged batches without padding; only
// where rows live changes, never what is computed -- pinned against the dense form).
// dtype 0 = IEEE fp32, dtype 1 = bfloat16 stored as raw uint16.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <thread>
#include <vector>

namespace {

constexpr int kF32 = 0;
constexpr int kBF16 = 1;

inline int elem_size(int dtype) { return dtype == kBF16 ? 2 : 4; }

// bfloat16 is the upper half of an fp32 bit pattern: widening is exact.
inline float bf16_to_float(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

inline float load_elem_f32(const void* base, int dtype, int64_t i) {
  if (dtype == kBF16) return bf16_to_float(static_cast<const uint16_t*>(base)[i]);
  return static_cast<const float*>(base)[i];
}

inline double load_elem(const void* base, int dtype, int64_t i) {
  return static_cast<double>(load_elem_f32(base, dtype, i));
}

// Sum of squares of one row, fp64, elements taken in index order.
double row_sumsq_f64(const void* K, int dtype, int64_t row_off, int D) {
  double s = 0.0;
  for (int d = 0; d < D; ++d) {
    const double x = load_elem(K, dtype, row_off + d);
    s += x * x;
  }
  return s;
}

// Sum of squares of one row in single precision, in the summation order the
// GPU library documents for its ordering key, so that the keep/evict decision
// can also be compared with no tolerance band at all:
//   * the row is cut into 16-byte pieces (8 bf16 or 4 fp32 elements);
//   * each piece is summed front to back with fused multiply-adds,
//     acc = fma(x, x, acc), starting from 0;
//   * the P piece sums are combined by a butterfly: for off = P/2, P/4, .., 1
//     every p[i] becomes p[i] + p[i ^ off]; the result is p[0].
float row_sumsq_f32_ordered(const void* K, int dtype, int64_t row_off, int D) {
  const int per_piece = 16 / elem_size(dtype);
  const int P = D / per_piece;
  std::vector<float> p(P), nxt(P);
  for (int i = 0; i < P; ++i) {
    float acc = 0.0f;
    for (int e = 0; e < per_piece; ++e) {
      const float x = load_elem_f32(K, dtype, row_off + int64_t(i) * per_piece + e);
      acc = std::fmaf(x, x, acc);
    }
    p[i] = acc;
  }
  for (int off = P / 2; off >= 1; off /= 2) {
    for (int i = 0; i < P; ++i) nxt[i] = p[i] + p[i ^ off];
    p.swap(nxt);
  }
  return p[0];
}

inline double row_key(const void* K, int dtype, int64_t row_off, int D, int key_mode) {
  if (key_mode == 1) return static_cast<double>(row_sumsq_f32_ordered(K, dtype, row_off, D));
  return row_sumsq_f64(K, dtype, row_off, D);
}

// The `keep` positions with the smallest key; equal keys go to the lower
// position (reading: the paper does not say how ties break).  policy 0 keeps
// the lowest norms (the method); policy 1 keeps the highest (the paper's
// ablation), ties again to the lower position.  Result sorted by position.
void select_positions(const double* key, int T, int keep, int policy, int32_t* out) {
  std::vector<int32_t> order(T);
  std::iota(order.begin(), order.end(), 0);
  if (policy == 0) {
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return key[a] < key[b]; });
  } else {
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return key[a] > key[b]; });
  }
  std::vector<int32_t> kept(order.begin(), order.begin() + keep);
  std::sort(kept.begin(), kept.end());
  std::copy(kept.begin(), kept.end(), out);
}

// Ordering key of the keep-random ablation (Section 4: "keeping random tokens"), made
// reproducible: the upper 32 bits of the SplitMix64 output function (Steele, Lea, Flood,
// "Fast splittable pseudorandom number generators", 2014) for the state
// seed + (unit * 2^32 + t), all arithmetic modulo 2^64.
uint32_t random_key(uint64_t seed, uint64_t unit, uint32_t t) {
  uint64_t z = seed + (unit * 4294967296ull + t);
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  z = z ^ (z >> 31);
  return static_cast<uint32_t>(z >> 32);
}

bool in_list(const int32_t* list, int n, int v) {
  for (int i = 0; i < n; ++i)
    if (list[i] == v) return true;
  return false;
}

// Run fn(unit) for unit in [0, n) on `nthreads` threads (units are independent).
template <class F>
void for_each_unit(int64_t n, int nthreads, F fn) {
  if (nthreads <= 1) {
    for (int64_t u = 0; u < n; ++u) fn(u);
    return;
  }
  std::vector<std::thread> pool;
  for (int w = 0; w < nthreads; ++w) {
    pool.emplace_back([=]() {
      for (int64_t u = w; u < n; u += nthreads) fn(u);
    });
  }
  for (auto& t : pool) t.join();
}

// Where the rows of unit u = (b * L + l) * H + h live on the row axis of a cache tensor
// (and of the per-row index map and keys, which have the same row axis).
struct Rows {
  int H;
  int64_t T_cap;              // dense: rows per unit
  const int64_t* row_off;     // packed: [B * L] first row of (b, l); null = dense
  const int32_t* row_cap;     // packed: [B * L] rows (b, l) may hold
  int64_t total_rows;         // packed: extent of the shared row axis
  int64_t first(int64_t u) const {
    return row_off ? (u % H) * total_rows + row_off[u / H] : u * T_cap;
  }
  int64_t cap(int64_t u) const { return row_off ? row_cap[u / H] : T_cap; }
};

Rows dense_rows(int H, int64_t T_cap) { return Rows{H, T_cap, nullptr, nullptr, 0}; }
Rows packed_rows(int H, const int64_t* off, const int32_t* cap, int64_t total) {
  return Rows{H, 0, off, cap, total};
}

int compress_impl(const void* K, const void* V, int dtype, int B, int L, int H, Rows rin, int D,
                  const int32_t* len, const int32_t* keep, const int32_t* uncompressed, int n_unc,
                  int key_mode, int policy, uint64_t seed, Rows rout, void* K_out, void* V_out,
                  int32_t* idx_out, double* key_out, int32_t* kept_len, const int32_t* keep_unit,
                  int32_t* kept_len_unit, int nthreads);
int attention_impl(const void* q, const void* K_c, const void* V_c, int dtype, int B, int L, int Hkv,
                   int Hq, Rows rows, int D, const int32_t* cur_len, double scale, double* out,
                   const int32_t* cur_len_unit, int nthreads);
int append_evict_impl(void* K_c, void* V_c, int32_t* idx, double* key_c, int dtype, int B, int L,
                      int H, Rows rows, int D, int32_t* cur_len, const int32_t* budget,
                      const int32_t* uncompressed, int n_unc, const void* k_new, const void* v_new,
                      const int32_t* pos_new, int key_mode, int per_head);

}  // namespace

extern "C" {

int l2kv_oracle_hardware_threads() {
  const unsigned n = std::thread::hardware_concurrency();
  return n == 0 ? 1 : static_cast<int>(n);
}

// a1: sum of squares (fp64) of n_rows rows of D elements.
void l2kv_oracle_key_sumsq(const void* K, int dtype, int64_t n_rows, int D, double* sumsq) {
  for (int64_t r = 0; r < n_rows; ++r) sumsq[r] = row_sumsq_f64(K, dtype, r * D, D);
}

// a1 in the GPU library's documented single-precision order (see above).
void l2kv_oracle_key_sumsq_f32(const void* K, int dtype, int64_t n_rows, int D, float* sumsq) {
  for (int64_t r = 0; r < n_rows; ++r) sumsq[r] = row_sumsq_f32_ordered(K, dtype, r * D, D);
}

uint32_t l2kv_oracle_random_key(uint64_t seed, uint64_t unit, uint32_t t) {
  return random_key(seed, unit, t);
}

// a2 on a bare key array.
void l2kv_oracle_select(const double* key, int T, int keep, int policy, int32_t* idx_out) {
  select_positions(key, T, keep, policy, idx_out);
}

// Reading (rounding of a keep ratio): keep = ceil(ratio * len), clamped to
// [1, len]; the paper quotes ratios only.
int32_t l2kv_oracle_keep_count(int32_t len, double keep_ratio) {
  if (len <= 0) return 0;
  double k = std::ceil(keep_ratio * static_cast<double>(len));
  if (k < 1.0) k = 1.0;
  if (k > len) k = len;
  return static_cast<int32_t>(k);
}

// a1-a4: compress a whole cache.
//   K, V        [B, L, H, T_cap, D]
//   len[b]      valid tokens of sequence b; keep[b] tokens kept per head in
//               every compressed layer (the paper uses one ratio for all heads)
//   uncompressed[0..n_unc)  layers copied whole (kept_len = len, identity map)
//   key_mode    0: fp64 sums (the definition); 1: the GPU's fp32 order
//   policy      0: keep the lowest norms (the method); 1: keep the highest; 2: keep the
//               lowest seeded random keys of unit (b * L + l) * H + h (`seed`)
//   outputs     K_out, V_out [B, L, H, T_cap_out, D] (rows >= kept_len untouched),
//               idx_out int32, key_out double [B, L, H, T_cap_out], kept_len [B, L]
//   keep_unit   optional [B, L, H]: a keep count of its own for every head (the per-head
//               ratios that the paper's discussion of future work names); it replaces
//               keep[b] in compressed layers, and kept_len_unit [B, L, H] then receives
//               every unit's length (kept_len holds head 0's)
// Returns 0, or -1 if an argument is out of range.
int l2kv_oracle_compress(const void* K, const void* V, int dtype, int B, int L, int H, int T_cap,
                         int D, const int32_t* len, const int32_t* keep,
                         const int32_t* uncompressed, int n_unc, int key_mode, int policy,
                         uint64_t seed, int T_cap_out, void* K_out, void* V_out, int32_t* idx_out,
                         double* key_out, int32_t* kept_len, const int32_t* keep_unit,
                         int32_t* kept_len_unit, int nthreads) {
  return compress_impl(K, V, dtype, B, L, H, dense_rows(H, T_cap), D, len, keep, uncompressed, n_unc,
                       key_mode, policy, seed, dense_rows(H, T_cap_out), K_out, V_out, idx_out,
                       key_out, kept_len, keep_unit, kept_len_unit, nthreads);
}

// The same on packed tensors: K, V [H, total_in, D] with rows (in_off, in_cap); K_out, V_out
// [H, total_out, D], idx_out / key_out [H, total_out] with rows (out_off, out_cap).
int l2kv_oracle_compress_packed(const void* K, const void* V, int dtype, int B, int L, int H,
                                const int64_t* in_off, const int32_t* in_cap, int64_t total_in, int D,
                                const int32_t* len, const int32_t* keep, const int32_t* uncompressed,
                                int n_unc, int key_mode, int policy, uint64_t seed,
                                const int64_t* out_off, const int32_t* out_cap, int64_t total_out,
                                void* K_out, void* V_out, int32_t* idx_out, double* key_out,
                                int32_t* kept_len, const int32_t* keep_unit, int32_t* kept_len_unit,
                                int nthreads) {
  return compress_impl(K, V, dtype, B, L, H, packed_rows(H, in_off, in_cap, total_in), D, len, keep,
                       uncompressed, n_unc, key_mode, policy, seed,
                       packed_rows(H, out_off, out_cap, total_out), K_out, V_out, idx_out, key_out,
                       kept_len, keep_unit, kept_len_unit, nthreads);
}

}  // extern "C"

namespace {

int compress_impl(const void* K, const void* V, int dtype, int B, int L, int H, Rows rin, int D,
                  const int32_t* len, const int32_t* keep, const int32_t* uncompressed, int n_unc,
                  int key_mode, int policy, uint64_t seed, Rows rout, void* K_out, void* V_out,
                  int32_t* idx_out, double* key_out, int32_t* kept_len, const int32_t* keep_unit,
                  int32_t* kept_len_unit, int nthreads) {
  if (keep_unit != nullptr && kept_len_unit == nullptr) return -1;
  for (int b = 0; b < B; ++b) {
    if (len[b] < 0) return -1;
    if (keep_unit == nullptr && (keep[b] < 0 || keep[b] > len[b])) return -1;
    for (int64_t u = int64_t(b) * L * H; u < int64_t(b + 1) * L * H; ++u) {
      const int l = static_cast<int>((u / H) % L);
      if (len[b] > rin.cap(u)) return -1;
      if (keep_unit != nullptr && (keep_unit[u] < 0 || keep_unit[u] > len[b])) return -1;
      const int n_out = in_list(uncompressed, n_unc, l) ? len[b]
                        : keep_unit != nullptr          ? keep_unit[u]
                                                        : keep[b];
      if (n_out > rout.cap(u)) return -1;
    }
  }
  const int es = elem_size(dtype);
  std::vector<int32_t> unit_keep_store(size_t(B) * L * H);
  int32_t* unit_keep = unit_keep_store.data();
  for (int b = 0; b < B; ++b)
    for (int l = 0; l < L; ++l)
      for (int h = 0; h < H; ++h) {
        const int64_t u = (int64_t(b) * L + l) * H + h;
        unit_keep[u] = in_list(uncompressed, n_unc, l) ? len[b]
                       : keep_unit != nullptr          ? keep_unit[u]
                                                       : keep[b];
        if (kept_len_unit != nullptr) kept_len_unit[u] = unit_keep[u];
        if (h == 0) kept_len[b * L + l] = unit_keep[u];
      }

  for_each_unit(int64_t(B) * L * H, nthreads, [=](int64_t u) {
    const int b = static_cast<int>(u / (int64_t(L) * H));
    const int l = static_cast<int>((u / H) % L);
    const int T = len[b];
    const int n_keep = unit_keep[u];
    const int64_t in_row0 = rin.first(u);     // first row of this unit, in rows
    const int64_t out_row0 = rout.first(u);
    std::vector<double> key(T);
    for (int t = 0; t < T; ++t) key[t] = row_key(K, dtype, (in_row0 + t) * D, D, key_mode);
    std::vector<int32_t> kept(n_keep);
    if (in_list(uncompressed, n_unc, l)) {
      std::iota(kept.begin(), kept.end(), 0);
    } else if (n_keep > 0 && policy == 2) {
      std::vector<double> rnd(T);
      for (int t = 0; t < T; ++t) rnd[t] = static_cast<double>(random_key(seed, uint64_t(u), uint32_t(t)));
      select_positions(rnd.data(), T, n_keep, 0, kept.data());
    } else if (n_keep > 0) {
      select_positions(key.data(), T, n_keep, policy, kept.data());
    }
    const size_t row_bytes = size_t(D) * es;
    for (int j = 0; j < n_keep; ++j) {
      const int64_t src = (in_row0 + kept[j]) * int64_t(row_bytes);
      const int64_t dst = (out_row0 + j) * int64_t(row_bytes);
      std::memcpy(static_cast<char*>(K_out) + dst, static_cast<const char*>(K) + src, row_bytes);
      std::memcpy(static_cast<char*>(V_out) + dst, static_cast<const char*>(V) + src, row_bytes);
      idx_out[out_row0 + j] = kept[j];
      key_out[out_row0 + j] = key[kept[j]];
    }
  });
  return 0;
}

}  // namespace

extern "C" {

// a5: one query per query head over the cached rows [0, cur_len[b, l]).
//   q [B, L, Hq, D]; K_c, V_c [B, L, Hkv, T_cap, D]; out double [B, L, Hq, D]
// Query head j reads KV head j / (Hq / Hkv) (reading: contiguous grouping; the
// paper cites grouped-query attention without giving the mapping).  No mask:
// a decode query sees every cached entry (Eq. 4).  scale <= 0 means
// 1 / sqrt(D) (Eq. 2).  An empty cache gives zeros (reading).  cur_len_unit, when not
// null, is [B, L, Hkv] and replaces cur_len (caches compressed with per-head keep counts).
int l2kv_oracle_attention(const void* q, const void* K_c, const void* V_c, int dtype, int B, int L,
                          int Hkv, int Hq, int T_cap, int D, const int32_t* cur_len, double scale,
                          double* out, const int32_t* cur_len_unit, int nthreads) {
  return attention_impl(q, K_c, V_c, dtype, B, L, Hkv, Hq, dense_rows(Hkv, T_cap), D, cur_len, scale,
                        out, cur_len_unit, nthreads);
}

// The same over a packed cache: K_c, V_c [Hkv, total_rows, D] with rows (row_off, row_cap).
int l2kv_oracle_attention_packed(const void* q, const void* K_c, const void* V_c, int dtype, int B,
                                 int L, int Hkv, int Hq, const int64_t* row_off,
                                 const int32_t* row_cap, int64_t total_rows, int D,
                                 const int32_t* cur_len, double scale, double* out,
                                 const int32_t* cur_len_unit, int nthreads) {
  return attention_impl(q, K_c, V_c, dtype, B, L, Hkv, Hq,
                        packed_rows(Hkv, row_off, row_cap, total_rows), D, cur_len, scale, out,
                        cur_len_unit, nthreads);
}

}  // extern "C"

namespace {

int attention_impl(const void* q, const void* K_c, const void* V_c, int dtype, int B, int L, int Hkv,
                   int Hq, Rows rows, int D, const int32_t* cur_len, double scale, double* out,
                   const int32_t* cur_len_unit, int nthreads) {
  if (Hkv <= 0 || Hq % Hkv != 0) return -1;
  const int G = Hq / Hkv;
  const double sc = scale > 0.0 ? scale : 1.0 / std::sqrt(static_cast<double>(D));
  for_each_unit(int64_t(B) * L * Hq, nthreads, [=](int64_t u) {
    const int hq = static_cast<int>(u % Hq);
    const int64_t bl = u / Hq;
    const int n = cur_len_unit != nullptr ? cur_len_unit[bl * Hkv + hq / G] : cur_len[bl];
    const int64_t kv_row0 = rows.first(bl * Hkv + hq / G);
    double* o = out + u * D;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    if (n <= 0) return;
    std::vector<double> z(n);
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
      double dot = 0.0;
      for (int d = 0; d < D; ++d)
        dot += load_elem(q, dtype, u * D + d) * load_elem(K_c, dtype, (kv_row0 + j) * D + d);
      z[j] = dot * sc;
      m = std::max(m, z[j]);
    }
    double denom = 0.0;
    for (int j = 0; j < n; ++j) {
      z[j] = std::exp(z[j] - m);
      denom += z[j];
    }
    for (int j = 0; j < n; ++j) {
      const double p = z[j] / denom;
      for (int d = 0; d < D; ++d) o[d] += p * load_elem(V_c, dtype, (kv_row0 + j) * D + d);
    }
  });
  return 0;
}

}  // namespace

extern "C" {

// Attention loss of the norm-based compression against the ideal one (Section 3, Eqs. 5-7),
// for one query per query head over the cached keys [0, cur_len[b, l]):
//   a_p        = softmax_p(scale * q . k_p)                                   (Eq. 2)
//   L^m        = sum of a_p over the m tokens the method drops first, i.e. the m largest in
//                the order (key, position)                                     (Eq. 5)
//   L^{m,ref}  = sum of the m smallest a_p (the ideal compression drops the lowest scores)
//   Y^m        = L^m - L^{m,ref},   Y = sum_{m=1..n} Y^m                      (Eqs. 6, 7)
// Outputs: alr [B, L, Hq]; optional curves loss / loss_ref [B, L, Hq, T_cap] with L^m at
// index m - 1 (entries at and beyond n untouched).  key_mode as in compression.
int l2kv_oracle_attention_loss(const void* q, const void* K, int dtype, int B, int L, int Hkv,
                               int Hq, int T_cap, int D, const int32_t* cur_len, double scale,
                               int key_mode, double* alr, double* loss, double* loss_ref,
                               int nthreads) {
  if (Hkv <= 0 || Hq % Hkv != 0) return -1;
  const int G = Hq / Hkv;
  const double sc = scale > 0.0 ? scale : 1.0 / std::sqrt(static_cast<double>(D));
  for_each_unit(int64_t(B) * L * Hq, nthreads, [=](int64_t u) {
    const int hq = static_cast<int>(u % Hq);
    const int64_t bl = u / Hq;
    const int n = cur_len[bl];
    const int64_t kv_row0 = (bl * Hkv + hq / G) * T_cap;
    alr[u] = 0.0;
    if (n <= 0) return;
    std::vector<double> a(n), key(n);
    double m = -INFINITY;
    for (int p = 0; p < n; ++p) {
      double dot = 0.0;
      for (int d = 0; d < D; ++d)
        dot += load_elem(q, dtype, u * D + d) * load_elem(K, dtype, (kv_row0 + p) * D + d);
      a[p] = dot * sc;
      m = std::max(m, a[p]);
      key[p] = row_key(K, dtype, (kv_row0 + p) * D, D, key_mode);
    }
    double denom = 0.0;
    for (int p = 0; p < n; ++p) { a[p] = std::exp(a[p] - m); denom += a[p]; }
    for (int p = 0; p < n; ++p) a[p] /= denom;
    // drop order of the method: largest (key, position) first
    std::vector<int32_t> by_norm(n);
    std::iota(by_norm.begin(), by_norm.end(), 0);
    std::sort(by_norm.begin(), by_norm.end(), [&](int32_t x, int32_t y) {
      return key[x] > key[y] || (key[x] == key[y] && x > y);
    });
    std::vector<double> asc(a);
    std::sort(asc.begin(), asc.end());
    double lm = 0.0, lref = 0.0, y = 0.0;
    for (int i = 0; i < n; ++i) {
      lm += a[by_norm[i]];
      lref += asc[i];
      y += lm - lref;
      if (loss) loss[u * T_cap + i] = lm;
      if (loss_ref) loss_ref[u * T_cap + i] = lref;
    }
    alr[u] = y;
  });
  return 0;
}

// a6: append one token per (b, l, h); over budget, evict the highest norm.
//   K_c, V_c [B, L, H, T_cap, D], idx [B, L, H, T_cap], key_c double (same
//   shape), cur_len [B, L] in/out, budget[b], k_new / v_new [B, L, H, D],
//   pos_new[b] = original position of the new token.
// Readings: (i) the new token competes like any other -- if it has the highest
// norm it is the one dropped; (ii) among equal norms the highest position goes
// first (the mirror of keeping the lower position); (iii) the new row takes the
// evicted slot, so the cache stays dense but is no longer position-ordered and
// idx carries the original positions; (iv) uncompressed layers only append.
// Returns 0, or -2 if a row would not fit T_cap (nothing is written for it).
int l2kv_oracle_append_evict(void* K_c, void* V_c, int32_t* idx, double* key_c, int dtype, int B,
                             int L, int H, int T_cap, int D, int32_t* cur_len,
                             const int32_t* budget, const int32_t* uncompressed, int n_unc,
                             const void* k_new, const void* v_new, const int32_t* pos_new,
                             int key_mode, int per_head) {
  return append_evict_impl(K_c, V_c, idx, key_c, dtype, B, L, H, dense_rows(H, T_cap), D, cur_len,
                           budget, uncompressed, n_unc, k_new, v_new, pos_new, key_mode, per_head);
}

// The same on a packed cache: K_c, V_c [H, total_rows, D], idx / key_c [H, total_rows] with rows
// (row_off, row_cap); a row that would not fit row_cap[b, l] is the overflow case.
int l2kv_oracle_append_evict_packed(void* K_c, void* V_c, int32_t* idx, double* key_c, int dtype,
                                    int B, int L, int H, const int64_t* row_off,
                                    const int32_t* row_cap, int64_t total_rows, int D,
                                    int32_t* cur_len, const int32_t* budget,
                                    const int32_t* uncompressed, int n_unc, const void* k_new,
                                    const void* v_new, const int32_t* pos_new, int key_mode,
                                    int per_head) {
  return append_evict_impl(K_c, V_c, idx, key_c, dtype, B, L, H,
                           packed_rows(H, row_off, row_cap, total_rows), D, cur_len, budget,
                           uncompressed, n_unc, k_new, v_new, pos_new, key_mode, per_head);
}

}  // extern "C"

namespace {

int append_evict_impl(void* K_c, void* V_c, int32_t* idx, double* key_c, int dtype, int B, int L,
                      int H, Rows rows, int D, int32_t* cur_len, const int32_t* budget,
                      const int32_t* uncompressed, int n_unc, const void* k_new, const void* v_new,
                      const int32_t* pos_new, int key_mode, int per_head) {
  // per_head != 0: cur_len and budget are [B, L, H] (caches compressed with a keep count per
  // head); otherwise cur_len is [B, L] and budget [B].
  const size_t row_bytes = size_t(D) * elem_size(dtype);
  int status = 0;
  for (int b = 0; b < B; ++b) {
    for (int l = 0; l < L; ++l) {
      bool any_grow = false;
      const int n_shared = per_head ? 0 : cur_len[b * L + l];
      for (int h = 0; h < H; ++h) {
        const int64_t u = (int64_t(b) * L + l) * H + h;
        const int n = per_head ? cur_len[u] : n_shared;
        const int cap = per_head ? budget[u] : budget[b];
        const bool grow = in_list(uncompressed, n_unc, l) || n < cap;
        const int64_t row0 = rows.first(u);
        if (grow && n >= rows.cap(u)) {
          status = -2;
          continue;
        }
        const double s_new = row_key(k_new, dtype, u * D, D, key_mode);
        int slot;
        if (grow) {
          slot = n;
          any_grow = true;
          if (per_head) cur_len[u] = n + 1;
        } else {
          // arg-max of (key, position) over the stored entries and the new one
          slot = -1;  // -1 = the new token itself
          double best = s_new;
          int32_t best_pos = pos_new[b];
          for (int j = 0; j < n; ++j) {
            const double s = key_c[row0 + j];
            const int32_t p = idx[row0 + j];
            if (s > best || (s == best && p > best_pos)) {
              best = s;
              best_pos = p;
              slot = j;
            }
          }
          if (slot < 0) continue;  // the new token is the one discarded
        }
        const int64_t dst = (row0 + slot) * int64_t(row_bytes);
        std::memcpy(static_cast<char*>(K_c) + dst,
                    static_cast<const char*>(k_new) + u * int64_t(row_bytes), row_bytes);
        std::memcpy(static_cast<char*>(V_c) + dst,
                    static_cast<const char*>(v_new) + u * int64_t(row_bytes), row_bytes);
        idx[row0 + slot] = pos_new[b];
        key_c[row0 + slot] = s_new;
      }
      if (!per_head && any_grow) cur_len[b * L + l] = n_shared + 1;
    }
  }
  return status;
}

}  // namespace

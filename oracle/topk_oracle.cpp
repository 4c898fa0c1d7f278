// CPU oracle for exact ragged Top-K (test infrastructure; not part of the product).
//
// Two independent selectors over the same ordering:
//   oracle_topk_stable_sort  - the plain definition: std::stable_sort of a row's
//                              indices by descending key, first min(K, L) kept.
//   oracle_topk_nth_element  - std::nth_element with the strict total order
//                              (key descending, index ascending); used to pin
//                              the first one and as an O(L) CPU baseline.
// Ordering (operator contract, Section 2.1, with ties resolved to the lower
// index and -0.0 placed below +0.0): the monotone key on the raw bit pattern.
// Rows are independent, so an OpenMP loop over rows is the only parallelism.
//
// Shares no code with the CUDA library.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <numeric>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline uint32_t bits_of(float x) {
  uint32_t u;
  std::memcpy(&u, &x, sizeof u);
  return u;
}

// larger score <=> larger key
inline uint32_t key_ascending(uint32_t u) {
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

const uint32_t kNegInfBits = 0xFF800000u;

void fill_row(const float* row, int64_t L, int32_t K, const std::vector<int32_t>& best,
              int32_t* out_idx, float* out_val) {
  const int64_t m = std::min<int64_t>(K, L);
  for (int64_t j = 0; j < m; ++j) {
    out_idx[j] = best[j];
    if (out_val) out_val[j] = row[best[j]];
  }
  for (int64_t j = m; j < K; ++j) {
    out_idx[j] = -1;
    if (out_val) std::memcpy(&out_val[j], &kNegInfBits, 4);
  }
}

}  // namespace

extern "C" {

int oracle_max_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Definition: stable sort by descending key.  Output best first, then (-1, -inf).
// num_threads <= 0 means "all cores".  Returns the number of threads used.
int oracle_topk_stable_sort(const float* scores, const int32_t* row_starts,
                            const int32_t* row_lengths, int32_t num_rows, int32_t K,
                            int32_t* out_idx, float* out_val, int num_threads) {
  int used = 1;
#ifdef _OPENMP
  if (num_threads <= 0) num_threads = omp_get_max_threads();
  used = num_threads;
#pragma omp parallel for schedule(dynamic, 1) num_threads(num_threads)
#endif
  for (int32_t r = 0; r < num_rows; ++r) {
    const int64_t L = std::max<int32_t>(row_lengths[r], 0);
    const float* row = scores + row_starts[r];
    std::vector<uint32_t> key(L);
    for (int64_t i = 0; i < L; ++i) key[i] = key_ascending(bits_of(row[i]));
    std::vector<int32_t> order(L);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return key[a] > key[b]; });
    fill_row(row, L, K, order, out_idx + (int64_t)r * K,
             out_val ? out_val + (int64_t)r * K : nullptr);
  }
  return used;
}

// Independent selector: nth_element under the strict total order
// (key descending, index ascending), then the first min(K, L) positions
// sorted by that same order so the output is comparable slot by slot.
int oracle_topk_nth_element(const float* scores, const int32_t* row_starts,
                            const int32_t* row_lengths, int32_t num_rows, int32_t K,
                            int32_t* out_idx, float* out_val, int num_threads) {
  int used = 1;
#ifdef _OPENMP
  if (num_threads <= 0) num_threads = omp_get_max_threads();
  used = num_threads;
#pragma omp parallel for schedule(dynamic, 1) num_threads(num_threads)
#endif
  for (int32_t r = 0; r < num_rows; ++r) {
    const int64_t L = std::max<int32_t>(row_lengths[r], 0);
    const float* row = scores + row_starts[r];
    std::vector<int32_t> order(L);
    std::iota(order.begin(), order.end(), 0);
    auto before = [&](int32_t a, int32_t b) {
      const uint32_t ka = key_ascending(bits_of(row[a]));
      const uint32_t kb = key_ascending(bits_of(row[b]));
      return ka != kb ? ka > kb : a < b;
    };
    const int64_t m = std::min<int64_t>(K, L);
    if (m < L) std::nth_element(order.begin(), order.begin() + m, order.end(), before);
    std::sort(order.begin(), order.begin() + m, before);
    fill_row(row, L, K, order, out_idx + (int64_t)r * K,
             out_val ? out_val + (int64_t)r * K : nullptr);
  }
  return used;
}

}  // extern "C"

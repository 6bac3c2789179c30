// Per-row selection of the k_hat largest values with a sorted list in registers (Sec. 3.1 "Grouped
// Top-k Selection", per-query grouping): shared by the stand-alone selection kernel and by the
// estimator's output kernel, which selects straight from the A_hat tile in tensor memory.
#pragma once

#include <stdint.h>

#include <utility>

namespace sea {
namespace select {

// x >= y afterwards when kDescending, x <= y otherwise
template <bool kDescending>
__device__ __forceinline__ void cmp_exchange(float& x, float& y) {
  const float hi = fmaxf(x, y), lo = fminf(x, y);
  x = kDescending ? hi : lo;
  y = kDescending ? lo : hi;
}
// Batcher's odd-even merge sort as a list of compare-exchange pairs built at compile time: 19 pairs
// for 8 values, 63 for 16, 191 for 32 (a bitonic sorter needs 24, 80 and 240).
template <int N>
struct BatcherNet {
  static constexpr int kMax = N * 8;
  int lo[kMax] = {}, hi[kMax] = {};
  int count = 0;
  constexpr BatcherNet() {
    for (int p = 1; p < N; p <<= 1)
      for (int k = p; k >= 1; k >>= 1)
        for (int j = k % p; j <= N - 1 - k; j += 2 * k)
          for (int i = 0; i < k && i <= N - j - k - 1; ++i)
            if ((i + j) / (2 * p) == (i + j + k) / (2 * p)) {
              lo[count] = i + j;
              hi[count] = i + j + k;
              ++count;
            }
  }
};
template <int N, int... I>
__device__ __forceinline__ void apply_net(float (&a)[N], std::integer_sequence<int, I...>) {
  constexpr BatcherNet<N> net{};
  (cmp_exchange<false>(a[net.lo[I]], a[net.hi[I]]), ...);  // every index is a compile-time constant
}
// Ascending sort of N registers (N a power of two).
template <int N>
__device__ __forceinline__ void sort_ascending(float (&a)[N]) {
  constexpr BatcherNet<N> net{};
  apply_net<N>(a, std::make_integer_sequence<int, net.count>{});
}
template <int N>
__device__ __forceinline__ void bitonic_merge_descending(float (&a)[N]) {
#pragma unroll
  for (int j = N >> 1; j > 0; j >>= 1)
#pragma unroll
    for (int i = 0; i < N; ++i) {
      const int l = i ^ j;
      if (l > i) cmp_exchange<true>(a[i], a[l]);
    }
}
// top (descending) <- the KMAX largest of top and grp (any order; destroyed)
template <int KMAX>
__device__ __forceinline__ void merge_group(float (&top)[KMAX], float (&grp)[KMAX]) {
  sort_ascending<KMAX>(grp);
#pragma unroll
  for (int s = 0; s < KMAX; ++s) top[s] = fmaxf(top[s], grp[s]);
  bitonic_merge_descending<KMAX>(top);
}

// One block of 32 columns starting at j0: `gt` marks the columns above the k_hat-th largest value,
// `eq` those equal to it, of which the lowest `ties_left` (over the whole row, in column order) are
// still to be taken.  Appends the selected columns to my_sel (ascending; may be null), adds their keys after
// up-sampling to cnt (column c covers keys c r .. c r + r - 1; a causal row i keeps those <= i) and
// stores the block's word of the bit mask.
__device__ __forceinline__ void emit_columns(uint32_t gt, uint32_t eq, int j0, int& ties_left, int32_t* my_sel, int& out,
                                             int& cnt, uint32_t* bits_word, int i, int r, int causal) {
  uint32_t eq_taken = eq;
  if (__popc(eq) > ties_left) {
    eq_taken = 0u;
    for (int t = 0; t < ties_left; ++t) {
      const uint32_t low = eq & (0u - eq);
      eq_taken |= low;
      eq ^= low;
    }
  }
  ties_left -= __popc(eq_taken);
  uint32_t word = gt | eq_taken;
  if (bits_word != nullptr) *bits_word = word;
  while (word) {
    const int j = j0 + __ffs(word) - 1;
    word &= word - 1u;
    if (my_sel != nullptr) my_sel[out] = j;
    ++out;
    cnt += causal ? max(0, min(r, i + 1 - j * r)) : r;
  }
}

}  // namespace select
}  // namespace sea

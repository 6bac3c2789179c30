// Mask generation: per-row top-k_hat over the compressed estimate (Sec. 3.1 "Grouped Top-k
// Selection", per-query grouping) and nearest-neighbour expansion of the selected columns to
// a flat CSR (Sec. 3.1 "Linear Sparse Attention Mask Generation", App. "Sparse Interpolation").
//
// Selection is exact and unique: every value is mapped to a 32-bit key whose unsigned order
// is the float order (with -0 folded onto +0), the k_hat-th largest key is found by a
// bit-by-bit search with warp-wide counts, and columns holding exactly that key are taken
// in ascending column order until k_hat are chosen.
#include "sea_common.cuh"
#include "sea_select.cuh"

namespace sea {
namespace {

using namespace select;

constexpr int kWarpsPerCta = 8;
constexpr int kScanThreads = 256;
constexpr int kScanPerThread = 8;
constexpr int kScanTile = kScanThreads * kScanPerThread;
constexpr int kThreadMaxKc = 128;  // shapes handled with one thread per row: the sorted-list walk costs
constexpr int kThreadMaxK = 32;    // Kc * k_hat min/max pairs per row, the bit search about 64 * Kc / 32 * 32

constexpr int kHistBins = 256;
constexpr int kHistShift = 17;

// ---- one warp per row ---------------------------------------------------------------------------
// Lane l holds the VPL consecutive columns l * VPL ..., so that column order is lane order and the
// selected columns of a lane can be emitted without looking at the others, after one prefix sum over
// the lanes.  `aware`: a causal row i only chooses among the columns that hold a key j <= i (columns
// 0 .. i / r) and keeps at most as many as there are; sel may be null then (rows keep differing
// numbers of columns).
//
// The row's keys: in registers, or (wide rows, which would need more registers than leave room for
// enough warps) in the warp's part of shared memory, lane l's t-th key at word l (VPL + 1) + t: the
// lanes read their t-th keys from different banks, and the row can be fetched with neighbouring lanes
// on neighbouring 16-byte pieces (a lane that fetched its own VPL columns instead would touch every
// cache line of the row with every load, and the rows of a CTA's warps do not fit the L1 cache).
template <int VPL, bool kShared>
struct RowKeys;
template <int VPL>
struct RowKeys<VPL, false> {
  static constexpr int kSlots = VPL;
  static constexpr bool kDense = true;  // slot t is column col0 + t
  uint32_t k[VPL];
  int col0;
  __device__ __forceinline__ RowKeys(uint32_t*, int first) : col0(first) {}
  __device__ __forceinline__ uint32_t get(int t) const { return k[t]; }
  __device__ __forceinline__ void set(int t, uint32_t v) { k[t] = v; }
};
template <int VPL>
struct RowKeys<VPL, true> {
  static constexpr int kSlots = VPL;
  static constexpr bool kDense = true;
  static constexpr int kStride = VPL + 1;
  uint32_t* base;
  uint32_t* p;
  int col0;
  __device__ __forceinline__ RowKeys(uint32_t* warp_keys, int first)
      : base(warp_keys), p(warp_keys + (threadIdx.x & 31) * kStride), col0(first) {}
  __device__ __forceinline__ uint32_t get(int t) const { return p[t]; }
  __device__ __forceinline__ void set(int t, uint32_t v) { p[t] = v; }
  // the key of column `col`, whichever lane owns it
  __device__ __forceinline__ void put(int col, uint32_t v) { base[(col / VPL) * kStride + (col % VPL)] = v; }
};
struct RowOut {
  int32_t* sel;      // the row's part of sel, or null
  uint32_t* words;   // the row's part of mask_bits, or null
  int n_words;
  int32_t* count;    // the row's entry of row_counts, or null
  int i, r, causal;  // query index inside the sequence, keys per column
};

// Selection of the k_hat largest keys among the slots of all lanes (an empty slot holds key 0, which
// sorts below every real value), ties to the lower column, and the row's outputs.  `hist`: the warp's
// kHistBins words of shared memory.
//
// The k_hat-th largest key tau (the largest tau with |{key >= tau}| >= k_hat) is found from the
// row's largest key `top`, a histogram of (top - key) >> kHistShift over the kHistBins steps below it
// (1/64 of an octave each: four octaves of magnitudes), a scan for the step that holds tau, and a
// search by ballots among the keys inside that step (one per lane); when the step holds more than
// 32 keys, or tau lies below the histogram, bit by bit with warp-wide counts over all keys.
template <typename Keys>
__device__ __forceinline__ void select_row(const Keys& key, int* hist, int lane, int k_hat, const RowOut& out) {
  constexpr int N = Keys::kSlots;
  uint32_t tau = 0u;
  bool found = false;
  {
    uint32_t top = 0u;
#pragma unroll
    for (int t = 0; t < N; ++t) top = max(top, key.get(t));
    top = __reduce_max_sync(0xffffffffu, top);
    // step x is kept at word (x & 7) * 32 + (x >> 3): lane x >> 3 owns it and reads it without conflicts
#pragma unroll
    for (int j = 0; j < kHistBins / 32; ++j) hist[j * 32 + lane] = 0;
    __syncwarp();
#pragma unroll
    for (int t = 0; t < N; ++t) {
      const uint32_t x = (top - key.get(t)) >> kHistShift;
      if (x < (uint32_t)kHistBins && key.get(t) != 0u) atomicAdd(&hist[(x & 7u) * 32u + (x >> 3)], 1);
    }
    __syncwarp();
    int bins[kHistBins / 32], mine = 0;
#pragma unroll
    for (int j = 0; j < kHistBins / 32; ++j) {
      bins[j] = hist[j * 32 + lane];
      mine += bins[j];
    }
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const int total = __shfl_sync(0xffffffffu, inc, 31);
    if (total >= k_hat) {
      int over = inc - mine;  // keys in the steps above this lane's
      const bool owner = over < k_hat && over + mine >= k_hat;
      int step = 0;
      if (owner) {
#pragma unroll
        for (int j = 0; j < kHistBins / 32; ++j)
          if (over + bins[j] < k_hat && step == j) {
            over += bins[j];
            ++step;
          }
        step += lane * (kHistBins / 32);
      }
      const int src = __ffs(__ballot_sync(0xffffffffu, owner)) - 1;
      step = __shfl_sync(0xffffffffu, step, src);
      const int above = __shfl_sync(0xffffffffu, over, src);
      // the keys inside the step, one per lane when there are at most 32
      int inside = 0;
#pragma unroll
      for (int t = 0; t < N; ++t) inside += key.get(t) != 0u && ((top - key.get(t)) >> kHistShift) == (uint32_t)step;  // 0: an empty slot
      int pos = inside;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, pos, o);
        if (lane >= o) pos += v;
      }
      const int n_in = __shfl_sync(0xffffffffu, pos, 31);
      if (n_in <= 32) {
        uint32_t* list = reinterpret_cast<uint32_t*>(hist);  // the counters are no longer needed
        __syncwarp();
        pos -= inside;
        constexpr uint32_t kFine = (1u << kHistShift) - 1u;
#pragma unroll
        for (int t = 0; t < N; ++t) {
          const uint32_t rel = top - key.get(t);
          if (key.get(t) != 0u && (rel >> kHistShift) == (uint32_t)step) list[pos++] = kFine - (rel & kFine);  // grows with the key
        }
        __syncwarp();
        const bool have = lane < n_in;
        const uint32_t fine_mine = have ? list[lane] : 0u;
        uint32_t fine = 0u;
#pragma unroll
        for (int bit = kHistShift - 1; bit >= 0; --bit) {
          const uint32_t cand = fine | (1u << bit);
          if (__popc(__ballot_sync(0xffffffffu, have && fine_mine >= cand)) + above >= k_hat) fine = cand;
        }
        tau = top - (((uint32_t)step << kHistShift) | (kFine - fine));
        found = true;
      }
    }
    __syncwarp();
  }
  if (!found) {
    // bit by bit with warp-wide counts over all keys
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
      const uint32_t cand = tau | (1u << bit);
      int c = 0;
#pragma unroll
      for (int t = 0; t < N; ++t) c += key.get(t) >= cand;
      c = __reduce_add_sync(0xffffffffu, c);
      if (c >= k_hat) tau = cand;
    }
  }
  // per lane: the bits of its slots above tau and equal to it
  uint64_t gt = 0ull, eq = 0ull;
#pragma unroll
  for (int t = 0; t < N; ++t) {
    gt |= (uint64_t)(key.get(t) > tau) << t;
    eq |= (uint64_t)(key.get(t) == tau) << t;
  }
  const int my_gt = __popcll(gt), my_eq = __popcll(eq);
  // inclusive prefix sums over the lanes of (slots above tau, slots equal to it), packed
  int inc = (my_gt << 16) | my_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += v;
  }
  const int tot = __shfl_sync(0xffffffffu, inc, 31);
  const int need = k_hat - (tot >> 16);  // how many columns equal to tau are taken (lowest first)
  // of this lane's equal columns, the first `mine` are taken
  const int eq_before = (inc & 0xffff) - my_eq;
  int mine = min(max(need - eq_before, 0), my_eq);
  uint64_t take = gt;
  for (uint64_t e = eq; mine > 0; --mine) {
    const uint64_t low = e & (0ull - e);
    take |= low;
    e ^= low;
  }
  const int taken_before = (inc >> 16) - my_gt + min(eq_before, max(need, 0));

  int cnt = 0;
  int32_t* my_sel = out.sel != nullptr ? out.sel + taken_before : nullptr;
  {
    for (uint64_t tk = take; tk != 0ull; tk &= tk - 1ull) {
      const int col = key.col0 + __ffsll((long long)tk) - 1;
      if (my_sel != nullptr) *my_sel++ = col;
      cnt += out.causal ? max(0, min(out.r, out.i + 1 - col * out.r)) : out.r;
    }
    if (out.words != nullptr) {
      if constexpr (N >= 32) {
#pragma unroll
        for (int j = 0; j < N / 32; ++j)
          if (lane * (N / 32) + j < out.n_words) out.words[lane * (N / 32) + j] = (uint32_t)(take >> (32 * j));
      } else {
        // 32 / N neighbouring lanes share a word
        constexpr int kLanes = 32 / N;
        uint32_t word = (uint32_t)take << ((lane % kLanes) * N);
#pragma unroll
        for (int o = 1; o < kLanes; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
        if (lane % kLanes == 0 && lane / kLanes < out.n_words) out.words[lane / kLanes] = word;
      }
    }
  }
  if (out.count != nullptr) {
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (lane == 0) *out.count = cnt;
  }
}

// Selection among a short list of candidates (a wide row's entries at or above a lower bound of
// its k_hat-th largest value): `list_key` / `list_col` hold n_c <= kListMax of them in ascending
// column order, at least k_hat.  The smallest keys are struck off, all entries of a value at a
// time, while k_hat would still remain: the value at which that stops is the k_hat-th largest key;
// entries above it are selected, and of those equal to it the first (lowest columns) that are still
// needed.  Lane l looks after entries l, l + 32, l + 64.
constexpr int kListMax = 96;
__device__ __forceinline__ void select_from_list(const uint32_t* list_key, const int* list_col, int n_c, uint32_t* words,
                                                 int lane, int k_hat, const RowOut& out) {
  constexpr uint32_t kGone = 0xffffffffu;  // no finite value has this key
  uint32_t a[3];
  int col[3];
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const int idx = lane + 32 * i;
    a[i] = idx < n_c ? list_key[idx] : kGone;
    col[i] = idx < n_c ? list_col[idx] : 0;
  }
  int remaining = n_c;
  uint32_t tau;
  int ties_needed;
  for (;;) {
    tau = __reduce_min_sync(0xffffffffu, min(a[0], min(a[1], a[2])));
    const int c = __popc(__ballot_sync(0xffffffffu, a[0] == tau)) + __popc(__ballot_sync(0xffffffffu, a[1] == tau)) +
                  __popc(__ballot_sync(0xffffffffu, a[2] == tau));
    if (remaining - c < k_hat) {
      ties_needed = k_hat - (remaining - c);
      break;
    }
    remaining -= c;
#pragma unroll
    for (int i = 0; i < 3; ++i) a[i] = a[i] == tau ? kGone : a[i];
  }
  for (int wv = lane; wv < out.n_words; wv += 32) words[wv] = 0u;
  __syncwarp();
  const uint32_t below = (1u << lane) - 1u;
  int ties_before = 0, taken_before = 0, cnt = 0;
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const bool alive = a[i] != kGone;
    const uint32_t eq = __ballot_sync(0xffffffffu, alive && a[i] == tau);
    const bool take = alive && (a[i] > tau || (a[i] == tau && ties_before + __popc(eq & below) < ties_needed));
    const uint32_t tk = __ballot_sync(0xffffffffu, take);
    if (take) {
      if (out.sel != nullptr) out.sel[taken_before + __popc(tk & below)] = col[i];
      cnt += out.causal ? max(0, min(out.r, out.i + 1 - col[i] * out.r)) : out.r;
      if (out.words != nullptr) atomicOr(&words[col[i] >> 5], 1u << (col[i] & 31));
    }
    ties_before += __popc(eq);
    taken_before += __popc(tk);
  }
  __syncwarp();
  if (out.words != nullptr)
    for (int wv = lane; wv < out.n_words; wv += 32) out.words[wv] = words[wv];
  if (out.count != nullptr) {
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (lane == 0) *out.count = cnt;
  }
}

template <int VPL, bool kShared>
__global__ void __launch_bounds__(kWarpsPerCta * 32, kShared ? 3 : 4)
topk_rows_kernel(const float* __restrict__ A_hat, int32_t* __restrict__ sel,
                 int32_t* __restrict__ row_counts, uint32_t* __restrict__ mask_bits, int rows, int Kc_all, int k_all,
                 int seq_len, int r, int causal, int aware) {
  static_assert(kHistBins >= 64, "the histogram words double as the row's bit words (Kc <= 2048)");
  __shared__ int hist_all[kWarpsPerCta][kHistBins];
  extern __shared__ uint32_t keys_all[];  // [kWarpsPerCta][32 * (VPL + 1)] when kShared
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  const float* a = A_hat + (size_t)row * Kc_all;
  const int Kc = aware ? min(Kc_all, (row % seq_len) / r + 1) : Kc_all;  // columns that compete
  const int k_hat = min(k_all, Kc);
  const int col0 = lane * VPL;  // this lane's first column
  RowKeys<VPL, kShared> key(keys_all + (kShared ? warp * (VPL + 1) * 32 : 0), col0);
  RowOut out;
  out.sel = sel != nullptr ? sel + (size_t)row * k_all : nullptr;
  out.n_words = (Kc_all + 31) / 32;
  out.words = mask_bits != nullptr ? mask_bits + (size_t)row * out.n_words : nullptr;
  out.count = row_counts != nullptr ? row_counts + row : nullptr;
  out.i = row % seq_len;
  out.r = r;
  out.causal = causal;

  if constexpr (kShared) {
    // A wide row first sheds most of its values.  The row is fetched as 16-byte pieces (lane l takes
    // pieces l, l + 32, ...) and parked in the warp's shared memory as it is; while fetching, every
    // lane keeps the two largest values it met.  Those are 64 different entries of the row, so the
    // k_hat-th largest of the 64 (found bit by bit with ballots on their keys) has at least k_hat
    // entries at or above it, and so has any bound L below it: every selected entry is >= L, and few
    // more than k_hat entries are (L = 0 when fewer than k_hat of the 64 hold a column: no shortcut
    // then).  Each lane then reads back its own VPL consecutive columns (piece q sits at q ^ (owner
    // lane & 7): neither the writes nor these reads meet bank conflicts); the entries >= L go, in
    // column order, to a short list and select_from_list finishes the row.
    if (k_hat <= 32 && Kc_all % 4 == 0) {
      constexpr int kPerLane = VPL / 4;  // pieces of a lane's own columns
      static_assert(kPerLane >= 4, "the swizzle needs at least four pieces per lane");
      // where piece q is parked: eight neighbouring pieces, and the j-th pieces of eight neighbouring
      // lanes, fall on eight different 16-byte bank groups
      auto parked = [](int q) { return kPerLane >= 8 ? q ^ ((q / kPerLane) & 7) : q ^ ((q >> 3) & 3); };
      float4* stage = reinterpret_cast<float4*>(keys_all + warp * (VPL + 1) * 32);
      float f1 = -INFINITY, f2 = -INFINITY;  // columns that do not compete count as -inf (inputs are finite)
#pragma unroll 4
      for (int q = lane; q < 8 * VPL; q += 32) {
        float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (4 * q < Kc) v = __ldg(reinterpret_cast<const float4*>(a + 4 * q));
        if (4 * q + 3 >= Kc) {  // the visible part of an aware row need not end on a piece
          if (4 * q + 1 >= Kc) v.y = -INFINITY;
          if (4 * q + 2 >= Kc) v.z = -INFINITY;
          v.w = -INFINITY;
        }
        stage[parked(q)] = v;
        const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          f2 = fmaxf(f2, fminf(f1, x[e]));
          f1 = fmaxf(f1, x[e]);
        }
      }
      const uint32_t top1 = f1 == -INFINITY ? 0u : order_key(f1), top2 = f2 == -INFINITY ? 0u : order_key(f2);
      // (the upper 16 bits of the k_hat-th largest key are bound enough: the values between that and
      // the key itself are a 128th of an octave)
      uint32_t low = 0u;
#pragma unroll 1
      for (int bit = 31; bit >= 16; --bit) {
        const uint32_t c = low | (1u << bit);
        if (__popc(__ballot_sync(0xffffffffu, top1 >= c)) + __popc(__ballot_sync(0xffffffffu, top2 >= c)) >= k_hat) low = c;
      }
      __syncwarp();
      if (low != 0u) {
        // from the key back to the value it stands for
        const float low_f = __uint_as_float((low & 0x80000000u) ? (low ^ 0x80000000u) : ~low);
        uint64_t cand = 0ull;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
          const float4 v = stage[parked(lane * kPerLane + j)];
          cand |= (uint64_t)((v.x >= low_f ? 1u : 0u) | (v.y >= low_f ? 2u : 0u) | (v.z >= low_f ? 4u : 0u) | (v.w >= low_f ? 8u : 0u))
                  << (4 * j);
        }
        // the candidates in column order: lane by lane, each lane's in ascending order
        const int mine = __popcll(cand);
        int inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += v;
        }
        const int n_c = __shfl_sync(0xffffffffu, inc, 31);
        if (n_c <= kListMax) {
          const float* vals = reinterpret_cast<const float*>(stage);
          uint32_t* list_key = reinterpret_cast<uint32_t*>(hist_all[warp]);
          int* list_col = hist_all[warp] + kListMax;
          uint32_t* words = reinterpret_cast<uint32_t*>(hist_all[warp]) + 2 * kListMax;
          static_assert(2 * kListMax + 64 <= kHistBins, "the lists and the row's bit words share the histogram's words");
          int at = inc - mine;
          for (; cand != 0ull; cand &= cand - 1ull, ++at) {
            const int t = __ffsll((long long)cand) - 1;
            list_key[at] = order_key(vals[4 * parked(lane * kPerLane + (t >> 2)) + (t & 3)]);
            list_col[at] = col0 + t;
          }
          __syncwarp();
          select_from_list(list_key, list_col, n_c, words, lane, k_hat, out);
          return;
        }
      }
      __syncwarp();  // the keys below go where the values were
    }
    // every key of the row, lane l's t-th at word l (VPL + 1) + t
    if (Kc_all % 4 == 0) {
#pragma unroll 4
      for (int c = 4 * lane; c < 32 * VPL; c += 128) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < Kc_all) v = __ldg(reinterpret_cast<const float4*>(a + c));
        const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) key.put(c + e, c + e < Kc ? order_key(x[e]) : 0u);  // empty slots sort below every real value
      }
    } else {
      for (int c = lane; c < 32 * VPL; c += 32) key.put(c, c < Kc ? order_key(__ldg(a + c)) : 0u);
    }
    __syncwarp();
  } else if (VPL % 4 == 0 && Kc_all % 4 == 0) {  // rows start on 16-byte boundaries
#pragma unroll
    for (int t = 0; t < VPL; t += 4) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (col0 + t < Kc_all) v = __ldg(reinterpret_cast<const float4*>(a + col0 + t));
      const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) key.set(t + e, col0 + t + e < Kc ? order_key(x[e]) : 0u);  // empty slots sort below every real value
    }
  } else {
#pragma unroll
    for (int t = 0; t < VPL; ++t) key.set(t, col0 + t < Kc ? order_key(__ldg(a + col0 + t)) : 0u);
  }
  select_row(key, hist_all[warp], lane, k_hat, out);
}

// Selection with one thread per row, for short rows and small k_hat: no cross-lane traffic at
// all.  Every thread walks its row (16-byte loads; a row is a few cache lines that the thread
// reads front to back) in groups of KMAX values and keeps the KMAX largest values seen so far as
// a descending list in registers: a group is sorted ascending by an odd-even merge network, the
// element-wise maximum with the list is then a bitonic sequence holding the KMAX largest of
// both, and a bitonic merge sorts it again - all compare-exchanges on fixed registers, no
// branches.  That leaves the k_hat-th largest value tau in the last slot; a second walk over
// the row builds, 32 columns at a time, the bit masks of the columns above tau and equal to it,
// keeps the first k_hat - |{value > tau}| of the equal ones, and emits the set bits in ascending
// column order: the same set as the bit search below, ties going to the lower column.  The walk
// works on the floats themselves: inputs are finite, and the float comparisons treat -0 and +0
// as equal exactly as the bit search's keys do.
constexpr int kThreadRows = 128;  // threads (= rows) per CTA

template <int KMAX, bool kVec, bool kAware>
__global__ void __launch_bounds__(kThreadRows)
topk_rows_thread_kernel(const float* __restrict__ A_hat, int32_t* __restrict__ sel,
                        int32_t* __restrict__ row_counts, uint32_t* __restrict__ mask_bits, int rows, int Kc_all,
                        int k_all, int seq_len, int r, int causal) {
  const int row = blockIdx.x * kThreadRows + threadIdx.x;
  if (row >= rows) return;
  const float* a = A_hat + (size_t)row * Kc_all;
  const int i = row % seq_len;
  // kAware: only the columns that hold a key j <= i compete, and at most as many are kept
  const int Kc = kAware ? min(Kc_all, i / r + 1) : Kc_all;
  const int k_hat = min(k_all, Kc);
  // Descending list.  Its first KMAX - k_hat slots hold +inf, above every (finite) value, so the
  // k_hat-th largest value of the row always ends up in the last slot; -inf stands for columns
  // beyond the row.
  float top[KMAX];
#pragma unroll
  for (int s = 0; s < KMAX; ++s) top[s] = s < KMAX - k_hat ? INFINITY : -INFINITY;
  for (int j0 = 0; j0 < Kc; j0 += KMAX) {
    float grp[KMAX];
    if (kVec) {  // Kc_all % 4 == 0: rows start on 16-byte boundaries
#pragma unroll
      for (int j = 0; j < KMAX; j += 4) {
        float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (j0 + j < Kc) v = __ldg(reinterpret_cast<const float4*>(a + j0 + j));
        grp[j] = v.x;
        grp[j + 1] = !kAware || j0 + j + 1 < Kc ? v.y : -INFINITY;  // Kc_all is a multiple of 4, the visible part need not be
        grp[j + 2] = !kAware || j0 + j + 2 < Kc ? v.z : -INFINITY;
        grp[j + 3] = !kAware || j0 + j + 3 < Kc ? v.w : -INFINITY;
      }
    } else {
#pragma unroll
      for (int j = 0; j < KMAX; ++j) grp[j] = j0 + j < Kc ? __ldg(a + j0 + j) : -INFINITY;
    }
    merge_group<KMAX>(top, grp);
  }
  const float tau = top[KMAX - 1];
  int n_gt = 0;
#pragma unroll
  for (int s = 0; s < KMAX; ++s) n_gt += (top[s] != INFINITY && top[s] > tau);
  int ties_left = k_hat - n_gt;  // how many columns equal to tau are still to be taken (lowest first)

  const int words = (Kc_all + 31) / 32;
  int32_t* my_sel = sel != nullptr ? sel + (size_t)row * k_all : nullptr;
  int out = 0, cnt = 0;
  for (int j0 = 0; j0 < Kc_all; j0 += 32) {
    uint32_t gt = 0u, eq = 0u;
    if (kVec) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (j0 + j < Kc) v = __ldg(reinterpret_cast<const float4*>(a + j0 + j));
        const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool in = !kAware || j0 + j + e < Kc;
          gt |= (in && x[e] > tau ? 1u : 0u) << (j + e);
          eq |= (in && x[e] == tau ? 1u : 0u) << (j + e);
        }
      }
    } else {
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float x = j0 + j < Kc ? __ldg(a + j0 + j) : -INFINITY;
        gt |= (x > tau ? 1u : 0u) << j;
        eq |= (x == tau ? 1u : 0u) << j;
      }
    }
    emit_columns(gt, eq, j0, ties_left, my_sel, out, cnt, mask_bits != nullptr ? mask_bits + (size_t)row * words + (j0 >> 5) : nullptr,
                 i, r, causal);
  }
  if (row_counts != nullptr) row_counts[row] = cnt;
}

// ---- exclusive scan of row_counts -> row_ptr (two small kernels) ---------------------
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int& block_total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  const int nwarps = blockDim.x >> 5;
  if (warp == 0) {
    int w = lane < nwarps ? warp_tot[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= o) winc += t;
    }
    if (lane < nwarps) warp_tot[lane] = winc - w;  // exclusive offset of each warp
    if (lane == 31) warp_tot[32] = winc;           // block total
  }
  __syncthreads();
  block_total = warp_tot[32];
  const int res = inc - v + warp_tot[warp];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kScanThreads)
scan_tile_sums_kernel(const int32_t* __restrict__ counts, int32_t* __restrict__ tile_sums, int rows) {
  __shared__ int warp_tot[33];
  const int base = blockIdx.x * kScanTile + threadIdx.x * kScanPerThread;
  int s = 0;
#pragma unroll
  for (int e = 0; e < kScanPerThread; ++e) s += (base + e < rows) ? counts[base + e] : 0;
  int total;
  block_exclusive_scan(s, warp_tot, total);
  if (threadIdx.x == 0) tile_sums[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kScanThreads)
scan_write_row_ptr_kernel(const int32_t* __restrict__ counts, const int32_t* __restrict__ tile_sums,
                          int32_t* __restrict__ row_ptr, int rows) {
  __shared__ int warp_tot[33];
  // the tile's offset: the sum of the tiles before it (a few hundred values at most)
  int before = 0;
  for (int t = threadIdx.x; t < (int)blockIdx.x; t += kScanThreads) before += tile_sums[t];
  int tile_off;
  block_exclusive_scan(before, warp_tot, tile_off);
  const int base = blockIdx.x * kScanTile + threadIdx.x * kScanPerThread;
  int v[kScanPerThread];
  int s = 0;
#pragma unroll
  for (int e = 0; e < kScanPerThread; ++e) {
    v[e] = (base + e < rows) ? counts[base + e] : 0;
    s += v[e];
  }
  int total;
  int run = block_exclusive_scan(s, warp_tot, total) + tile_off;
#pragma unroll
  for (int e = 0; e < kScanPerThread; ++e) {
    if (base + e < rows) row_ptr[base + e] = run;
    run += v[e];
    if (base + e == rows - 1) row_ptr[rows] = run;
  }
}

__global__ void uniform_row_ptr_kernel(int32_t* __restrict__ row_ptr, int rows, int per_row) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i <= rows) row_ptr[i] = i * per_row;
}

// One warp per row: col_idx[row_ptr[row] + n] = sel[n / r] * r + n % r.  For a causal row the
// kept keys are a prefix of that sequence, because sel is ascending and only the run that
// contains the diagonal is cut.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
fill_col_idx_kernel(const int32_t* __restrict__ sel, const int32_t* __restrict__ row_ptr,
                    int32_t* __restrict__ col_idx, long long nnz_cap, int rows, int k_hat, int r, int log2r,
                    int32_t* __restrict__ status) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_warps = gridDim.x * kWarpsPerCta;
  int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  if (log2r >= 0 && k_hat <= 32) {
    // r a power of two: the run and the offset inside it are a shift and a mask; the row's
    // selected columns sit one per lane and are fetched by shuffles.  A warp walks rows row,
    // row + n_warps, ...: the next row's pointers and columns are requested before this row's
    // keys are written, so that their latency hides under the stores.
    int base = __ldg(row_ptr + row), end = __ldg(row_ptr + row + 1);
    int mine = lane < k_hat ? __ldg(sel + (size_t)row * k_hat + lane) << log2r : 0;
    for (;;) {
      const int next = row + n_warps;
      int base_n = 0, end_n = 0, mine_n = 0;
      if (next < rows) {
        base_n = __ldg(row_ptr + next), end_n = __ldg(row_ptr + next + 1);
        mine_n = lane < k_hat ? __ldg(sel + (size_t)next * k_hat + lane) << log2r : 0;
      }
      int n = end - base;
      if ((long long)base + n > nnz_cap) {
        if (lane == 0) atomicOr(status, SEA_DEV_ROW_OVERFLOW);
        n = (int)max(0ll, min((long long)n, nnz_cap - base));
      }
      int32_t* out = col_idx + base;
      const int n_up = (n + 31) & ~31;  // every lane takes part in the shuffles
#pragma unroll 4
      for (int pos = lane; pos < n_up; pos += 32) {
        const int start = __shfl_sync(0xffffffffu, mine, (pos >> log2r) & 31);
        if (pos < n) out[pos] = start + (pos & (r - 1));
      }
      if (next >= rows) break;
      row = next, base = base_n, end = end_n, mine = mine_n;
    }
    return;
  }
  for (; row < rows; row += n_warps) {
    const int base = row_ptr[row];
    int n = row_ptr[row + 1] - base;
    if ((long long)base + n > nnz_cap) {
      if (lane == 0) atomicOr(status, SEA_DEV_ROW_OVERFLOW);
      n = (int)max(0ll, min((long long)n, nnz_cap - base));
    }
    const int32_t* my_sel = sel + (size_t)row * k_hat;
    if (log2r >= 0) {
      for (int pos = lane; pos < n; pos += 32)
        col_idx[(size_t)base + pos] = (__ldg(my_sel + (pos >> log2r)) << log2r) + (pos & (r - 1));
    } else {
      for (int pos = lane; pos < n; pos += 32) {
        const int b = pos / r;
        col_idx[(size_t)base + pos] = __ldg(my_sel + b) * r + (pos - b * r);
      }
    }
  }
}

template <int VPL>
bool launch_topk(const float* A_hat, int32_t* sel, int32_t* counts, uint32_t* mask_bits, int rows,
                 const sea_shape& s, bool aware, cudaStream_t st) {
  const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  constexpr bool kShared = VPL >= 16;  // from 512 columns on the row is parked in shared memory (beyond that its keys would not fit the registers)
  const size_t smem = kShared ? (size_t)kWarpsPerCta * (VPL + 1) * 32 * sizeof(uint32_t) : 0;
  auto kern = topk_rows_kernel<VPL, kShared>;
  if (smem > 40 * 1024 && cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return false;
  kern<<<grid, kWarpsPerCta * 32, smem, st>>>(A_hat, sel, counts, mask_bits, rows, s.Kc, s.k_hat, s.T, s.T / s.Kc,
                                              s.causal, aware ? 1 : 0);
  return true;
}

// The warp-per-row kernel for a row of `vpl` values per lane.
bool launch_topk_rows(const float* A_hat, int32_t* sel, int32_t* counts, uint32_t* mask_bits, int rows,
                      const sea_shape& s, bool aware, cudaStream_t st) {
  const int vpl = (s.Kc + 31) / 32;
  if (vpl <= 1) return launch_topk<1>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  if (vpl <= 2) return launch_topk<2>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  if (vpl <= 4) return launch_topk<4>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  if (vpl <= 8) return launch_topk<8>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  if (vpl <= 16) return launch_topk<16>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  if (vpl <= 32) return launch_topk<32>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  if (vpl <= 64) return launch_topk<64>(A_hat, sel, counts, mask_bits, rows, s, aware, st);
  return false;
}

}  // namespace

// row_ptr = exclusive prefix sums of the per-row counts, row_ptr[rows] = their total.
sea_status launch_row_ptr_scan(const int32_t* row_counts, int32_t* tile_sums, int32_t* row_ptr, int rows,
                               cudaStream_t st) {
  sea_status rc;
  const int ntiles = (rows + kScanTile - 1) / kScanTile;
  scan_tile_sums_kernel<<<ntiles, kScanThreads, 0, st>>>(row_counts, tile_sums, rows);
  if ((rc = check_launch()) != SEA_OK) return rc;
  scan_write_row_ptr_kernel<<<ntiles, kScanThreads, 0, st>>>(row_counts, tile_sums, row_ptr, rows);
  return check_launch();
}

sea_status launch_topk_mask(const sea_shape& s, const float* A_hat, int32_t* sel, int32_t* row_ptr,
                            int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts,
                            int32_t* tile_sums, uint32_t* mask_bits, bool selected, int32_t* status,
                            cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
  int32_t* counts = s.causal ? row_counts : nullptr;
  sea_status rc = SEA_OK;
  if (selected) {
    // sel, the counts and the bits are in place already
  } else if (s.Kc <= kThreadMaxKc && s.k_hat <= kThreadMaxK) {
    // a short row and few columns to keep: one thread per row
    const int grid = (rows + kThreadRows - 1) / kThreadRows;
#define SEA_TOPK_THREAD(KM)                                                                                     \
  do {                                                                                                          \
    if (s.Kc % 4 == 0)                                                                                          \
      topk_rows_thread_kernel<KM, true, false><<<grid, kThreadRows, 0, st>>>(A_hat, sel, counts, mask_bits,    \
                                                                             rows, s.Kc, s.k_hat, s.T, r,      \
                                                                             s.causal);                        \
    else                                                                                                        \
      topk_rows_thread_kernel<KM, false, false><<<grid, kThreadRows, 0, st>>>(A_hat, sel, counts, mask_bits,   \
                                                                              rows, s.Kc, s.k_hat, s.T, r,     \
                                                                              s.causal);                       \
  } while (0)
    if (s.k_hat <= 8) SEA_TOPK_THREAD(8);
    else if (s.k_hat <= 16) SEA_TOPK_THREAD(16);
    else SEA_TOPK_THREAD(32);
#undef SEA_TOPK_THREAD
  }
  else if (!launch_topk_rows(A_hat, sel, counts, mask_bits, rows, s, false, st)) return SEA_ERR_UNSUPPORTED;
  if (!selected && (rc = check_launch()) != SEA_OK) return rc;

  if (s.causal) {
    if ((rc = launch_row_ptr_scan(row_counts, tile_sums, row_ptr, rows, st)) != SEA_OK) return rc;
  } else {
    uniform_row_ptr_kernel<<<(rows + 1 + 255) / 256, 256, 0, st>>>(row_ptr, rows, s.k_hat * r);
    if ((rc = check_launch()) != SEA_OK) return rc;
  }
  if (col_idx != nullptr) {
    const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
    int log2r = -1;
    for (int l = 0; l < 31; ++l)
      if ((1 << l) == r) log2r = l;
    // a grid that fills the machine once: each warp then walks several rows
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      return SEA_ERR_CUDA;
    const int resident = sms * (2048 / (kWarpsPerCta * 32));
    fill_col_idx_kernel<<<grid < resident ? grid : resident, kWarpsPerCta * 32, 0, st>>>(
        sel, row_ptr, col_idx, (long long)nnz_cap, rows, s.k_hat, r, log2r, status);
    if ((rc = check_launch()) != SEA_OK) return rc;
  }
  return SEA_OK;
}

// ---- capped replication (App. "Sparse Interpolation", the case k K / T < 1) --------------------
// A selected column c keeps at most k_star of its r keys, spaced uniformly over the run:
// c r + floor(u r / k_star), u = 0 .. k_star - 1.  A causal row i keeps those <= i: with
// m = i - c r >= 0 that is min(k_star, ceil((m + 1) k_star / r)) of them, a prefix.
__global__ void capped_counts_kernel(const int32_t* __restrict__ sel, int32_t* __restrict__ row_counts, int rows,
                                     int k_hat, int seq_len, int r, int k_star, int causal) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const int i = row % seq_len;
  int cnt = 0;
  for (int e = 0; e < k_hat; ++e) {
    if (!causal) {
      cnt += k_star;
    } else {
      const long long m = (long long)i - (long long)__ldg(sel + (size_t)row * k_hat + e) * r;
      if (m >= 0) cnt += (int)min((long long)k_star, ((m + 1) * k_star + r - 1) / r);
    }
  }
  row_counts[row] = cnt;
}

// One warp per row: position n of the row is key number n % k_star of its (n / k_star)-th column.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
fill_col_idx_capped_kernel(const int32_t* __restrict__ sel, const int32_t* __restrict__ row_ptr,
                           int32_t* __restrict__ col_idx, long long nnz_cap, int rows, int k_hat, int r, int k_star,
                           int32_t* __restrict__ status) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  const int base = row_ptr[row];
  int n = row_ptr[row + 1] - base;
  if ((long long)base + n > nnz_cap) {
    if (lane == 0) atomicOr(status, SEA_DEV_ROW_OVERFLOW);
    n = (int)max(0ll, min((long long)n, nnz_cap - base));
  }
  const int32_t* my_sel = sel + (size_t)row * k_hat;
  for (int pos = lane; pos < n; pos += 32) {
    const int b = pos / k_star, u = pos - b * k_star;
    col_idx[(size_t)base + pos] = __ldg(my_sel + b) * r + (int)(((long long)u * r) / k_star);
  }
}

sea_status launch_topk_mask_capped(const sea_shape& s, int k_star, const float* A_hat, int32_t* sel, int32_t* row_ptr,
                                   int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts, int32_t* tile_sums,
                                   int32_t* status, cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
  if (k_star >= r)  // no cap: the whole run
    return launch_topk_mask(s, A_hat, sel, row_ptr, col_idx, nnz_cap, row_counts, tile_sums, nullptr, false, status, st);
  // the selection as usual (its row pointers are those of whole runs and are replaced below)
  sea_status rc = launch_topk_mask(s, A_hat, sel, row_ptr, nullptr, 0, row_counts, tile_sums, nullptr, false, status, st);
  if (rc != SEA_OK) return rc;
  capped_counts_kernel<<<(rows + 255) / 256, 256, 0, st>>>(sel, row_counts, rows, s.k_hat, s.T, r, k_star, s.causal);
  if ((rc = check_launch()) != SEA_OK) return rc;
  if ((rc = launch_row_ptr_scan(row_counts, tile_sums, row_ptr, rows, st)) != SEA_OK) return rc;
  const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  fill_col_idx_capped_kernel<<<grid, kWarpsPerCta * 32, 0, st>>>(sel, row_ptr, col_idx, (long long)nnz_cap, rows, s.k_hat, r,
                                                                 k_star, status);
  return check_launch();
}

// ---- nearest-neighbour resize at any ratio (App. "Sparse Interpolation"; App. "Visualization of
// intermediate buffers": every causal row is resized to its own width) --------------------------
// Row i of the compressed mask (Kc pixels) is resized to W pixels, W = T or, with row_widths, i + 1:
// key j looks at pixel floor(j Kc / W), so a selected pixel c covers the keys
// ceil(c W / Kc) .. ceil((c + 1) W / Kc) - 1 (none when W < Kc skips the pixel).  Causal rows keep j <= i.
__device__ __forceinline__ int resized_first_key(int c, int W, int Kc) { return (int)(((long long)c * W + Kc - 1) / Kc); }
__device__ __forceinline__ void resized_run(int c, int i, int T, int Kc, int causal, int row_widths, int& start, int& len) {
  const int W = row_widths ? i + 1 : T;
  start = resized_first_key(c, W, Kc);
  int end = resized_first_key(c + 1, W, Kc);
  if (causal) end = min(end, i + 1);
  len = max(0, end - start);
}

__global__ void resized_counts_kernel(const int32_t* __restrict__ sel, int32_t* __restrict__ row_counts, int rows, int k_hat,
                                      int T, int Kc, int causal, int row_widths) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const int i = row % T;
  int cnt = 0;
  for (int e = 0; e < k_hat; ++e) {
    int start, len;
    resized_run(__ldg(sel + (size_t)row * k_hat + e), i, T, Kc, causal, row_widths, start, len);
    cnt += len;
  }
  row_counts[row] = cnt;
}

// One warp per row, 32 selected pixels at a time: the lanes hold the pixels' runs and the running
// sum of their lengths; every entry of the row finds its run by a search over those sums.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
fill_col_idx_resized_kernel(const int32_t* __restrict__ sel, const int32_t* __restrict__ row_ptr,
                            int32_t* __restrict__ col_idx, long long nnz_cap, int rows, int k_hat, int T, int Kc, int causal,
                            int row_widths, int32_t* __restrict__ status) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  const int i = row % T;
  const long long base = row_ptr[row];
  long long room = nnz_cap - base;  // entries of this row that still fit
  if (base + (row_ptr[row + 1] - base) > nnz_cap && lane == 0) atomicOr(status, SEA_DEV_ROW_OVERFLOW);
  int done = 0;
  for (int e0 = 0; e0 < k_hat; e0 += 32) {
    int start = 0, len = 0;
    if (e0 + lane < k_hat) resized_run(__ldg(sel + (size_t)row * k_hat + e0 + lane), i, T, Kc, causal, row_widths, start, len);
    int inc = len;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    const int total = __shfl_sync(0xffffffffu, inc, 31);
    const int n_up = (total + 31) & ~31;  // every lane takes part in the shuffles
    for (int pos = lane; pos < n_up; pos += 32) {
      // the first lane whose running sum exceeds pos
      int lo = 0;
#pragma unroll
      for (int step = 16; step > 0; step >>= 1) {
        const int v = __shfl_sync(0xffffffffu, inc, lo + step - 1);
        if (v <= pos) lo += step;
      }
      const int run_start = __shfl_sync(0xffffffffu, start, lo);
      const int before = __shfl_sync(0xffffffffu, inc - len, lo);
      if (pos < total && (long long)(done + pos) < room) col_idx[base + done + pos] = run_start + (pos - before);
    }
    done += total;
  }
}

sea_status launch_topk_mask_resized(const sea_shape& s, int row_widths, const float* A_hat, int32_t* sel, int32_t* row_ptr,
                                    int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts, int32_t* tile_sums,
                                    int32_t* status, cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  // the selection as usual, on a copy of the shape that asks for no row lengths (the row pointers it
  // writes are replaced below)
  sea_shape plain = s;
  plain.causal = 0;
  sea_status rc = launch_topk_mask(plain, A_hat, sel, row_ptr, nullptr, 0, row_counts, tile_sums, nullptr, false, status, st);
  if (rc != SEA_OK) return rc;
  resized_counts_kernel<<<(rows + 255) / 256, 256, 0, st>>>(sel, row_counts, rows, s.k_hat, s.T, s.Kc, s.causal, row_widths);
  if ((rc = check_launch()) != SEA_OK) return rc;
  if ((rc = launch_row_ptr_scan(row_counts, tile_sums, row_ptr, rows, st)) != SEA_OK) return rc;
  if (col_idx == nullptr) return SEA_OK;
  const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  fill_col_idx_resized_kernel<<<grid, kWarpsPerCta * 32, 0, st>>>(sel, row_ptr, col_idx, (long long)nnz_cap, rows, s.k_hat, s.T,
                                                                  s.Kc, s.causal, row_widths, status);
  return check_launch();
}

// Causal-aware per-query selection: bits, row lengths, row pointers and (optionally) column indices.
sea_status launch_topk_mask_aware(const sea_shape& s, const float* A_hat, uint32_t* mask_bits, int32_t* row_ptr,
                                  int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts, int32_t* tile_sums,
                                  int32_t* status, cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  if (s.Kc <= kThreadMaxKc && s.k_hat <= kThreadMaxK) {
    // a short row and few columns to keep: one thread per row
    const int grid = (rows + kThreadRows - 1) / kThreadRows;
    const int r = s.T / s.Kc;
#define SEA_AWARE_THREAD(KM)                                                                                          \
  do {                                                                                                                \
    if (s.Kc % 4 == 0)                                                                                                \
      topk_rows_thread_kernel<KM, true, true><<<grid, kThreadRows, 0, st>>>(A_hat, nullptr, row_counts, mask_bits,   \
                                                                            rows, s.Kc, s.k_hat, s.T, r, s.causal);  \
    else                                                                                                              \
      topk_rows_thread_kernel<KM, false, true><<<grid, kThreadRows, 0, st>>>(A_hat, nullptr, row_counts, mask_bits,  \
                                                                             rows, s.Kc, s.k_hat, s.T, r, s.causal); \
  } while (0)
    if (s.k_hat <= 8) SEA_AWARE_THREAD(8);
    else if (s.k_hat <= 16) SEA_AWARE_THREAD(16);
    else SEA_AWARE_THREAD(32);
#undef SEA_AWARE_THREAD
  } else if (!launch_topk_rows(A_hat, nullptr, row_counts, mask_bits, rows, s, true, st)) {
    return SEA_ERR_UNSUPPORTED;
  }
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;
  if ((rc = launch_row_ptr_scan(row_counts, tile_sums, row_ptr, rows, st)) != SEA_OK) return rc;
  if (col_idx != nullptr) return launch_fill_col_idx_bits(s, mask_bits, row_ptr, col_idx, nnz_cap, status, st);
  return SEA_OK;
}

}  // namespace sea

// ---- sea_topk_mask_static: the same stage without a caller-provided workspace ----------------
//
// For callers that can neither allocate device memory nor hand over a workspace: an inference
// plugin whose memory plan was frozen when the engine was built, or a serving loop that must not
// call cudaMalloc because it synchronises the device and can fail under a fixed memory budget.
// The scratch the stage needs (per-row counts and the partial sums of their scan) lives in the
// file-scope device array below, sized for at most kStaticMaxRows rows; every GPU that loads the
// library holds these 4.2 MB until the process exits.
#include <mutex>

namespace sea {
namespace {

constexpr int kStaticMaxRows = 1 << 20;  // B*H*T limit of the static variant
constexpr int kStaticTiles = kStaticMaxRows / kScanTile + 1;
constexpr int kStaticHead = 64;  // int32 words reserved ahead of the counts (word 0: status)
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) int32_t g_static_scratch[kStaticHead + kStaticMaxRows + kStaticTiles + 63];

// In host code the array's name is only a handle; the device address is looked up once per
// device, with that device current, and remembered here.
std::mutex g_static_mutex;
int32_t* g_static_ptr[kStaticMaxDevices] = {};

sea_status static_scratch(int32_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) return SEA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[dev] == nullptr) {
    int32_t* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch) != cudaSuccess || p == nullptr)
      return SEA_ERR_CUDA;
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return SEA_OK;
}

}  // namespace
}  // namespace sea

extern "C" sea_status sea_topk_mask_static(const sea_shape* shape, const float* A_hat, int32_t* sel,
                                           int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                           void* cuda_stream) {
  using namespace sea;
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, false);
  if (rc != SEA_OK) return rc;
  if (!A_hat || !sel || !row_ptr) return SEA_ERR_INVALID_ARG;
  auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (misaligned(A_hat) || misaligned(sel) || misaligned(row_ptr) || (col_idx && misaligned(col_idx)))
    return SEA_ERR_INVALID_ARG;
  const long long rows = (long long)shape->B * shape->H * shape->T;
  if (rows > kStaticMaxRows) return SEA_ERR_TOO_LARGE;  // beyond the static scratch
  const long long full = rows * shape->k_hat * (shape->T / shape->Kc);
  // without a status word to report a truncated row, col_idx must be able to hold every row in full
  if (col_idx && (nnz_cap < full || nnz_cap > 2147483647ll)) return SEA_ERR_TOO_LARGE;
  int32_t* scratch = nullptr;
  const sea_status rs = static_scratch(&scratch);
  if (rs != SEA_OK) return rs;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps the previous call's contents: counts and partial sums are rewritten in full
  // by the kernels, the status word is the one thing that has to start at zero
  if (cudaMemsetAsync(scratch, 0, sizeof(int32_t), st) != cudaSuccess) return SEA_ERR_CUDA;
  return launch_topk_mask(*shape, A_hat, sel, row_ptr, col_idx, nnz_cap, scratch + kStaticHead,
                          scratch + kStaticHead + kStaticMaxRows, nullptr, false, scratch, st);
}

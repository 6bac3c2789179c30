// Mask generation with the causal-per-batch grouping (Sec. 3.1 "Grouped Top-k Selection"):
// the estimate of a batch element is viewed as [T, H, Kc] and, for every query position, the
// H * k_hat largest of its H * Kc entries are kept - the heads of a position compete for one
// budget, positions never exchange anything.  Rows (b, h, t) then keep differing numbers of
// columns; the selection leaves as one bit per compressed column, and the up-sampled mask as the
// same flat CSR the per-query grouping produces (App. "FlatCSR" keeps one row per (b, t) over the
// flattened (head, key) axis instead and transposes inside its kernels).
//
// One CTA per (b, t): its H * Kc values stay in registers as order-preserving 32-bit keys, the
// (H * k_hat)-th largest key is found bit by bit, and keys equal to it are taken in ascending
// flattened index h * Kc + c until the budget is used up.
#include "sea_common.cuh"

namespace sea {
namespace {

constexpr int kMaxThreads = 1024;
constexpr int kMaxVI = 8;           // 16-byte groups per thread
constexpr int kWarpsPerCta = 8;     // row-per-warp kernels

// Sum of v over the CTA.  `red` is one of two alternating 32-word buffers, so a single barrier
// per call is enough.
__device__ __forceinline__ int block_sum(int v, int* red, int nwarps) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = __reduce_add_sync(0xffffffffu, v);
  if (lane == 0) red[warp] = v;
  __syncthreads();
  const int t = lane < nwarps ? red[lane] : 0;
  return __reduce_add_sync(0xffffffffu, t);
}

// Exclusive prefix of v over the threads of the CTA in thread order, and the CTA's total.
__device__ __forceinline__ int block_exclusive_scan(int v, int* tot, int nwarps, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();  // the previous call's readers are done with tot[]
  if (lane == 31) tot[warp] = inc;
  __syncthreads();
  int w = lane < nwarps ? tot[lane] : 0;
  int winc = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += t;
  }
  total = __shfl_sync(0xffffffffu, winc, 31);
  const int warp_off = __shfl_sync(0xffffffffu, winc - w, warp);
  return inc - v + warp_off;
}

// Thread `tid` holds the 16-byte groups q = i * blockDim.x + tid (i < VI) of the position's
// H * Kc / 4 groups; group q covers flattened indices 4 q .. 4 q + 3, all of one head because
// Kc % 4 == 0.
//
// The search for the k_sel-th largest key tau:
//   1  the position's largest key `top` (one CTA-wide maximum);
//   2  a histogram of the distances top - key in steps of 2^kFineBits, over the kBins steps below
//      `top` (for positive values that is every magnitude down to top / 65536; the keys spread
//      widely over it, so the shared-memory counters rarely collide), and a scan over it that
//      finds the step holding tau and the number of keys in the steps above it;
//   3  the keys inside that step (a handful for spread-out data) go to a list and one warp finds
//      tau among them, bit by bit, without CTA-wide barriers.
// When fewer than k_sel keys lie inside the histogram's span (tau is negative while `top` is not)
// or the step does not fit the list (many equal values), tau is found bit by bit with CTA-wide
// counts over all keys instead.
constexpr int kFineBits = 15;
constexpr int kBinBits = 12;
constexpr int kBins = 1 << kBinBits;
constexpr uint32_t kFineMask = (1u << kFineBits) - 1u;
constexpr int kListCap = 1024;

//
// kStream: the position holds more keys than VI groups per thread (H * Kc > 4 VI blockDim.x).  The
// threads then take the groups in n_pass passes of VI, and every step below that walks the keys
// fetches them again pass by pass (from L2: a position's values are a few hundred KB) instead of
// keeping them in registers; group (pass VI + i) blockDim.x + tid keeps the flattened order.
template <int VI, int kThreadsMax, int kMinCtas, bool kStream>
__global__ void __launch_bounds__(kThreadsMax, kMinCtas)
topk_grouped_kernel(const float* __restrict__ A_hat, uint32_t* __restrict__ mask_bits,
                    int32_t* __restrict__ row_counts, int32_t* __restrict__ park_off, int H, int T, int Kc, int log2Kc,
                    int k_sel, int r, int causal, int n_pass) {
  extern __shared__ uint32_t sh_dyn[];  // [H][words] bits, then [H] selected columns per head
  __shared__ int hist[kBins];
  __shared__ uint32_t list[kListCap];
  __shared__ int red[2][32];
  __shared__ int scan_tot[32];
  __shared__ int list_n;
  __shared__ uint32_t found[3];  // after 2: step, |{key above it}|; after 3: tau, |{key > tau}|, |{key == tau}|
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nthreads = blockDim.x, nwarps = nthreads >> 5;
  const int bt = blockIdx.x;
  const int b = bt / T, t = bt - b * T;
  const int words = (Kc + 31) >> 5;
  const int n4 = (H * Kc) >> 2;
  uint32_t* sh_bits = sh_dyn;
  int* head_pc = reinterpret_cast<int*>(sh_dyn + H * words);
  // head and column of flattened index f
  auto split = [&](int f, int& h, int& c) {
    if (log2Kc >= 0) {
      h = f >> log2Kc;
      c = f & (Kc - 1);
    } else {
      h = f / Kc;
      c = f - h * Kc;
    }
  };

  for (int w = 4 * tid; w < kBins; w += 4 * nthreads) *reinterpret_cast<int4*>(&hist[w]) = make_int4(0, 0, 0, 0);
  for (int w = tid; w < H * words; w += nthreads) sh_bits[w] = 0u;
  if (tid == 0) list_n = 0;
  // Step x of the histogram is owned by thread x >> log2per (a power of two of steps per thread,
  // `owners` threads own some) and kept at word (x & (per - 1)) * owners + (x >> log2per): when the
  // owners read their j-th steps, neighbouring lanes read neighbouring words.
  int log2per = 0;
  while ((nthreads << log2per) < kBins) ++log2per;
  const int per = 1 << log2per, log2owners = kBinBits - log2per, owners = 1 << log2owners;

  uint32_t key[VI][4];
  // the keys of the thread's groups of pass `pass` (all of its groups when the keys stay in registers)
  auto load_keys = [&](int pass) {
#pragma unroll
    for (int i = 0; i < VI; ++i) {
      const int q = (pass * VI + i) * nthreads + tid;
      key[i][0] = key[i][1] = key[i][2] = key[i][3] = 0u;  // below the key of every finite value
      if (q < n4) {
        int h, c;
        split(4 * q, h, c);
        const float4 v = __ldg(reinterpret_cast<const float4*>(A_hat + ((size_t)(b * H + h) * T + t) * Kc + c));
        key[i][0] = order_key(v.x);
        key[i][1] = order_key(v.y);
        key[i][2] = order_key(v.z);
        key[i][3] = order_key(v.w);
      }
    }
  };
  const int passes = kStream ? n_pass : 1;
  // SEA_EACH_PASS { body }: the body once per pass, with that pass's keys in key[][]
#define SEA_EACH_PASS for (int pass = 0; pass < passes; ++pass) if (kStream ? (load_keys(pass), true) : true)
  uint32_t top = 0u;
  for (int pass = 0; pass < passes; ++pass) {
    load_keys(pass);
#pragma unroll
    for (int i = 0; i < VI; ++i) top = max(max(top, key[i][0]), max(key[i][1], max(key[i][2], key[i][3])));
  }
  // ---- 1: the largest key
  top = __reduce_max_sync(0xffffffffu, top);
  if (lane == 0) red[0][warp] = (int)top;
  __syncthreads();  // also: the counters are zero
  top = __reduce_max_sync(0xffffffffu, lane < nwarps ? (uint32_t)red[0][lane] : 0u);
  // ---- 2: histogram of (top - key) >> kFineBits over the keys less than kBins steps below top
  SEA_EACH_PASS {
#pragma unroll
    for (int i = 0; i < VI; ++i)
      if ((pass * VI + i) * nthreads + tid < n4) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const uint32_t x = (top - key[i][e]) >> kFineBits;
          if (x < (uint32_t)kBins) atomicAdd(&hist[((x & (per - 1)) << log2owners) + (x >> log2per)], 1);
        }
      }
  }
  __syncthreads();
  int n_gt = 0, n_eq = 0;
  uint32_t tau = 0u;
  bool searched = false;
  {
    // the first step (from the top) at which the running count reaches k_sel
    int mine = 0;
    if (tid < owners)
      for (int j = 0; j < per; ++j) mine += hist[j * owners + tid];
    int total;
    int over = block_exclusive_scan(mine, scan_tot, nwarps, total);  // keys in the steps above this thread's
    if (over < k_sel && over + mine >= k_sel) {
      int j = 0;
      while (over + hist[j * owners + tid] < k_sel) over += hist[j++ * owners + tid];
      found[0] = (uint32_t)(tid * per + j);
      found[1] = (uint32_t)over;
    }
    __syncthreads();
    if (total >= k_sel) {
      // ---- 3: the keys inside the step
      const uint32_t step = found[0];
      const int above = (int)found[1];
      int inside = 0;
      SEA_EACH_PASS {
#pragma unroll
        for (int i = 0; i < VI; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) inside += key[i][e] != 0u && ((top - key[i][e]) >> kFineBits) == step;
  }  // 0: a padding slot
      if (inside > 0) {
        int at = atomicAdd(&list_n, inside);
        if (at + inside <= kListCap) {
          SEA_EACH_PASS {
#pragma unroll
            for (int i = 0; i < VI; ++i)
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t rel = top - key[i][e];
                if (key[i][e] != 0u && (rel >> kFineBits) == step) list[at++] = kFineMask - (rel & kFineMask);  // grows with the key
              }
  }
        }
      }
      __syncthreads();  // also: every thread has read found[] before it is written again
      const int n_list = list_n;
      if (n_list <= kListCap) {
        if (warp == 0) {
          uint32_t fine = 0u;  // the k_sel-th largest key's position inside the step
          int g = 0, e = 0;
          if (n_list <= 32) {
            // an entry per lane: counts are ballots
            const bool have = lane < n_list;
            const uint32_t mine = have ? list[lane] : 0u;
            for (int bit = kFineBits - 1; bit >= 0; --bit) {
              const uint32_t cand = fine | (1u << bit);
              if (__popc(__ballot_sync(0xffffffffu, have && mine >= cand)) + above >= k_sel) fine = cand;
            }
            g = __popc(__ballot_sync(0xffffffffu, have && mine > fine));
            e = __popc(__ballot_sync(0xffffffffu, have && mine == fine));
          } else {
            for (int bit = kFineBits - 1; bit >= 0; --bit) {
              const uint32_t cand = fine | (1u << bit);
              int c = 0;
              for (int idx = lane; idx < n_list; idx += 32) c += list[idx] >= cand;
              if (__reduce_add_sync(0xffffffffu, c) + above >= k_sel) fine = cand;
            }
            for (int idx = lane; idx < n_list; idx += 32) {
              g += list[idx] > fine;
              e += list[idx] == fine;
            }
            g = __reduce_add_sync(0xffffffffu, g);
            e = __reduce_add_sync(0xffffffffu, e);
          }
          if (lane == 0) {
            found[0] = top - ((step << kFineBits) | (kFineMask - fine));
            found[1] = (uint32_t)(above + g);
            found[2] = (uint32_t)e;
          }
        }
        __syncthreads();
        tau = found[0];
        n_gt = (int)found[1];
        n_eq = (int)found[2];
        searched = true;
      }
    }
  }
  if (!searched) {
    // the largest tau with |{key >= tau}| >= k_sel, bit by bit over all keys
    int rb = 0;  // which of the two reduction buffers the next CTA-wide sum uses
    for (int bit = 31; bit >= 0; --bit) {
      const uint32_t cand = tau | (1u << bit);
      int c = 0;
      SEA_EACH_PASS {
#pragma unroll
        for (int i = 0; i < VI; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) c += key[i][e] >= cand;
  }
      if (block_sum(c, red[rb], nwarps) >= k_sel) tau = cand;
      rb ^= 1;
    }
    SEA_EACH_PASS {
#pragma unroll
      for (int i = 0; i < VI; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          n_gt += key[i][e] > tau;
          n_eq += key[i][e] == tau;
        }
  }
    n_gt = block_sum(n_gt, red[rb], nwarps);
    n_eq = block_sum(n_eq, red[rb ^ 1], nwarps);
  }
  const int need = k_sel - n_gt;  // how many keys equal to tau are taken (lowest flattened index first)

  // the selected elements of a group, as bits of its head's string
  auto emit = [&](int q, uint32_t nib) {
    if (nib != 0u && q < n4) {
      int h, c;
      split(4 * q, h, c);
      atomicOr(&sh_bits[h * words + (c >> 5)], nib << (c & 31));
    }
  };
  if (n_eq == need) {
    SEA_EACH_PASS {
#pragma unroll
      for (int i = 0; i < VI; ++i) {
        uint32_t nib = 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) nib |= (key[i][e] >= tau ? 1u : 0u) << e;
        emit((pass * VI + i) * nthreads + tid, nib);
      }
  }
  } else {
    // more equal keys than places: rank them in flattened order (group index major, then thread)
    int seen = 0;
    SEA_EACH_PASS {
#pragma unroll
      for (int i = 0; i < VI; ++i) {
        int mine = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) mine += key[i][e] == tau;
        int total;
        int rank = seen + block_exclusive_scan(mine, scan_tot, nwarps, total);
        uint32_t nib = 0u;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const bool eq = key[i][e] == tau;
          const bool take = key[i][e] > tau || (eq && rank < need);
          rank += eq;
          nib |= (take ? 1u : 0u) << e;
        }
        emit((pass * VI + i) * nthreads + tid, nib);
        seen += total;
      }
  }
  }
#undef SEA_EACH_PASS
  __syncthreads();

  // a thread per head: the row's bit string and its number of keys after up-sampling.  Column c
  // covers keys c r .. c r + r - 1; a causal row keeps those <= t: the columns below
  // (t + 1) / r in full and (t + 1) % r keys of the column at (t + 1) / r.
  const int c_full = causal ? (t + 1) / r : Kc;
  const int rem = causal ? (t + 1) - c_full * r : 0;
  for (int h = tid; h < H; h += nthreads) {
    const size_t row = (size_t)(b * H + h) * T + t;
    const uint32_t* src = sh_bits + h * words;
    int cnt = 0, pc = 0;
    for (int w = 0; w < words; ++w) {
      const uint32_t word = src[w];
      const int lo = 32 * w;
      const uint32_t full = c_full >= lo + 32 ? 0xffffffffu : (c_full <= lo ? 0u : (1u << (c_full - lo)) - 1u);
      pc += __popc(word);
      cnt += r * __popc(word & full);
      if (c_full >= lo && c_full < lo + 32 && ((word >> (c_full - lo)) & 1u)) cnt += rem;
    }
    if (mask_bits != nullptr) {
      uint32_t* dst = mask_bits + row * words;
      if ((words & 3) == 0) {  // rows of whole 16-byte pieces
        for (int w = 0; w < words; w += 4)
          *reinterpret_cast<uint4*>(dst + w) = make_uint4(src[w], src[w + 1], src[w + 2], src[w + 3]);
      } else {
        for (int w = 0; w < words; ++w) dst[w] = src[w];
      }
    }
    row_counts[row] = cnt;
    head_pc[h] = pc;
  }
  if (park_off != nullptr) {
    // where each row parks its unnormalised probabilities: the heads of this position one after
    // the other inside the position's slab of k_sel * r values
    __syncthreads();
    for (int h = tid; h < H; h += nthreads) {
      int before = 0;
      for (int g = 0; g < h; ++g) before += head_pc[g];
      park_off[(size_t)(b * H + h) * T + t] = (bt * k_sel + before) * r;
    }
  }
}

// One warp per row: the set bits in ascending order, r keys each, cut at the row's length (for a
// causal row the kept keys are a prefix of that sequence).  Word by word, the lanes whose bit is
// set note their position under their rank, which turns "the j-th selected column" into a lookup.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
fill_col_idx_bits_kernel(const uint32_t* __restrict__ mask_bits, const int32_t* __restrict__ row_ptr,
                         int32_t* __restrict__ col_idx, long long nnz_cap, int rows, int words, int r, int log2r,
                         int32_t* __restrict__ status) {
  __shared__ int col_of[kWarpsPerCta][32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  const int base = row_ptr[row];
  int n = row_ptr[row + 1] - base;
  if ((long long)base + n > nnz_cap) {
    if (lane == 0) atomicOr(status, SEA_DEV_ROW_OVERFLOW);
    n = (int)max(0ll, min((long long)n, nnz_cap - base));
  }
  const uint32_t* my_bits = mask_bits + (size_t)row * words;
  int32_t* out = col_idx + base;
  int done = 0;
  for (int w = 0; w < words && done < n; ++w) {
    const uint32_t word = __ldg(my_bits + w);
    if (word == 0u) continue;
    if ((word >> lane) & 1u) col_of[warp][__popc(word & ((1u << lane) - 1u))] = 32 * w + lane;
    __syncwarp();
    const int lim = min(__popc(word) * r, n - done);
    for (int pos = lane; pos < lim; pos += 32) {
      const int j = log2r >= 0 ? pos >> log2r : pos / r;
      out[done + pos] = col_of[warp][j] * r + (pos - j * r);
    }
    done += lim;
    __syncwarp();
  }
}

// One thread per (b, t): running offsets of its heads inside the position's slab of the parking
// area.
__global__ void park_offsets_kernel(const uint32_t* __restrict__ mask_bits, int32_t* __restrict__ park_off, int B,
                                    int H, int T, int words, int r, int per_slab, int32_t* __restrict__ status) {
  const int bt = blockIdx.x * blockDim.x + threadIdx.x;
  if (bt >= B * T) return;
  const int b = bt / T, t = bt - b * T;
  int used = 0;
  bool over = false;
  for (int h = 0; h < H; ++h) {
    const size_t row = (size_t)(b * H + h) * T + t;
    int pc = 0;
    if ((words & 3) == 0) {  // rows of whole 16-byte pieces (the caller's array is 16-byte aligned)
      for (int w = 0; w < words; w += 4) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(mask_bits + row * words + w));
        pc += __popc(v.x) + __popc(v.y) + __popc(v.z) + __popc(v.w);
      }
    } else {
      for (int w = 0; w < words; ++w) pc += __popc(__ldg(mask_bits + row * words + w));
    }
    const int next = used + pc * r;
    if (next > per_slab) over = true;
    park_off[row] = over ? -1 : bt * per_slab + used;
    used = next;
  }
  if (over) atomicOr(status, SEA_DEV_ROW_OVERFLOW);
}

template <int VI, int kThreadsMax, int kMinCtas, bool kStream = false>
void launch_grouped(const float* A_hat, uint32_t* mask_bits, int32_t* counts, int32_t* park_off, const sea_shape& s,
                    int threads, cudaStream_t st) {
  const size_t smem = ((size_t)s.H * ((s.Kc + 31) / 32) + s.H) * sizeof(uint32_t);
  int log2Kc = -1;
  for (int l = 0; l < 31; ++l)
    if ((1 << l) == s.Kc) log2Kc = l;
  const int n_pass = (s.H * s.Kc / 4 + VI * threads - 1) / (VI * threads);
  topk_grouped_kernel<VI, kThreadsMax, kMinCtas, kStream><<<s.B * s.T, threads, smem, st>>>(
      A_hat, mask_bits, counts, park_off, s.H, s.T, s.Kc, log2Kc, s.H * s.k_hat, s.T / s.Kc, s.causal, n_pass);
}

}  // namespace

// Rows of whole 16-byte groups, and the position's bit strings (with a word per head) within the
// 48 KB of dynamic shared memory a kernel gets without asking.
bool topk_grouped_supported(const sea_shape& s) {
  return s.Kc % 4 == 0 && ((long long)s.H * ((s.Kc + 31) / 32) + s.H) * 4 <= 48 * 1024 && (long long)s.H * s.Kc < (1ll << 30);
}

sea_status launch_topk_mask_grouped(const sea_shape& s, const float* A_hat, uint32_t* mask_bits, int32_t* row_ptr,
                                    int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts, int32_t* tile_sums,
                                    int32_t* park_off, int32_t* status, cudaStream_t st) {
  if (!topk_grouped_supported(s)) return SEA_ERR_UNSUPPORTED;
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
  const int n4 = s.H * s.Kc / 4;
  // four groups per thread while the CTA stays within its size limit
  int threads = ((n4 + 3) / 4 + 31) / 32 * 32;
  if (threads < 128) threads = 128;
  if (threads > kMaxThreads) threads = kMaxThreads;
  const int vi = (n4 + threads - 1) / threads;
  if (threads <= 256) {  // small CTAs: several per SM
    if (vi <= 1) launch_grouped<1, 256, 6>(A_hat, mask_bits, row_counts, park_off, s, threads, st);
    else if (vi <= 2) launch_grouped<2, 256, 6>(A_hat, mask_bits, row_counts, park_off, s, threads, st);
    else launch_grouped<4, 256, 6>(A_hat, mask_bits, row_counts, park_off, s, threads, st);
  } else if (vi <= 4) {
    launch_grouped<4, kMaxThreads, 1>(A_hat, mask_bits, row_counts, park_off, s, threads, st);
  } else if (vi <= kMaxVI) {
    launch_grouped<8, kMaxThreads, 1>(A_hat, mask_bits, row_counts, park_off, s, threads, st);
  } else {  // more keys than a CTA's registers hold: several passes over the position's values
    launch_grouped<8, kMaxThreads, 1, true>(A_hat, mask_bits, row_counts, park_off, s, threads, st);
  }
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;
  if ((rc = launch_row_ptr_scan(row_counts, tile_sums, row_ptr, rows, st)) != SEA_OK) return rc;
  if (col_idx != nullptr) return launch_fill_col_idx_bits(s, mask_bits, row_ptr, col_idx, nnz_cap, status, st);
  return SEA_OK;
}

sea_status launch_fill_col_idx_bits(const sea_shape& s, const uint32_t* mask_bits, const int32_t* row_ptr,
                                    int32_t* col_idx, int64_t nnz_cap, int32_t* status, cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
  int log2r = -1;
  for (int l = 0; l < 31; ++l)
    if ((1 << l) == r) log2r = l;
  const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  fill_col_idx_bits_kernel<<<grid, kWarpsPerCta * 32, 0, st>>>(mask_bits, row_ptr, col_idx, (long long)nnz_cap, rows,
                                                               (s.Kc + 31) / 32, r, log2r, status);
  return check_launch();
}

sea_status launch_park_offsets(const sea_shape& s, const uint32_t* mask_bits, int32_t* park_off, int32_t* status,
                               cudaStream_t st) {
  const int n = s.B * s.T;
  park_offsets_kernel<<<(n + 127) / 128, 128, 0, st>>>(mask_bits, park_off, s.B, s.H, s.T, (s.Kc + 31) / 32,
                                                       s.T / s.Kc, s.H * s.k_hat * (s.T / s.Kc), status);
  return check_launch();
}

}  // namespace sea

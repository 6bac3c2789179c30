// Sparse attention as masked dense tiles on the 5th-generation tensor cores (bf16, mask given
// as `sel`, r = T / Kc a power of two >= 4, T a multiple of 128).
//
// Same result as the per-row kernels (Sec. 3.1.1: scores at the mask's positions, row softmax,
// product with V), computed tile by tile: a work item is 128 consecutive queries of one head;
// for every 128-key tile S = Q K^T is formed by tcgen05.mma into tensor memory, each query's
// thread keeps only the keys of its selected columns (a bit per compressed column, App. "Sparse
// Interpolation": column c covers keys c*r .. c*r+r-1; causal rows drop keys j > i), and
// O += P V is a second tcgen05.mma whose A operand (the probabilities, as a bf16 head plus a
// bf16 remainder) is written back into the tensor-memory columns that held S.  With the
// selections of neighbouring rows uncorrelated the union of the selected columns of 128 rows
// is every column, so all tiles are visited; at the densities this layer runs at (k_hat / Kc
// of 1/8 to 1/64) the dense products cost less than gathering every row's K and V rows.
//
// One pass over the key tiles of a work item with an online softmax.  The two threads of a row
// (one per half of a tile's columns) each keep a reference value m of their own: probabilities are
// formed as exp2((s - m) * scale * log2 e), summed in fp32, and accumulated by the P V product into
// an output buffer of the thread's half (two accumulators of 64 columns per item).  m starts as the
// maximum of the first tile that holds a kept score and is only raised when a later tile's maximum
// exceeds it by more than 2^8 in the exponent's units; the thread then waits for the P V products
// issued so far, multiplies its accumulator row and its sum by exp2((m_old - m_new) * ...) and goes
// on - a rare event, since a reference within 2^8 of the maximum keeps every probability and sum
// far inside the fp32 range.  When the item ends the halves exchange (m, sum), and the output row is
// (O_0 w_0 + O_1 w_1) / (l_0 w_0 + l_1 w_1) with w_h = exp2((m_h - max(m_0, m_1)) * ...).
// The raw scores of kept keys are parked in a scratch array as they are read; the last warpgroup
// turns them into P = exp2((s - M) * ...) / l, rounded once, when the item ends.
//
// Warp roles (warpgroups that re-balance their registers): warp 0 issues the TMA copies (the
// item's mask bits and Q tile, K and V tiles through rings of 16 KB stages), warp 1 issues the
// Q K^T MMAs, warp 2 the P V MMAs (whole warps, so that what feeds the MMAs stays in uniform
// registers; one elected lane issues); the row warpgroups own the query rows (per thread a row and 128 / kSplit of every
// tile's columns); the last warpgroup turns the parked scores into P.  All hand-offs are
// mbarriers; every wait is bounded by a clock and a wait that runs out sets SEA_DEV_TIMEOUT,
// after which all roles drain and leave.
#include <cuda.h>

#include "sea_common.cuh"
#include "sea_tc.cuh"

namespace sea {
namespace {

using namespace tc;

constexpr int kTile = 128;                // queries per work item, keys per tile
constexpr int kTileBytes = kTile * 128;   // 128 rows x 64 bf16
constexpr int kNK = 4;                    // K ring stages
constexpr int kNV = 3;                    // V ring stages
constexpr int kSplit = 2;                 // row warpgroups: each takes 128 / kSplit columns of every tile
constexpr int kRowWarps = 4 * kSplit;
constexpr int kRowThreads = 32 * kRowWarps;
constexpr int kThreads = 128 * (kSplit + 2);  // warpgroups: control, kSplit x row warps, P writers
constexpr int kChunks = 4 / kSplit;       // 32-column chunks per row thread and tile
// Registers per thread after the warpgroups re-balance.  A warpgroup can only grow by what the
// others of this CTA have given back, so over the warpgroups they sum to no more than the launch
// allocation (kSplit 2: 4 x 128, kSplit 4: 6 x 80), or the growing warps would wait for ever.
constexpr int kRegsLaunch = kSplit == 2 ? 128 : 80;
constexpr int kRegsCtl = kSplit == 2 ? 40 : 32;
constexpr int kRegsRow = kSplit == 2 ? 200 : 96;
constexpr int kRegsFix = kSplit == 2 ? 72 : 64;
static_assert(kRegsCtl + kSplit * kRegsRow + kRegsFix <= kRegsLaunch * (kSplit + 2), "register re-balance exceeds the launch allocation");
static_assert(kRegsLaunch * kThreads <= 65536, "launch allocation exceeds the register file");
constexpr uint32_t kTmemCols = 512;
constexpr int kNS = 3;                    // S / P buffers of 128 columns: the MMAs run up to two tiles ahead of the rows
constexpr uint32_t kColS = 0;
constexpr uint32_t kColO = 128 * kNS;     // the output accumulators of the two column halves, 64 columns each
constexpr float kLazyBits = 8.f;          // the reference may lag the running maximum by 2^8
static_assert(kColO + 128 <= kTmemCols, "tensor memory budget");

// Barrier indices inside the shared-memory barrier block.
enum {
  kBarQFull = 0,                 // [2]
  kBarQEmpty = 2,                // [2]
  kBarKFull = 4,                 // [kNK]
  kBarKEmpty = kBarKFull + kNK,  // [kNK]
  kBarVFull = kBarKEmpty + kNK,  // [kNV]
  kBarVEmpty = kBarVFull + kNV,  // [kNV]
  kBarSFull = kBarVEmpty + kNV,  // [kNS]  S tile written by the MMA
  kBarSDone = kBarSFull + kNS,   // [kNS][kSplit]  a column half of P written over the S tile (and, for an item's first tile, the previous item's output read)
  kBarOFull = kBarSDone + kNS * kSplit,  // [2]  the item's last P V product has finished (items alternate between the two)
  kBarBitsFull = kBarOFull + 2,       // [2]  the item's mask bits have landed
  kBarBitsEmpty = kBarBitsFull + 2,   // [2]
  kBarFixFull = kBarBitsEmpty + 2,    // [2]  row normalisers handed to the P writers
  kBarFixEmpty = kBarFixFull + 2,     // [2]
  kBarPFree = kBarFixEmpty + 2,       // [kNS]  the P V product has consumed the buffer
  kBarDrain = kBarPFree + kNS,        // [1]
  kBarDrain2 = kBarDrain + 1,         // [1]
  kNumBars = kBarDrain2 + 1
};

__device__ __forceinline__ float ex2(float x) {  // 2^x; x = -inf gives 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// Instruction descriptors (kind::f16): fp32 accumulator, bf16 operands, M = 128.
constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
// B = V tile read MN-major (keys are its K index), N = 64.
constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

// The four MMAs of S = Q K^T (contraction steps of 16 along d; a step moves both descriptors on by
// 32 bytes).  All operands are formed before the block, so that the issuing thread, which shares
// its scheduler with row warps, spends one instruction per MMA inside it.
__device__ __forceinline__ void issue_qk_mmas(uint32_t d_tmem, uint64_t q_desc, uint64_t k_desc) {
  const uint64_t q1 = q_desc + 2, q2 = q_desc + 4, q3 = q_desc + 6;
  const uint64_t k1 = k_desc + 2, k2 = k_desc + 4, k3 = k_desc + 6;
  asm volatile(
      "{\n .reg .pred pz, pt;\n"
      "setp.ne.b32 pz, %0, %0;\n setp.eq.b32 pt, %0, %0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %5, %9, pz;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %2, %6, %9, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %3, %7, %9, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %4, %8, %9, pt;\n"
      "}\n"
      ::"r"(d_tmem), "l"(q_desc), "l"(q1), "l"(q2), "l"(q3), "l"(k_desc), "l"(k1), "l"(k2), "l"(k3), "r"(kIdescQK)
      : "memory");
}
// Eight of the sixteen MMAs of O += P V for one key tile (contraction steps 4 h .. 4 h + 3): step
// k takes the head of P from columns 32 (k / 2) + 8 (k % 2) of the buffer, the remainder from 16
// columns further on, and keys 16 k .. 16 k + 15 of the V stage (2048 bytes per step).
// `accumulate` is 0 only for the very first MMA of a work item.
__device__ __forceinline__ void issue_pv_half(uint32_t d_tmem, uint32_t p_tmem, uint64_t v_desc, int h, uint32_t accumulate) {
  const uint32_t pa = p_tmem + 64 * h;
  const uint64_t vd = v_desc + 512 * h;
  const uint32_t a1 = pa + 16, a2 = pa + 8, a3 = pa + 24, a4 = pa + 32, a5 = pa + 48, a6 = pa + 40, a7 = pa + 56;
  const uint64_t v1 = vd + 128, v2 = vd + 256, v3 = vd + 384;
  asm volatile(
      "{\n .reg .pred pf, pt;\n"
      "setp.ne.b32 pf, %14, 0;\n setp.eq.b32 pt, %0, %0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %9, %13, pf;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%2], %9, %13, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%3], %10, %13, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%4], %10, %13, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%5], %11, %13, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%6], %11, %13, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%7], %12, %13, pt;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%8], %12, %13, pt;\n"
      "}\n"
      ::"r"(d_tmem), "r"(pa), "r"(a1), "r"(a2), "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7), "l"(vd), "l"(v1), "l"(v2),
        "l"(v3), "r"(kIdescPV), "r"(accumulate)
      : "memory");
}

struct TcParams {
  const __nv_bfloat16* Q;       // unused by the kernel body (TMA reads it); kept for clarity
  const int32_t* row_ptr;
  const uint32_t* mask_bits;    // [rows][words] one bit per compressed column
  __nv_bfloat16* O;
  __nv_bfloat16* P;
  float* p_scratch;             // unnormalised probabilities of kept keys: row `row` parks its runs at
  const int32_t* park_off;      // park_off[row] (negative: nowhere), or at row * k_hat * r when this is null
  int32_t* status;
  const uint32_t* tile_live;    // [work items][live_words] a bit per key tile: some row of the item keeps a key of it
  const uint32_t* some_tile_unused;  // [n_unused_flags] non-zero: some item has a key tile in which none of its rows keeps a key
  int n_unused_flags;
  int BH, T, words, log2r, k_hat, causal, live_words;
  float scale_log2;
};

// The key tiles of a work item that its rows keep a key of, a bit per tile, read an item ahead.
// Tiles that no row of the item selected anything in are not visited at all: no copy, no product,
// no row work.  Walking a list that is only known on the device costs every role time on every tile
// (the loops' bounds and counters no longer live in uniform registers), so the kernel exists twice:
// kSkip = true walks the lists, kSkip = false visits every tile; both are launched, and the one
// that the mask does not call for (tile_live[-1]: some tile of some item is unused) returns at once.
constexpr int kLiveWords = 8;  // T <= 32768
template <bool kSkip>
struct LiveTiles {
  uint32_t w[kSkip ? kLiveWords : 1];
};
template <bool kSkip>
__device__ __forceinline__ LiveTiles<kSkip> load_live_tiles(const TcParams& p, int item) {  // item < 0: none
  LiveTiles<kSkip> lt;
  if constexpr (kSkip) {
    const uint32_t* src = p.tile_live + (size_t)(item < 0 ? 0 : item) * p.live_words;
#pragma unroll
    for (int i = 0; i < kLiveWords; ++i) lt.w[i] = (item >= 0 && i < p.live_words) ? __ldg(src + i) : 0u;
  } else {
    lt.w[0] = 0u;
  }
  return lt;
}
// The first tile to visit that is >= from (from >= 0), or -1.
template <bool kSkip>
__device__ __forceinline__ int next_live_tile(const LiveTiles<kSkip>& lt, int from, int nt) {
  if constexpr (!kSkip) return from < nt ? from : -1;
  int t = -1;
#pragma unroll
  for (int i = 0; i < (kSkip ? kLiveWords : 1); ++i) {
    const int skip = from - 32 * i;  // bits of this word below `from`
    uint32_t m = lt.w[i];
    if (skip >= 32) m = 0u;
    else if (skip > 0) m &= 0xffffffffu << skip;
    if (t < 0 && m != 0u) t = 32 * i + __ffs((int)m) - 1;
  }
  return t < nt ? t : -1;
}

// The k-th work item of this CTA, or -1 when it has no more.  Items are numbered in order of
// descending cost and dealt out to the CTAs stripe by stripe, back and forth (the CTA that got a
// stripe's most expensive item gets the next stripe's cheapest), which evens out the CTAs' totals
// without any exchange between them.
__device__ __forceinline__ int cta_item(int k, int n_items) {
  const int g = (int)gridDim.x, c = (int)blockIdx.x;
  const int item = k * g + ((k & 1) ? g - 1 - c : c);
  return item < n_items ? item : -1;
}

struct Item {
  int bh, qt, nt, row0;
};
__device__ __forceinline__ Item decode_item(int item, const TcParams& p) {
  // items in order of descending cost: the last query tile of every head first
  Item it;
  const int ntq = p.T / kTile;
  it.qt = ntq - 1 - item / p.BH;
  it.bh = item - (item / p.BH) * p.BH;
  it.nt = p.causal ? it.qt + 1 : ntq;
  it.row0 = it.bh * p.T + it.qt * kTile;
  return it;
}

// Bits of the compressed columns that key tile t touches (L < 7: 128 >> L columns; else 1),
// and the offset (in keys) inside the row's run list at which the tile's first column starts
// if it is selected.  my_bits: the row's bit string, `words` consecutive words.
template <int L>
__device__ __forceinline__ uint32_t tile_bits(const uint32_t* my_bits, int t, int log2r, int rank_base, int& off0) {
  if constexpr (L < 7) {
    constexpr int G = 128 >> L;
    const int first = t * G;
    const uint32_t w = my_bits[first >> 5];
    off0 = rank_base << L;
    return G == 32 ? w : (w >> (first & 31)) & ((1u << G) - 1u);
  } else {
    const int sh = log2r - 7;
    const int col = t >> sh;
    off0 = (rank_base << log2r) + ((t - (col << sh)) << 7);
    return (my_bits[col >> 5] >> (col & 31)) & 1u;
  }
}
template <int L>
__device__ __forceinline__ int next_rank(int rank_base, uint32_t tb, int t, int log2r) {
  if constexpr (L < 7) return rank_base + __popc(tb);
  const int sh = log2r - 7;
  return (((t + 1) >> sh) != (t >> sh)) ? rank_base + (int)tb : rank_base;
}

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;\n" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// Exponents of one 32-column chunk (kept apart from the scores, which the parking stores still
// read): x = s * cs + bias with bias = -(reference, in the
// exponent's units) for kept columns and -inf otherwise (chunk cg of the tile; lim = last kept
// column inside the chunk on the diagonal tile).  Returns the maximum of mx and the exponents.
template <int L, bool kDiag>
__device__ __forceinline__ float chunk_exponents(const uint32_t (&v)[32], uint32_t (&x)[32], uint32_t tb, int cg, int lim,
                                                 float cs, float neg_ref, float mx) {
  constexpr int R = 1 << (L < 5 ? L : 5);  // columns of this chunk per group
  const float2 cs2 = make_float2(cs, cs);
  float m0 = mx, m1 = -INFINITY;
#pragma unroll
  for (int gi = 0; gi < 32 / R; ++gi) {
    const int g = L >= 7 ? 0 : ((32 * cg) >> L) + (L < 5 ? gi : 0);
    const float bias = (tb >> g) & 1u ? neg_ref : -INFINITY;
#pragma unroll
    for (int e2 = gi * R / 2; e2 < (gi + 1) * R / 2; ++e2) {
      const float b0 = (!kDiag || 2 * e2 <= lim) ? bias : -INFINITY;
      const float b1 = (!kDiag || 2 * e2 + 1 <= lim) ? bias : -INFINITY;
      const float2 xx = __ffma2_rn(make_float2(__uint_as_float(v[2 * e2]), __uint_as_float(v[2 * e2 + 1])), cs2, make_float2(b0, b1));
      x[2 * e2] = __float_as_uint(xx.x);
      x[2 * e2 + 1] = __float_as_uint(xx.y);
      if (e2 & 1) m1 = fmax3(m1, xx.x, xx.y); else m0 = fmax3(m0, xx.x, xx.y);
    }
  }
  return fmaxf(m0, m1);
}

// Probabilities of one 32-column chunk from its exponents: p = 2^(x - adj); the row sum grows by
// them; hi / lo receive the bf16 head (truncated) and the bf16 remainder, two columns per word.
__device__ __forceinline__ void chunk_probs(const uint32_t (&v)[32], float adj, float2& la, float2& lb, uint32_t (&hi)[16],
                                            uint32_t (&lo)[16]) {
  const float2 m1 = make_float2(-1.f, -1.f);
#pragma unroll
  for (int e2 = 0; e2 < 16; ++e2) {
    const float2 pp = make_float2(ex2(__uint_as_float(v[2 * e2]) - adj), ex2(__uint_as_float(v[2 * e2 + 1]) - adj));
    if (e2 & 1) lb = __fadd2_rn(lb, pp); else la = __fadd2_rn(la, pp);
    const uint32_t h0 = __float_as_uint(pp.x) & 0xffff0000u, h1 = __float_as_uint(pp.y) & 0xffff0000u;
    hi[e2] = __byte_perm(h0, h1, 0x7632);
    const float2 rem = __ffma2_rn(make_float2(__uint_as_float(h0), __uint_as_float(h1)), m1, pp);  // p - head, exact
    const __nv_bfloat162 l2 = __floats2bfloat162_rn(rem.x, rem.y);
    lo[e2] = *reinterpret_cast<const uint32_t*>(&l2);
  }
}

// Parks the raw scores of the kept groups of one 32-column chunk: run `rank` of the row starts at
// rank * r floats inside the row's part of the scratch array (the writers cut a causal row's last
// run by the row's length, so whole groups are stored).
template <int L>
__device__ __forceinline__ void chunk_park(const uint32_t (&v)[32], uint32_t tb, int cg, float* my_scratch, int rank_base,
                                           int off0) {
  constexpr int R = 1 << (L < 5 ? L : 5);
#pragma unroll
  for (int gi = 0; gi < 32 / R; ++gi) {
    const int g = L >= 7 ? 0 : ((32 * cg) >> L) + (L < 5 ? gi : 0);
    if ((tb >> g) & 1u) {
      const int off = L >= 7 ? off0 + 32 * cg
                             : ((rank_base + __popc(tb & ((1u << g) - 1u))) << L) + (32 * cg + gi * R - (g << L));
      uint4* dst = reinterpret_cast<uint4*>(my_scratch + off);
#pragma unroll
      for (int e4 = 0; e4 < R / 4; ++e4)
        dst[e4] = make_uint4(v[gi * R + 4 * e4], v[gi * R + 4 * e4 + 1], v[gi * R + 4 * e4 + 2], v[gi * R + 4 * e4 + 3]);
    }
  }
}

// AND of a predicate over the row threads (named barrier 1); also orders their memory accesses.
__device__ __forceinline__ bool rows_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.and.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(r) : "r"((uint32_t)ok), "n"(kRowThreads) : "memory");
  return r != 0;
}

constexpr int kBarBlockBytes = (8 * kNumBars + 8 + 15) / 16 * 16;  // barriers, tensor-memory slot, abort flag

template <int kRegs>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegs)); }
template <int kRegs>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegs)); }

template <int L, bool kWriteP, bool kSkip>
__global__ void __launch_bounds__(kThreads, 1)
sparse_attn_tiles_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                            const __grid_constant__ CUtensorMap map_v, const TcParams p) {
  {
    int unused = 0;
    for (int i = threadIdx.x; i < p.n_unused_flags; i += kThreads) unused |= (int)__ldg(p.some_tile_unused + i);
    if (kSkip != (__syncthreads_or(unused) != 0)) return;  // the other instance of the kernel does the work
  }
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* sm = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const uint32_t sQ = smem_u32(sm);                          // 2 x 16 KB
  const uint32_t sK = sQ + 2 * kTileBytes;                   // kNK x 16 KB
  const uint32_t sV = sK + kNK * kTileBytes;                 // kNV x 16 KB
  unsigned char* tail = sm + (2 + kNK + kNV) * kTileBytes;
  const uint32_t bars = smem_u32(tail);                      // kNumBars x 8 B
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8 * kNumBars + 4);
  // the arrays begin on a 16-byte boundary: the mask bits at their end are the target of a bulk copy
  float* xch_m = reinterpret_cast<float*>(tail + kBarBlockBytes);       // [2 items][kSplit][128] the halves' references
  float* xch_l = xch_m + 2 * kSplit * kTile;                             // [2 items][kSplit][128] the halves' sums
  float* fix_inv = xch_l + 2 * kSplit * kTile;                           // [2 slots][128] 1 / row sum
  float* fix_nmc = fix_inv + 2 * kTile;                                  // [2][128] -(row reference, in the exponent's units)
  int* fix_base = reinterpret_cast<int*>(fix_nmc + 2 * kTile);           // [2][128]
  int* fix_cnt = fix_base + 2 * kTile;                                   // [2][128]
  int* fix_off = fix_cnt + 2 * kTile;                                    // [2][128]
  uint32_t* bits = reinterpret_cast<uint32_t*>(fix_off + 2 * kTile);     // [2 slots][128 rows][words]
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < kNumBars; ++i) {
      uint32_t count = 1;
      if (i >= kBarBitsEmpty && i < kBarBitsEmpty + 2) count = kRowWarps;  // one arrival per row warp
      if (i >= kBarSDone && i < kBarSDone + kNS * kSplit) count = 4;       // one arrival per row warp of the half
      if ((i >= kBarFixFull && i < kBarFixFull + 2) || (i >= kBarFixEmpty && i < kBarFixEmpty + 2)) count = 4;
      mbar_init(bar(i), count);
    }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_items = p.BH * (p.T / kTile);
  const uint32_t bits_bytes = (uint32_t)(kTile * p.words * 4);

  if (warp < 4) {
    reg_dec<kRegsCtl>();
    if (warp == 0 && lane == 0) {
      // ---------------------------------------------------------------- TMA producer
      uint32_t q_it = 0, k_it = 0, v_it = 0;
      bool ok = true;
      LiveTiles<kSkip> live_next = load_live_tiles<kSkip>(p, cta_item(0, n_items));  // read an item ahead: the latency hides behind the item before
      for (int k = 0, item; (item = cta_item(k, n_items)) >= 0 && ok; ++k) {
        const Item it = decode_item(item, p);
        const uint32_t qb = q_it & 1;
        ok = mbar_wait<100>(bar(kBarBitsEmpty + qb), ((q_it >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(bar(kBarBitsFull + qb), bits_bytes);
        bulk_load(smem_u32(bits) + qb * bits_bytes, p.mask_bits + (size_t)it.row0 * p.words, bits_bytes, bar(kBarBitsFull + qb));
        ok = mbar_wait<100>(bar(kBarQEmpty + qb), ((q_it >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(bar(kBarQFull + qb), kTileBytes);
        tma_load_2d(sQ + qb * kTileBytes, &map_q, 0, it.row0, bar(kBarQFull + qb));
        ++q_it;
        const LiveTiles<kSkip> live = live_next;
        live_next = load_live_tiles<kSkip>(p, cta_item(k + 1, n_items));
        for (int t = next_live_tile<kSkip>(live, 0, it.nt); t >= 0; t = next_live_tile<kSkip>(live, t + 1, it.nt)) {
          const uint32_t ks = k_it % kNK;
          ok = mbar_wait<100>(bar(kBarKEmpty + ks), ((k_it / kNK) & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(bar(kBarKFull + ks), kTileBytes);
          tma_load_2d(sK + ks * kTileBytes, &map_k, 0, it.bh * p.T + t * kTile, bar(kBarKFull + ks));
          ++k_it;
          const uint32_t vs = v_it % kNV;
          ok = mbar_wait<100>(bar(kBarVEmpty + vs), ((v_it / kNV) & 1) ^ 1, abort_flag);
          if (!ok) break;
          mbar_expect_tx(bar(kBarVFull + vs), kTileBytes);
          tma_load_2d(sV + vs * kTileBytes, &map_v, 0, it.bh * p.T + t * kTile, bar(kBarVFull + vs));
          ++v_it;
        }
      }
      // copies still in flight must land before the CTA may leave: wait for the last use of every stage
      for (uint32_t i = (k_it > kNK ? k_it - kNK : 0); i < k_it; ++i) mbar_wait_drain(bar(kBarKFull + i % kNK), (i / kNK) & 1);
      for (uint32_t i = (v_it > kNV ? v_it - kNV : 0); i < v_it; ++i) mbar_wait_drain(bar(kBarVFull + i % kNV), (i / kNV) & 1);
      for (uint32_t i = (q_it > 2 ? q_it - 2 : 0); i < q_it; ++i) {
        mbar_wait_drain(bar(kBarQFull + (i & 1)), (i >> 1) & 1);
        mbar_wait_drain(bar(kBarBitsFull + (i & 1)), (i >> 1) & 1);
      }
    } else if (warp == 1) {
      // ---------------------------------------------------------------- issuer of S = Q K^T
      // S/P buffer u % kNS serves use u (tile after tile, item after item).  Before a buffer is
      // written again the P V product of its previous use must have consumed it (barrier PFree,
      // committed by the other issuer, one phase per use).
      uint32_t q_it = 0, k_it = 0;
      uint32_t b = 0, round = 0;  // use round * kNS + b occupies buffer b
      const uint64_t k_desc0 = smem_desc(sK, 16, 1024);  // a stage further on: + 16 KB / 16
      bool ok = true;
      LiveTiles<kSkip> live_next = load_live_tiles<kSkip>(p, cta_item(0, n_items));  // read an item ahead: the latency hides behind the item before
      for (int k = 0, item; (item = cta_item(k, n_items)) >= 0 && ok; ++k) {
        const Item it = decode_item(item, p);
        const uint32_t qb = q_it & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarQFull + qb), (q_it >> 1) & 1, abort_flag));
        const uint64_t q_desc = smem_desc(sQ + qb * kTileBytes, 16, 1024);
        const LiveTiles<kSkip> live = live_next;
        live_next = load_live_tiles<kSkip>(p, cta_item(k + 1, n_items));
        for (int t = next_live_tile<kSkip>(live, 0, it.nt), t_next; t >= 0 && ok; t = t_next) {
          t_next = next_live_tile<kSkip>(live, t + 1, it.nt);
          const uint32_t ks = k_it % kNK;
          const uint32_t kbar = bar(kBarKFull + ks), kpar = (k_it / kNK) & 1;
          if (round > 0) ok = __all_sync(0xffffffffu, mbar_wait2(bar(kBarPFree + b), (round & 1u) ^ 1u, kbar, kpar, abort_flag));
          else ok = __all_sync(0xffffffffu, mbar_wait(kbar, kpar, abort_flag));
          if (!ok) break;
          fence_after();
          if (elect_one()) {
            issue_qk_mmas(tmem + kColS + 128 * b, q_desc, k_desc0 + 1024ull * ks);
            mma_commit(bar(kBarKEmpty + ks));
            mma_commit(bar(kBarSFull + b));
            if (t_next < 0) mma_commit(bar(kBarQEmpty + qb));
          }
          __syncwarp();
          ++k_it;
          if (++b == (uint32_t)kNS) {
            b = 0;
            ++round;
          }
        }
        ++q_it;
      }
      // every MMA issued by this thread must have finished before tensor memory is released
      if (elect_one()) mma_commit(bar(kBarDrain));
      __syncwarp();
      mbar_wait(bar(kBarDrain), 0, abort_flag);
      __syncwarp();
    } else if (warp == 2) {
      // ---------------------------------------------------------------- issuer of O_h += P_h V
      uint32_t v_it = 0, o_it = 0;
      uint32_t b = 0, round = 0;
      const uint64_t v_desc0 = smem_desc(sV, 8192, 1024);  // a stage further on: + 16 KB / 16
      bool ok = true;
      LiveTiles<kSkip> live_next = load_live_tiles<kSkip>(p, cta_item(0, n_items));  // read an item ahead: the latency hides behind the item before
      for (int k = 0, item; (item = cta_item(k, n_items)) >= 0 && ok; ++k) {
        const Item it = decode_item(item, p);
        const LiveTiles<kSkip> live = live_next;
        live_next = load_live_tiles<kSkip>(p, cta_item(k + 1, n_items));
        const int t_first = next_live_tile<kSkip>(live, 0, it.nt);
        for (int t = t_first, t_next; t >= 0 && ok; t = t_next) {
          t_next = next_live_tile<kSkip>(live, t + 1, it.nt);
          const bool first = t == t_first;
          // the rows have written P (and, before an item's first tile, read the previous item's output)
          // Each column half has its own accumulator and its own barrier, so a half's product starts as
          // soon as its rows are done.  Every row thread reads both accumulators when an item ends: the
          // first product of an item waits for both halves.
          const uint32_t vs = v_it % kNV;
          ok = __all_sync(0xffffffffu, mbar_wait2(bar(kBarSDone + kSplit * b), round & 1u, bar(kBarVFull + vs), (v_it / kNV) & 1, abort_flag));
          if (ok && first) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSDone + kSplit * b + 1), round & 1u, abort_flag));
          if (!ok) break;
          fence_after();
          const uint64_t vd = v_desc0 + 1024ull * vs;
          if (elect_one()) issue_pv_half(tmem + kColO, tmem + kColS + 128 * b, vd, 0, first ? 0u : 1u);
          __syncwarp();
          if (!first) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSDone + kSplit * b + 1), round & 1u, abort_flag));
            if (!ok) break;
            fence_after();
          }
          if (elect_one()) {
            issue_pv_half(tmem + kColO + 64, tmem + kColS + 128 * b, vd, 1, first ? 0u : 1u);
            mma_commit(bar(kBarVEmpty + vs));
            mma_commit(bar(kBarPFree + b));
            if (t_next < 0) mma_commit(bar(kBarOFull + (o_it & 1)));
          }
          __syncwarp();
          ++v_it;
          if (++b == (uint32_t)kNS) {
            b = 0;
            ++round;
          }
        }
        ++o_it;
      }
      if (elect_one()) mma_commit(bar(kBarDrain2));
      __syncwarp();
      mbar_wait(bar(kBarDrain2), 0, abort_flag);
      __syncwarp();
    }
  } else if (warp < 4 + kRowWarps) {
    // ---------------------------------------------------------------- row warps: a query row and
    // 128 / kSplit of every tile's columns per thread
    reg_inc<kRegsRow>();
    const int quarter = warp & 3;          // tensor-memory lanes 32*quarter .. +31
    const int part = (warp - 4) >> 2;      // columns (128 / kSplit) * part .. of every tile
    const int rt = quarter * 32 + lane;    // row inside the work item
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const uint32_t my_o = lane_addr + kColO + 64 * part;  // this half's accumulator row
    const int log2r = p.log2r;
    const int KR = p.k_hat << log2r;
    const float cs = p.scale_log2;
    uint32_t b = 0, round = 0, it_cnt = 0;  // use round * kNS + b of the S / P buffers
    bool ok = true;
    struct {
      bool active;
      float w0, w1, inv, nmc;  // weights of the two halves' accumulators (normaliser included), 1 / sum, -(row reference)
      int row, p_base, p_cnt, p_off;
      uint32_t it_cnt;
    } pend = {false, 0.f, 0.f, 0.f, 0.f, 0, 0, 0, 0, 0u};
    // Output row of the pending item (this thread: 32 of its columns, from both halves'
    // accumulators), and the hand-over of the rows' normalisers to the warps that write P.
    auto epilogue = [&]() -> bool {
      if (!pend.active) return true;
      pend.active = false;
      const uint32_t pslot = pend.it_cnt & 1;
      bool good = __all_sync(0xffffffffu, mbar_wait(bar(kBarOFull + pslot), (pend.it_cnt >> 1) & 1, abort_flag));
      if (!good) return false;
      fence_after();
      constexpr int kOC = 64 / kSplit;
      static_assert(kOC == 32, "the output row is read 32 columns at a time");
      uint32_t o0[kOC], o1[kOC];
      tmem_ld32(lane_addr + kColO + kOC * part, o0);
      tmem_ld32(lane_addr + kColO + 64 + kOC * part, o1);
      tmem_ld_wait();
      fence_before();
      uint4* out = reinterpret_cast<uint4*>(p.O + (size_t)pend.row * kHeadDim + kOC * part);
#pragma unroll
      for (int e = 0; e < kOC / 8; ++e) {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float x = __uint_as_float(o0[8 * e + 2 * k]) * pend.w0 + __uint_as_float(o1[8 * e + 2 * k]) * pend.w1;
          const float y = __uint_as_float(o0[8 * e + 2 * k + 1]) * pend.w0 + __uint_as_float(o1[8 * e + 2 * k + 1]) * pend.w1;
          const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
          w[k] = *reinterpret_cast<const uint32_t*>(&h);
        }
        out[e] = make_uint4(w[0], w[1], w[2], w[3]);
      }
      if (kWriteP && part == 0) {
        good = __all_sync(0xffffffffu, mbar_wait(bar(kBarFixEmpty + pslot), ((pend.it_cnt >> 1) & 1) ^ 1, abort_flag));
        if (!good) return false;
        fix_inv[pslot * kTile + rt] = pend.inv;
        fix_nmc[pslot * kTile + rt] = pend.nmc;
        fix_base[pslot * kTile + rt] = pend.p_base;
        fix_cnt[pslot * kTile + rt] = pend.p_cnt;
        fix_off[pslot * kTile + rt] = pend.p_off;
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarFixFull + pslot));
      }
      return true;
    };
    LiveTiles<kSkip> live_next = load_live_tiles<kSkip>(p, cta_item(0, n_items));  // read an item ahead: the latency hides behind the item before
    for (int k = 0, item; (item = cta_item(k, n_items)) >= 0; ++k, ++it_cnt) {
      const Item it = decode_item(item, p);
      const int row = it.row0 + rt;
      const uint32_t slot = it_cnt & 1;
      int p_base = 0, p_cnt = 0, p_off = 0;
      bool park = kWriteP;
      if (kWriteP) {
        p_off = p.park_off != nullptr ? __ldg(p.park_off + row) : row * KR;
        if (p_off < 0) {  // the row has no place in the parking area: its P entries are not produced
          park = false;
          p_off = 0;
        }
        if (part == 0 && park) {
          p_base = __ldg(p.row_ptr + row);
          p_cnt = __ldg(p.row_ptr + row + 1) - p_base;
        }
      }
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarBitsFull + slot), (it_cnt >> 1) & 1, abort_flag));
      const uint32_t* my_bits = bits + slot * (kTile * p.words) + rt * p.words;
      float* my_scratch = kWriteP ? p.p_scratch + p_off : nullptr;
      float mb = -INFINITY;  // this half's reference in the exponent's units (score * cs); -inf while it has met no kept score
      float2 la = make_float2(0.f, 0.f), lb = make_float2(0.f, 0.f);
      int rank_base = 0;
      const LiveTiles<kSkip> live = live_next;
      live_next = load_live_tiles<kSkip>(p, cta_item(k + 1, n_items));
      const int t_first = next_live_tile<kSkip>(live, 0, it.nt);
      for (int t = t_first; t >= 0 && ok; t = next_live_tile<kSkip>(live, t + 1, it.nt)) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull + b), round & 1u, abort_flag));
        if (!ok) break;
        fence_after();
        int off0;
        const uint32_t tb = tile_bits<L>(my_bits, t, log2r, rank_base, off0);
        const uint32_t src = lane_addr + kColS + 128 * b + 32 * kChunks * part;
        uint32_t v[kChunks][32];
#pragma unroll
        for (int c = 0; c < kChunks; ++c) tmem_ld32(src + 32 * c, v[c]);
        tmem_ld_wait();
        const bool diag = p.causal && t == it.qt;
        // exponents under the current reference (0 while there is none), and their maximum
        const float neg_ref = mb == -INFINITY ? 0.f : -mb;
        float mx = -INFINITY;
        uint32_t x[kChunks][32];
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          const int cg = kChunks * part + c;
          if (kWriteP && park) chunk_park<L>(v[c], tb, cg, my_scratch, rank_base, off0);
          if (diag) mx = chunk_exponents<L, true>(v[c], x[c], tb, cg, rt - 32 * cg, cs, neg_ref, mx);
          else mx = chunk_exponents<L, false>(v[c], x[c], tb, cg, 0, cs, neg_ref, mx);
        }
        // The reference moves to the tile's maximum when that lies more than kLazyBits above it, or
        // when this is the row half's first kept score; the exponents then shift by adj.
        const bool raise = mb == -INFINITY ? mx > -INFINITY : mx > kLazyBits;
        float adj = 0.f;
        if (__any_sync(0xffffffffu, raise)) {
          // What the row has accumulated under the old reference is multiplied by 2^-adj; with no
          // kept score so far the sum and the accumulator row are exactly zero and stay so.
          const bool rescale = raise && mb != -INFINITY;
          if (raise) {
            adj = mx;
            mb = rescale ? mb + mx : mx;
          }
          const float f = rescale ? ex2(-adj) : 1.f;
          la.x *= f; la.y *= f; lb.x *= f; lb.y *= f;
          if (__any_sync(0xffffffffu, rescale)) {
            // rare: the P V products issued so far (the last one belongs to the previous use) must have finished
            const uint32_t pb = b == 0 ? kNS - 1 : b - 1, pround = b == 0 ? round - 1 : round;
            ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarPFree + pb), pround & 1u, abort_flag));
            if (!ok) break;
            fence_after();
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t o[16];
              tmem_ld16(my_o + 16 * c, o);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
              tmem_st16(my_o + 16 * c, o);
            }
          }
        }
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          uint32_t hi[16], lo[16];
          chunk_probs(x[c], adj, la, lb, hi, lo);
          tmem_st16(src + 32 * c, hi);
          tmem_st16(src + 32 * c + 16, lo);
        }
        rank_base = next_rank<L>(rank_base, tb, t, log2r);
        // the previous item's output row leaves the accumulators before this item's first product
        // may overwrite them: by now that item's last product has long finished
        if (t == t_first && !epilogue()) {
          ok = false;
          break;
        }
        tmem_st_wait();
        fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarSDone + kSplit * b + part));
        if (++b == (uint32_t)kNS) {
          b = 0;
          ++round;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(kBarBitsEmpty + slot));
      // The halves exchange their references and sums.  Items alternate between two exchange areas:
      // a thread can only write an area again after the barrier of the item in between, which every
      // thread reaches after it has read what it needs here.
      float* xm = xch_m + slot * (kSplit * kTile);
      float* xl = xch_l + slot * (kSplit * kTile);
      xm[part * kTile + rt] = mb;
      xl[part * kTile + rt] = (la.x + la.y) + (lb.x + lb.y);
      ok = rows_all(ok);
      if (!ok) break;
      {
        const float m0 = xm[rt], m1 = xm[kTile + rt];
        const float M = fmaxf(m0, m1);
        const float w0 = m0 == -INFINITY ? 0.f : ex2(m0 - M);  // a half without kept scores has weight 0
        const float w1 = m1 == -INFINITY ? 0.f : ex2(m1 - M);
        const float l = xl[rt] * w0 + xl[kTile + rt] * w1;
        const float inv = l > 0.f ? 1.f / l : 0.f;
        // the item's output row is written while the next item's first tile is worked on; remember
        // what that needs
        pend.active = true;
        pend.w0 = w0 * inv;
        pend.w1 = w1 * inv;
        pend.inv = inv;
        pend.nmc = M == -INFINITY ? 0.f : -M;
        pend.row = row;
        pend.it_cnt = it_cnt;
        pend.p_base = p_base;
        pend.p_cnt = p_cnt;
        pend.p_off = p_off;
      }
    }
    if (ok) ok = epilogue();
  } else {
    // ---------------------------------------------------------------- P writers: 32 rows per warp
    reg_dec<kRegsFix>();
    if (kWriteP) {
      const int w4 = warp - (4 + kRowWarps);
      const float cs = p.scale_log2;
      uint32_t it_cnt = 0;
      bool ok = true;
      for (int k = 0, item; (item = cta_item(k, n_items)) >= 0 && ok; ++k, ++it_cnt) {
        const uint32_t slot = it_cnt & 1;
        ok = __all_sync(0xffffffffu, mbar_wait<500>(bar(kBarFixFull + slot), (it_cnt >> 1) & 1, abort_flag));
        if (!ok) break;
        // P = 2^((parked score - M) cs) / row sum, rounded once.  Rows are taken eight at a time, in
        // slices of 128 keys (one 16-byte load per lane and row), so that eight loads are in flight.
        const int* cnt_s = fix_cnt + slot * kTile + 32 * w4;
        const int* base_s = fix_base + slot * kTile + 32 * w4;
        const float* inv_s = fix_inv + slot * kTile + 32 * w4;
        const float* nmc_s = fix_nmc + slot * kTile + 32 * w4;
        const int* off_s = fix_off + slot * kTile + 32 * w4;
        const int longest_all = __reduce_max_sync(0xffffffffu, cnt_s[lane]);
        for (int u0 = 0; u0 < longest_all; u0 += 128) {
          const int u = u0 + 4 * lane;
          for (int r0 = 0; r0 < 32; r0 += 8) {
            int longest = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) longest = max(longest, cnt_s[r0 + j]);
            if (longest <= u0) continue;  // none of these rows reaches this slice
            float4 val[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
              val[j] = u < cnt_s[r0 + j] ? __ldcg(reinterpret_cast<const float4*>(p.p_scratch + off_s[r0 + j] + u))
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int n = cnt_s[r0 + j];
              const float inv = inv_s[r0 + j], nmc = nmc_s[r0 + j];
              __nv_bfloat16* dst = p.P + (size_t)base_s[r0 + j] + u;
              const float f[4] = {ex2(fmaf(val[j].x, cs, nmc)) * inv, ex2(fmaf(val[j].y, cs, nmc)) * inv,
                                  ex2(fmaf(val[j].z, cs, nmc)) * inv, ex2(fmaf(val[j].w, cs, nmc)) * inv};
#pragma unroll
              for (int e = 0; e < 4; ++e)
                if (u + e < n) dst[e] = __float2bfloat16_rn(f[e]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(kBarFixEmpty + slot));
      }
    }
  }
  // ---------------------------------------------------------------- teardown
  fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && *abort_flag) atomicOr(p.status, SEA_DEV_TIMEOUT);
}

// One warp per work item (128 query rows): which key tiles does any of its rows keep a key of?
// The union of the rows' bit strings, then a bit per key tile; an item whose rows keep nothing at
// all still visits one tile, so that its output rows are written (as zeros) the usual way.
// unused_flags [gridDim.x]: whether some item of this block has a key tile that it does not use.
__global__ void __launch_bounds__(128)
tile_live_kernel(const uint32_t* __restrict__ mask_bits, uint32_t* __restrict__ tile_live, uint32_t* __restrict__ unused_flags,
                 int n_items, int BH, int T, int words, int log2r, int causal, int live_words) {
  __shared__ uint32_t uni_all[4][32];  // Kc <= 1024: at most 32 words
  const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int item = blockIdx.x * 4 + wid;
  int unused = 0;
  if (item < n_items) {
    uint32_t* uni = uni_all[wid];
    const int ntq = T / kTile;
    const int qt = ntq - 1 - item / BH, bh = item % BH;
    const int nt = causal ? qt + 1 : ntq;
    const uint32_t* rows = mask_bits + ((size_t)bh * T + (size_t)qt * kTile) * words;
    for (int w = 0; w < words; ++w) {
      uint32_t acc = 0u;
      for (int r = lane; r < kTile; r += 32) acc |= __ldg(rows + (size_t)r * words + w);
      acc = __reduce_or_sync(0xffffffffu, acc);
      if (lane == 0) uni[w] = acc;
    }
    __syncwarp();
    uint32_t* out = tile_live + (size_t)item * live_words;
    int n_live = 0;
    for (int w0 = 0; w0 < live_words; ++w0) {
      const int t = 32 * w0 + lane;
      bool mine = false;
      if (t < nt) {
        if (log2r >= 7) {
          const int c = t >> (log2r - 7);
          mine = (uni[c >> 5] >> (c & 31)) & 1u;
        } else {
          const int G = 128 >> log2r;  // compressed columns per key tile: 1 .. 32, never across a word
          const int c0 = t * G;
          const uint32_t m = G >= 32 ? 0xffffffffu : ((1u << G) - 1u);
          mine = ((uni[c0 >> 5] >> (c0 & 31)) & m) != 0u;
        }
      }
      const uint32_t word = __ballot_sync(0xffffffffu, mine);
      n_live += __popc(word);
      if (lane == 0) out[w0] = word;
    }
    if (n_live == 0 && lane == 0) out[0] = 1u;
    unused = n_live < nt;
  }
  unused = __syncthreads_or(unused);
  if (threadIdx.x == 0) unused_flags[blockIdx.x] = unused ? 1u : 0u;
}

// One thread per row: the ascending selected columns become a bit string of `words` words.
__global__ void sel_to_bits_kernel(const int32_t* __restrict__ sel, uint32_t* __restrict__ mask_bits, int rows, int k_hat,
                                   int words) {
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const int32_t* s = sel + (size_t)row * k_hat;
  uint32_t* out = mask_bits + (size_t)row * words;
  int cur = 0;
  uint32_t acc = 0;
  for (int e = 0; e < k_hat; ++e) {
    const int c = __ldg(s + e);
    const int w = c >> 5;
    while (cur < w && cur < words) {
      out[cur++] = acc;
      acc = 0;
    }
    acc |= 1u << (c & 31);
  }
  while (cur < words) {
    out[cur++] = acc;
    acc = 0;
  }
}

int log2_exact(int x) {
  int l = 0;
  while ((1 << l) < x) ++l;
  return (1 << l) == x ? l : -1;
}

template <int L, bool kWriteP, bool kSkip>
sea_status launch_tc_one(const sea_shape& s, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                     const TcParams& prm, cudaStream_t st) {
  const size_t smem = 1024 + (size_t)(2 + kNK + kNV) * kTileBytes + kBarBlockBytes + (size_t)(4 * kSplit + 10) * kTile * 4 +
                      2 * (size_t)prm.words * kTile * 4;
  auto kern = sparse_attn_tiles_tc_kernel<L, kWriteP, kSkip>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return SEA_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SEA_ERR_CUDA;
  const int n_items = prm.BH * (s.T / kTile);
  const int grid = n_items < sms ? n_items : sms;  // persistent: one CTA per SM (it owns all of the SM's tensor memory)
  kern<<<grid, kThreads, smem, st>>>(mq, mk, mv, prm);
  return check_launch();
}
// Both instances: the one that the mask does not call for returns at once.
template <int L, bool kWriteP>
sea_status launch_tc(const sea_shape& s, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                     const TcParams& prm, cudaStream_t st) {
  const sea_status rc = launch_tc_one<L, kWriteP, false>(s, mq, mk, mv, prm, st);
  if (rc != SEA_OK) return rc;
  return launch_tc_one<L, kWriteP, true>(s, mq, mk, mv, prm, st);
}

}  // namespace

size_t sparse_attn_tc_bits_bytes(const sea_shape& s) {
  return (size_t)s.B * s.H * s.T * (size_t)((s.Kc + 31) / 32) * sizeof(uint32_t);
}
size_t sparse_attn_tc_live_bytes(const sea_shape& s) {
  const size_t ntq = (size_t)(s.T + kTile - 1) / kTile;
  const size_t n_items = (size_t)s.B * s.H * ntq;
  return n_items * ((ntq + 31) / 32) * sizeof(uint32_t) + ((n_items + 3) / 4) * sizeof(uint32_t);  // the lists, then the flags
}
size_t sparse_attn_tc_scratch_bytes(const sea_shape& s) {
  return (size_t)s.B * s.H * s.T * (size_t)s.k_hat * (size_t)(s.T / s.Kc) * sizeof(float);
}

bool sparse_attn_tc_shape_ok(const sea_shape& s) {
  if (s.io != SEA_BF16) return false;
  const int r = s.T / s.Kc;
  if (s.T % s.Kc != 0 || s.T % kTile != 0 || log2_exact(r) < 2) return false;
  if (s.T / kTile > 32 * kLiveWords) return false;  // a bit per key tile of a work item, held in registers
  // dense tiles pay off while a row keeps at least about 1/40 of the keys it may see: measured at
  // k_hat / Kc = 1/32 the tiles take 0.77 of the per-row gather's time, at 1/64 they take 1.43 of it
  return (long long)s.k_hat * 40 >= s.Kc;
}

bool sparse_attn_tc_applicable(const sea_shape& s, const int32_t* sel, bool have_bits, const int32_t* status,
                               const void* mask_bits, const void* p_scratch) {
  if ((sel == nullptr && !have_bits) || status == nullptr || mask_bits == nullptr || p_scratch == nullptr) return false;
  return sparse_attn_tc_shape_ok(s) && tc::encode_fn() != nullptr;
}

sea_status launch_sparse_attn_tc(const sea_shape& s, const void* Q, const void* K, const void* V, const int32_t* row_ptr,
                                 const int32_t* sel, void* O, void* P, uint32_t* mask_bits, bool bits_valid,
                                 float* p_scratch, const int32_t* park_off, uint32_t* tile_live, int32_t* status,
                                 cudaStream_t st) {
  const unsigned long long rows = (unsigned long long)s.B * s.H * s.T;
  CUtensorMap mq, mk, mv;
  if (!make_rows_map_bf16(&mq, Q, rows, kTile) || !make_rows_map_bf16(&mk, K, rows, kTile) || !make_rows_map_bf16(&mv, V, rows, kTile)) return SEA_ERR_CUDA;
  TcParams prm{};
  prm.Q = static_cast<const __nv_bfloat16*>(Q);
  prm.row_ptr = row_ptr;
  prm.mask_bits = mask_bits;
  prm.O = static_cast<__nv_bfloat16*>(O);
  prm.P = static_cast<__nv_bfloat16*>(P);
  prm.p_scratch = p_scratch;
  prm.park_off = park_off;
  prm.status = status;
  prm.BH = s.B * s.H;
  prm.T = s.T;
  prm.words = (s.Kc + 31) / 32;
  prm.log2r = log2_exact(s.T / s.Kc);
  prm.k_hat = s.k_hat;
  prm.causal = s.causal;
  const float scale = s.scale != 0.f ? s.scale : 0.125f;
  prm.scale_log2 = scale * 1.4426950408889634f;

  if (!bits_valid) {
    sel_to_bits_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(sel, mask_bits, (int)rows, s.k_hat, prm.words);
    const sea_status rc = check_launch();
    if (rc != SEA_OK) return rc;
  }
  {
    const int n_items = prm.BH * (s.T / kTile);
    prm.live_words = (s.T / kTile + 31) / 32;
    prm.tile_live = tile_live;
    uint32_t* flags = tile_live + (size_t)n_items * prm.live_words;  // a word per block of the kernel below, after the lists
    prm.some_tile_unused = flags;
    prm.n_unused_flags = (n_items + 3) / 4;
    tile_live_kernel<<<prm.n_unused_flags, 128, 0, st>>>(mask_bits, tile_live, flags, n_items, prm.BH, s.T, prm.words, prm.log2r,
                                                        s.causal, prm.live_words);
    const sea_status rc = check_launch();
    if (rc != SEA_OK) return rc;
  }
  Launch::sparse_kernel() = "sparse_attn_tiles_tc_kernel";
  {
    // (an upper bound when the mask leaves whole key tiles unused: those are skipped)
    // every (query tile, key tile) pair a query tile may see: S = Q K^T and P V with P as a bf16
    // head plus a bf16 remainder, 2 * 128 * 128 * 64 FLOPs each
    const double nq = s.T / kTile;
    const double pairs = (double)s.B * s.H * (s.causal ? nq * (nq + 1) / 2 : nq * nq);
    Launch::sparse_flops() = pairs * 3.0 * (2.0 * kTile * kTile * kHeadDim);
  }
  const int L = prm.log2r < 7 ? prm.log2r : 7;
#define SEA_TC(LL)                                                                   \
  case LL:                                                                           \
    return P ? launch_tc<LL, true>(s, mq, mk, mv, prm, st) : launch_tc<LL, false>(s, mq, mk, mv, prm, st)
  switch (L) {
    SEA_TC(2);
    SEA_TC(3);
    SEA_TC(4);
    SEA_TC(5);
    SEA_TC(6);
    SEA_TC(7);
  }
#undef SEA_TC
  return SEA_ERR_UNSUPPORTED;
}

}  // namespace sea

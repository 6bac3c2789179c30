// Attention estimation for bf16 inputs on tensor-core tiles (mma.sync m16n8k16, fp32 accumulate).
//
// Same three-kernel structure as the fp32 reference form in sea_estimate.cu (chunk key states,
// fixed-order scan over chunks, per-chunk output), with every contraction on the tensor cores.
// Precision: the estimate has to agree with fp64 to 1e-3, and the feature map exponentiates a
// projection of magnitude ~10, so bf16 operands alone (2^-9) are not enough.  Every fp32 operand
// is therefore carried as a bf16 head plus a bf16 remainder (x ~ hi + lo, 2^-17 relative) and a
// product A B is evaluated as A_hi B_hi + A_hi B_lo + A_lo B_hi; Q, K and V are exact in bf16
// and need no remainder.  The scaling d^(-1/4) is folded into omega beforehand so that the
// projection's left operand stays exact.
//
// A CTA of four warps owns a chunk of 64 rows, one warp per 16 rows, FlashAttention-2 style:
// accumulator fragments of one product are repacked in registers as the A fragments of the
// next, and only operands shared between warps (omega, phi(K), V, the prefix state S, W_dec)
// live in shared memory, padded so that ldmatrix is conflict-free.
#include "sea_common.cuh"

namespace sea {
namespace {

constexpr int kC = kEstChunk;          // 64 rows per chunk
constexpr int kThreads = 128;          // 4 warps x 16 rows
constexpr int kStateCols = kHeadDim + 1;
constexpr int kPad = 8;                // bf16 elements of row padding (16 bytes)
constexpr int kLd64 = kHeadDim + kPad; // pitch of 64-wide bf16 tiles
constexpr int kWTile = 128;            // decoder columns staged per pass

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x2_t(uint32_t (&r)[2], const void* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];\n"
               : "=r"(r[0]), "=r"(r[1]) : "r"(a));
}

// (hi, lo) bf16x2 words of two floats: x ~ hi + lo.
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - __uint_as_float(hi << 16), y - __uint_as_float(hi & 0xffff0000u));
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// omega * d^(-1/4) and W_dec as bf16 head / remainder, zero padded to [MP][64] and [64][KcP].
__global__ void favor_prep_kernel(const float* __restrict__ omega, const float* __restrict__ W_dec,
                                  __nv_bfloat16* __restrict__ om_hi, __nv_bfloat16* __restrict__ om_lo,
                                  __nv_bfloat16* __restrict__ w_hi, __nv_bfloat16* __restrict__ w_lo,
                                  int m, int MP, int Kc, int KcP, float in_scale) {
  const int n_om = MP * kHeadDim, n_w = kHeadDim * KcP;
  for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < n_om + n_w; v += gridDim.x * blockDim.x) {
    float x;
    __nv_bfloat16 *hi, *lo;
    if (v < n_om) {
      x = (v / kHeadDim) < m ? omega[v] * in_scale : 0.f;
      hi = om_hi + v; lo = om_lo + v;
    } else {
      const int u = v - n_om, e = u / KcP, c = u - e * KcP;
      x = c < Kc ? W_dec[(size_t)e * Kc + c] : 0.f;
      hi = w_hi + u; lo = w_lo + u;
    }
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    *hi = h;
    *lo = __float2bfloat16_rn(x - __bfloat162float(h));
  }
}

// Copies a [rows][64] bf16 matrix (row pitch 64) into shared memory with pitch kLd64.
__device__ __forceinline__ void stage_rows64(__nv_bfloat16* dst, const __nv_bfloat16* src, int rows, int valid_rows) {
  for (int v = threadIdx.x; v < rows * 8; v += kThreads) {
    const int rr = v >> 3, cc = (v & 7) * 8;
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (rr < valid_rows) x = __ldg(reinterpret_cast<const uint4*>(src + (size_t)rr * kHeadDim + cc));
    *reinterpret_cast<uint4*>(dst + rr * kLd64 + cc) = x;
  }
}

// A fragments (4 k-steps over d = 64) of this warp's 16 rows of a bf16 [T][64] matrix, read
// straight from global memory, and |u|^2 / 16 = |x|^2 / 2 of rows g and g+8.
__device__ __forceinline__ void load_rows_frag(uint32_t (&a)[4][4], float& sq_g, float& sq_g8,
                                               const __nv_bfloat16* head, int row_g, int seq_len, int t) {
  const bool ok0 = row_g < seq_len, ok1 = row_g + 8 < seq_len;
  const uint32_t* p0 = reinterpret_cast<const uint32_t*>(head + (size_t)row_g * kHeadDim) + t;
  const uint32_t* p1 = p0 + 8 * (kHeadDim / 2);
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    a[s][0] = ok0 ? __ldg(p0 + 8 * s) : 0u;
    a[s][1] = ok1 ? __ldg(p1 + 8 * s) : 0u;
    a[s][2] = ok0 ? __ldg(p0 + 8 * s + 4) : 0u;
    a[s][3] = ok1 ? __ldg(p1 + 8 * s + 4) : 0u;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float lo = __uint_as_float(a[s][i] << 16), hi = __uint_as_float(a[s][i] & 0xffff0000u);
      if (i & 1) s1 = fmaf(lo, lo, fmaf(hi, hi, s1)); else s0 = fmaf(lo, lo, fmaf(hi, hi, s0));
    }
  }
  s0 += __shfl_xor_sync(0xffffffffu, s0, 1); s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
  s1 += __shfl_xor_sync(0xffffffffu, s1, 1); s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
  sq_g = s0 * (1.f / 16.f);
  sq_g8 = s1 * (1.f / 16.f);
}

// acc[n-tile] = rows(16) x omega'^T: the projection onto all MP features.
template <int MP>
__device__ __forceinline__ void project(float (&acc)[MP / 8][4], const uint32_t (&a)[4][4],
                                        const __nv_bfloat16* om_hi, const __nv_bfloat16* om_lo, int lane) {
#pragma unroll
  for (int j = 0; j < MP / 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
  // B = omega' stored [n = f][k = dim]; x4 covers two n-tiles x two k-halves
  const int lrow = (lane & 7) + 8 * (lane >> 4), lcol = 8 * ((lane >> 3) & 1);
#pragma unroll
  for (int s = 0; s < 4; ++s) {
#pragma unroll
    for (int j = 0; j < MP / 16; ++j) {
      uint32_t bh[4], bl[4];
      const int off = (16 * j + lrow) * kLd64 + 16 * s + lcol;
      ldsm_x4(bh, om_hi + off);
      ldsm_x4(bl, om_lo + off);
      mma16816(acc[2 * j], a[s], bh[0], bh[1]);
      mma16816(acc[2 * j + 1], a[s], bh[2], bh[3]);
      mma16816(acc[2 * j], a[s], bl[0], bl[1]);
      mma16816(acc[2 * j + 1], a[s], bl[2], bl[3]);
    }
  }
}

// phi = exp(proj - |x|^2/2) / sqrt(m), zero for padded features and rows beyond the sequence;
// returned as A fragments (head and remainder) over the feature index.
template <int MP>
__device__ __forceinline__ void features_frag(uint32_t (&fh)[MP / 16][4], uint32_t (&fl)[MP / 16][4],
                                              const float (&acc)[MP / 8][4], float sq_g, float sq_g8,
                                              bool ok_g, bool ok_g8, int m, float inv_sqrt_m, int t) {
#pragma unroll
  for (int j = 0; j < MP / 8; ++j) {
    const int f = 8 * j + 2 * t;
    float v[4];
    v[0] = __expf(acc[j][0] - sq_g) * inv_sqrt_m;
    v[1] = __expf(acc[j][1] - sq_g) * inv_sqrt_m;
    v[2] = __expf(acc[j][2] - sq_g8) * inv_sqrt_m;
    v[3] = __expf(acc[j][3] - sq_g8) * inv_sqrt_m;
    if (!(ok_g && f < m)) v[0] = 0.f;
    if (!(ok_g && f + 1 < m)) v[1] = 0.f;
    if (!(ok_g8 && f < m)) v[2] = 0.f;
    if (!(ok_g8 && f + 1 < m)) v[3] = 0.f;
    // n-tile j is k-step j/2 of the next product; even tiles fill a0/a1, odd tiles a2/a3
    const int ks = j >> 1, o = (j & 1) * 2;
    split2(v[0], v[1], fh[ks][o], fl[ks][o]);
    split2(v[2], v[3], fh[ks][o + 1], fl[ks][o + 1]);
  }
}

// Writes this warp's 16 rows of phi (head / remainder) to shared [64][MP + kPad].
template <int MP>
__device__ __forceinline__ void store_features(__nv_bfloat16* ph, __nv_bfloat16* pl, const uint32_t (&fh)[MP / 16][4],
                                               const uint32_t (&fl)[MP / 16][4], int r0, int g, int t) {
  constexpr int LD = MP + kPad;
#pragma unroll
  for (int ks = 0; ks < MP / 16; ++ks) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = r0 + g + 8 * (i & 1), col = 16 * ks + 8 * (i >> 1) + 2 * t;
      *reinterpret_cast<uint32_t*>(ph + row * LD + col) = fh[ks][i];
      *reinterpret_cast<uint32_t*>(pl + row * LD + col) = fl[ks][i];
    }
  }
}

template <int MP>
struct SmemKeyState {
  // one region holds omega' during the projection and phi(K) afterwards
  static constexpr int kR = (MP * kLd64 > kC * (MP + kPad)) ? MP * kLd64 : kC * (MP + kPad);
  __nv_bfloat16 r_hi[kR], r_lo[kR];
  __nv_bfloat16 v[kC * kLd64];
};

// Kernel 1: S_c = phi(K_c)^T [V_c | 1] for every chunk.
template <int MP>
__global__ void __launch_bounds__(kThreads)
favor_key_state_mma_kernel(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                           const __nv_bfloat16* __restrict__ om_hi_g, const __nv_bfloat16* __restrict__ om_lo_g,
                           float* __restrict__ state, int seq_len, int m, int nchunk) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SmemKeyState<MP>& sm = *reinterpret_cast<SmemKeyState<MP>*>(smem_raw);
  constexpr int LDP = MP + kPad;
  const int chunk = blockIdx.x, bh = blockIdx.y, row0 = chunk * kC;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const size_t head = (size_t)bh * seq_len * kHeadDim;
  const int valid = min(kC, seq_len - row0);

  stage_rows64(sm.r_hi, om_hi_g, MP, MP);
  stage_rows64(sm.r_lo, om_lo_g, MP, MP);
  stage_rows64(sm.v, V + head + (size_t)row0 * kHeadDim, kC, valid);
  __syncthreads();

  {
    uint32_t a[4][4];
    float sq_g, sq_g8;
    const int r0 = 16 * warp;
    load_rows_frag(a, sq_g, sq_g8, K + head, row0 + r0 + g, seq_len, t);
    float acc[MP / 8][4];
    project<MP>(acc, a, sm.r_hi, sm.r_lo, lane);
    uint32_t fh[MP / 16][4], fl[MP / 16][4];
    features_frag<MP>(fh, fl, acc, sq_g, sq_g8, r0 + g < valid, r0 + g + 8 < valid, m, rsqrtf((float)m), t);
    __syncthreads();  // every warp is done reading omega'; the region now takes phi(K)
    store_features<MP>(sm.r_hi, sm.r_lo, fh, fl, r0, g, t);
  }
  __syncthreads();

  float* st = state + ((size_t)bh * nchunk + chunk) * (size_t)m * kStateCols;
  const uint32_t ones = g == 0 ? 0x3f803f80u : 0u;  // B fragment of a column of ones (n = 0)
  for (int mt = warp; mt < MP / 16; mt += 4) {
    float acc[9][4];
#pragma unroll
    for (int j = 0; j < 9; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[j][e] = 0.f;
#pragma unroll
    for (int ks = 0; ks < 4; ++ks) {
      // A = phi^T: stored [k = row][m = feature] -> transposed load
      uint32_t ah[4], al[4];
      const int arow = 16 * ks + (lane & 7) + 8 * (lane >> 4), acol = 16 * mt + 8 * ((lane >> 3) & 1);
      ldsm_x4_t(ah, sm.r_hi + arow * LDP + acol);
      ldsm_x4_t(al, sm.r_lo + arow * LDP + acol);
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t b[4];  // V stored [k = row][n = dim]
        const int brow = 16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1), bcol = 16 * np + 8 * (lane >> 4);
        ldsm_x4_t(b, sm.v + brow * kLd64 + bcol);
        mma16816(acc[2 * np], ah, b[0], b[1]);
        mma16816(acc[2 * np + 1], ah, b[2], b[3]);
        mma16816(acc[2 * np], al, b[0], b[1]);
        mma16816(acc[2 * np + 1], al, b[2], b[3]);
      }
      mma16816(acc[8], ah, ones, ones);
      mma16816(acc[8], al, ones, ones);
    }
    const int f0 = 16 * mt + g, f1 = f0 + 8;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int e = 8 * j + 2 * t;
      if (f0 < m) { st[(size_t)f0 * kStateCols + e] = acc[j][0]; st[(size_t)f0 * kStateCols + e + 1] = acc[j][1]; }
      if (f1 < m) { st[(size_t)f1 * kStateCols + e] = acc[j][2]; st[(size_t)f1 * kStateCols + e + 1] = acc[j][3]; }
    }
    if (t == 0) {
      if (f0 < m) st[(size_t)f0 * kStateCols + kHeadDim] = acc[8][0];
      if (f1 < m) st[(size_t)f1 * kStateCols + kHeadDim] = acc[8][2];
    }
  }
}

// Kernel 2: fixed-order combination of the chunk states of each head (exclusive prefix when
// causal, total otherwise), written as the bf16 head / remainder operand that kernel 3 copies
// straight into shared memory: per (head, chunk) two [MP][72] matrices, columns 0..63 the value
// part, column 64 the normaliser part z, the rest (and feature rows >= m) zero.
constexpr int kSLd = kHeadDim + 8;  // 72 columns: 144-byte pitch

__global__ void favor_state_scan_mma_kernel(const float* __restrict__ state, __nv_bfloat16* __restrict__ split,
                                            int nchunk, int m, int MP, long long total_threads, int causal) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_threads) return;
  const int per_head = MP * (kSLd / 2);
  const long long bh = gid / per_head;
  const int v = (int)(gid - bh * per_head);
  const int f = v / (kSLd / 2), c = (v - f * (kSLd / 2)) * 2;
  const bool in0 = f < m && c < kStateCols, in1 = f < m && c + 1 < kStateCols;
  const size_t per_chunk = (size_t)m * kStateCols;
  const float* p = state + (size_t)bh * nchunk * per_chunk + (size_t)f * kStateCols + c;
  const size_t out_chunk = 2 * (size_t)MP * kSLd;
  __nv_bfloat16* q = split + (size_t)bh * nchunk * out_chunk + (size_t)f * kSLd + c;
  float r0 = 0.f, r1 = 0.f;
#pragma unroll 4
  for (int ch = 0; ch < nchunk; ++ch) {
    const float x = in0 ? p[ch * per_chunk] : 0.f;
    const float y = in1 ? p[ch * per_chunk + 1] : 0.f;
    if (causal) {
      uint32_t hi, lo;
      split2(r0, r1, hi, lo);
      *reinterpret_cast<uint32_t*>(q + ch * out_chunk) = hi;
      *reinterpret_cast<uint32_t*>(q + ch * out_chunk + (size_t)MP * kSLd) = lo;
    }
    r0 += x;
    r1 += y;
  }
  if (!causal) {
    uint32_t hi, lo;
    split2(r0, r1, hi, lo);
    *reinterpret_cast<uint32_t*>(q) = hi;
    *reinterpret_cast<uint32_t*>(q + (size_t)MP * kSLd) = lo;
  }
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

template <int MP>
struct SmemOutput {
  // omega' (pitch 72) during the projections, then the prefix state S (pitch 72)
  __nv_bfloat16 r1_hi[MP * kSLd], r1_lo[MP * kSLd];
  __nv_bfloat16 ph_hi[kC * (MP + kPad)], ph_lo[kC * (MP + kPad)];
  __nv_bfloat16 v[kC * kLd64];
};

// Kernel 3: per chunk, num = phi(Q) S + (phi(Q) phi(K)^T . tril) V, den likewise with the ones
// column, C = num / den, written as bf16 head / remainder [rows][64] for the decoder product.
template <int MP>
__global__ void __launch_bounds__(kThreads, 2)
favor_output_mma_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                        const __nv_bfloat16* __restrict__ V, const __nv_bfloat16* __restrict__ om_hi_g,
                        const __nv_bfloat16* __restrict__ om_lo_g, const __nv_bfloat16* __restrict__ s_split,
                        __nv_bfloat16* __restrict__ c_hi, __nv_bfloat16* __restrict__ c_lo,
                        int32_t* __restrict__ status, int seq_len, int m, int nchunk, int causal) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SmemOutput<MP>& sm = *reinterpret_cast<SmemOutput<MP>*>(smem_raw);
  constexpr int LDP = MP + kPad;
  constexpr int LDS = kSLd;
  static_assert(kLd64 == kSLd, "omega' and S share one region and one pitch");
  const int chunk = blockIdx.x, bh = blockIdx.y, row0 = chunk * kC;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const size_t head = (size_t)bh * seq_len * kHeadDim;
  const int valid = min(kC, seq_len - row0);
  const int r0 = 16 * warp;
  const float inv_sqrt_m = rsqrtf((float)m);

  stage_rows64(sm.r1_hi, om_hi_g, MP, MP);
  stage_rows64(sm.r1_lo, om_lo_g, MP, MP);
  if (causal) stage_rows64(sm.v, V + head + (size_t)row0 * kHeadDim, kC, valid);
  __syncthreads();

  uint32_t qh[MP / 16][4], ql[MP / 16][4];  // phi(Q) rows of this warp as A fragments
  {
    uint32_t a[4][4];
    float sq_g, sq_g8;
    load_rows_frag(a, sq_g, sq_g8, Q + head, row0 + r0 + g, seq_len, t);
    float acc[MP / 8][4];
    project<MP>(acc, a, sm.r1_hi, sm.r1_lo, lane);
    features_frag<MP>(qh, ql, acc, sq_g, sq_g8, true, true, m, inv_sqrt_m, t);
  }
  if (causal) {
    uint32_t a[4][4];
    float sq_g, sq_g8;
    load_rows_frag(a, sq_g, sq_g8, K + head, row0 + r0 + g, seq_len, t);
    float acc[MP / 8][4];
    project<MP>(acc, a, sm.r1_hi, sm.r1_lo, lane);
    uint32_t fh[MP / 16][4], fl[MP / 16][4];
    features_frag<MP>(fh, fl, acc, sq_g, sq_g8, r0 + g < valid, r0 + g + 8 < valid, m, inv_sqrt_m, t);
    store_features<MP>(sm.ph_hi, sm.ph_lo, fh, fl, r0, g, t);
  }
  __syncthreads();  // phi(K) visible; omega' no longer needed: its region takes the state S

  {  // asynchronous copy of the prefix (or total) state, overlapped with the in-chunk part
    const __nv_bfloat16* src = s_split + ((size_t)bh * nchunk + (causal ? chunk : 0)) * (2 * (size_t)MP * kSLd);
    constexpr int kVecs = MP * kSLd / 8;  // 16-byte pieces per matrix
    for (int v = threadIdx.x; v < kVecs; v += kThreads) {
      cp_async16(sm.r1_hi + v * 8, src + v * 8);
      cp_async16(sm.r1_lo + v * 8, src + (size_t)MP * kSLd + v * 8);
    }
  }

  // num[0..7] = 64 value columns, num[8] = normaliser column (n = 0 of the ninth tile)
  float num[9][4];
#pragma unroll
  for (int j = 0; j < 9; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) num[j][e] = 0.f;

  float den_g = 0.f, den_g8 = 0.f;  // this lane's share of the in-chunk normaliser
  if (causal) {
    // keys 16jp .. 16jp+15 of the chunk; pairs beyond this warp's last row are fully masked
    for (int jp = 0; jp <= warp; ++jp) {
      float sc[2][4];
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int e = 0; e < 4; ++e) sc[u][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < MP / 16; ++ks) {
        uint32_t bh_[4], bl_[4];  // phi(K) stored [n = key][k = f]
        const int off = (16 * jp + (lane & 7) + 8 * (lane >> 4)) * LDP + 16 * ks + 8 * ((lane >> 3) & 1);
        ldsm_x4(bh_, sm.ph_hi + off);
        ldsm_x4(bl_, sm.ph_lo + off);
        mma16816(sc[0], qh[ks], bh_[0], bh_[1]);
        mma16816(sc[1], qh[ks], bh_[2], bh_[3]);
        mma16816(sc[0], qh[ks], bl_[0], bl_[1]);
        mma16816(sc[1], qh[ks], bl_[2], bl_[3]);
        mma16816(sc[0], ql[ks], bh_[0], bh_[1]);
        mma16816(sc[1], ql[ks], bh_[2], bh_[3]);
      }
      uint32_t ph[4], pl[4];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int j = 16 * jp + 8 * u + 2 * t, i0 = r0 + g, i1 = r0 + g + 8;
        if (j > i0) sc[u][0] = 0.f;
        if (j + 1 > i0) sc[u][1] = 0.f;
        if (j > i1) sc[u][2] = 0.f;
        if (j + 1 > i1) sc[u][3] = 0.f;
        den_g += sc[u][0] + sc[u][1];
        den_g8 += sc[u][2] + sc[u][3];
        split2(sc[u][0], sc[u][1], ph[2 * u], pl[2 * u]);
        split2(sc[u][2], sc[u][3], ph[2 * u + 1], pl[2 * u + 1]);
      }
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t b[4];  // V stored [k = key][n = dim]
        const int off = (16 * jp + (lane & 7) + 8 * ((lane >> 3) & 1)) * kLd64 + 16 * np + 8 * (lane >> 4);
        ldsm_x4_t(b, sm.v + off);
        mma16816(num[2 * np], ph, b[0], b[1]);
        mma16816(num[2 * np + 1], ph, b[2], b[3]);
        mma16816(num[2 * np], pl, b[0], b[1]);
        mma16816(num[2 * np + 1], pl, b[2], b[3]);
      }
    }
    den_g += __shfl_xor_sync(0xffffffffu, den_g, 1); den_g += __shfl_xor_sync(0xffffffffu, den_g, 2);
    den_g8 += __shfl_xor_sync(0xffffffffu, den_g8, 1); den_g8 += __shfl_xor_sync(0xffffffffu, den_g8, 2);
  }

  cp_async_wait_all();
  __syncthreads();  // S complete and visible to every warp
#pragma unroll
  for (int ks = 0; ks < MP / 16; ++ks) {
    const int brow = 16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t bh_[4], bl_[4];  // S stored [k = f][n = e]
      const int off = brow * LDS + 16 * np + 8 * (lane >> 4);
      ldsm_x4_t(bh_, sm.r1_hi + off);
      ldsm_x4_t(bl_, sm.r1_lo + off);
      mma16816(num[2 * np], qh[ks], bh_[0], bh_[1]);
      mma16816(num[2 * np + 1], qh[ks], bh_[2], bh_[3]);
      mma16816(num[2 * np], qh[ks], bl_[0], bl_[1]);
      mma16816(num[2 * np + 1], qh[ks], bl_[2], bl_[3]);
      mma16816(num[2 * np], ql[ks], bh_[0], bh_[1]);
      mma16816(num[2 * np + 1], ql[ks], bh_[2], bh_[3]);
    }
    uint32_t zh[2], zl[2];
    const int zoff = (16 * ks + (lane & 15)) * LDS + kHeadDim;
    ldsm_x2_t(zh, sm.r1_hi + zoff);
    ldsm_x2_t(zl, sm.r1_lo + zoff);
    mma16816(num[8], qh[ks], zh[0], zh[1]);
    mma16816(num[8], qh[ks], zl[0], zl[1]);
    mma16816(num[8], ql[ks], zh[0], zh[1]);
  }

  // the prefix normaliser sits in column 0 of the ninth tile, i.e. in the lane with t == 0
  den_g += __shfl_sync(0xffffffffu, num[8][0], lane & ~3);
  den_g8 += __shfl_sync(0xffffffffu, num[8][2], lane & ~3);
  const bool ok_g = r0 + g < valid, ok_g8 = r0 + g + 8 < valid;
  if ((ok_g && !(den_g > 0.f && den_g < INFINITY)) || (ok_g8 && !(den_g8 > 0.f && den_g8 < INFINITY)))
    atomicOr(status, SEA_DEV_NONFINITE);
  const float inv_g = 1.f / den_g, inv_g8 = 1.f / den_g8;

  const size_t o_g = ((size_t)bh * seq_len + row0 + r0 + g) * kHeadDim, o_g8 = o_g + 8 * kHeadDim;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e = 8 * j + 2 * t;
    uint32_t hi, lo;
    if (ok_g) {
      split2(num[j][0] * inv_g, num[j][1] * inv_g, hi, lo);
      *reinterpret_cast<uint32_t*>(c_hi + o_g + e) = hi;
      *reinterpret_cast<uint32_t*>(c_lo + o_g + e) = lo;
    }
    if (ok_g8) {
      split2(num[j][2] * inv_g8, num[j][3] * inv_g8, hi, lo);
      *reinterpret_cast<uint32_t*>(c_hi + o_g8 + e) = hi;
      *reinterpret_cast<uint32_t*>(c_lo + o_g8 + e) = lo;
    }
  }
}

// Kernel 4: decoder head A_hat = C W_dec on the bf16 head / remainder operands.  A CTA of four
// warps owns 64 rows (one warp per 16) and walks the Kc columns in tiles of 128.
__global__ void __launch_bounds__(kThreads)
favor_decoder_mma_kernel(const __nv_bfloat16* __restrict__ c_hi, const __nv_bfloat16* __restrict__ c_lo,
                         const __nv_bfloat16* __restrict__ w_hi_g, const __nv_bfloat16* __restrict__ w_lo_g,
                         float* __restrict__ A_hat, long long rows, int Kc, int KcP) {
  constexpr int LDW = kWTile + kPad;  // 136: 272-byte pitch
  __shared__ __align__(16) __nv_bfloat16 wt_hi[kHeadDim * LDW];
  __shared__ __align__(16) __nv_bfloat16 wt_lo[kHeadDim * LDW];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const long long row_g = (long long)blockIdx.x * kC + 16 * warp + g;
  const bool ok_g = row_g < rows, ok_g8 = row_g + 8 < rows;
  uint32_t ch[4][4], cl[4][4];
  {
    const uint32_t* h0 = reinterpret_cast<const uint32_t*>(c_hi + (size_t)row_g * kHeadDim) + t;
    const uint32_t* l0 = reinterpret_cast<const uint32_t*>(c_lo + (size_t)row_g * kHeadDim) + t;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      ch[s][0] = ok_g ? __ldg(h0 + 8 * s) : 0u;
      ch[s][1] = ok_g8 ? __ldg(h0 + 256 + 8 * s) : 0u;
      ch[s][2] = ok_g ? __ldg(h0 + 8 * s + 4) : 0u;
      ch[s][3] = ok_g8 ? __ldg(h0 + 256 + 8 * s + 4) : 0u;
      cl[s][0] = ok_g ? __ldg(l0 + 8 * s) : 0u;
      cl[s][1] = ok_g8 ? __ldg(l0 + 256 + 8 * s) : 0u;
      cl[s][2] = ok_g ? __ldg(l0 + 8 * s + 4) : 0u;
      cl[s][3] = ok_g8 ? __ldg(l0 + 256 + 8 * s + 4) : 0u;
    }
  }
  float* out_g = A_hat + (size_t)row_g * Kc;
  float* out_g8 = out_g + (size_t)8 * Kc;
  const bool vec2 = (Kc & 1) == 0;
  for (int c0 = 0; c0 < Kc; c0 += kWTile) {
    if (c0 > 0) __syncthreads();  // the previous tile is no longer being read
    for (int v = threadIdx.x; v < kHeadDim * (kWTile / 8); v += kThreads) {
      const int e = v / (kWTile / 8), cc = (v - e * (kWTile / 8)) * 8;
      uint4 xh = make_uint4(0u, 0u, 0u, 0u), xl = xh;
      if (c0 + cc < KcP) {
        xh = __ldg(reinterpret_cast<const uint4*>(w_hi_g + (size_t)e * KcP + c0 + cc));
        xl = __ldg(reinterpret_cast<const uint4*>(w_lo_g + (size_t)e * KcP + c0 + cc));
      }
      *reinterpret_cast<uint4*>(wt_hi + e * LDW + cc) = xh;
      *reinterpret_cast<uint4*>(wt_lo + e * LDW + cc) = xl;
    }
    __syncthreads();
    const int ncols = min(kWTile, Kc - c0);
    for (int np = 0; np * 16 < ncols; ++np) {
      float acc[2][4];
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[u][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        uint32_t bh_[4], bl_[4];  // W stored [k = e][n = c]
        const int off = (16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1)) * LDW + 16 * np + 8 * (lane >> 4);
        ldsm_x4_t(bh_, wt_hi + off);
        ldsm_x4_t(bl_, wt_lo + off);
        mma16816(acc[0], ch[ks], bh_[0], bh_[1]);
        mma16816(acc[1], ch[ks], bh_[2], bh_[3]);
        mma16816(acc[0], ch[ks], bl_[0], bl_[1]);
        mma16816(acc[1], ch[ks], bl_[2], bl_[3]);
        mma16816(acc[0], cl[ks], bh_[0], bh_[1]);
        mma16816(acc[1], cl[ks], bh_[2], bh_[3]);
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int c = c0 + 16 * np + 8 * u + 2 * t;
        if (vec2) {
          if (ok_g && c < Kc) *reinterpret_cast<float2*>(out_g + c) = make_float2(acc[u][0], acc[u][1]);
          if (ok_g8 && c < Kc) *reinterpret_cast<float2*>(out_g8 + c) = make_float2(acc[u][2], acc[u][3]);
        } else {
          if (ok_g) {
            if (c < Kc) out_g[c] = acc[u][0];
            if (c + 1 < Kc) out_g[c + 1] = acc[u][1];
          }
          if (ok_g8) {
            if (c < Kc) out_g8[c] = acc[u][2];
            if (c + 1 < Kc) out_g8[c + 1] = acc[u][3];
          }
        }
      }
    }
  }
}

template <int MP>
sea_status launch_mp(const sea_shape& s, const __nv_bfloat16* Q, const __nv_bfloat16* K, const __nv_bfloat16* V,
                     const float* omega, const float* W_dec, float* A_hat, float* state,
                     __nv_bfloat16* split_buf, int32_t* status, cudaStream_t st) {
  const int BH = s.B * s.H, m = s.m;
  const int nchunk = (s.T + kC - 1) / kC;
  const long long rows = (long long)BH * s.T;
  const int KcP = (s.Kc + 15) / 16 * 16;
  // carve-up of the split buffer (see estimate_split_bytes)
  __nv_bfloat16* om_hi = split_buf;
  __nv_bfloat16* om_lo = om_hi + 128 * kHeadDim;
  __nv_bfloat16* w_hi = om_lo + 128 * kHeadDim;
  __nv_bfloat16* w_lo = w_hi + (size_t)kHeadDim * KcP;
  __nv_bfloat16* c_hi = w_lo + (size_t)kHeadDim * KcP;
  __nv_bfloat16* c_lo = c_hi + (size_t)rows * kHeadDim;
  __nv_bfloat16* s_split = c_lo + (size_t)rows * kHeadDim;
  const size_t smem1 = sizeof(SmemKeyState<MP>), smem3 = sizeof(SmemOutput<MP>);
  if (cudaFuncSetAttribute(favor_key_state_mma_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess ||
      cudaFuncSetAttribute(favor_output_mma_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem3) != cudaSuccess)
    return SEA_ERR_CUDA;
  const int n_prep = MP * kHeadDim + kHeadDim * KcP;
  favor_prep_kernel<<<(n_prep + 255) / 256, 256, 0, st>>>(omega, W_dec, om_hi, om_lo, w_hi, w_lo, m, MP, s.Kc, KcP,
                                                          0.35355339059327373f);
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;
  const dim3 grid(nchunk, BH);
  favor_key_state_mma_kernel<MP><<<grid, kThreads, smem1, st>>>(K, V, om_hi, om_lo, state, s.T, m, nchunk);
  if ((rc = check_launch()) != SEA_OK) return rc;
  const long long total = (long long)BH * MP * (kSLd / 2);
  favor_state_scan_mma_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(state, s_split, nchunk, m, MP, total, s.causal);
  if ((rc = check_launch()) != SEA_OK) return rc;
  favor_output_mma_kernel<MP><<<grid, kThreads, smem3, st>>>(Q, K, V, om_hi, om_lo, s_split, c_hi, c_lo, status, s.T, m,
                                                             nchunk, s.causal);
  if ((rc = check_launch()) != SEA_OK) return rc;
  favor_decoder_mma_kernel<<<(unsigned)((rows + kC - 1) / kC), kThreads, 0, st>>>(c_hi, c_lo, w_hi, w_lo, A_hat, rows, s.Kc, KcP);
  return check_launch();
}

}  // namespace

// bf16 scratch of the tensor-core estimator: omega' and W_dec (head / remainder), C (head /
// remainder, [rows][64]) and the scanned chunk states ([BH][nchunk][2][128][72]).
size_t estimate_split_bytes(const sea_shape& s) {
  const size_t KcP = ((size_t)s.Kc + 15) / 16 * 16;
  const size_t rows = (size_t)s.B * s.H * s.T;
  const size_t nchunk = ((size_t)s.T + kC - 1) / kC;
  const size_t elems = 2 * (size_t)128 * kHeadDim + 2 * (size_t)kHeadDim * KcP + 2 * rows * kHeadDim +
                       (size_t)s.B * s.H * nchunk * 2 * 128 * kSLd;
  return elems * sizeof(__nv_bfloat16);
}

sea_status launch_estimate_bf16(const sea_shape& s, const void* Q, const void* K, const void* V,
                                const float* omega, const float* W_dec, float* A_hat, float* est_state,
                                void* split_buf, int32_t* status, cudaStream_t st) {
  using T = __nv_bfloat16;
  if (s.m <= 32)
    return launch_mp<32>(s, (const T*)Q, (const T*)K, (const T*)V, omega, W_dec, A_hat, est_state, (T*)split_buf, status, st);
  if (s.m <= 64)
    return launch_mp<64>(s, (const T*)Q, (const T*)K, (const T*)V, omega, W_dec, A_hat, est_state, (T*)split_buf, status, st);
  return launch_mp<128>(s, (const T*)Q, (const T*)K, (const T*)V, omega, W_dec, A_hat, est_state, (T*)split_buf, status, st);
}

}  // namespace sea

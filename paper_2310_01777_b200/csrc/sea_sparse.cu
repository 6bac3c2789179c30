// Sparse attention stage: scores at the mask's positions, row softmax, product with V
// (Sec. 3.1.1 "Sparse Attention Mechanism": rho, sigma, C = A* V), fused in one kernel.
//
// One warp owns one query row; the row's scores are parked in shared memory (log2 domain),
// the softmax runs with one lane per key (pair), and rows longer than the shared-memory
// chunk take a first statistics-only pass over K.
//
// fp32 I/O: plain FMA arithmetic.  A key row (256 B) is read by 16 neighbouring lanes with
// one 16-byte load each, so every fetched byte is used.
//
// bf16 I/O: the gathered products run on the tensor cores (mma.sync m16n8k16, fp32
// accumulate) even though each query is a single vector: 16 gathered keys form the M side of
// S^T = K_g q^T (4 MMAs per 16 keys, q replicated over the 8 columns), and O^T = V_g^T p
// takes V_g^T as the M side (4 tiles of 16 dims) with the probabilities, split into a bf16
// head and a bf16 remainder so that O is accumulated from (almost) unrounded p, replicated
// over the columns.  The contraction index of an MMA may be permuted freely as long as both
// operands agree, which lets every lane fetch whole 16-byte pieces of a key row: there is no
// shared-memory staging of K or V and every fetched byte is used.  This cuts the issued
// instructions per gathered key by an order of magnitude against the FMA form, which was
// issue-bound.
#include "sea_common.cuh"

namespace sea {
namespace {

constexpr int kWarpsPerCta = 8;

template <typename T, bool kWriteP, bool kUseSel>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
sparse_attn_rows_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                        const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                        const int32_t* __restrict__ sel, T* __restrict__ O, T* __restrict__ P,
                        int rows, int seq_len, int r, int k_hat, float scale_log2, int chunk) {
  using IO = Io<T>;
  constexpr int EPL = IO::kElemsPerLane;
  constexpr int LPR = IO::kLanesPerRow;
  constexpr int KPI = 32 / LPR;  // keys per warp-wide load
  extern __shared__ float smem[];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  float* sc = smem + warp * chunk;
  const int g = lane / LPR, sub = lane % LPR;

  const int bh = row / seq_len;
  const T* Kh = K + (size_t)bh * seq_len * kHeadDim;
  const T* Vh = V + (size_t)bh * seq_len * kHeadDim;
  const int base = __ldg(row_ptr + row);
  const int n = __ldg(row_ptr + row + 1) - base;
  const int32_t* my_sel = kUseSel ? sel + (size_t)row * k_hat : nullptr;
  const int32_t* my_col = kUseSel ? nullptr : col_idx + base;

  auto key_at = [&](int pos) -> int {
    if (kUseSel) {
      const int b = pos / r;
      return __ldg(my_sel + b) * r + (pos - b * r);
    }
    return __ldg(my_col + pos);
  };

  float o[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) o[e] = 0.f;

  if (n > 0) {
    float q[EPL];
    IO::load(Q + (size_t)row * kHeadDim + sub * EPL, q);

    // scores of positions [c0, c0+cn) -> sc[0..cn), returns their maximum
    auto scores_chunk = [&](int c0, int cn) -> float {
      float mx = -INFINITY;
#pragma unroll 4
      for (int it = 0; it * KPI < cn; ++it) {
        const int pos = it * KPI + g;
        const bool valid = pos < cn;
        const int j = valid ? key_at(c0 + pos) : 0;
        float kv[EPL];
        IO::load(Kh + (size_t)j * kHeadDim + sub * EPL, kv);
        float dot = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) dot = fmaf(q[e], kv[e], dot);
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        dot *= scale_log2;
        if (valid) {
          mx = fmaxf(mx, dot);
          if (sub == 0) sc[pos] = dot;
        }
      }
      return warp_max(mx);
    };

    float m_run = -INFINITY, l_run = 0.f;
    if (n > chunk) {  // statistics pass for rows that do not fit one chunk
      for (int c0 = 0; c0 < n; c0 += chunk) {
        const int cn = min(chunk, n - c0);
        const float mx = scores_chunk(c0, cn);
        __syncwarp();
        const float m_new = fmaxf(m_run, mx);
        float part = 0.f;
        for (int pos = lane; pos < cn; pos += 32) part += exp2f(sc[pos] - m_new);
        part = warp_sum(part);
        l_run = l_run * exp2f(m_run - m_new) + part;
        m_run = m_new;
        __syncwarp();
      }
    }
    for (int c0 = 0; c0 < n; c0 += chunk) {
      const int cn = min(chunk, n - c0);
      const float mx = scores_chunk(c0, cn);
      __syncwarp();
      const bool single = n <= chunk;
      if (single) m_run = mx;
      float part = 0.f;
      for (int pos = lane; pos < cn; pos += 32) {
        const float e = exp2f(sc[pos] - m_run);
        sc[pos] = e;
        part += e;
      }
      if (single) l_run = warp_sum(part);
      const float inv = 1.f / l_run;
      if (kWriteP) {
        for (int pos = lane; pos < cn; pos += 32) P[(size_t)base + c0 + pos] = IO::to_io(sc[pos] * inv);
      }
      __syncwarp();
#pragma unroll 4
      for (int it = 0; it * KPI < cn; ++it) {
        const int pos = it * KPI + g;
        const bool valid = pos < cn;
        const int j = valid ? key_at(c0 + pos) : 0;
        const float p = valid ? sc[pos] : 0.f;
        float vv[EPL];
        IO::load(Vh + (size_t)j * kHeadDim + sub * EPL, vv);
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[e] = fmaf(p, vv[e], o[e]);
      }
      __syncwarp();
    }
    const float inv = 1.f / l_run;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
#pragma unroll
      for (int off = LPR; off < 32; off <<= 1) o[e] += __shfl_xor_sync(0xffffffffu, o[e], off);
      o[e] *= inv;
    }
  }
  if (g == 0) IO::store(O + (size_t)row * kHeadDim + sub * EPL, o);
}


// ---- bf16 tensor-core form ------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Lane (g = lane/4, t = lane%4).  Per position p of the row the key index sits in idx[p]; sc[p]
// holds the score and is overwritten in place, two positions at a time, by the packed
// probabilities {bf16x2 head, bf16x2 remainder}.
template <bool kWriteP, bool kUseSel>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
sparse_attn_rows_mma_kernel(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
                            const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ row_ptr,
                            const int32_t* __restrict__ col_idx, const int32_t* __restrict__ sel,
                            __nv_bfloat16* __restrict__ O, __nv_bfloat16* __restrict__ P, int rows,
                            int seq_len, int r, int k_hat, float scale_log2, int chunk) {
  extern __shared__ float smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * kWarpsPerCta + warp;
  if (row >= rows) return;
  int32_t* idx = reinterpret_cast<int32_t*>(smem) + warp * 2 * chunk;
  float* sc = smem + warp * 2 * chunk + chunk;
  uint2* pairs = reinterpret_cast<uint2*>(sc);
  const int g = lane >> 2, t = lane & 3;

  const int bh = row / seq_len;
  const char* Kh = reinterpret_cast<const char*>(K + (size_t)bh * seq_len * kHeadDim);
  const char* Vh = reinterpret_cast<const char*>(V + (size_t)bh * seq_len * kHeadDim);
  const int base = __ldg(row_ptr + row);
  const int n = __ldg(row_ptr + row + 1) - base;
  __nv_bfloat16* out = O + (size_t)row * kHeadDim;
  if (n <= 0) {
    if (t == 0) *reinterpret_cast<uint4*>(out + 8 * g) = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const int32_t* my_sel = kUseSel ? sel + (size_t)row * k_hat : nullptr;
  const int32_t* my_col = kUseSel ? nullptr : col_idx + base;

  // q as the B operand: words 0..3 = dims 8t..8t+7, words 4..7 = dims 32+8t..32+8t+7
  uint32_t qw[8];
  {
    const char* qp = reinterpret_cast<const char*>(Q + (size_t)row * kHeadDim);
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(qp + 16 * t));
    const uint4 b = __ldg(reinterpret_cast<const uint4*>(qp + 64 + 16 * t));
    qw[0] = a.x; qw[1] = a.y; qw[2] = a.z; qw[3] = a.w;
    qw[4] = b.x; qw[5] = b.y; qw[6] = b.z; qw[7] = b.w;
  }

  auto fill_idx = [&](int c0, int cn16, int cn) {
    for (int p = lane; p < cn16; p += 32) {
      int j = 0;
      if (p < cn) {
        if (kUseSel) {
          const int b = (c0 + p) / r;
          j = __ldg(my_sel + b) * r + (c0 + p - b * r);
        } else {
          j = __ldg(my_col + c0 + p);
        }
      }
      idx[p] = j;
    }
    __syncwarp();
  };

  // scores of the chunk -> sc[0..cn16) (-inf beyond cn); returns the chunk maximum
  auto scores_chunk = [&](int cn16, int cn) -> float {
    float mx = -INFINITY;
#pragma unroll 2
    for (int p0 = 0; p0 < cn16; p0 += 16) {
      const int j0 = idx[p0 + g], j1 = idx[p0 + g + 8];
      const char* k0 = Kh + (size_t)j0 * (kHeadDim * 2) + 16 * t;
      const char* k1 = Kh + (size_t)j1 * (kHeadDim * 2) + 16 * t;
      const uint4 a_lo = __ldg(reinterpret_cast<const uint4*>(k0));
      const uint4 a_hi = __ldg(reinterpret_cast<const uint4*>(k0 + 64));
      const uint4 b_lo = __ldg(reinterpret_cast<const uint4*>(k1));
      const uint4 b_hi = __ldg(reinterpret_cast<const uint4*>(k1 + 64));
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      mma_bf16_16816(acc, a_lo.x, b_lo.x, a_lo.y, b_lo.y, qw[0], qw[1]);
      mma_bf16_16816(acc, a_lo.z, b_lo.z, a_lo.w, b_lo.w, qw[2], qw[3]);
      mma_bf16_16816(acc, a_hi.x, b_hi.x, a_hi.y, b_hi.y, qw[4], qw[5]);
      mma_bf16_16816(acc, a_hi.z, b_hi.z, a_hi.w, b_hi.w, qw[6], qw[7]);
      const float s0 = p0 + g < cn ? acc[0] * scale_log2 : -INFINITY;
      const float s1 = p0 + g + 8 < cn ? acc[2] * scale_log2 : -INFINITY;
      mx = fmaxf(mx, fmaxf(s0, s1));
      if (t == 0) {
        sc[p0 + g] = s0;
        sc[p0 + g + 8] = s1;
      }
    }
    mx = warp_max(mx);
    __syncwarp();
    return mx;
  };

  float m_run = -INFINITY, l_run = 0.f;
  if (n > chunk) {  // statistics pass for rows that do not fit one chunk
    for (int c0 = 0; c0 < n; c0 += chunk) {
      const int cn = min(chunk, n - c0), cn16 = (cn + 15) & ~15;
      fill_idx(c0, cn16, cn);
      const float mx = scores_chunk(cn16, cn);
      const float m_new = fmaxf(m_run, mx);
      float part = 0.f;
      for (int p = lane; p < cn; p += 32) part += exp2f(sc[p] - m_new);
      part = warp_sum(part);
      l_run = l_run * exp2f(m_run - m_new) + part;
      m_run = m_new;
      __syncwarp();
    }
  }

  float acc_o[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc_o[i][e] = 0.f;

  for (int c0 = 0; c0 < n; c0 += chunk) {
    const int cn = min(chunk, n - c0), cn16 = (cn + 15) & ~15;
    fill_idx(c0, cn16, cn);
    const float mx = scores_chunk(cn16, cn);
    const bool single = n <= chunk;
    if (single) m_run = mx;
    // exponentials in place (positions >= cn hold -inf and give 0)
    float part = 0.f;
    for (int u = lane; u < cn16 / 2; u += 32) {
      float2 s = reinterpret_cast<float2*>(sc)[u];
      s.x = exp2f(s.x - m_run);
      s.y = exp2f(s.y - m_run);
      part += s.x + s.y;
      reinterpret_cast<float2*>(sc)[u] = s;
    }
    if (single) l_run = warp_sum(part);
    const float inv = 1.f / l_run;
    for (int u = lane; u < cn16 / 2; u += 32) {
      const float2 e = reinterpret_cast<float2*>(sc)[u];
      const float p0 = e.x * inv, p1 = e.y * inv;
      const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
      const uint32_t hw = *reinterpret_cast<const uint32_t*>(&h);
      const uint32_t lw = pack_bf16(p0 - __bfloat162float(h.x), p1 - __bfloat162float(h.y));
      pairs[u] = make_uint2(hw, lw);
      if (kWriteP) {
        __nv_bfloat16* pp = P + (size_t)base + c0 + 2 * u;
        if (2 * u < cn) pp[0] = h.x;
        if (2 * u + 1 < cn) pp[1] = h.y;
      }
    }
    __syncwarp();
#pragma unroll 2
    for (int p0 = 0; p0 < cn16; p0 += 16) {
      const int2 ja = *reinterpret_cast<const int2*>(idx + p0 + 2 * t);
      const int2 jb = *reinterpret_cast<const int2*>(idx + p0 + 8 + 2 * t);
      const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(Vh + (size_t)ja.x * (kHeadDim * 2) + 16 * g));
      const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(Vh + (size_t)ja.y * (kHeadDim * 2) + 16 * g));
      const uint4 v2 = __ldg(reinterpret_cast<const uint4*>(Vh + (size_t)jb.x * (kHeadDim * 2) + 16 * g));
      const uint4 v3 = __ldg(reinterpret_cast<const uint4*>(Vh + (size_t)jb.y * (kHeadDim * 2) + 16 * g));
      const uint2 pa = pairs[p0 / 2 + t];      // positions p0+2t, p0+2t+1
      const uint2 pb = pairs[p0 / 2 + 4 + t];  // positions p0+8+2t, p0+9+2t
      const uint32_t w0[4] = {v0.x, v0.y, v0.z, v0.w}, w1[4] = {v1.x, v1.y, v1.z, v1.w};
      const uint32_t w2[4] = {v2.x, v2.y, v2.z, v2.w}, w3[4] = {v3.x, v3.y, v3.z, v3.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {  // tile i: rows g / g+8 = dims 8g+2i / 8g+2i+1
        const uint32_t a0 = __byte_perm(w0[i], w1[i], 0x5410);
        const uint32_t a1 = __byte_perm(w0[i], w1[i], 0x7632);
        const uint32_t a2 = __byte_perm(w2[i], w3[i], 0x5410);
        const uint32_t a3 = __byte_perm(w2[i], w3[i], 0x7632);
        mma_bf16_16816(acc_o[i], a0, a1, a2, a3, pa.x, pb.x);
        mma_bf16_16816(acc_o[i], a0, a1, a2, a3, pa.y, pb.y);
      }
    }
    __syncwarp();
  }
  if (t == 0) {
    uint4 o;
    o.x = pack_bf16(acc_o[0][0], acc_o[0][2]);
    o.y = pack_bf16(acc_o[1][0], acc_o[1][2]);
    o.z = pack_bf16(acc_o[2][0], acc_o[2][2]);
    o.w = pack_bf16(acc_o[3][0], acc_o[3][2]);
    *reinterpret_cast<uint4*>(out + 8 * g) = o;
  }
}

template <typename T>
sea_status launch_typed(const sea_shape& s, const T* Q, const T* K, const T* V,
                        const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel, T* O,
                        T* P, cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  const int r = (s.T + s.Kc - 1) / s.Kc;  // a column's keys (the most, when T is no multiple of Kc)
  const long long cap = (long long)s.k_hat * r;
  int chunk = (int)((cap + 31) / 32 * 32);
  if (chunk > 1024) chunk = 1024;
  const size_t smem = (size_t)kWarpsPerCta * chunk * sizeof(float);
  const float scale = s.scale != 0.f ? s.scale : 0.125f;  // 1/sqrt(64)
  const float scale_log2 = scale * 1.4426950408889634f;
  const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
  const dim3 block(kWarpsPerCta * 32);
#define SEA_LAUNCH(WP, US)                                                                     \
  sparse_attn_rows_kernel<T, WP, US><<<grid, block, smem, st>>>(Q, K, V, row_ptr, col_idx, sel, O, P, \
                                                                rows, s.T, r, s.k_hat, scale_log2, chunk)
  if (sel) {
    if (P) SEA_LAUNCH(true, true); else SEA_LAUNCH(false, true);
  } else {
    if (P) SEA_LAUNCH(true, false); else SEA_LAUNCH(false, false);
  }
#undef SEA_LAUNCH
  return check_launch();
}

}  // namespace

sea_status launch_sparse_attn(const sea_shape& s, const void* Q, const void* K, const void* V,
                              const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel,
                              void* O, void* P, uint32_t* mask_bits, bool bits_valid, float* p_scratch,
                              uint32_t* tile_live, int32_t* status, cudaStream_t st) {
  if (tile_live != nullptr && sparse_attn_tc_applicable(s, sel, false, status, mask_bits, p_scratch))
    return launch_sparse_attn_tc(s, Q, K, V, row_ptr, sel, O, P, mask_bits, bits_valid, p_scratch, nullptr, tile_live, status, st);
  if (sparse_attn_tma_applicable(s, sel, status))
    return launch_sparse_attn_tma(s, Q, K, V, row_ptr, sel, O, P, status, st);
  return launch_sparse_attn_rows(s, Q, K, V, row_ptr, col_idx, sel, O, P, st);
}

sea_status launch_sparse_attn_masked(const sea_shape& s, const void* Q, const void* K, const void* V,
                                     const int32_t* row_ptr, const int32_t* col_idx, const uint32_t* mask_bits,
                                     void* O, void* P, int32_t* park_off, bool park_valid, bool rows_within_k_hat,
                                     float* p_scratch, uint32_t* tile_live, int32_t* status, cudaStream_t st) {
  if (park_off != nullptr && tile_live != nullptr && sparse_attn_tc_applicable(s, nullptr, true, status, mask_bits, p_scratch)) {
    if (P != nullptr && rows_within_k_hat)  // every row fits the per-query parking layout
      return launch_sparse_attn_tc(s, Q, K, V, row_ptr, nullptr, O, P, const_cast<uint32_t*>(mask_bits), true, p_scratch,
                                   nullptr, tile_live, status, st);
    if (P != nullptr && !park_valid) {
      const sea_status rc = launch_park_offsets(s, mask_bits, park_off, status, st);
      if (rc != SEA_OK) return rc;
    }
    // the bits are only read: bits_valid keeps the launcher from deriving them from a selection list
    return launch_sparse_attn_tc(s, Q, K, V, row_ptr, nullptr, O, P, const_cast<uint32_t*>(mask_bits), true, p_scratch,
                                 P != nullptr ? park_off : nullptr, tile_live, status, st);
  }
  if (col_idx == nullptr) return SEA_ERR_INVALID_ARG;
  return launch_sparse_attn_rows(s, Q, K, V, row_ptr, col_idx, nullptr, O, P, st);
}

// The per-row kernels: any CSR, rows of any length.
sea_status launch_sparse_attn_rows(const sea_shape& s, const void* Q, const void* K, const void* V,
                                   const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel, void* O,
                                   void* P, cudaStream_t st) {
  Launch::sparse_kernel() = s.io == SEA_BF16 ? "sparse_attn_rows_mma_kernel" : "sparse_attn_rows_kernel";
  Launch::sparse_flops() = 0.0;  // depends on the mask: 4 * nnz * d
  if (s.io == SEA_BF16) {
    using T = __nv_bfloat16;
    const int rows = s.B * s.H * s.T;
    const int r = (s.T + s.Kc - 1) / s.Kc;  // a column's keys (the most, when T is no multiple of Kc)
    const long long cap = (long long)s.k_hat * r;
    int chunk = (int)((cap + 63) / 64 * 64);
    if (chunk > 1024) chunk = 1024;
    const size_t smem = (size_t)kWarpsPerCta * chunk * 2 * sizeof(float);
    const float scale = s.scale != 0.f ? s.scale : 0.125f;  // 1/sqrt(64)
    const float scale_log2 = scale * 1.4426950408889634f;
    const int grid = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
    const dim3 block(kWarpsPerCta * 32);
#define SEA_LAUNCH(WP, US)                                                                          \
  do {                                                                                              \
    if (smem > 48 * 1024 &&                                                                         \
        cudaFuncSetAttribute(sparse_attn_rows_mma_kernel<WP, US>,                                   \
                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) \
      return SEA_ERR_CUDA;                                                                          \
    sparse_attn_rows_mma_kernel<WP, US><<<grid, block, smem, st>>>(                                 \
        (const T*)Q, (const T*)K, (const T*)V, row_ptr, col_idx, sel, (T*)O, (T*)P, rows, s.T, r,   \
        s.k_hat, scale_log2, chunk);                                                                \
  } while (0)
    if (sel) {
      if (P) SEA_LAUNCH(true, true); else SEA_LAUNCH(false, true);
    } else {
      if (P) SEA_LAUNCH(true, false); else SEA_LAUNCH(false, false);
    }
#undef SEA_LAUNCH
    return check_launch();
  }
  return launch_typed<float>(s, (const float*)Q, (const float*)K, (const float*)V, row_ptr, col_idx,
                             sel, (float*)O, (float*)P, st);
}

}  // namespace sea

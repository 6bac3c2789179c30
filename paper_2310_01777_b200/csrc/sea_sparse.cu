// Sparse attention stage: scores at the mask's positions, row softmax, product with V
// (Sec. 3.1.1 "Sparse Attention Mechanism": rho, sigma, C = A* V), fused in one kernel.
//
// One warp owns one query row.  A key row of d = 64 elements is 128 B (bf16) or 256 B
// (fp32) and is read by 8 (16) neighbouring lanes with one 16-byte load each, so a warp
// load instruction covers 4 (2) whole keys and every fetched byte is used.  The row's
// scores are parked in shared memory (log2 domain), the softmax runs with one lane per
// key, and the probabilities are then broadcast back to the lane groups for the V pass.
// Rows longer than the shared-memory chunk take a first statistics-only pass over K.
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

template <typename T>
sea_status launch_typed(const sea_shape& s, const T* Q, const T* K, const T* V,
                        const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel, T* O,
                        T* P, cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
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
                              void* O, void* P, cudaStream_t st) {
  if (s.io == SEA_BF16) {
    using T = __nv_bfloat16;
    return launch_typed<T>(s, (const T*)Q, (const T*)K, (const T*)V, row_ptr, col_idx, sel, (T*)O, (T*)P, st);
  }
  return launch_typed<float>(s, (const float*)Q, (const float*)K, (const float*)V, row_ptr, col_idx,
                             sel, (float*)O, (float*)P, st);
}

}  // namespace sea

// Attention estimation (Sec. 3.1 "Attention Matrix Estimation"): FAVOR+ linear attention
// (Sec. 3 "Performer (FAVOR+)") followed by one linear decoder head.
//
//   x = u d^(-1/4);  phi_f(u) = exp(omega_f.x - |x|^2/2) / sqrt(m)
//   C_i = sum_j phi(q_i).phi(k_j) v_j / sum_j phi(q_i).phi(k_j);   A_hat = C W_dec
//
// The sequence is cut into chunks of 64 rows.  Kernel 1 forms each chunk's key state
// S_c = phi(K_c)^T [V_c | 1]  (m x 65).  Kernel 2 combines the states along the sequence
// in a fixed order: an exclusive prefix for causal attention, the total otherwise.
// Kernel 3 computes, per chunk, phi(Q_c) S + (phi(Q_c) phi(K_c)^T . tril) [V_c | 1]
// (the second term only when causal), divides, applies W_dec and writes A_hat.
// This file is the plain fp32 FMA form used for fp32 inputs (chunks of 64 rows); bf16 inputs
// take the tensor-core form in sea_estimate_tc.cu (chunks of 128 rows).
#include "sea_common.cuh"

namespace sea {
namespace {

constexpr int kC = kEstChunk;       // rows per chunk
constexpr int kLd = kHeadDim + 1;   // padded leading dimension of 64-wide tiles
constexpr int kThreads = 256;
constexpr int kStateCols = kHeadDim + 1;  // [V | 1]

// acc[a][b] += sum_k A(i_a, k) B(k, j_b) with i_a = ty + 16a, j_b = tx + 16b (j clamped to
// ncols-1 so that partial tiles stay inside the array; the caller discards those columns).
__device__ __forceinline__ void tile_mma(float (&acc)[4][4], const float* A, int sai, int sak,
                                         const float* B, int sbk, int sbj, int kd, int ncols,
                                         int ty, int tx) {
  int ao[4], bo[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    ao[x] = (ty + 16 * x) * sai;
    bo[x] = min(tx + 16 * x, ncols - 1) * sbj;
  }
#pragma unroll 4
  for (int k = 0; k < kd; ++k) {
    float a[4], b[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      a[x] = A[ao[x] + k * sak];
      b[x] = B[bo[x] + k * sbk];
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
  }
}

__device__ __forceinline__ void zero_acc(float (&acc)[4][4]) {
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) acc[x][y] = 0.f;
}

// Loads rows [row0, row0+64) of one head into a padded fp32 tile, times `mul`; rows >= seq_len are 0.
template <typename T>
__device__ __forceinline__ void load_chunk(float* dst, const T* head, int row0, int seq_len, float mul) {
  using IO = Io<T>;
  constexpr int EPL = IO::kElemsPerLane;
  constexpr int VEC_PER_ROW = kHeadDim / EPL;
  for (int v = threadIdx.x; v < kC * VEC_PER_ROW; v += kThreads) {
    const int rr = v / VEC_PER_ROW, cc = (v % VEC_PER_ROW) * EPL;
    float x[EPL];
    if (row0 + rr < seq_len) {
      IO::load(head + (size_t)(row0 + rr) * kHeadDim + cc, x);
    } else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) x[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) dst[rr * kLd + cc + e] = x[e] * mul;
  }
}

// phi[i][f] = exp(x_i . omega_f - |x_i|^2/2) / sqrt(m) for the 64 rows of a chunk; rows at or
// beyond `valid_rows` get 0.  x: [64][kLd], om: [m][kLd], phi: [64][m+1].
__device__ __forceinline__ void features(float* phi, const float* x, const float* om, float* sq,
                                         int m, int valid_rows, float inv_sqrt_m) {
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  if (threadIdx.x < kC) {
    float s = 0.f;
    for (int t = 0; t < kHeadDim; ++t) {
      const float v = x[threadIdx.x * kLd + t];
      s = fmaf(v, v, s);
    }
    sq[threadIdx.x] = 0.5f * s;
  }
  __syncthreads();
  const int ldp = m + 1;
  for (int f0 = 0; f0 < m; f0 += 64) {
    float acc[4][4];
    zero_acc(acc);
    tile_mma(acc, x, kLd, 1, om + f0 * kLd, 1, kLd, kHeadDim, m - f0, ty, tx);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int i = ty + 16 * a, f = f0 + tx + 16 * b;
        if (f < m) phi[i * ldp + f] = i < valid_rows ? __expf(acc[a][b] - sq[i]) * inv_sqrt_m : 0.f;
      }
  }
  __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
favor_key_state_kernel(const T* __restrict__ K, const T* __restrict__ V, const float* __restrict__ omega,
                       float* __restrict__ state, int seq_len, int m, int nchunk, float in_scale) {
  extern __shared__ float sm[];
  float* xk = sm;                    // [64][65]
  float* vv = xk + kC * kLd;         // [64][65]
  float* om = vv + kC * kLd;         // [m][65]
  float* phi = om + m * kLd;         // [64][m+1]
  float* sq = phi + kC * (m + 1);    // [64]
  const int chunk = blockIdx.x, bh = blockIdx.y;
  const int row0 = chunk * kC;
  const size_t head = (size_t)bh * seq_len * kHeadDim;
  load_chunk<T>(xk, K + head, row0, seq_len, in_scale);
  load_chunk<T>(vv, V + head, row0, seq_len, 1.f);
  for (int v = threadIdx.x; v < m * kHeadDim; v += kThreads)
    om[(v / kHeadDim) * kLd + (v % kHeadDim)] = __ldg(omega + v);
  __syncthreads();
  features(phi, xk, om, sq, m, min(kC, seq_len - row0), rsqrtf((float)m));

  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float* st = state + ((size_t)bh * nchunk + chunk) * (size_t)m * kStateCols;
  const int ldp = m + 1;
  for (int f0 = 0; f0 < m; f0 += 64) {
    float acc[4][4];
    zero_acc(acc);
    // S[f][e] = sum_i phi[i][f] v[i][e]   (A(i=f,k=i) = phi[k][f0+f])
    const int nf = min(64, m - f0);
    int fcl[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) fcl[a] = min(ty + 16 * a, nf - 1);
#pragma unroll 4
    for (int k = 0; k < kC; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        a[x] = phi[k * ldp + f0 + fcl[x]];
        b[x] = vv[k * kLd + tx + 16 * x];
      }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int f = f0 + ty + 16 * a;
        if (f < m) st[(size_t)f * kStateCols + tx + 16 * b] = acc[a][b];
      }
  }
  for (int f = threadIdx.x; f < m; f += kThreads) {
    float z = 0.f;
    for (int i = 0; i < kC; ++i) z += phi[i * ldp + f];
    st[(size_t)f * kStateCols + kHeadDim] = z;
  }
}

// Fixed-order combination of the chunk states of each head.
__global__ void favor_state_scan_kernel(float* __restrict__ state, int nchunk, int per_chunk,
                                        long long total_threads, int causal) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_threads) return;
  const long long bh = gid / per_chunk;
  const int e = (int)(gid - bh * per_chunk);
  float* p = state + (size_t)bh * nchunk * per_chunk + e;
  float run = 0.f;
  for (int c = 0; c < nchunk; ++c) {
    const float t = p[(size_t)c * per_chunk];
    if (causal) p[(size_t)c * per_chunk] = run;
    run += t;
  }
  if (!causal) p[0] = run;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
favor_output_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V,
                    const float* __restrict__ omega, const float* __restrict__ W_dec,
                    const float* __restrict__ state, float* __restrict__ A_hat,
                    int32_t* __restrict__ status, int seq_len, int m, int Kc, int nchunk, int causal,
                    float in_scale) {
  extern __shared__ float sm[];
  float* xq = sm;                       // [64][65]  later: C tile
  float* xk = xq + kC * kLd;            // [64][65]  later: masked kernel tile A, then W_dec tile
  float* vv = xk + kC * kLd;            // [64][65]
  float* om = vv + kC * kLd;            // [m][65]   later: prefix state S
  float* phiq = om + m * kLd;           // [64][m+1]
  float* phik = phiq + kC * (m + 1);    // [64][m+1]
  float* sq = phik + kC * (m + 1);      // [64]
  float* den = sq + kC;                 // [64]
  const int chunk = blockIdx.x, bh = blockIdx.y;
  const int row0 = chunk * kC;
  const int valid = min(kC, seq_len - row0);
  const size_t head = (size_t)bh * seq_len * kHeadDim;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int ldp = m + 1;
  const float inv_sqrt_m = rsqrtf((float)m);

  load_chunk<T>(xq, Q + head, row0, seq_len, in_scale);
  if (causal) {
    load_chunk<T>(xk, K + head, row0, seq_len, in_scale);
    load_chunk<T>(vv, V + head, row0, seq_len, 1.f);
  }
  for (int v = threadIdx.x; v < m * kHeadDim; v += kThreads)
    om[(v / kHeadDim) * kLd + (v % kHeadDim)] = __ldg(omega + v);
  __syncthreads();
  features(phiq, xq, om, sq, m, kC, inv_sqrt_m);
  if (causal) features(phik, xk, om, sq, m, valid, inv_sqrt_m);

  // prefix (or total) key state of this chunk -> om region as S [m][65]
  const float* st = state + ((size_t)bh * nchunk + (causal ? chunk : 0)) * (size_t)m * kStateCols;
  for (int v = threadIdx.x; v < m * kStateCols; v += kThreads) om[v] = st[v];
  __syncthreads();

  float num[4][4];
  zero_acc(num);
  tile_mma(num, phiq, ldp, 1, om, kStateCols, 1, m, kHeadDim, ty, tx);
  if (threadIdx.x < kC) {
    float s = 0.f;
    for (int f = 0; f < m; ++f) s = fmaf(phiq[threadIdx.x * ldp + f], om[f * kStateCols + kHeadDim], s);
    den[threadIdx.x] = s;
  }
  if (causal) {
    float acc[4][4];
    zero_acc(acc);
    tile_mma(acc, phiq, ldp, 1, phik, 1, ldp, m, kC, ty, tx);  // phi(q_i).phi(k_j)
    __syncthreads();  // every thread is done with xk as key tile
    float* At = xk;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int i = ty + 16 * a, j = tx + 16 * b;
        At[i * kLd + j] = j <= i ? acc[a][b] : 0.f;
      }
    __syncthreads();
    tile_mma(num, At, kLd, 1, vv, kLd, 1, kC, kHeadDim, ty, tx);
    if (threadIdx.x < kC) {
      float s = den[threadIdx.x];
      for (int j = 0; j < kC; ++j) s += At[threadIdx.x * kLd + j];
      den[threadIdx.x] = s;
    }
  }
  __syncthreads();
  float* Ct = xq;
  bool bad = false;
#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int i = ty + 16 * a;
    const float dn = den[i];
    if (i < valid && !(dn > 0.f && dn < INFINITY)) bad = true;
    const float inv = 1.f / dn;
#pragma unroll
    for (int b = 0; b < 4; ++b) Ct[i * kLd + tx + 16 * b] = num[a][b] * inv;
  }
  if (bad) atomicOr(status, SEA_DEV_NONFINITE);
  __syncthreads();

  float* Wt = xk;  // [64 (e)][65] tile of W_dec columns
  float* out = A_hat + ((size_t)bh * seq_len + row0) * Kc;
  for (int c0 = 0; c0 < Kc; c0 += 64) {
    const int nc = min(64, Kc - c0);
    for (int v = threadIdx.x; v < kHeadDim * 64; v += kThreads) {
      const int e = v >> 6, c = v & 63;
      Wt[e * kLd + c] = c < nc ? __ldg(W_dec + (size_t)e * Kc + c0 + c) : 0.f;
    }
    __syncthreads();
    float acc[4][4];
    zero_acc(acc);
    tile_mma(acc, Ct, kLd, 1, Wt, kLd, 1, kHeadDim, 64, ty, tx);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int i = ty + 16 * a, c = tx + 16 * b;
        if (i < valid && c < nc) out[(size_t)i * Kc + c0 + c] = acc[a][b];
      }
    __syncthreads();
  }
}

template <typename T>
sea_status launch_typed(const sea_shape& s, const T* Q, const T* K, const T* V, const float* omega,
                        const float* W_dec, float* A_hat, float* state, int32_t* status,
                        cudaStream_t st) {
  const int BH = s.B * s.H, m = s.m;
  const int nchunk = (s.T + kC - 1) / kC;
  const float in_scale = 0.35355339059327373f;  // 64^(-1/4)
  const size_t smem1 = sizeof(float) * (2 * kC * kLd + (size_t)m * kLd + (size_t)kC * (m + 1) + kC);
  const size_t smem3 = sizeof(float) * (3 * kC * kLd + (size_t)m * kLd + 2 * (size_t)kC * (m + 1) + 2 * kC);
  if (cudaFuncSetAttribute(favor_key_state_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess ||
      cudaFuncSetAttribute(favor_output_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem3) != cudaSuccess)
    return SEA_ERR_CUDA;
  const dim3 grid(nchunk, BH);
  favor_key_state_kernel<T><<<grid, kThreads, smem1, st>>>(K, V, omega, state, s.T, m, nchunk, in_scale);
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;
  const int per_chunk = m * kStateCols;
  const long long total = (long long)BH * per_chunk;
  favor_state_scan_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(state, nchunk, per_chunk, total, s.causal);
  if ((rc = check_launch()) != SEA_OK) return rc;
  favor_output_kernel<T><<<grid, kThreads, smem3, st>>>(Q, K, V, omega, W_dec, state, A_hat, status, s.T,
                                                        m, s.Kc, nchunk, s.causal, in_scale);
  return check_launch();
}

}  // namespace

sea_status launch_estimate_f32(const sea_shape& s, const void* Q, const void* K, const void* V,
                               const float* omega, const float* W_dec, float* A_hat, float* est_state,
                               int32_t* status, cudaStream_t st) {
  return launch_typed<float>(s, (const float*)Q, (const float*)K, (const float*)V, omega, W_dec, A_hat,
                             est_state, status, st);
}

sea_status launch_estimate(const sea_shape& s, const void* Q, const void* K, const void* V,
                           const float* omega, const float* W_dec, float* A_hat, float* est_state,
                           void* est_split, const SelectOut* select_out, bool* selected, int32_t* status,
                           cudaStream_t st) {
  if (selected != nullptr) *selected = false;
  if (s.io == SEA_BF16) {
    // the tensor-core form needs the driver's tensor-map encoder; there is no other bf16 path
    if (!estimate_tc_applicable(s)) return SEA_ERR_CUDA;
    const bool sel = select_out != nullptr && select_out->sel != nullptr && estimate_tc_selects(s);
    if (selected != nullptr) *selected = sel;
    return launch_estimate_tc(s, Q, K, V, omega, W_dec, A_hat, est_state, est_split, sel ? select_out : nullptr, status, st);
  }
  return launch_estimate_f32(s, Q, K, V, omega, W_dec, A_hat, est_state, status, st);
}

}  // namespace sea

// The paper's estimator head and output mixing with caller-given (random-init) weights:
//
//   V_cat = [V_I ; V], C_perf = FAVOR+(Q, K, V_cat)                 (Sec. 3.1 "Attention Matrix Estimation")
//   Z = mu([C_perf ; V]), Z_hat = nu(Z) -> image [H c_h, T, K / c_s]  (Sec. 3.1 "CNN Decoder")
//   A_hat = softmax(conv3(resize(conv2(conv1(image)))))               (App. "Attention Estimator CNN")
//   s_prob = sigmoid(f_prob(Z)), s_mix = sigmoid(f_pool(Z)), C_avg, C_sea = s_mix s_prob C + (1 - s_mix) C_avg
//                                                                     (Sec. 3.1.1)
//
// FAVOR+ is linear in the values, so C_perf is two runs of the library's own estimator (whose
// decoder is set to the identity): one on V_I (causal: the positional embedding), one on V.  The
// MLPs and the convolutions are plain fp32 kernels (the estimate has to agree with fp64 to 1e-3
// through three convolutions of 9 C terms each, which rules out bf16 operands without a remainder
// term); they are written for correctness first and are the slowest part of this path by far.
#include "sea_common.cuh"

namespace sea {
namespace {

// ---- V_I / positional embedding as a [B, H, T, 64] tensor in the io dtype ------------------------
template <typename T>
__global__ void first_values_kernel(T* __restrict__ out, const T* __restrict__ pos_emb, long long rows, int seq_len, int causal) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * kHeadDim) return;
  const int t = (int)((i / kHeadDim) % seq_len), c = (int)(i % kHeadDim);
  if (causal) out[i] = pos_emb[(size_t)t * kHeadDim + c];
  else out[i] = Io<T>::to_io(c == (int)(((long long)t * kHeadDim) / seq_len) ? 1.f : 0.f);
}

__global__ void identity64_kernel(float* __restrict__ w) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < kHeadDim * kHeadDim) w[i] = (i / kHeadDim == i % kHeadDim) ? 1.f : 0.f;
}

// ---- y = act(x W + b) for 64 rows per block; x is the concatenation of up to three 64-wide
// sources (two fp32, one in the io dtype) or one fp32 source of width k_in ----------------------
// image != 0: the output row (b, h, t) of width c_h * wr goes to the image [B][H c_h][T][wr] instead
// (entry j * wr + x -> channel h c_h + j, column x).
// A thread: 16 rows of one output column at a time (a warp shares its rows: their inputs come
// from shared memory as broadcasts, four values of k per load; the weights' reads run along n).
constexpr int kLinRows = 64, kLinRowsPerThread = 16, kLinCols = 64;

template <typename T>
__global__ void __launch_bounds__(256)
linear_kernel(const float* __restrict__ x0, const float* __restrict__ x1, const T* __restrict__ x2, int k_in,
              const float* __restrict__ W, const float* __restrict__ b, float* __restrict__ out, long long rows, int n_out,
              int relu, int image, int H, int seq_len, int c_h, int wr) {
  extern __shared__ __align__(16) float xs[];  // [kLinRows][k_pad], k_pad = k_in rounded up to a multiple of 4
  const int k_pad = (k_in + 3) & ~3;
  const long long row0 = (long long)blockIdx.x * kLinRows;
  for (int i = threadIdx.x; i < kLinRows * k_pad; i += blockDim.x) {
    const int r = i / k_pad, k = i - r * k_pad;
    const long long row = row0 + r;
    float v = 0.f;
    if (row < rows && k < k_in) {
      if (x1 == nullptr && x2 == nullptr) v = x0[row * k_in + k];
      else if (k < kHeadDim) v = x0[row * kHeadDim + k];
      else if (k < 2 * kHeadDim) v = x1[row * kHeadDim + k - kHeadDim];
      else v = Io<T>::from_io(x2[row * kHeadDim + k - 2 * kHeadDim]);
    }
    xs[i] = v;
  }
  __syncthreads();
  const int tn = threadIdx.x % kLinCols, tr = threadIdx.x / kLinCols;
  const float* my_x = xs + (size_t)tr * kLinRowsPerThread * k_pad;
  for (int n = tn; n < n_out; n += kLinCols) {
    float acc[kLinRowsPerThread];
    const float bn = b[n];
#pragma unroll
    for (int r = 0; r < kLinRowsPerThread; ++r) acc[r] = bn;
    for (int k = 0; k < k_pad; k += 4) {
      float w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) w[q] = (k + q < k_in) ? __ldg(W + (size_t)(k + q) * n_out + n) : 0.f;
#pragma unroll
      for (int r = 0; r < kLinRowsPerThread; ++r) {
        const float4 x = *reinterpret_cast<const float4*>(my_x + r * k_pad + k);
        acc[r] = fmaf(x.x, w[0], acc[r]);
        acc[r] = fmaf(x.y, w[1], acc[r]);
        acc[r] = fmaf(x.z, w[2], acc[r]);
        acc[r] = fmaf(x.w, w[3], acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < kLinRowsPerThread; ++r) {
      const long long row = row0 + tr * kLinRowsPerThread + r;
      if (row >= rows) break;
      const float y = relu ? fmaxf(acc[r], 0.f) : acc[r];
      if (!image) {
        out[row * n_out + n] = y;
      } else {
        const long long bh = row / seq_len;
        const int t = (int)(row - bh * seq_len), bb = (int)(bh / H), h = (int)(bh - (long long)bb * H);
        const int j = n / wr, xcol = n - j * wr;
        out[(((size_t)bb * H * c_h + (size_t)h * c_h + j) * seq_len + t) * wr + xcol] = y;
      }
    }
  }
}

// ---- 3 x 3 convolution, NCHW fp32 ------------------------------------------------------------------
// Logical input: [C_in][H_in * up_h][W_in * up_w], entry (y, x) = in[y / up_h][x / up_w] (a nearest
// resize folded into the read).  Width padded by one on both sides; height: pad_top rows above, as
// many below as the kernel needs to reach h_out rows at stride_h.  Output [C_out][h_out][w_out],
// w_out = W_in * up_w.  A block: 8 output channels x 16 rows x 32 columns; a thread: 4 rows of
// one column for the 8 channels.
constexpr int kCvCo = 8, kCvCi = 8, kCvTw = 32, kCvTh = 16, kCvPx = 4;

__global__ void __launch_bounds__(128)
conv3x3_kernel(const float* __restrict__ in, const float* __restrict__ w, const float* __restrict__ bias, float* __restrict__ out,
               int c_in, int h_in, int w_in, int up_h, int up_w, int stride_h, int pad_top, int c_out, int h_out, int relu) {
  extern __shared__ float sm[];
  const int w_log = w_in * up_w, h_log = h_in * up_h;
  const int patch_h = (kCvTh - 1) * stride_h + 3, patch_w = kCvTw + 2;
  float* s_in = sm;                                  // [kCvCi][patch_h][patch_w]
  float* s_w = sm + kCvCi * patch_h * patch_w;       // [kCvCo][kCvCi][9]
  const int tiles_w = (w_log + kCvTw - 1) / kCvTw;
  const int tx0 = (blockIdx.x % tiles_w) * kCvTw, ty0 = (blockIdx.x / tiles_w) * kCvTh;
  const int co0 = blockIdx.y * kCvCo, n = blockIdx.z;
  const int lx = threadIdx.x % kCvTw, ly = threadIdx.x / kCvTw;  // column, group of four rows
  const float* in_n = in + (size_t)n * c_in * h_in * w_in;
  float acc[kCvCo][kCvPx];
#pragma unroll
  for (int o = 0; o < kCvCo; ++o)
#pragma unroll
    for (int q = 0; q < kCvPx; ++q) acc[o][q] = 0.f;
  const int y_in0 = ty0 * stride_h - pad_top;  // logical input row of the patch's first row
  for (int ci0 = 0; ci0 < c_in; ci0 += kCvCi) {
    __syncthreads();
    for (int i = threadIdx.x; i < kCvCi * patch_h * patch_w; i += blockDim.x) {
      const int c = i / (patch_h * patch_w), rem = i - c * patch_h * patch_w;
      const int py = rem / patch_w, px = rem - py * patch_w;
      const int y = y_in0 + py, x = tx0 - 1 + px;
      float v = 0.f;
      if (ci0 + c < c_in && y >= 0 && y < h_log && x >= 0 && x < w_log)
        v = __ldg(in_n + ((size_t)(ci0 + c) * h_in + y / up_h) * w_in + x / up_w);
      s_in[i] = v;
    }
    for (int i = threadIdx.x; i < kCvCo * kCvCi * 9; i += blockDim.x) {
      const int o = i / (kCvCi * 9), rem = i - o * kCvCi * 9, c = rem / 9, tap = rem - c * 9;
      s_w[i] = (co0 + o < c_out && ci0 + c < c_in) ? __ldg(w + ((size_t)(co0 + o) * c_in + ci0 + c) * 9 + tap) : 0.f;
    }
    __syncthreads();
#pragma unroll 1
    for (int c = 0; c < kCvCi; ++c) {
      // the strip of the patch this thread's four output rows read: rows (4 ly + q) stride + ky, columns lx + kx
      const float* strip = s_in + c * patch_h * patch_w + (kCvPx * ly * stride_h) * patch_w + lx;
#pragma unroll
      for (int o = 0; o < kCvCo; ++o) {
        const float* wv = s_w + (o * kCvCi + c) * 9;
#pragma unroll
        for (int ky = 0; ky < 3; ++ky)
#pragma unroll
          for (int kx = 0; kx < 3; ++kx) {
            const float wgt = wv[3 * ky + kx];
#pragma unroll
            for (int q = 0; q < kCvPx; ++q) acc[o][q] = fmaf(strip[(q * stride_h + ky) * patch_w + kx], wgt, acc[o][q]);
          }
      }
    }
  }
  const int x = tx0 + lx;
  if (x >= w_log) return;
#pragma unroll
  for (int o = 0; o < kCvCo; ++o) {
    if (co0 + o >= c_out) break;
    const float bv = bias[co0 + o];
#pragma unroll
    for (int q = 0; q < kCvPx; ++q) {
      const int y = ty0 + kCvPx * ly + q;
      if (y < h_out) {
        const float v = acc[o][q] + bv;
        out[(((size_t)n * c_out + co0 + o) * h_out + y) * w_log + x] = relu ? fmaxf(v, 0.f) : v;
      }
    }
  }
}

// ---- row softmax in place (one warp per row) -----------------------------------------------------
__global__ void __launch_bounds__(256)
softmax_rows_kernel(float* __restrict__ a, long long rows, int width) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  float* p = a + row * width;
  float mx = -INFINITY;
  for (int c = lane; c < width; c += 32) mx = fmaxf(mx, p[c]);
  mx = warp_max(mx);
  float sum = 0.f;
  for (int c = lane; c < width; c += 32) sum += __expf(p[c] - mx);
  sum = warp_sum(sum);
  const float inv = 1.f / sum;
  for (int c = lane; c < width; c += 32) p[c] = __expf(p[c] - mx) * inv;
}

// the decoder's logits [B][H][T][Kc] are already in A_hat's layout (channel = head): nothing to transpose

// ---- scalers: s = sigmoid(Z . w + b) for both heads, one thread per row ---------------------------
__global__ void scalers_kernel(const float* __restrict__ Z, const float* __restrict__ w_prob, const float* __restrict__ w_mix,
                               float b_prob, float b_mix, float* __restrict__ s_prob, float* __restrict__ s_mix, long long rows,
                               int d_hidden) {
  const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  float a = b_prob, m = b_mix;
  for (int k = 0; k < d_hidden; ++k) {
    const float z = Z[row * d_hidden + k];
    a = fmaf(z, __ldg(w_prob + k), a);
    m = fmaf(z, __ldg(w_mix + k), m);
  }
  s_prob[row] = 1.f / (1.f + __expf(-a));
  s_mix[row] = 1.f / (1.f + __expf(-m));
}

// ---- pooled context ---------------------------------------------------------------------------------
// causal: running mean of V along the sequence.  One block per head: its 64 x 16 threads split the
// sequence into 16 segments per column, sum their segments, take the sums of the segments before
// theirs from shared memory and walk their segments again.
constexpr int kMeanSegs = 16;
template <typename T>
__global__ void __launch_bounds__(kHeadDim * kMeanSegs)
running_mean_kernel(const T* __restrict__ V, float* __restrict__ c_avg, int seq_len) {
  __shared__ float seg_sum[kMeanSegs][kHeadDim];
  const int bh = blockIdx.x, c = threadIdx.x % kHeadDim, sg = threadIdx.x / kHeadDim;
  const int seg_len = (seq_len + kMeanSegs - 1) / kMeanSegs;
  const int t0 = min(seq_len, sg * seg_len), t1 = min(seq_len, t0 + seg_len);
  const T* v = V + (size_t)bh * seq_len * kHeadDim + c;
  float* o = c_avg + (size_t)bh * seq_len * kHeadDim + c;
  float sum = 0.f;
  for (int t = t0; t < t1; ++t) sum += Io<T>::from_io(v[(size_t)t * kHeadDim]);
  seg_sum[sg][c] = sum;
  __syncthreads();
  sum = 0.f;
  for (int q = 0; q < sg; ++q) sum += seg_sum[q][c];
  for (int t = t0; t < t1; ++t) {
    sum += Io<T>::from_io(v[(size_t)t * kHeadDim]);
    o[(size_t)t * kHeadDim] = sum / (float)(t + 1);
  }
}
// not causal: importance i_hat = column means of A_hat, resized to T keys by nearest neighbour,
// C_avg = i^T V; one block per head, its 64 x 4 threads split the keys four ways
template <typename T>
__global__ void __launch_bounds__(256)
pooled_kernel(const float* __restrict__ A_hat, const T* __restrict__ V, float* __restrict__ c_avg, int seq_len, int Kc) {
  extern __shared__ float i_hat[];  // [Kc]
  __shared__ float part[4][kHeadDim];
  const int bh = blockIdx.x;
  const float* a = A_hat + (size_t)bh * seq_len * Kc;
  for (int c = threadIdx.x; c < Kc; c += blockDim.x) {
    float s = 0.f;
    for (int t = 0; t < seq_len; ++t) s += a[(size_t)t * Kc + c];
    i_hat[c] = s / (float)seq_len;
  }
  __syncthreads();
  const int c = threadIdx.x & 63, q = threadIdx.x >> 6;
  const T* v = V + (size_t)bh * seq_len * kHeadDim + c;
  float s = 0.f;
  for (int j = q; j < seq_len; j += 4) s = fmaf(i_hat[(int)(((long long)j * Kc) / seq_len)], Io<T>::from_io(v[(size_t)j * kHeadDim]), s);
  part[q][c] = s;
  __syncthreads();
  if (q == 0) c_avg[(size_t)bh * kHeadDim + c] = (part[0][c] + part[1][c]) + (part[2][c] + part[3][c]);
}

// ---- C_sea = s_mix (s_prob C) + (1 - s_mix) C_avg, in place over O; P *= s_prob --------------------
template <typename T>
__global__ void mix_kernel(T* __restrict__ O, const float* __restrict__ s_prob, const float* __restrict__ s_mix,
                           const float* __restrict__ c_avg, long long rows, int seq_len, int causal) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * kHeadDim) return;
  const long long row = i / kHeadDim;
  const int c = (int)(i - row * kHeadDim);
  const float avg = causal ? c_avg[i] : c_avg[(row / seq_len) * kHeadDim + c];
  const float sm_ = s_mix[row];
  O[i] = Io<T>::to_io(sm_ * (s_prob[row] * Io<T>::from_io(O[i])) + (1.f - sm_) * avg);
}
template <typename T>
__global__ void __launch_bounds__(256)
scale_p_kernel(T* __restrict__ P, const int32_t* __restrict__ row_ptr, const float* __restrict__ s_prob, long long rows) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int lo = row_ptr[row], hi = row_ptr[row + 1];
  const float s = s_prob[row];
  for (int j = lo + lane; j < hi; j += 32) P[j] = Io<T>::to_io(s * Io<T>::from_io(P[j]));
}

int conv_out_h(int h_log, int stride_h) { return (h_log + 2 - 3) / stride_h + 1; }  // two rows of padding in all

sea_status conv3x3(const float* in, const float* w, const float* b, float* out, int n, int c_in, int h_in, int w_in, int up_h,
                   int up_w, int stride_h, int pad_top, int c_out, int relu, cudaStream_t st) {
  const int h_log = h_in * up_h, w_log = w_in * up_w;
  const int h_out = conv_out_h(h_log, stride_h);
  const int patch_h = (kCvTh - 1) * stride_h + 3;
  const size_t smem = (size_t)(kCvCi * patch_h * (kCvTw + 2) + kCvCo * kCvCi * 9) * sizeof(float);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(conv3x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return SEA_ERR_CUDA;
  const dim3 grid(((w_log + kCvTw - 1) / kCvTw) * ((h_out + kCvTh - 1) / kCvTh), (c_out + kCvCo - 1) / kCvCo, n);
  conv3x3_kernel<<<grid, 128, smem, st>>>(in, w, b, out, c_in, h_in, w_in, up_h, up_w, stride_h, pad_top, c_out, h_out, relu);
  return check_launch();
}

template <typename T>
sea_status linear(const float* x0, const float* x1, const T* x2, int k_in, const float* W, const float* b, float* out,
                  long long rows, int n_out, int relu, int image, int H, int seq_len, int c_h, int wr, cudaStream_t st) {
  const size_t smem = (size_t)kLinRows * ((k_in + 3) & ~3) * sizeof(float);
  if (smem > 48 * 1024 &&
      cudaFuncSetAttribute(linear_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return SEA_ERR_CUDA;
  linear_kernel<T><<<(unsigned)((rows + kLinRows - 1) / kLinRows), 256, smem, st>>>(x0, x1, x2, k_in, W, b, out, rows, n_out,
                                                                                   relu, image, H, seq_len, c_h, wr);
  return check_launch();
}

}  // namespace

// True when all three convolutions of this shape run in the tensor-core form.
static bool decoder_conv_tc(const sea_shape& s, const sea_decoder& dec) {
  const int C = s.H * dec.c_h, wr = s.Kc / dec.c_s;
  const int stride1 = s.causal ? 1 : dec.c_s;
  const int t1 = conv_out_h(s.T, stride1);
  if (t1 <= 0 || s.T % t1 != 0) return false;
  return conv_tc_shape_ok(C, C, s.T, wr, 1, 1, stride1, false) && conv_tc_shape_ok(C, C, t1, wr, 1, 1, 1, false) &&
         conv_tc_shape_ok(C, s.H, t1, wr, s.T / t1, dec.c_s, 1, true);
}

// Buffers of the decoder path inside its part of the workspace (all offsets 256-byte aligned).
DecoderLayout decoder_layout(const sea_shape& s, const sea_decoder& dec) {
  DecoderLayout L{};
  const size_t rows = (size_t)s.B * s.H * s.T;
  const size_t elem = s.io == SEA_BF16 ? 2 : 4;
  const size_t C = (size_t)s.H * dec.c_h, wr = (size_t)s.Kc / dec.c_s;
  const size_t t1 = s.causal ? (size_t)s.T : (size_t)conv_out_h(s.T, dec.c_s);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes, 256);
    return at;
  };
  L.ident = take((size_t)kHeadDim * kHeadDim * sizeof(float));
  L.first = take(rows * kHeadDim * elem);
  L.c_first = take(rows * kHeadDim * sizeof(float));
  L.c_value = take(rows * kHeadDim * sizeof(float));
  L.z = take(rows * (size_t)dec.d_hidden * sizeof(float));
  L.hidden = take(rows * (size_t)dec.d_hidden * sizeof(float));
  L.image = take((size_t)s.B * C * s.T * wr * sizeof(float));
  // (in the tensor-core form the buffers hold bf16 head / remainder planes of whole blocks of 64 channels)
  const size_t Cs = decoder_conv_tc(s, dec) ? (size_t)conv_tc_channels((int)C) : C;
  L.conv_a = take((size_t)s.B * Cs * t1 * wr * sizeof(float));
  L.conv_b = take((size_t)s.B * Cs * t1 * wr * sizeof(float));
  L.s_prob = take(rows * sizeof(float));
  L.s_mix = take(rows * sizeof(float));
  L.c_avg = take((s.causal ? rows : (size_t)s.B * s.H) * kHeadDim * sizeof(float));
  if (decoder_conv_tc(s, dec)) {
    L.act0 = take((size_t)s.B * Cs * s.T * wr * 2 * sizeof(__nv_bfloat16));
    L.w_tiles = take(3 * align_up(conv_tc_weight_bytes((int)C), 256));
    if (mlp_tc_shape_ok(dec.d_hidden, (int)wr * dec.c_h)) L.mlp_w = take(mlp_tc_weight_bytes((int)wr * dec.c_h));
  }
  L.total = off;
  return L;
}

template <typename T>
static sea_status estimate_decoder_typed(const sea_shape& s, const sea_decoder& dec, const T* Q, const T* K, const T* V,
                                         const float* omega, float* A_hat, float* Z, char* dws, float* est_state,
                                         void* est_split, int32_t* status, cudaStream_t st) {
  const DecoderLayout L = decoder_layout(s, dec);
  const long long rows = (long long)s.B * s.H * s.T;
  float* ident = reinterpret_cast<float*>(dws + L.ident);
  T* first = reinterpret_cast<T*>(dws + L.first);
  float* c_first = reinterpret_cast<float*>(dws + L.c_first);
  float* c_value = reinterpret_cast<float*>(dws + L.c_value);
  float* hidden = reinterpret_cast<float*>(dws + L.hidden);
  float* image = reinterpret_cast<float*>(dws + L.image);
  float* conv_a = reinterpret_cast<float*>(dws + L.conv_a);
  float* conv_b = reinterpret_cast<float*>(dws + L.conv_b);
  sea_status rc;
  identity64_kernel<<<(kHeadDim * kHeadDim + 255) / 256, 256, 0, st>>>(ident);
  if ((rc = check_launch()) != SEA_OK) return rc;
  first_values_kernel<T><<<(unsigned)((rows * kHeadDim + 255) / 256), 256, 0, st>>>(first, static_cast<const T*>(dec.pos_emb), rows,
                                                                                  s.T, s.causal);
  if ((rc = check_launch()) != SEA_OK) return rc;
  // C_perf: the library's estimator with the identity as its decoder, on V_I (or the embedding) and on V
  sea_shape e = s;
  e.Kc = kHeadDim;
  e.k_hat = 1;
  if ((rc = launch_estimate(e, Q, K, first, omega, ident, c_first, est_state, est_split, nullptr, nullptr, status, st)) != SEA_OK)
    return rc;
  if ((rc = launch_estimate(e, Q, K, V, omega, ident, c_value, est_state, est_split, nullptr, nullptr, status, st)) != SEA_OK)
    return rc;
  const int wr = s.Kc / dec.c_s, C = s.H * dec.c_h;
  // with the convolutions in their tensor-core form the MLPs can run in theirs, writing the CNN's input as bf16 planes
  const bool mlp_tc = decoder_conv_tc(s, dec) && mlp_tc_shape_ok(dec.d_hidden, wr * dec.c_h);
  // Z = relu([C_perf ; V] W_mu + b_mu); Z_hat = relu(Z W_1 + b_1) W_2 + b_2, written as the image
  if (mlp_tc) {
    if ((rc = launch_mlp_tc(s, dec, c_first, c_value, V, Z, dws + L.act0, dws + L.mlp_w, status, st)) != SEA_OK) return rc;
  } else {
    if ((rc = linear<T>(c_first, c_value, V, 3 * kHeadDim, dec.W_mu, dec.b_mu, Z, rows, dec.d_hidden, 1, 0, 0, 0, 0, 0, st)) != SEA_OK)
      return rc;
    if ((rc = linear<T>(Z, nullptr, nullptr, dec.d_hidden, dec.W_nu1, dec.b_nu1, hidden, rows, dec.d_hidden, 1, 0, 0, 0, 0, 0, st)) !=
        SEA_OK)
      return rc;
    if ((rc = linear<T>(hidden, nullptr, nullptr, dec.d_hidden, dec.W_nu2, dec.b_nu2, image, rows, wr * dec.c_h, 0, 1, s.H, s.T,
                        dec.c_h, wr, st)) != SEA_OK)
      return rc;
  }
  // the CNN: causal layers see rows t-2 .. t (two rows of padding above), the others pad one row on either side
  const int pad_top = s.causal ? 2 : 1;
  const int stride1 = s.causal ? 1 : dec.c_s;
  const int t1 = conv_out_h(s.T, stride1);
  if (decoder_conv_tc(s, dec)) {
    // tensor-core form: activations as bf16 head / remainder planes, pixel-major
    char* act0 = dws + L.act0;
    char* wt = dws + L.w_tiles;
    const size_t wt_step = align_up(conv_tc_weight_bytes(C), 256);
    if (!mlp_tc && (rc = launch_nchw_to_nhwc_split(image, act0, s.B, C, s.T, wr, st)) != SEA_OK) return rc;
    if ((rc = launch_conv_tc(act0, s.B, C, s.T, wr, 1, 1, stride1, pad_top, dec.conv1_w, dec.conv1_b, C, 1, wt, conv_a, nullptr,
                             status, st)) != SEA_OK)
      return rc;
    if ((rc = launch_conv_tc(conv_a, s.B, C, t1, wr, 1, 1, 1, pad_top, dec.conv2_w, dec.conv2_b, C, 1, wt + wt_step, conv_b, nullptr,
                             status, st)) != SEA_OK)
      return rc;
    if ((rc = launch_conv_tc(conv_b, s.B, C, t1, wr, s.T / t1, dec.c_s, 1, pad_top, dec.conv3_w, dec.conv3_b, s.H, 0,
                             wt + 2 * wt_step, nullptr, A_hat, status, st)) != SEA_OK)
      return rc;
    softmax_rows_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(A_hat, rows, s.Kc);
    return check_launch();
  }
  if ((rc = conv3x3(image, dec.conv1_w, dec.conv1_b, conv_a, s.B, C, s.T, wr, 1, 1, stride1, pad_top, C, 1, st)) != SEA_OK) return rc;
  if ((rc = conv3x3(conv_a, dec.conv2_w, dec.conv2_b, conv_b, s.B, C, t1, wr, 1, 1, 1, pad_top, C, 1, st)) != SEA_OK) return rc;
  // nearest resize to [T, Kc] folded into the last layer's reads (integer factors: T = t1 * up_h, Kc = wr * c_s)
  if ((rc = conv3x3(conv_b, dec.conv3_w, dec.conv3_b, A_hat, s.B, C, t1, wr, s.T / t1, dec.c_s, 1, pad_top, s.H, 0, st)) != SEA_OK)
    return rc;
  softmax_rows_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(A_hat, rows, s.Kc);
  return check_launch();
}

sea_status launch_estimate_decoder(const sea_shape& s, const sea_decoder& dec, const void* Q, const void* K, const void* V,
                                   const float* omega, float* A_hat, float* Z, char* dws, float* est_state, void* est_split,
                                   int32_t* status, cudaStream_t st) {
  if (s.io == SEA_BF16)
    return estimate_decoder_typed<__nv_bfloat16>(s, dec, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K,
                                                 (const __nv_bfloat16*)V, omega, A_hat, Z, dws, est_state, est_split, status, st);
  return estimate_decoder_typed<float>(s, dec, (const float*)Q, (const float*)K, (const float*)V, omega, A_hat, Z, dws, est_state,
                                       est_split, status, st);
}

template <typename T>
static sea_status mix_typed(const sea_shape& s, const sea_decoder& dec, const float* Z, const float* A_hat, const T* V,
                            const int32_t* row_ptr, T* O, T* P, char* dws, cudaStream_t st) {
  const DecoderLayout L = decoder_layout(s, dec);
  const long long rows = (long long)s.B * s.H * s.T;
  float* s_prob = reinterpret_cast<float*>(dws + L.s_prob);
  float* s_mix = reinterpret_cast<float*>(dws + L.s_mix);
  float* c_avg = reinterpret_cast<float*>(dws + L.c_avg);
  sea_status rc;
  scalers_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(Z, dec.w_prob, dec.w_mix, dec.b_prob, dec.b_mix, s_prob, s_mix, rows,
                                                               dec.d_hidden);
  if ((rc = check_launch()) != SEA_OK) return rc;
  const int BH = s.B * s.H;
  if (s.causal) running_mean_kernel<T><<<BH, kHeadDim * kMeanSegs, 0, st>>>(V, c_avg, s.T);
  else pooled_kernel<T><<<BH, 256, (size_t)s.Kc * sizeof(float), st>>>(A_hat, V, c_avg, s.T, s.Kc);
  if ((rc = check_launch()) != SEA_OK) return rc;
  mix_kernel<T><<<(unsigned)((rows * kHeadDim + 255) / 256), 256, 0, st>>>(O, s_prob, s_mix, c_avg, rows, s.T, s.causal);
  if ((rc = check_launch()) != SEA_OK) return rc;
  if (P != nullptr) {
    scale_p_kernel<T><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(P, row_ptr, s_prob, rows);
    rc = check_launch();
  }
  return rc;
}

sea_status launch_mix_output(const sea_shape& s, const sea_decoder& dec, const float* Z, const float* A_hat, const void* V,
                             const int32_t* row_ptr, void* O, void* P, char* dws, cudaStream_t st) {
  if (s.io == SEA_BF16)
    return mix_typed<__nv_bfloat16>(s, dec, Z, A_hat, (const __nv_bfloat16*)V, row_ptr, (__nv_bfloat16*)O, (__nv_bfloat16*)P, dws, st);
  return mix_typed<float>(s, dec, Z, A_hat, (const float*)V, row_ptr, (float*)O, (float*)P, dws, st);
}

}  // namespace sea

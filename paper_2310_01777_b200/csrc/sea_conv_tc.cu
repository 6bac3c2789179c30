// Tensor-core form of the estimator head's 3 x 3 convolutions (Sec. 3.1 "CNN Decoder", App.
// "Attention Estimator CNN"): an implicit GEMM per tap on tcgen05, fp32 accumulators in tensor memory.
//
// A layer is out[pixel][n] = sum over taps (a, b) and input channels c of
//     act[pixel shifted by tap (a, b)][c] * w_eff[(a, b)][n][c],
// i.e. nine GEMMs of [pixels x C_in] by [C_in x N] accumulated into one tile: M = 128 pixels (a
// box of bh rows x bw columns of the feature map), N <= 128, K = 64 input channels per block.
//   * Activations live as NHWC bf16 in two planes, head and remainder (x ~ hi + lo, 2^-17
//     relative), so that a pixel's 64 channels are one 128-byte row of a K-major operand tile and
//     a tap's shift is just another box coordinate of the same tensor map: rows and columns
//     outside the map read as zero, which is the layer's zero padding.  The stride of the first
//     (non-causal) layer is a view [Y][s] of the input rows, row = Y stride + s.
//   * Three products per step: hi hi + hi lo + lo hi (the lo lo term is below fp32 rounding).
//   * The nearest resize before the last layer is folded into its weights: an output pixel
//     (Y up_h + py, X up_w + px) reads stored pixels (Y + dY, X + dX) only, with dY, dX in a set of
//     at most three values, so the layer is a 3 x 3 convolution on the stored grid with
//     N = up_h up_w C_out outputs per pixel, one group of C_out per phase (py, px), and weights that
//     are the sums of the original taps that fall on the same stored pixel.
//   * Roles of the 192 threads: warp 0 copies (TMA), warp 1 issues the MMAs (one elected lane),
//     warps 2-5 take finished tiles out of tensor memory (bias, ReLU, split or phase scatter).  Two
//     accumulator tiles per work item share the weights' tiles; accumulators are double-buffered so
//     that the epilogue of one item runs under the products of the next.
// Every wait is bounded (abort flag + SEA_DEV_TIMEOUT in the status word).
#include "sea_common.cuh"
#include "sea_tc.cuh"

namespace sea {
using namespace tc;

namespace {

constexpr int kCtTiles = 2;           // accumulator tiles (of 128 pixels) per work item
constexpr int kCtStages = 2;
constexpr int kCtTileBytes = 16384;   // 128 rows x 64 bf16
constexpr int kCtStageBytes = (2 * kCtTiles + 2) * kCtTileBytes;  // A: tiles x {hi, lo}; B: hi, lo
constexpr int kCtThreads = 192;
constexpr int kCtMaxN = 128;

struct ConvTcParams {
  int n_cblk;             // C_in / 64
  int n_out;              // accumulator columns N (a multiple of 32): n_real outputs and columns of zeros
  int n_real;
  int bw, bh;             // pixel tile: bh rows of bw columns, bh * bw = 128
  int tiles_x, tiles_y;   // tiles_y counts groups of kCtTiles tile rows
  int n_items;
  int batch;              // plane p of batch element b is slice p * batch + b of the activations
  int h_out, w_out;       // grid of output pixels (before the phase scatter)
  int ny, nx;             // taps per axis
  int tap_s[3], tap_y[3], tap_x[3];
  const float* bias;      // [c_out]
  int c_out, relu;
  __nv_bfloat16* out_split;  // [2][batch][h_out][w_out][n_out]   (kLogits == false; channels c_out .. n_out - 1 are zero)
  float* out_logits;         // [batch][c_out][h_out up_h][w_out up_w]   (kLogits == true)
  int up_h, up_w;
  int32_t* status;
};

enum { kCt_Full = 0, kCt_Empty = kCt_Full + kCtStages, kCt_AccFull = kCt_Empty + kCtStages, kCt_AccEmpty = kCt_AccFull + 2,
       kCt_Drain = kCt_AccEmpty + 2, kCt_NumBars };

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, int c4,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];\n"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar) : "memory");
}
__device__ __forceinline__ void ct_warp_arrive(uint32_t bar, int lane) {
  fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}
__host__ __device__ inline int floor_div(int a, int b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }

template <bool kLogits>
__global__ void __launch_bounds__(kCtThreads, 1)
conv_taps_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const ConvTcParams p) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* sm = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  unsigned char* tail = sm + kCtStages * kCtStageBytes;
  const uint32_t bars = smem_u32(tail);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kCt_NumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8 * kCt_NumBars + 4);
  float* bias_s = reinterpret_cast<float*>(tail + 128);  // [kCtMaxN], by accumulator column
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < kCt_NumBars; ++i) mbar_init(bar(i), (i >= kCt_AccEmpty && i < kCt_AccEmpty + 2) ? 4 : 1);
    *abort_flag = 0;
    mbar_init_fence();
  }
  for (int n = tid; n < kCtMaxN; n += kCtThreads) bias_s[n] = n < p.n_real ? p.bias[n % p.c_out] : 0.f;
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), 512);
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_kblk = p.ny * p.nx * p.n_cblk;
  const uint32_t b_bytes = (uint32_t)p.n_out * 128u;

  if (warp == 0) {
    // ---------------------------------------------------------------- copies
    const bool leader = elect_one();
    bool ok = true;
    uint32_t kb = 0;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
      const int tx = item % p.tiles_x, rest = item / p.tiles_x, ty = rest % p.tiles_y, b = rest / p.tiles_y;
      const int x0 = tx * p.bw, y0 = ty * kCtTiles * p.bh;
      for (int a = 0; a < p.ny && ok; ++a)
        for (int bx = 0; bx < p.nx && ok; ++bx)
          for (int cb = 0; cb < p.n_cblk; ++cb, ++kb) {
            const uint32_t s = kb % kCtStages, use = kb / kCtStages;
            if (use > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(kCt_Empty + s), (use - 1) & 1, abort_flag));
            if (!ok) break;
            if (leader) {
              const uint32_t dst = smem_u32(sm) + s * kCtStageBytes;
              mbar_expect_tx(bar(kCt_Full + s), 2 * kCtTiles * kCtTileBytes + 2 * b_bytes);
#pragma unroll
              for (int m = 0; m < kCtTiles; ++m)
#pragma unroll
                for (int plane = 0; plane < 2; ++plane)
                  tma_load_5d(dst + (2 * m + plane) * kCtTileBytes, &map_a, cb * 64, x0 + p.tap_x[bx], p.tap_s[a],
                              y0 + m * p.bh + p.tap_y[a], plane * p.batch + b, bar(kCt_Full + s));
              const int wt = ((a * p.nx + bx) * p.n_cblk + cb) * 2;
#pragma unroll
              for (int plane = 0; plane < 2; ++plane)
                tma_load_3d(dst + (2 * kCtTiles + plane) * kCtTileBytes, &map_w, 0, 0, wt + plane, bar(kCt_Full + s));
            }
            __syncwarp();
          }
    }
    // copies still in flight must land before the CTA may leave (only after a wait ran out can the
    // consumer have stopped short of them)
    if (!ok)
      for (uint32_t j = (kb >= kCtStages ? kb - kCtStages : 0); j < kb; ++j)
        mbar_wait_drain(bar(kCt_Full + j % kCtStages), (j / kCtStages) & 1);
  } else if (warp == 1) {
    // ---------------------------------------------------------------- products
    const bool leader = elect_one();
    bool ok = true;
    uint32_t kb = 0, it = 0;
    const uint32_t idesc = idesc_bf16(p.n_out, false, false);
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++it) {
      const uint32_t buf = it & 1, v = it >> 1;
      if (v > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(kCt_AccEmpty + buf), (v - 1) & 1, abort_flag));
      for (int j = 0; j < n_kblk && ok; ++j, ++kb) {
        const uint32_t s = kb % kCtStages, use = kb / kCtStages;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kCt_Full + s), use & 1, abort_flag));
        if (!ok) break;
        fence_after();
        const uint32_t base = smem_u32(sm) + s * kCtStageBytes;
        const uint64_t wh = smem_desc(base + 2 * kCtTiles * kCtTileBytes, 16, 1024);
        const uint64_t wl = smem_desc(base + (2 * kCtTiles + 1) * kCtTileBytes, 16, 1024);
        if (leader) {
#pragma unroll
          for (int m = 0; m < kCtTiles; ++m) {
            const uint64_t ah = smem_desc(base + 2 * m * kCtTileBytes, 16, 1024);
            const uint64_t al = smem_desc(base + (2 * m + 1) * kCtTileBytes, 16, 1024);
            const uint32_t d = tmem + buf * (kCtTiles * kCtMaxN) + m * kCtMaxN;
#pragma unroll
            for (int k = 0; k < 4; ++k) {  // 16 channels = 32 bytes = 2 descriptor units per step
              mma_ss(d, ah + 2 * k, wh + 2 * k, idesc, (j > 0 || k > 0) ? 1u : 0u);
              mma_ss(d, ah + 2 * k, wl + 2 * k, idesc, 1);
              mma_ss(d, al + 2 * k, wh + 2 * k, idesc, 1);
            }
          }
          mma_commit(bar(kCt_Empty + s));
        }
        __syncwarp();
      }
      if (ok && leader) mma_commit(bar(kCt_AccFull + buf));
      __syncwarp();
    }
    // every product issued has completed before tensor memory is given back
    if (leader) mma_commit(bar(kCt_Drain));
    __syncwarp();
    mbar_wait(bar(kCt_Drain), 0, abort_flag);
  } else {
    // ---------------------------------------------------------------- finished tiles
    const int quarter = warp & 3, r = quarter * 32 + lane;  // the warp's lanes of tensor memory; the thread's pixel of a tile
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const int py_t = r / p.bw, px_t = r - py_t * p.bw;
    bool ok = true;
    uint32_t it = 0;
    for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++it) {
      const int tx = item % p.tiles_x, rest = item / p.tiles_x, ty = rest % p.tiles_y, b = rest / p.tiles_y;
      const uint32_t buf = it & 1, v = it >> 1;
      ok = __all_sync(0xffffffffu, mbar_wait_idle(bar(kCt_AccFull + buf), v & 1, abort_flag));
      if (!ok) break;
      fence_after();
      const int x = tx * p.bw + px_t;
#pragma unroll 1
      for (int m = 0; m < kCtTiles; ++m) {
        const int y = (ty * kCtTiles + m) * p.bh + py_t;
        const bool live = y < p.h_out;
#pragma unroll 1
        for (int c = 0; c < p.n_out / 32; ++c) {
          uint32_t e[32];
          tmem_ld32(lane_addr + buf * (kCtTiles * kCtMaxN) + m * kCtMaxN + 32 * c, e);
          tmem_ld_wait();
          float vals[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float t = __uint_as_float(e[i]) + bias_s[32 * c + i];
            vals[i] = p.relu ? fmaxf(t, 0.f) : t;
          }
          if (!live) {
            // rows past the map's end: nothing to store
          } else if constexpr (!kLogits) {
            uint32_t hi[16], lo[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) split_pair(vals[2 * i], vals[2 * i + 1], hi[i], lo[i]);
            const size_t plane_elems = (size_t)p.batch * p.h_out * p.w_out * p.n_out;
            __nv_bfloat16* dst = p.out_split + (((size_t)b * p.h_out + y) * p.w_out + x) * p.n_out + 32 * c;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              reinterpret_cast<uint4*>(dst)[q] = make_uint4(hi[4 * q], hi[4 * q + 1], hi[4 * q + 2], hi[4 * q + 3]);
              reinterpret_cast<uint4*>(dst + plane_elems)[q] = make_uint4(lo[4 * q], lo[4 * q + 1], lo[4 * q + 2], lo[4 * q + 3]);
            }
          } else {
            const int h_full = p.h_out * p.up_h, w_full = p.w_out * p.up_w;
            int n = 32 * c, ph = n / p.c_out, co = n - ph * p.c_out;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int py = ph / p.up_w, px = ph - py * p.up_w;
              if (32 * c + i < p.n_real)
                p.out_logits[(((size_t)b * p.c_out + co) * h_full + (size_t)y * p.up_h + py) * w_full + (size_t)x * p.up_w + px] = vals[i];
              if (++co == p.c_out) {
                co = 0;
                ++ph;
              }
            }
          }
          __syncwarp();  // the next load from tensor memory is warp-wide
        }
      }
      ct_warp_arrive(bar(kCt_AccEmpty + buf), lane);
    }
  }
  fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && *abort_flag) atomicOr(p.status, SEA_DEV_TIMEOUT);
}

// ---- operand preparation -----------------------------------------------------------------------
// Weights [c_out][c_in][3][3] fp32 -> tiles [ny nx][cs_in / 64][hi, lo][n_out][64] bf16 of the
// effective taps (cs_in = c_in rounded up to whole blocks of 64 channels): column n = phase
// (py, px) * c_out + co takes, at tap (a, bx), the sum of the original taps (ky, kx) whose logical
// input pixel falls on stored offset (min_y + a, min_x + bx); columns n >= n_real and channels
// >= c_in hold zeros.
__global__ void conv_weights_split_kernel(const float* __restrict__ w, __nv_bfloat16* __restrict__ out, int c_in, int cs_in,
                                          int c_out, int n_real, int n_out, int ny, int nx, int up_h, int up_w, int pad_top) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int half_c = cs_in / 2;
  if (idx >= (long long)ny * nx * n_out * half_c) return;
  const int cpair = (int)(idx % half_c);
  const int n = (int)((idx / half_c) % n_out), tap = (int)(idx / ((long long)half_c * n_out));
  const int a = tap / nx, bx = tap - a * nx;
  const int ph = n / c_out, co = n - ph * c_out, py = ph / up_w, px = ph - py * up_w;
  const int min_y = floor_div(-pad_top, up_h), min_x = floor_div(-1, up_w);
  float sum[2] = {0.f, 0.f};
  if (n < n_real)
    for (int ky = 0; ky < 3; ++ky) {
      if (floor_div(py + ky - pad_top, up_h) - min_y != a) continue;
      for (int kx = 0; kx < 3; ++kx) {
        if (floor_div(px + kx - 1, up_w) - min_x != bx) continue;
        for (int q = 0; q < 2; ++q)
          if (2 * cpair + q < c_in) sum[q] += w[(((size_t)co * c_in + 2 * cpair + q) * 3 + ky) * 3 + kx];
      }
    }
  uint32_t hi, lo;
  split_pair(sum[0], sum[1], hi, lo);
  const int ci = 2 * cpair, cb = ci / 64, within = ci % 64;
  const size_t tile = ((size_t)tap * (cs_in / 64) + cb) * 2;
  uint32_t* o = reinterpret_cast<uint32_t*>(out);
  o[((tile * n_out + n) * 64 + within) / 2] = hi;
  o[(((tile + 1) * n_out + n) * 64 + within) / 2] = lo;
}

// Feature map [batch][C][h][w] fp32 -> [hi, lo][batch][h][w][cs] bf16, cs = C rounded up to whole
// blocks of 64 channels (the added channels are zero).  A block: 64 channels x 32 columns of one row
// through shared memory (reads run along w, writes along the channels).
__global__ void __launch_bounds__(256)
nchw_to_nhwc_split_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, int C, int cs, int h, int w, int batch) {
  __shared__ float t[64][33];
  const int tiles_w = (w + 31) / 32;
  const int x0 = (blockIdx.x % tiles_w) * 32, y = blockIdx.x / tiles_w, c0 = blockIdx.y * 64, b = blockIdx.z;
  const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = grp + 8 * i;
    t[c][lane] = (x0 + lane < w && c0 + c < C) ? in[(((size_t)b * C + c0 + c) * h + y) * w + x0 + lane] : 0.f;
  }
  __syncthreads();
  const size_t plane_words = (size_t)batch * h * w * cs / 2;
  uint32_t* o = reinterpret_cast<uint32_t*>(out);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int xl = grp + 8 * i;
    if (x0 + xl >= w) continue;
    uint32_t hi, lo;
    split_pair(t[2 * lane][xl], t[2 * lane + 1][xl], hi, lo);
    const size_t word = ((((size_t)b * h + y) * w + x0 + xl) * cs + c0 + 2 * lane) / 2;
    o[word] = hi;
    o[plane_words + word] = lo;
  }
}

// [planes][d3][d2][d1][d0] bf16, boxes of b3 x 1 x b1 x 64 elements of one plane, 128-byte swizzle.
bool make_map_bf16_5d(CUtensorMap* map, const void* ptr, unsigned long long d0, unsigned long long d1, unsigned long long d2,
                      unsigned long long d3, unsigned long long d4, unsigned b1, unsigned b3) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[5] = {d0, d1, d2, d3, d4};
  const cuuint64_t strides[4] = {d0 * 2, d0 * d1 * 2, d0 * d1 * d2 * 2, d0 * d1 * d2 * d3 * 2};
  const cuuint32_t box[5] = {64, b1, 1, b3, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Channel strides and accumulator widths: channels come in whole blocks of 64 (a row of an operand
// tile), accumulator columns in whole chunks of 32; what is added holds zeros.
int conv_tc_channels(int c) { return (c + 63) / 64 * 64; }
static int conv_tc_columns(int c_out, int up_h, int up_w, bool logits) {
  return logits ? (up_h * up_w * c_out + 31) / 32 * 32 : conv_tc_channels(c_out);
}

// Shapes this form takes: at most 128 input channels and 128 accumulator columns after rounding
// up, a row of the stored map made of whole boxes of min(w, 128) columns that divide 128, and
// (strided layer) a height that is a multiple of the stride, at least as many rows as a box has.  `logits`: the layer writes fp32 logits
// with the resize's phases scattered; else bf16 planes for the next layer (no resize).
bool conv_tc_shape_ok(int c_in, int c_out, int h_in, int w_in, int up_h, int up_w, int stride_h, bool logits) {
  if (c_in <= 0 || c_out <= 0 || up_h < 1 || up_w < 1 || stride_h < 1 || h_in <= 0 || w_in <= 0) return false;
  if (!logits && (up_h != 1 || up_w != 1)) return false;
  const int bw = w_in < 128 ? w_in : 128;
  if (conv_tc_channels(c_in) > 128 || conv_tc_columns(c_out, up_h, up_w, logits) > kCtMaxN) return false;
  if (128 % bw != 0 || w_in % bw != 0) return false;
  if (stride_h != 1 && (up_h != 1 || up_w != 1 || h_in % stride_h != 0)) return false;
  if (h_in / stride_h < 128 / bw) return false;  // a copy box (128 / bw rows) no taller than the map
  return true;
}

size_t conv_tc_weight_bytes(int c_in) { return (size_t)9 * (conv_tc_channels(c_in) / 64) * 2 * kCtMaxN * 64 * sizeof(__nv_bfloat16); }

sea_status launch_nchw_to_nhwc_split(const float* in, void* out, int batch, int C, int h, int w, cudaStream_t st) {
  const int cs = conv_tc_channels(C);
  const dim3 grid(((w + 31) / 32) * h, cs / 64, batch);
  nchw_to_nhwc_split_kernel<<<grid, 256, 0, st>>>(in, static_cast<__nv_bfloat16*>(out), C, cs, h, w, batch);
  return check_launch();
}

// One layer.  act_in: [hi, lo][batch][h_in][w_in][cs_in] bf16 (cs_in = c_in rounded up to a multiple of
// 64, the added channels zero); the layer's logical input is its nearest resize by (up_h, up_w),
// padded by pad_top rows above (2 - pad_top below) and one column on either side, read at row stride
// stride_h.  Output: out_split ([hi, lo][batch][h_out][w_in][cs_out] bf16, ReLU per `relu`, added
// channels zero) or, when out_logits is given, fp32 [batch][c_out][h_in up_h][w_in up_w].
sea_status launch_conv_tc(const void* act_in, int batch, int c_in, int h_in, int w_in, int up_h, int up_w, int stride_h,
                          int pad_top, const float* w, const float* bias, int c_out, int relu, void* w_tiles, void* out_split,
                          float* out_logits, int32_t* status, cudaStream_t st) {
  const bool logits = out_logits != nullptr;
  if (!conv_tc_shape_ok(c_in, c_out, h_in, w_in, up_h, up_w, stride_h, logits)) return SEA_ERR_UNSUPPORTED;
  const int cs_in = conv_tc_channels(c_in);
  ConvTcParams p{};
  p.n_cblk = cs_in / 64;
  p.n_real = up_h * up_w * c_out;
  p.n_out = conv_tc_columns(c_out, up_h, up_w, logits);
  p.bw = w_in < 128 ? w_in : 128;
  p.bh = 128 / p.bw;
  p.h_out = stride_h > 1 ? h_in / stride_h : h_in;
  p.w_out = w_in;
  p.tiles_x = w_in / p.bw;
  p.tiles_y = (p.h_out + kCtTiles * p.bh - 1) / (kCtTiles * p.bh);
  p.n_items = batch * p.tiles_x * p.tiles_y;
  p.batch = batch;
  const int min_y = floor_div(-pad_top, up_h), max_y = floor_div(up_h - 1 + 2 - pad_top, up_h);
  const int min_x = floor_div(-1, up_w), max_x = floor_div(up_w, up_w);
  p.ny = max_y - min_y + 1;
  p.nx = max_x - min_x + 1;
  for (int a = 0; a < p.ny; ++a) {
    const int v = min_y + a;
    p.tap_y[a] = floor_div(v, stride_h);
    p.tap_s[a] = v - p.tap_y[a] * stride_h;
  }
  for (int bx = 0; bx < p.nx; ++bx) p.tap_x[bx] = min_x + bx;
  p.bias = bias;
  p.c_out = c_out;
  p.relu = relu;
  p.out_split = static_cast<__nv_bfloat16*>(out_split);
  p.out_logits = out_logits;
  p.up_h = up_h;
  p.up_w = up_w;
  p.status = status;

  const long long w_threads = (long long)p.ny * p.nx * p.n_out * (cs_in / 2);
  conv_weights_split_kernel<<<(unsigned)((w_threads + 255) / 256), 256, 0, st>>>(w, static_cast<__nv_bfloat16*>(w_tiles), c_in, cs_in,
                                                                               c_out, p.n_real, p.n_out, p.ny, p.nx, up_h, up_w, pad_top);
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;

  CUtensorMap map_a, map_w;
  if (!make_map_bf16_5d(&map_a, act_in, cs_in, w_in, stride_h, h_in / stride_h, 2ull * batch, p.bw, p.bh)) return SEA_ERR_CUDA;
  if (!make_map_bf16_3d(&map_w, w_tiles, 64, p.n_out, (unsigned long long)p.ny * p.nx * p.n_cblk * 2, 64, p.n_out)) return SEA_ERR_CUDA;
  const size_t smem = 1024 + (size_t)kCtStages * kCtStageBytes + 128 + kCtMaxN * sizeof(float);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SEA_ERR_CUDA;
  const int grid = p.n_items < sms ? p.n_items : sms;
  if (out_logits != nullptr) {
    if (cudaFuncSetAttribute(conv_taps_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SEA_ERR_CUDA;
    conv_taps_tc_kernel<true><<<grid, kCtThreads, smem, st>>>(map_a, map_w, p);
  } else {
    if (cudaFuncSetAttribute(conv_taps_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SEA_ERR_CUDA;
    conv_taps_tc_kernel<false><<<grid, kCtThreads, smem, st>>>(map_a, map_w, p);
  }
  return check_launch();
}

}  // namespace sea

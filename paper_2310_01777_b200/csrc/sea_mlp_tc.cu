// Tensor-core form of the estimator head's two MLPs (Sec. 3.1 "Attention Matrix Estimation"):
//     Z     = relu([C_perf ; V] W_mu + b_mu)            [rows x 192] -> [rows x 64]
//     Z_hat = relu(Z W_1 + b_1) W_2 + b_2               [rows x 64]  -> [rows x c_h (K / c_s)]
// for the hidden width d' = 64, one 128-row tile at a time, all three products on tcgen05 with
// bf16 head / remainder operands (x ~ hi + lo: hi hi + hi lo + lo hi) and fp32 accumulators in
// tensor memory.  Z goes to global memory (the output mixing reads it); the hidden layer never
// leaves the SM; Z_hat is written straight as the CNN's input feature map in the tensor-core
// convolutions' layout, [hi, lo][B][T][K / c_s][H c_h] bf16 (row (b, h, t), entry j (K / c_s) + x
// -> pixel (t, x), channel h c_h + j).
// A tile is 128 rows: hg neighbouring heads (a power of two dividing H, at most 32) at 128 / hg
// positions, heads fastest, so that a warp's stores of Z_hat fall on neighbouring channels of the
// same pixels.
// Roles: warps 0-3 own the tile's rows (thread = row = lane of tensor memory): they stage the
// inputs, and take each product out (bias, ReLU, split) to feed the next; warp 4 copies the weights
// in (once, or per 256-column chunk of W_2 when Z_hat is wider than that) and issues the MMAs.
// Every wait is bounded (abort flag + SEA_DEV_TIMEOUT in the status word).
#include "sea_common.cuh"
#include "sea_tc.cuh"

namespace sea {
using namespace tc;

namespace {

constexpr int kMlHidden = 64;          // d'
constexpr int kMlIn = 3 * kHeadDim;    // C_perf (2 d) and V
constexpr int kMlChunk = 256;          // columns of Z_hat per product
constexpr int kMlThreads = 160;
constexpr int kMlTile = 16384;         // 128 rows x 64 bf16
constexpr int kMlWmuBytes = 3 * 2 * kMlHidden * 128, kMlW1Bytes = 2 * kMlHidden * 128, kMlW2Bytes = 2 * kMlChunk * 128;

enum { kMl_W = 0, kMl_W2, kMl_X, kMl_M1, kMl_Z, kMl_M2, kMl_H, kMl_M3, kMl_Free3, kMl_Drain, kMl_NumBars };

struct MlpTcParams {
  const float *c_first, *c_value;   // [rows][64] each: the two halves of C_perf
  const void* V;                    // [rows][64], io dtype
  const float *b_mu, *b_1, *b_2;
  float* Z;                         // [rows][64]
  __nv_bfloat16* act;               // [2][B][T][wr][cs]
  long long rows;
  int n_tiles, n3, n_chunks, chunk;
  int H, seq_len, c_h, wr, batch;
  int cs;                           // channels per pixel of act: H c_h rounded up to a multiple of 64 (the rest stays zero)
  int hg, tiles_t;                  // heads per tile (a power of two dividing H, at most 32); tiles along the sequence per group of heads
  int32_t* status;
};

__device__ __forceinline__ void ml_warp_arrive(uint32_t bar, int lane) {
  fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}
// 32 consecutive values of row r (columns 32 c .. 32 c + 31 of a 64-column K-major tile with the
// 128-byte swizzle), as 16 packed words.
__device__ __forceinline__ void store_half_row(unsigned char* tile, int r, int c, const uint32_t (&w)[16]) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    *reinterpret_cast<uint4*>(tile + r * 128 + (((4 * c + q) ^ (r & 7)) << 4)) = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
}

template <typename T>
__global__ void __launch_bounds__(kMlThreads, 1)
mlp_tc_kernel(const __grid_constant__ CUtensorMap map_wmu, const __grid_constant__ CUtensorMap map_w1,
              const __grid_constant__ CUtensorMap map_w2, const MlpTcParams p) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* sm = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  unsigned char* sX = sm;                       // [3 blocks of 64 inputs][hi, lo] tiles; later Z (block 0) and the hidden layer (block 1)
  unsigned char* sWmu = sX + 6 * kMlTile;       // [3][hi, lo][64 outputs][64 inputs]
  unsigned char* sW1 = sWmu + kMlWmuBytes;      // [hi, lo][64][64]
  unsigned char* sW2 = sW1 + kMlW1Bytes;        // [hi, lo][chunk outputs][64]
  unsigned char* tail = sW2 + kMlW2Bytes;
  const uint32_t bars = smem_u32(tail);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kMl_NumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8 * kMl_NumBars + 4);
  float* bias_s = reinterpret_cast<float*>(tail + 128);  // b_mu [64], b_1 [64]
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  constexpr uint32_t kCol1 = 0, kCol2 = 128, kCol3 = 256;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int i = 0; i < kMl_NumBars; ++i) mbar_init(bar(i), (i == kMl_X || i == kMl_Z || i == kMl_H || i == kMl_Free3) ? 4 : 1);
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (tid < 2 * kMlHidden) bias_s[tid] = tid < kMlHidden ? p.b_mu[tid] : p.b_1[tid - kMlHidden];
  if (warp == 4) tmem_alloc(smem_u32(tmem_slot), 512);
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t w2_bytes = 2u * (uint32_t)p.chunk * 128u;

  if (warp == 4) {
    // ---------------------------------------------------------------- weights in, products out
    const bool leader = elect_one();
    bool ok = true;
    auto load_w2 = [&](int c) {
      if (!leader) return;
      mbar_expect_tx(bar(kMl_W2), w2_bytes);
      for (int plane = 0; plane < 2; ++plane)
        tma_load_3d(smem_u32(sW2) + plane * (uint32_t)p.chunk * 128u, &map_w2, 0, c * p.chunk, plane, bar(kMl_W2));
    };
    if (blockIdx.x < p.n_tiles) {
      if (leader) {
        mbar_expect_tx(bar(kMl_W), kMlWmuBytes + kMlW1Bytes);
        for (int t = 0; t < 6; ++t) tma_load_3d(smem_u32(sWmu) + t * 8192, &map_wmu, 0, 0, t, bar(kMl_W));
        for (int t = 0; t < 2; ++t) tma_load_3d(smem_u32(sW1) + t * 8192, &map_w1, 0, 0, t, bar(kMl_W));
      }
      if (p.n_chunks == 1) load_w2(0);
      __syncwarp();
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_W), 0, abort_flag));
    }
    constexpr uint32_t id64 = idesc_bf16(kMlHidden, false, false);
    const uint32_t id3 = idesc_bf16(p.chunk, false, false);
    uint32_t it = 0, c_it = 0;
    bool w2_pending = p.n_chunks == 1 && blockIdx.x < p.n_tiles;  // a copy of W_2 is in flight
    for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
      const uint32_t par = it & 1;
      // Z = [C_perf ; V] W_mu
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_X), par, abort_flag));
      if (!ok) break;
      fence_after();
      if (leader) {
#pragma unroll
        for (int kb = 0; kb < 3; ++kb) {
          const uint64_t ah = smem_desc(smem_u32(sX) + (2 * kb) * kMlTile, 16, 1024), al = smem_desc(smem_u32(sX) + (2 * kb + 1) * kMlTile, 16, 1024);
          const uint64_t wh = smem_desc(smem_u32(sWmu) + (2 * kb) * 8192, 16, 1024), wl = smem_desc(smem_u32(sWmu) + (2 * kb + 1) * 8192, 16, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            mma_ss(tmem + kCol1, ah + 2 * k, wh + 2 * k, id64, (kb > 0 || k > 0) ? 1u : 0u);
            mma_ss(tmem + kCol1, ah + 2 * k, wl + 2 * k, id64, 1);
            mma_ss(tmem + kCol1, al + 2 * k, wh + 2 * k, id64, 1);
          }
        }
        mma_commit(bar(kMl_M1));
      }
      __syncwarp();
      // hidden = Z W_1 (Z sits where the first block of inputs was)
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_Z), par, abort_flag));
      if (!ok) break;
      fence_after();
      if (leader) {
        const uint64_t ah = smem_desc(smem_u32(sX), 16, 1024), al = smem_desc(smem_u32(sX) + kMlTile, 16, 1024);
        const uint64_t wh = smem_desc(smem_u32(sW1), 16, 1024), wl = smem_desc(smem_u32(sW1) + 8192, 16, 1024);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          mma_ss(tmem + kCol2, ah + 2 * k, wh + 2 * k, id64, k > 0 ? 1u : 0u);
          mma_ss(tmem + kCol2, ah + 2 * k, wl + 2 * k, id64, 1);
          mma_ss(tmem + kCol2, al + 2 * k, wh + 2 * k, id64, 1);
        }
        mma_commit(bar(kMl_M2));
      }
      __syncwarp();
      // Z_hat = hidden W_2, a chunk of columns at a time (the hidden layer sits in the second block)
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_H), par, abort_flag));
      if (!ok) break;
      fence_after();
      for (int c = 0; c < p.n_chunks && ok; ++c, ++c_it) {
        if (p.n_chunks > 1) {
          // the chunk's columns of W_2 go where the previous chunk's were: its products are complete
          if (c_it > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_M3), (c_it - 1) & 1, abort_flag));
          if (!ok) break;
          load_w2(c);
          w2_pending = true;
          __syncwarp();
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_W2), c_it & 1, abort_flag));
          if (ok) w2_pending = false;
        } else if (c_it == 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_W2), 0, abort_flag));
          if (ok) w2_pending = false;
        }
        // the rows have taken the previous chunk out of tensor memory
        if (ok && c_it > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_Free3), (c_it - 1) & 1, abort_flag));
        if (!ok) break;
        fence_after();
        if (leader) {
          const uint64_t ah = smem_desc(smem_u32(sX) + 2 * kMlTile, 16, 1024), al = smem_desc(smem_u32(sX) + 3 * kMlTile, 16, 1024);
          const uint64_t wh = smem_desc(smem_u32(sW2), 16, 1024), wl = smem_desc(smem_u32(sW2) + (uint32_t)p.chunk * 128u, 16, 1024);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            mma_ss(tmem + kCol3, ah + 2 * k, wh + 2 * k, id3, k > 0 ? 1u : 0u);
            mma_ss(tmem + kCol3, ah + 2 * k, wl + 2 * k, id3, 1);
            mma_ss(tmem + kCol3, al + 2 * k, wh + 2 * k, id3, 1);
          }
          mma_commit(bar(kMl_M3));
        }
        __syncwarp();
      }
    }
    // every product issued has completed before tensor memory is given back; copies still in
    // flight must land before the CTA may leave
    if (leader) mma_commit(bar(kMl_Drain));
    __syncwarp();
    mbar_wait(bar(kMl_Drain), 0, abort_flag);
    if (!ok && blockIdx.x < p.n_tiles) {
      mbar_wait_drain(bar(kMl_W), 0);
      if (w2_pending) mbar_wait_drain(bar(kMl_W2), c_it & 1);
    }
  } else {
    // ---------------------------------------------------------------- rows
    const int r = warp * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    const T* V = static_cast<const T*>(p.V);
    const int C = p.cs;  // channel stride of the feature map (H c_h rounded up to a multiple of 64)
    const size_t plane_elems = (size_t)p.batch * p.seq_len * p.wr * C;
    const bool fast = p.n_chunks == 1 && p.c_h == 4 && p.wr % 16 == 0;
    bool ok = true;
    uint32_t it = 0, c_it = 0;
    for (int tile = blockIdx.x; tile < p.n_tiles && ok; tile += gridDim.x, ++it) {
      const uint32_t par = it & 1;
      // Row r of the tile is head h0 + r % hg at position t0 + r / hg: the threads of a warp hold
      // neighbouring heads of the same positions, whose channels are neighbours in the feature map
      const int tt = tile % p.tiles_t, grp = tile / p.tiles_t, groups = p.H / p.hg;
      const int b = grp / groups, h = (grp - b * groups) * p.hg + r % p.hg, t = tt * (128 / p.hg) + r / p.hg;
      const bool live = t < p.seq_len;
      const long long row = ((long long)b * p.H + h) * p.seq_len + (live ? t : 0);
      // inputs: C_perf's two halves (fp32) and V, as head / remainder rows of the three blocks
#pragma unroll 1
      for (int kb = 0; kb < 3; ++kb) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float v[32];
          if (!live) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = 0.f;
          } else if (kb < 2) {
            const float4* src = reinterpret_cast<const float4*>((kb == 0 ? p.c_first : p.c_value) + row * kHeadDim + 32 * c);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 t = __ldg(src + q);
              v[4 * q] = t.x, v[4 * q + 1] = t.y, v[4 * q + 2] = t.z, v[4 * q + 3] = t.w;
            }
          } else if constexpr (sizeof(T) == 2) {
            const uint4* src = reinterpret_cast<const uint4*>(V + row * kHeadDim + 32 * c);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 t = __ldg(src + q);
              const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                v[8 * q + 2 * u] = __uint_as_float(w[u] << 16);
                v[8 * q + 2 * u + 1] = __uint_as_float(w[u] & 0xffff0000u);
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = Io<T>::from_io(V[row * kHeadDim + 32 * c + i]);
          }
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) split_pair(v[2 * i], v[2 * i + 1], hi[i], lo[i]);
          store_half_row(sX + (2 * kb) * kMlTile, r, c, hi);
          store_half_row(sX + (2 * kb + 1) * kMlTile, r, c, lo);
        }
      }
      fence_async_smem();
      ml_warp_arrive(bar(kMl_X), lane);
      // Z = relu(. + b_mu): to global memory, and as the next product's operand
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_M1), par, abort_flag));
      if (!ok) break;
      fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t e[32];
        tmem_ld32(lane_addr + kCol1 + 32 * c, e);
        tmem_ld_wait();
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = fmaxf(__uint_as_float(e[i]) + bias_s[32 * c + i], 0.f);
        if (live) {
          float4* dst = reinterpret_cast<float4*>(p.Z + row * kMlHidden + 32 * c);
#pragma unroll
          for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        }
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) split_pair(v[2 * i], v[2 * i + 1], hi[i], lo[i]);
        store_half_row(sX, r, c, hi);
        store_half_row(sX + kMlTile, r, c, lo);
      }
      fence_async_smem();
      ml_warp_arrive(bar(kMl_Z), lane);
      // hidden = relu(. + b_1)
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_M2), par, abort_flag));
      if (!ok) break;
      fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t e[32];
        tmem_ld32(lane_addr + kCol2 + 32 * c, e);
        tmem_ld_wait();
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int i = 0; i < 16; ++i)
          split_pair(fmaxf(__uint_as_float(e[2 * i]) + bias_s[kMlHidden + 32 * c + 2 * i], 0.f),
                     fmaxf(__uint_as_float(e[2 * i + 1]) + bias_s[kMlHidden + 32 * c + 2 * i + 1], 0.f), hi[i], lo[i]);
        store_half_row(sX + 2 * kMlTile, r, c, hi);
        store_half_row(sX + 3 * kMlTile, r, c, lo);
      }
      fence_async_smem();
      ml_warp_arrive(bar(kMl_H), lane);
      // Z_hat + b_2 -> the feature map
      __nv_bfloat16* pix = p.act + ((size_t)b * p.seq_len + (live ? t : 0)) * p.wr * C + (size_t)h * p.c_h;  // pixel (t, 0), channel h c_h
      for (int c = 0; c < p.n_chunks && ok; ++c, ++c_it) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kMl_M3), c_it & 1, abort_flag));
        if (!ok) break;
        fence_after();
        if (fast) {
          for (int x0 = 0; x0 < p.wr; x0 += 16) {
            uint32_t e[4][16];
#pragma unroll
            for (int j = 0; j < 4; ++j) tmem_ld16(lane_addr + kCol3 + j * p.wr + x0, e[j]);
            tmem_ld_wait();
            if (live) {
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                float v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = __uint_as_float(e[j][i]) + __ldg(p.b_2 + j * p.wr + x0 + i);
                uint2 hi, lo;
                split_pair(v[0], v[1], hi.x, lo.x);
                split_pair(v[2], v[3], hi.y, lo.y);
                __nv_bfloat16* dst = pix + (size_t)(x0 + i) * C;
                *reinterpret_cast<uint2*>(dst) = hi;
                *reinterpret_cast<uint2*>(dst + plane_elems) = lo;
              }
            }
            __syncwarp();
          }
        } else {
          for (int q = 0; q < p.chunk / 16; ++q) {
            uint32_t e[16];
            tmem_ld16(lane_addr + kCol3 + 16 * q, e);
            tmem_ld_wait();
            if (live) {
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const int n = c * p.chunk + 16 * q + i, j = n / p.wr, x = n - j * p.wr;
                uint32_t hi, lo;
                split_pair(__uint_as_float(e[i]) + __ldg(p.b_2 + n), 0.f, hi, lo);
                unsigned short* dst = reinterpret_cast<unsigned short*>(pix + (size_t)x * C + j);
                dst[0] = (unsigned short)(hi & 0xffffu);
                dst[plane_elems] = (unsigned short)(lo & 0xffffu);
              }
            }
            __syncwarp();
          }
        }
        ml_warp_arrive(bar(kMl_Free3), lane);
      }
    }
  }
  fence_before();
  __syncthreads();
  if (warp == 4) {
    __syncwarp();
    fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && *abort_flag) atomicOr(p.status, SEA_DEV_TIMEOUT);
}

// W [k_in][n_out] fp32 -> tiles [k_in / 64][hi, lo][n_out][64] bf16 (the transpose, in blocks of 64 inputs)
__global__ void linear_weights_split_kernel(const float* __restrict__ W, __nv_bfloat16* __restrict__ out, int k_in, int n_out) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_out * (k_in / 2)) return;
  const int n = idx % n_out, k = 2 * (idx / n_out);
  uint32_t hi, lo;
  split_pair(W[(size_t)k * n_out + n], W[(size_t)(k + 1) * n_out + n], hi, lo);
  const size_t tile = (size_t)(k / 64) * 2;
  uint32_t* o = reinterpret_cast<uint32_t*>(out);
  o[((tile * n_out + n) * 64 + k % 64) / 2] = hi;
  o[(((tile + 1) * n_out + n) * 64 + k % 64) / 2] = lo;
}

}  // namespace

// The fused form takes d' = 64 and a Z_hat width that is one product of at most 256 columns (a
// multiple of 16) or whole chunks of 256.
bool mlp_tc_shape_ok(int d_hidden, int n3) {
  if (d_hidden != kMlHidden || n3 <= 0) return false;
  return n3 <= kMlChunk ? n3 % 16 == 0 : n3 % kMlChunk == 0;
}
size_t mlp_tc_weight_bytes(int n3) { return (size_t)(kMlIn * kMlHidden + kMlHidden * kMlHidden + kMlHidden * n3) * 2 * sizeof(__nv_bfloat16); }

template <typename T>
static sea_status launch_mlp_tc_typed(const sea_shape& s, const sea_decoder& dec, const float* c_first, const float* c_value, const T* V,
                                      float* Z, void* act, void* w_tiles, int32_t* status, cudaStream_t st) {
  const int wr = s.Kc / dec.c_s, n3 = wr * dec.c_h;
  if (!mlp_tc_shape_ok(dec.d_hidden, n3)) return SEA_ERR_UNSUPPORTED;
  __nv_bfloat16* wmu = static_cast<__nv_bfloat16*>(w_tiles);
  __nv_bfloat16* w1 = wmu + (size_t)kMlIn * kMlHidden * 2;
  __nv_bfloat16* w2 = w1 + (size_t)kMlHidden * kMlHidden * 2;
  linear_weights_split_kernel<<<(kMlHidden * kMlIn / 2 + 255) / 256, 256, 0, st>>>(dec.W_mu, wmu, kMlIn, kMlHidden);
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;
  linear_weights_split_kernel<<<(kMlHidden * kMlHidden / 2 + 255) / 256, 256, 0, st>>>(dec.W_nu1, w1, kMlHidden, kMlHidden);
  if ((rc = check_launch()) != SEA_OK) return rc;
  linear_weights_split_kernel<<<(n3 * kMlHidden / 2 + 255) / 256, 256, 0, st>>>(dec.W_nu2, w2, kMlHidden, n3);
  if ((rc = check_launch()) != SEA_OK) return rc;
  MlpTcParams p{};
  p.c_first = c_first;
  p.c_value = c_value;
  p.V = V;
  p.b_mu = dec.b_mu;
  p.b_1 = dec.b_nu1;
  p.b_2 = dec.b_nu2;
  p.Z = Z;
  p.act = static_cast<__nv_bfloat16*>(act);
  p.rows = (long long)s.B * s.H * s.T;
  p.hg = 1;
  while (p.hg < 32 && s.H % (2 * p.hg) == 0) p.hg *= 2;
  p.tiles_t = (s.T + 128 / p.hg - 1) / (128 / p.hg);
  p.n_tiles = s.B * (s.H / p.hg) * p.tiles_t;
  p.n3 = n3;
  p.chunk = n3 <= kMlChunk ? n3 : kMlChunk;
  p.n_chunks = n3 / p.chunk;
  p.H = s.H;
  p.seq_len = s.T;
  p.c_h = dec.c_h;
  p.wr = wr;
  p.batch = s.B;
  p.status = status;
  p.cs = conv_tc_channels(s.H * dec.c_h);
  if (p.cs != s.H * dec.c_h &&  // the channels beyond H c_h are written by nobody: zero
      cudaMemsetAsync(act, 0, (size_t)2 * s.B * s.T * wr * p.cs * sizeof(__nv_bfloat16), st) != cudaSuccess)
    return SEA_ERR_CUDA;
  CUtensorMap map_wmu, map_w1, map_w2;
  if (!make_map_bf16_3d(&map_wmu, wmu, 64, kMlHidden, 6, 64, kMlHidden) || !make_map_bf16_3d(&map_w1, w1, 64, kMlHidden, 2, 64, kMlHidden) ||
      !make_map_bf16_3d(&map_w2, w2, 64, n3, 2, 64, p.chunk))
    return SEA_ERR_CUDA;
  const size_t smem = 1024 + 6 * kMlTile + kMlWmuBytes + kMlW1Bytes + kMlW2Bytes + 128 + 2 * kMlHidden * sizeof(float);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SEA_ERR_CUDA;
  if (cudaFuncSetAttribute(mlp_tc_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return SEA_ERR_CUDA;
  mlp_tc_kernel<T><<<p.n_tiles < sms ? p.n_tiles : sms, kMlThreads, smem, st>>>(map_wmu, map_w1, map_w2, p);
  return check_launch();
}

sea_status launch_mlp_tc(const sea_shape& s, const sea_decoder& dec, const float* c_first, const float* c_value, const void* V, float* Z,
                         void* act, void* w_tiles, int32_t* status, cudaStream_t st) {
  if (s.io == SEA_BF16)
    return launch_mlp_tc_typed<__nv_bfloat16>(s, dec, c_first, c_value, static_cast<const __nv_bfloat16*>(V), Z, act, w_tiles, status, st);
  return launch_mlp_tc_typed<float>(s, dec, c_first, c_value, static_cast<const float*>(V), Z, act, w_tiles, status, st);
}

}  // namespace sea

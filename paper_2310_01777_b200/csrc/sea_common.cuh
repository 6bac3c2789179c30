// Shared device/host helpers of libsea (internal; the public interface is include/sea.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sea.h"

namespace sea {

constexpr int kHeadDim = 64;        // d, fixed by the interface
constexpr int kStatusBytes = 256;   // head of every workspace: the device status word
constexpr int kEstChunk = 64;       // rows per estimator chunk (prefix-state granularity)

struct Launch {  // per-thread launch bookkeeping behind sea_last_launch_count() / sea_last_sparse_kernel()
  static int& count() {
    static thread_local int c = 0;
    return c;
  }
  static const char*& sparse_kernel() {
    static thread_local const char* k = "none";
    return k;
  }
  static double& sparse_flops() {
    static thread_local double f = 0.0;
    return f;
  }
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace carve-up shared by the entry points (all offsets 256-byte aligned).
struct WsLayout {
  size_t status;      // int32 status word
  size_t est_state;   // float [BH][nchunk][m*(d+1)]  chunk states of the estimator
  size_t est_split;   // bf16 head/remainder copies of omega and W_dec (bf16 estimator)
  size_t row_counts;  // int32 [rows]                 per-row nnz before the scan
  size_t tile_sums;   // int32 [ceil(rows/2048)]      scan partials
  size_t a_hat;       // float [rows][Kc]             estimate when the caller keeps none
  size_t sel;         // int32 [rows][k_hat]
  size_t row_ptr;     // int32 [rows+1]
  size_t mask_bits;   // uint32 [rows][ceil(Kc/32)]   selected columns as bits (tensor-core sparse stage)
  size_t p_scratch;   // float [rows][k_hat*r]        unnormalised probabilities (tensor-core sparse stage)
  size_t park_off;    // int32 [rows]                 offsets into p_scratch (masks with rows of differing lengths)
  size_t tile_live;   // uint32 [BH*T/128][..]        a bit per (work item, key tile) that holds a kept key (tensor-core sparse stage)
  size_t total;
};

WsLayout ws_layout(const sea_shape& s);
// k_star > 0: a selected column keeps at most k_star keys (capped replication), which bounds the mask.
// ragged: T need not be a multiple of Kc (the resized expansion); a column then covers up to ceil(T / Kc) keys.
sea_status validate_shape(const sea_shape* s, bool need_estimator, int k_star = 0, bool ragged = false);
long long mask_entries_bound(const sea_shape& s, int k_star);

// Where the per-query selection goes when the estimator's output kernel performs it (see
// estimate_tc_selects): the same three arrays launch_topk_mask's selection kernel writes.
struct SelectOut {
  int32_t* sel;         // [rows][k_hat]
  int32_t* row_counts;  // [rows], causal shapes only (null otherwise)
  uint32_t* mask_bits;  // [rows][ceil(Kc/32)] or null
};

// Stage launchers (defined one per .cu file).  All are asynchronous on `st`.  select_out may be
// null; *selected tells whether the selection was performed.
sea_status launch_estimate(const sea_shape& s, const void* Q, const void* K, const void* V,
                           const float* omega, const float* W_dec, float* A_hat,
                           float* est_state, void* est_split, const SelectOut* select_out, bool* selected,
                           int32_t* status, cudaStream_t st);
sea_status launch_estimate_f32(const sea_shape& s, const void* Q, const void* K, const void* V,
                               const float* omega, const float* W_dec, float* A_hat,
                               float* est_state, int32_t* status, cudaStream_t st);
// bf16 estimator on tcgen05 (sea_estimate_tc.cu)
bool estimate_tc_applicable(const sea_shape& s);
bool estimate_tc_selects(const sea_shape& s);
size_t estimate_tc_state_bytes(const sea_shape& s);
size_t estimate_tc_split_bytes(const sea_shape& s);
sea_status launch_estimate_tc(const sea_shape& s, const void* Q, const void* K, const void* V,
                              const float* omega, const float* W_dec, float* A_hat, float* est_state,
                              void* est_split, const SelectOut* select_out, int32_t* status, cudaStream_t st);
// selected: sel, row_counts and mask_bits already hold the selection (the estimator wrote them);
// only the row pointers and the column indices are produced then.
sea_status launch_topk_mask(const sea_shape& s, const float* A_hat, int32_t* sel,
                            int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                            int32_t* row_counts, int32_t* tile_sums, uint32_t* mask_bits, bool selected,
                            int32_t* status, cudaStream_t st);
sea_status launch_row_ptr_scan(const int32_t* row_counts, int32_t* tile_sums, int32_t* row_ptr, int rows,
                               cudaStream_t st);
// Causal-per-batch grouping (sea_topk_grouped.cu).  mask_bits is written in full; park_off, when
// not null, receives the rows' offsets into the parking area of the tile kernel (see below).
bool topk_grouped_supported(const sea_shape& s);
sea_status launch_topk_mask_grouped(const sea_shape& s, const float* A_hat, uint32_t* mask_bits,
                                    int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                    int32_t* row_counts, int32_t* tile_sums, int32_t* park_off,
                                    int32_t* status, cudaStream_t st);
// Column indices of a mask given as bits and row pointers (rows of any length).
sea_status launch_fill_col_idx_bits(const sea_shape& s, const uint32_t* mask_bits, const int32_t* row_ptr,
                                    int32_t* col_idx, int64_t nnz_cap, int32_t* status, cudaStream_t st);
// Causal-aware per-query selection (sea_topk.cu): a causal row only chooses among the columns
// that hold a key it may see.  mask_bits is written in full.
sea_status launch_topk_mask_aware(const sea_shape& s, const float* A_hat, uint32_t* mask_bits,
                                  int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                  int32_t* row_counts, int32_t* tile_sums, int32_t* status,
                                  cudaStream_t st);
// Per-query selection whose selected columns are replicated to at most k_star uniformly spaced keys
// (sea_topk.cu); col_idx is required, the sparse stage then walks the CSR.
sea_status launch_topk_mask_capped(const sea_shape& s, int k_star, const float* A_hat, int32_t* sel,
                                   int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts,
                                   int32_t* tile_sums, int32_t* status, cudaStream_t st);
// Nearest-neighbour resize of the compressed mask at any ratio of T to Kc; row_widths: a causal row
// is resized to its own width i + 1 (sea_topk.cu).  col_idx may be null.
sea_status launch_topk_mask_resized(const sea_shape& s, int row_widths, const float* A_hat, int32_t* sel, int32_t* row_ptr,
                                    int32_t* col_idx, int64_t nnz_cap, int32_t* row_counts, int32_t* tile_sums,
                                    int32_t* status, cudaStream_t st);
// Where each row parks its unnormalised probabilities when rows keep differing numbers of columns:
// the (b, t) slabs of H*k_hat*r floats follow one another, the heads inside a slab.  Rows of a slab
// that keeps more than H*k_hat columns get -1 and SEA_DEV_ROW_OVERFLOW is raised.
sea_status launch_park_offsets(const sea_shape& s, const uint32_t* mask_bits, int32_t* park_off,
                               int32_t* status, cudaStream_t st);
// Sparse stage for a mask given as bits with its row_ptr (rows of any length).  park_valid:
// park_off already holds the offsets that belong to mask_bits.  rows_within_k_hat: no row keeps
// more than k_hat columns, so the per-query parking layout serves and no offsets are needed.
sea_status launch_sparse_attn_masked(const sea_shape& s, const void* Q, const void* K, const void* V,
                                     const int32_t* row_ptr, const int32_t* col_idx,
                                     const uint32_t* mask_bits, void* O, void* P, int32_t* park_off,
                                     bool park_valid, bool rows_within_k_hat, float* p_scratch, uint32_t* tile_live,
                                     int32_t* status, cudaStream_t st);
// mask_bits and p_scratch (workspace areas of the tensor-core kernel) may be null: the per-row
// kernels are used then.  bits_valid: mask_bits already holds the bit strings of `sel`
// (launch_topk_mask wrote them); otherwise they are derived from `sel` first.
sea_status launch_sparse_attn(const sea_shape& s, const void* Q, const void* K, const void* V,
                              const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel,
                              void* O, void* P, uint32_t* mask_bits, bool bits_valid, float* p_scratch,
                              uint32_t* tile_live, int32_t* status, cudaStream_t st);
sea_status launch_sparse_attn_rows(const sea_shape& s, const void* Q, const void* K, const void* V,
                                   const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel,
                                   void* O, void* P, cudaStream_t st);
// the shape alone allows the tensor-core tile kernel (dtype, T, r, density)
bool sparse_attn_tc_shape_ok(const sea_shape& s);
size_t sparse_attn_tc_bits_bytes(const sea_shape& s);
size_t sparse_attn_tc_scratch_bytes(const sea_shape& s);
size_t sparse_attn_tc_live_bytes(const sea_shape& s);
// have_bits: mask_bits already holds the mask (sel may then be null)
bool sparse_attn_tc_applicable(const sea_shape& s, const int32_t* sel, bool have_bits, const int32_t* status,
                               const void* mask_bits, const void* p_scratch);
// park_off: per-row offsets into p_scratch (null: row * k_hat * r, the per-query layout)
sea_status launch_sparse_attn_tc(const sea_shape& s, const void* Q, const void* K, const void* V,
                                 const int32_t* row_ptr, const int32_t* sel, void* O, void* P,
                                 uint32_t* mask_bits, bool bits_valid, float* p_scratch,
                                 const int32_t* park_off, uint32_t* tile_live, int32_t* status, cudaStream_t st);
bool sparse_attn_tma_applicable(const sea_shape& s, const int32_t* sel, const int32_t* status);
sea_status launch_sparse_attn_tma(const sea_shape& s, const void* Q, const void* K, const void* V,
                                  const int32_t* row_ptr, const int32_t* sel, void* O, void* P,
                                  int32_t* status, cudaStream_t st);

// The paper's estimator head and output mixing (sea_decoder.cu).  dws: the decoder's own part of
// the workspace (decoder_layout), est_state / est_split: the estimator's scratch of the base layout.
struct DecoderLayout {
  size_t ident, first, c_first, c_value, z, hidden, image, conv_a, conv_b, s_prob, s_mix, c_avg;
  size_t act0, w_tiles;  // tensor-core form of the convolutions only: the image as bf16 planes, the layers' weight tiles
  size_t mlp_w;          // tensor-core form of the MLPs only: their weight tiles
  size_t total;
};
// Tensor-core form of the estimator head's MLPs (sea_mlp_tc.cu): Z and the CNN's input feature map.
bool mlp_tc_shape_ok(int d_hidden, int n3);
size_t mlp_tc_weight_bytes(int n3);
sea_status launch_mlp_tc(const sea_shape& s, const sea_decoder& dec, const float* c_first, const float* c_value, const void* V, float* Z,
                         void* act, void* w_tiles, int32_t* status, cudaStream_t st);
// Tensor-core form of a 3 x 3 convolution layer (sea_conv_tc.cu).
int conv_tc_channels(int c);  // channel stride of the bf16 planes: c rounded up to a multiple of 64
bool conv_tc_shape_ok(int c_in, int c_out, int h_in, int w_in, int up_h, int up_w, int stride_h, bool logits);
size_t conv_tc_weight_bytes(int c_in);
sea_status launch_nchw_to_nhwc_split(const float* in, void* out, int batch, int C, int h, int w, cudaStream_t st);
sea_status launch_conv_tc(const void* act_in, int batch, int c_in, int h_in, int w_in, int up_h, int up_w, int stride_h,
                          int pad_top, const float* w, const float* bias, int c_out, int relu, void* w_tiles, void* out_split,
                          float* out_logits, int32_t* status, cudaStream_t st);
DecoderLayout decoder_layout(const sea_shape& s, const sea_decoder& dec);
sea_status launch_estimate_decoder(const sea_shape& s, const sea_decoder& dec, const void* Q, const void* K, const void* V,
                                   const float* omega, float* A_hat, float* Z, char* dws, float* est_state, void* est_split,
                                   int32_t* status, cudaStream_t st);
sea_status launch_mix_output(const sea_shape& s, const sea_decoder& dec, const float* Z, const float* A_hat, const void* V,
                             const int32_t* row_ptr, void* O, void* P, char* dws, cudaStream_t st);

inline sea_status check_launch() {
  Launch::count()++;
  return cudaGetLastError() == cudaSuccess ? SEA_OK : SEA_ERR_CUDA;
}

#ifdef __CUDACC__
// ---- 16-byte vector access to a row of d elements in the io dtype ------------------
template <typename T>
struct Io;

template <>
struct Io<float> {
  static constexpr int kElemsPerLane = 4;   // one 16-byte load
  static constexpr int kLanesPerRow = 16;   // 64 floats = 256 B
  __device__ static void load(const float* p, float (&v)[4]) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
  __device__ static void store(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
  __device__ static float to_io(float x) { return x; }
  __device__ static float from_io(float x) { return x; }
};

template <>
struct Io<__nv_bfloat16> {
  static constexpr int kElemsPerLane = 8;
  static constexpr int kLanesPerRow = 8;    // 64 bf16 = 128 B
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 t;
    uint32_t* w = reinterpret_cast<uint32_t*>(&t);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = t;
  }
  __device__ static __nv_bfloat16 to_io(float x) { return __float2bfloat16_rn(x); }
  __device__ static float from_io(__nv_bfloat16 x) { return __bfloat162float(x); }
};

// 32-bit key whose unsigned order is the float order, with -0 folded onto +0.
__device__ __forceinline__ uint32_t order_key(float v) {
  const uint32_t u = __float_as_uint(v + 0.f);  // -0 + 0 = +0: the two zeros tie; every other value is unchanged
  return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);  // negative: all bits flip; else: the sign bit
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
#endif  // __CUDACC__

}  // namespace sea

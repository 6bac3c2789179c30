// C ABI of libsea: argument checks, workspace carve-up and the chaining of the stages.
#include "sea_common.cuh"

namespace sea {

namespace {
constexpr int kScanTileRows = 2048;
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
size_t io_bytes(const sea_shape& s) { return s.io == SEA_BF16 ? 2 : 4; }
}  // namespace

// Largest number of CSR entries the mask of this shape can hold: every row keeps k_hat columns of
// min(r, k_star) keys (k_star <= 0: whole runs).
long long mask_entries_bound(const sea_shape& s, int k_star) {
  const long long r = (s.T + s.Kc - 1) / s.Kc;
  const long long per_col = k_star > 0 && k_star < r ? k_star : r;
  return (long long)s.B * s.H * s.T * s.k_hat * per_col;
}

sea_status validate_shape(const sea_shape* s, bool need_estimator, int k_star, bool ragged) {
  if (s == nullptr) return SEA_ERR_INVALID_ARG;
  if (s->B <= 0 || s->H <= 0 || s->T <= 0 || s->Kc <= 0 || s->k_hat <= 0) return SEA_ERR_INVALID_ARG;
  if (s->causal != 0 && s->causal != 1) return SEA_ERR_INVALID_ARG;
  if (s->io != SEA_F32 && s->io != SEA_BF16) return SEA_ERR_INVALID_ARG;
  if (!(s->scale >= 0.f) || s->scale > 3.0e38f) return SEA_ERR_INVALID_ARG;
  if (s->m < 0) return SEA_ERR_INVALID_ARG;
  if (s->k_hat > s->Kc) return SEA_ERR_INVALID_ARG;
  if (s->d != kHeadDim) return SEA_ERR_UNSUPPORTED;
  if (!ragged && s->T % s->Kc != 0) return SEA_ERR_UNSUPPORTED;
  if (s->Kc > 2048) return SEA_ERR_UNSUPPORTED;
  if (need_estimator && (s->m < 16 || s->m > 128 || s->m % 16 != 0)) return SEA_ERR_UNSUPPORTED;
  const long long rows = (long long)s->B * s->H * s->T;
  const long long lim = 2147483647ll;
  if (rows + 1 > lim || mask_entries_bound(*s, k_star) > lim) return SEA_ERR_TOO_LARGE;
  return SEA_OK;
}

WsLayout ws_layout(const sea_shape& s) {
  WsLayout L{};
  const size_t rows = (size_t)s.B * s.H * s.T;
  const size_t BH = (size_t)s.B * s.H;
  const size_t nchunk = ((size_t)s.T + kEstChunk - 1) / kEstChunk;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes, 256);
    return at;
  };
  L.status = take(kStatusBytes);
  auto larger = [](size_t a, size_t b) { return a > b ? a : b; };
  L.est_state = take(s.m > 0 ? larger(BH * nchunk * (size_t)s.m * (kHeadDim + 1) * sizeof(float), estimate_tc_state_bytes(s)) : 0);
  L.est_split = take(s.m > 0 ? estimate_tc_split_bytes(s) : 0);
  L.row_counts = take(rows * sizeof(int32_t));
  L.tile_sums = take(((rows + kScanTileRows - 1) / kScanTileRows + 1) * sizeof(int32_t));
  L.a_hat = take(rows * (size_t)s.Kc * sizeof(float));
  L.sel = take(rows * (size_t)s.k_hat * sizeof(int32_t));
  L.row_ptr = take((rows + 1) * sizeof(int32_t));
  L.mask_bits = take(sparse_attn_tc_bits_bytes(s));
  L.p_scratch = take(sparse_attn_tc_shape_ok(s) ? sparse_attn_tc_scratch_bytes(s) : 0);  // only the tile kernel parks
  L.park_off = take(s.io == SEA_BF16 ? rows * sizeof(int32_t) : 0);
  L.tile_live = take(sparse_attn_tc_shape_ok(s) ? sparse_attn_tc_live_bytes(s) : 0);
  L.total = off;
  return L;
}

}  // namespace sea

using namespace sea;

namespace {
// The two copy streams and the events of sea_attention_host's pipeline.  Creating them costs more
// than a slice of the pipeline takes, so a host thread creates them once per device it calls from
// and keeps them until it exits.
constexpr int kMaxSlices = 8;
struct HostPipe {
  int device = -1;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_begin = nullptr, ev_in[kMaxSlices] = {}, ev_done[kMaxSlices] = {};
  void release() {
    for (int c = 0; c < kMaxSlices; ++c) {
      if (ev_in[c]) cudaEventDestroy(ev_in[c]);
      if (ev_done[c]) cudaEventDestroy(ev_done[c]);
      ev_in[c] = ev_done[c] = nullptr;
    }
    if (ev_begin) cudaEventDestroy(ev_begin);
    if (s_in) cudaStreamDestroy(s_in);
    if (s_out) cudaStreamDestroy(s_out);
    ev_begin = nullptr;
    s_in = s_out = nullptr;
    device = -1;
  }
  bool prepare() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev == device) return true;
    release();
    bool good = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess &&
                cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess &&
                cudaEventCreateWithFlags(&ev_begin, cudaEventDisableTiming) == cudaSuccess;
    for (int c = 0; c < kMaxSlices && good; ++c)
      good = cudaEventCreateWithFlags(&ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&ev_done[c], cudaEventDisableTiming) == cudaSuccess;
    if (!good) {
      release();
      return false;
    }
    device = dev;
    return true;
  }
  ~HostPipe() {}  // at thread exit the CUDA runtime may already be gone: the handles are left to it
};
HostPipe& host_pipe() {
  static thread_local HostPipe pipe;
  return pipe;
}
}  // namespace

extern "C" {

sea_status sea_workspace_bytes(const sea_shape* shape, size_t* bytes) {
  if (bytes == nullptr) return SEA_ERR_INVALID_ARG;
  const sea_status rc = validate_shape(shape, false);
  if (rc != SEA_OK) return rc;
  *bytes = ws_layout(*shape).total;
  return SEA_OK;
}

sea_status sea_estimate(const sea_shape* shape, const void* Q, const void* K, const void* V,
                        const float* omega, const float* W_dec, float* A_hat, void* ws,
                        size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, true, 0, true);  // the estimate does not depend on the ratio of T to Kc
  if (rc != SEA_OK) return rc;
  if (!Q || !K || !V || !omega || !W_dec || !A_hat || !ws) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(omega) || !aligned16(W_dec) ||
      !aligned16(A_hat) || !aligned16(ws))
    return SEA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  return launch_estimate(*shape, Q, K, V, omega, W_dec, A_hat, reinterpret_cast<float*>(w + L.est_state),
                         w + L.est_split, nullptr, nullptr, reinterpret_cast<int32_t*>(w + L.status),
                         static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_topk_mask(const sea_shape* shape, const float* A_hat, int32_t* sel, int32_t* row_ptr,
                         int32_t* col_idx, int64_t nnz_cap, void* ws, size_t ws_bytes,
                         void* cuda_stream) {
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, false);
  if (rc != SEA_OK) return rc;
  if (!A_hat || !row_ptr || !ws) return SEA_ERR_INVALID_ARG;
  if (!aligned16(A_hat) || !aligned16(row_ptr) || !aligned16(ws) || (sel && !aligned16(sel)) ||
      (col_idx && !aligned16(col_idx)))
    return SEA_ERR_INVALID_ARG;
  if (col_idx && nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  return launch_topk_mask(*shape, A_hat, sel_buf, row_ptr, col_idx, nnz_cap,
                          reinterpret_cast<int32_t*>(w + L.row_counts),
                          reinterpret_cast<int32_t*>(w + L.tile_sums), nullptr, false,
                          reinterpret_cast<int32_t*>(w + L.status), static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_sparse_attn(const sea_shape* shape, const void* Q, const void* K, const void* V,
                           const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel, void* O,
                           void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, false, 0, sel == nullptr);  // a plain CSR may come from any up-sampling
  if (rc != SEA_OK) return rc;
  if (!Q || !K || !V || !row_ptr || !O || (!col_idx && !sel)) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(row_ptr) ||
      (P && !aligned16(P)) || (sel && !aligned16(sel)) || (col_idx && !aligned16(col_idx)))
    return SEA_ERR_INVALID_ARG;
  if (ws && !aligned16(ws)) return SEA_ERR_INVALID_ARG;
  if (ws && ws_bytes < (size_t)kStatusBytes) return SEA_ERR_WORKSPACE;
  // With a full workspace every kernel is available; with only the status word at its head the
  // per-row kernels run; without ws, those of them that have no device-side waits.
  char* w = static_cast<char*>(ws);
  const WsLayout L = ws_layout(*shape);
  const bool full = ws && ws_bytes >= L.total;
  return launch_sparse_attn(*shape, Q, K, V, row_ptr, col_idx, sel, O, P,
                            full ? reinterpret_cast<uint32_t*>(w + L.mask_bits) : nullptr, false,
                            full ? reinterpret_cast<float*>(w + L.p_scratch) : nullptr,
                            full ? reinterpret_cast<uint32_t*>(w + L.tile_live) : nullptr,
                            static_cast<int32_t*>(ws), static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_attention(const sea_shape* shape, const void* Q, const void* K, const void* V,
                         const float* omega, const float* W_dec, const float* A_hat_in, void* O,
                         float* A_hat, int32_t* sel, int32_t* row_ptr, int32_t* col_idx,
                         int64_t nnz_cap, void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const bool estimate = A_hat_in == nullptr;
  sea_status rc = validate_shape(shape, estimate);
  if (rc != SEA_OK) return rc;
  if (!Q || !K || !V || !O || !ws) return SEA_ERR_INVALID_ARG;
  if (estimate && (!omega || !W_dec)) return SEA_ERR_INVALID_ARG;
  if (P && !col_idx) return SEA_ERR_INVALID_ARG;  // probabilities are only meaningful beside their indices
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(ws) ||
      (omega && !aligned16(omega)) || (W_dec && !aligned16(W_dec)) || (A_hat_in && !aligned16(A_hat_in)) ||
      (A_hat && !aligned16(A_hat)) || (sel && !aligned16(sel)) || (row_ptr && !aligned16(row_ptr)) ||
      (col_idx && !aligned16(col_idx)) || (P && !aligned16(P)))
    return SEA_ERR_INVALID_ARG;
  if (col_idx && nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  // The sparse stage writes P at the positions row_ptr gives and never learns nnz_cap: a capacity
  // that a long mask could exceed is refused here.  (col_idx alone may be shorter: the fill
  // truncates and reports, and the sparse stage walks `sel`, not col_idx.)
  if (P && nnz_cap < mask_entries_bound(*shape, 0)) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t* status = reinterpret_cast<int32_t*>(w + L.status);

  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  int32_t* rp_buf = row_ptr ? row_ptr : reinterpret_cast<int32_t*>(w + L.row_ptr);
  uint32_t* bits = reinterpret_cast<uint32_t*>(w + L.mask_bits);
  int32_t* counts = reinterpret_cast<int32_t*>(w + L.row_counts);
  const float* a_use = A_hat_in;
  bool selected = false;
  if (estimate) {
    // where the estimator can, it selects each row's columns while the row is still on chip; the
    // estimate then only leaves the chip if the caller asked for it
    const bool on_chip = shape->io == SEA_BF16 && estimate_tc_selects(*shape);
    float* a_out = A_hat ? A_hat : (on_chip ? nullptr : reinterpret_cast<float*>(w + L.a_hat));
    const SelectOut so{sel_buf, shape->causal ? counts : nullptr, bits};
    rc = launch_estimate(*shape, Q, K, V, omega, W_dec, a_out, reinterpret_cast<float*>(w + L.est_state),
                         w + L.est_split, &so, &selected, status, st);
    if (rc != SEA_OK) return rc;
    a_use = a_out;
  }
  rc = launch_topk_mask(*shape, a_use, sel_buf, rp_buf, col_idx, nnz_cap, counts,
                        reinterpret_cast<int32_t*>(w + L.tile_sums), bits, selected, status, st);
  if (rc != SEA_OK) return rc;
  return launch_sparse_attn(*shape, Q, K, V, rp_buf, col_idx, sel_buf, O, P, bits, true,
                            reinterpret_cast<float*>(w + L.p_scratch), reinterpret_cast<uint32_t*>(w + L.tile_live), status, st);
}

}  // extern "C"

namespace {
// The two selections whose rows keep differing numbers of columns (the result leaves as bits).
enum class BitsMode { kPerBatch, kCausalAware };
bool bits_mode_supported(const sea_shape& s, BitsMode mode) {
  return mode == BitsMode::kPerBatch ? topk_grouped_supported(s) : s.causal == 1;
}

sea_status topk_mask_bits(BitsMode mode, const sea_shape* shape, const float* A_hat, uint32_t* mask_bits,
                          int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* ws, size_t ws_bytes,
                          void* cuda_stream) {
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, false);
  if (rc != SEA_OK) return rc;
  if (!bits_mode_supported(*shape, mode)) return SEA_ERR_UNSUPPORTED;
  if (!A_hat || !row_ptr || !ws) return SEA_ERR_INVALID_ARG;
  if (!aligned16(A_hat) || !aligned16(row_ptr) || !aligned16(ws) || (mask_bits && !aligned16(mask_bits)) ||
      (col_idx && !aligned16(col_idx)))
    return SEA_ERR_INVALID_ARG;
  if (col_idx && nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  uint32_t* bits = mask_bits ? mask_bits : reinterpret_cast<uint32_t*>(w + L.mask_bits);
  int32_t* counts = reinterpret_cast<int32_t*>(w + L.row_counts);
  int32_t* sums = reinterpret_cast<int32_t*>(w + L.tile_sums);
  int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (mode == BitsMode::kPerBatch)
    return launch_topk_mask_grouped(*shape, A_hat, bits, row_ptr, col_idx, nnz_cap, counts, sums, nullptr, status, st);
  return launch_topk_mask_aware(*shape, A_hat, bits, row_ptr, col_idx, nnz_cap, counts, sums, status, st);
}
}  // namespace

extern "C" {

sea_status sea_topk_mask_grouped(const sea_shape* shape, const float* A_hat, uint32_t* mask_bits,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* ws,
                                 size_t ws_bytes, void* cuda_stream) {
  return topk_mask_bits(BitsMode::kPerBatch, shape, A_hat, mask_bits, row_ptr, col_idx, nnz_cap, ws, ws_bytes,
                        cuda_stream);
}

sea_status sea_topk_mask_causal_aware(const sea_shape* shape, const float* A_hat, uint32_t* mask_bits,
                                      int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* ws,
                                      size_t ws_bytes, void* cuda_stream) {
  return topk_mask_bits(BitsMode::kCausalAware, shape, A_hat, mask_bits, row_ptr, col_idx, nnz_cap, ws, ws_bytes,
                        cuda_stream);
}

sea_status sea_sparse_attn_masked(const sea_shape* shape, const void* Q, const void* K, const void* V,
                                  const int32_t* row_ptr, const int32_t* col_idx, const uint32_t* mask_bits,
                                  void* O, void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, false);
  if (rc != SEA_OK) return rc;
  if (!Q || !K || !V || !row_ptr || !O || !mask_bits) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(row_ptr) ||
      !aligned16(mask_bits) || (P && !aligned16(P)) || (col_idx && !aligned16(col_idx)))
    return SEA_ERR_INVALID_ARG;
  if (ws && !aligned16(ws)) return SEA_ERR_INVALID_ARG;
  if (ws && ws_bytes < (size_t)kStatusBytes) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  const WsLayout L = ws_layout(*shape);
  const bool full = ws && ws_bytes >= L.total && shape->io == SEA_BF16;
  return launch_sparse_attn_masked(*shape, Q, K, V, row_ptr, col_idx, mask_bits, O, P,
                                   full ? reinterpret_cast<int32_t*>(w + L.park_off) : nullptr, false, false,
                                   full ? reinterpret_cast<float*>(w + L.p_scratch) : nullptr,
                                   full ? reinterpret_cast<uint32_t*>(w + L.tile_live) : nullptr,
                                   static_cast<int32_t*>(ws), static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

namespace {
sea_status attention_bits(BitsMode mode, const sea_shape* shape, const void* Q, const void* K, const void* V,
                          const float* omega, const float* W_dec, const float* A_hat_in, void* O, float* A_hat,
                          uint32_t* mask_bits, int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* P, void* ws,
                          size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const bool estimate = A_hat_in == nullptr;
  sea_status rc = validate_shape(shape, estimate);
  if (rc != SEA_OK) return rc;
  if (!bits_mode_supported(*shape, mode)) return SEA_ERR_UNSUPPORTED;
  if (!Q || !K || !V || !O || !ws) return SEA_ERR_INVALID_ARG;
  if (estimate && (!omega || !W_dec)) return SEA_ERR_INVALID_ARG;
  if (P && !col_idx) return SEA_ERR_INVALID_ARG;  // probabilities are only meaningful beside their indices
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(ws) ||
      (omega && !aligned16(omega)) || (W_dec && !aligned16(W_dec)) || (A_hat_in && !aligned16(A_hat_in)) ||
      (A_hat && !aligned16(A_hat)) || (mask_bits && !aligned16(mask_bits)) || (row_ptr && !aligned16(row_ptr)) ||
      (col_idx && !aligned16(col_idx)) || (P && !aligned16(P)))
    return SEA_ERR_INVALID_ARG;
  if (col_idx && nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
  // without col_idx the sparse stage must be able to work from the bits alone
  uint32_t* bits = mask_bits ? mask_bits : reinterpret_cast<uint32_t*>(w + L.mask_bits);
  float* scratch = shape->io == SEA_BF16 ? reinterpret_cast<float*>(w + L.p_scratch) : nullptr;
  int32_t* park = shape->io == SEA_BF16 ? reinterpret_cast<int32_t*>(w + L.park_off) : nullptr;
  const bool tiles_ok = park && sparse_attn_tc_applicable(*shape, nullptr, true, status, bits, scratch);
  if (!col_idx && !tiles_ok) return SEA_ERR_INVALID_ARG;
  // P is written at the positions row_ptr gives, and without the tile kernel the sparse stage walks
  // col_idx; neither learns nnz_cap, so a capacity that the mask could exceed is refused here
  if (col_idx && (P || !tiles_ok) && nnz_cap < mask_entries_bound(*shape, 0)) return SEA_ERR_TOO_LARGE;

  const float* a_use = A_hat_in;
  if (estimate) {
    float* a_out = A_hat ? A_hat : reinterpret_cast<float*>(w + L.a_hat);
    rc = launch_estimate(*shape, Q, K, V, omega, W_dec, a_out, reinterpret_cast<float*>(w + L.est_state),
                         w + L.est_split, nullptr, nullptr, status, st);
    if (rc != SEA_OK) return rc;
    a_use = a_out;
  }
  int32_t* rp_buf = row_ptr ? row_ptr : reinterpret_cast<int32_t*>(w + L.row_ptr);
  int32_t* counts = reinterpret_cast<int32_t*>(w + L.row_counts);
  int32_t* sums = reinterpret_cast<int32_t*>(w + L.tile_sums);
  if (mode == BitsMode::kPerBatch) {
    // the selection also lays out the parking area of the tile kernel when P is wanted
    rc = launch_topk_mask_grouped(*shape, a_use, bits, rp_buf, col_idx, nnz_cap, counts, sums, tiles_ok && P ? park : nullptr,
                                  status, st);
    if (rc != SEA_OK) return rc;
    return launch_sparse_attn_masked(*shape, Q, K, V, rp_buf, col_idx, bits, O, P, park, true, false, scratch, reinterpret_cast<uint32_t*>(w + L.tile_live), status, st);
  }
  rc = launch_topk_mask_aware(*shape, a_use, bits, rp_buf, col_idx, nnz_cap, counts, sums, status, st);
  if (rc != SEA_OK) return rc;
  return launch_sparse_attn_masked(*shape, Q, K, V, rp_buf, col_idx, bits, O, P, park, false, true, scratch, reinterpret_cast<uint32_t*>(w + L.tile_live), status, st);
}
}  // namespace

extern "C" {

sea_status sea_attention_grouped(const sea_shape* shape, const void* Q, const void* K, const void* V,
                                 const float* omega, const float* W_dec, const float* A_hat_in, void* O,
                                 float* A_hat, uint32_t* mask_bits, int32_t* row_ptr, int32_t* col_idx,
                                 int64_t nnz_cap, void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  return attention_bits(BitsMode::kPerBatch, shape, Q, K, V, omega, W_dec, A_hat_in, O, A_hat, mask_bits, row_ptr,
                        col_idx, nnz_cap, P, ws, ws_bytes, cuda_stream);
}

sea_status sea_attention_causal_aware(const sea_shape* shape, const void* Q, const void* K, const void* V,
                                      const float* omega, const float* W_dec, const float* A_hat_in, void* O,
                                      float* A_hat, uint32_t* mask_bits, int32_t* row_ptr, int32_t* col_idx,
                                      int64_t nnz_cap, void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  return attention_bits(BitsMode::kCausalAware, shape, Q, K, V, omega, W_dec, A_hat_in, O, A_hat, mask_bits, row_ptr,
                        col_idx, nnz_cap, P, ws, ws_bytes, cuda_stream);
}

sea_status sea_workspace_bytes_capped(const sea_shape* shape, int32_t k_star, size_t* bytes) {
  if (bytes == nullptr || k_star < 1) return SEA_ERR_INVALID_ARG;
  const sea_status rc = validate_shape(shape, false, k_star);
  if (rc != SEA_OK) return rc;
  *bytes = ws_layout(*shape).total;
  return SEA_OK;
}

sea_status sea_topk_mask_capped(const sea_shape* shape, int32_t k_star, const float* A_hat, int32_t* sel,
                                int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* ws, size_t ws_bytes,
                                void* cuda_stream) {
  Launch::count() = 0;
  if (k_star < 1) return SEA_ERR_INVALID_ARG;
  const sea_status rc = validate_shape(shape, false, k_star);
  if (rc != SEA_OK) return rc;
  if (!A_hat || !row_ptr || !col_idx || !ws) return SEA_ERR_INVALID_ARG;
  if (!aligned16(A_hat) || !aligned16(row_ptr) || !aligned16(col_idx) || !aligned16(ws) || (sel && !aligned16(sel)))
    return SEA_ERR_INVALID_ARG;
  if (nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  return launch_topk_mask_capped(*shape, k_star, A_hat, sel_buf, row_ptr, col_idx, nnz_cap,
                                 reinterpret_cast<int32_t*>(w + L.row_counts),
                                 reinterpret_cast<int32_t*>(w + L.tile_sums), reinterpret_cast<int32_t*>(w + L.status),
                                 static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_attention_capped(const sea_shape* shape, int32_t k_star, const void* Q, const void* K, const void* V,
                                const float* omega, const float* W_dec, const float* A_hat_in, void* O, float* A_hat,
                                int32_t* sel, int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* P, void* ws,
                                size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const bool estimate = A_hat_in == nullptr;
  if (k_star < 1) return SEA_ERR_INVALID_ARG;
  sea_status rc = validate_shape(shape, estimate, k_star);
  if (rc != SEA_OK) return rc;
  if (!Q || !K || !V || !O || !ws || !col_idx) return SEA_ERR_INVALID_ARG;
  if (estimate && (!omega || !W_dec)) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(ws) || !aligned16(col_idx) ||
      (omega && !aligned16(omega)) || (W_dec && !aligned16(W_dec)) || (A_hat_in && !aligned16(A_hat_in)) ||
      (A_hat && !aligned16(A_hat)) || (sel && !aligned16(sel)) || (row_ptr && !aligned16(row_ptr)) || (P && !aligned16(P)))
    return SEA_ERR_INVALID_ARG;
  if (nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  // the sparse stage walks col_idx (and writes P) by row_ptr alone: the capacity must hold any mask
  if (nnz_cap < mask_entries_bound(*shape, k_star)) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
  const float* a_use = A_hat_in;
  if (estimate) {
    float* a_out = A_hat ? A_hat : reinterpret_cast<float*>(w + L.a_hat);
    rc = launch_estimate(*shape, Q, K, V, omega, W_dec, a_out, reinterpret_cast<float*>(w + L.est_state),
                         w + L.est_split, nullptr, nullptr, status, st);
    if (rc != SEA_OK) return rc;
    a_use = a_out;
  }
  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  int32_t* rp_buf = row_ptr ? row_ptr : reinterpret_cast<int32_t*>(w + L.row_ptr);
  rc = launch_topk_mask_capped(*shape, k_star, a_use, sel_buf, rp_buf, col_idx, nnz_cap,
                               reinterpret_cast<int32_t*>(w + L.row_counts),
                               reinterpret_cast<int32_t*>(w + L.tile_sums), status, st);
  if (rc != SEA_OK) return rc;
  // rows keep scattered keys, not runs: the per-row kernels walk the CSR
  return launch_sparse_attn_rows(*shape, Q, K, V, rp_buf, col_idx, nullptr, O, P, st);
}

sea_status sea_workspace_bytes_resized(const sea_shape* shape, size_t* bytes) {
  if (bytes == nullptr) return SEA_ERR_INVALID_ARG;
  const sea_status rc = validate_shape(shape, false, 0, true);
  if (rc != SEA_OK) return rc;
  *bytes = ws_layout(*shape).total;
  return SEA_OK;
}

sea_status sea_topk_mask_resized(const sea_shape* shape, int32_t row_widths, const float* A_hat, int32_t* sel,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* ws, size_t ws_bytes,
                                 void* cuda_stream) {
  Launch::count() = 0;
  const sea_status rc = validate_shape(shape, false, 0, true);
  if (rc != SEA_OK) return rc;
  if (row_widths != 0 && row_widths != 1) return SEA_ERR_INVALID_ARG;
  if (row_widths && !shape->causal) return SEA_ERR_UNSUPPORTED;  // a row's own width is a causal notion
  if (!A_hat || !row_ptr || !ws) return SEA_ERR_INVALID_ARG;
  if (!aligned16(A_hat) || !aligned16(row_ptr) || !aligned16(ws) || (sel && !aligned16(sel)) || (col_idx && !aligned16(col_idx)))
    return SEA_ERR_INVALID_ARG;
  if (col_idx && nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  return launch_topk_mask_resized(*shape, row_widths, A_hat, sel_buf, row_ptr, col_idx, nnz_cap,
                                  reinterpret_cast<int32_t*>(w + L.row_counts), reinterpret_cast<int32_t*>(w + L.tile_sums),
                                  reinterpret_cast<int32_t*>(w + L.status), static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_attention_resized(const sea_shape* shape, int32_t row_widths, const void* Q, const void* K, const void* V,
                                 const float* omega, const float* W_dec, const float* A_hat_in, void* O, float* A_hat,
                                 int32_t* sel, int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* P, void* ws,
                                 size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  const bool estimate = A_hat_in == nullptr;
  sea_status rc = validate_shape(shape, estimate, 0, true);
  if (rc != SEA_OK) return rc;
  if (row_widths != 0 && row_widths != 1) return SEA_ERR_INVALID_ARG;
  if (row_widths && !shape->causal) return SEA_ERR_UNSUPPORTED;
  if (!Q || !K || !V || !O || !ws || !col_idx) return SEA_ERR_INVALID_ARG;
  if (estimate && (!omega || !W_dec)) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(ws) || !aligned16(col_idx) ||
      (omega && !aligned16(omega)) || (W_dec && !aligned16(W_dec)) || (A_hat_in && !aligned16(A_hat_in)) ||
      (A_hat && !aligned16(A_hat)) || (sel && !aligned16(sel)) || (row_ptr && !aligned16(row_ptr)) || (P && !aligned16(P)))
    return SEA_ERR_INVALID_ARG;
  if (nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  // the sparse stage walks col_idx (and writes P) by row_ptr alone: the capacity must hold any mask
  if (nnz_cap < mask_entries_bound(*shape, 0)) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  if (ws_bytes < L.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
  const float* a_use = A_hat_in;
  if (estimate) {
    float* a_out = A_hat ? A_hat : reinterpret_cast<float*>(w + L.a_hat);
    rc = launch_estimate(*shape, Q, K, V, omega, W_dec, a_out, reinterpret_cast<float*>(w + L.est_state),
                         w + L.est_split, nullptr, nullptr, status, st);
    if (rc != SEA_OK) return rc;
    a_use = a_out;
  }
  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  int32_t* rp_buf = row_ptr ? row_ptr : reinterpret_cast<int32_t*>(w + L.row_ptr);
  rc = launch_topk_mask_resized(*shape, row_widths, a_use, sel_buf, rp_buf, col_idx, nnz_cap,
                                reinterpret_cast<int32_t*>(w + L.row_counts), reinterpret_cast<int32_t*>(w + L.tile_sums),
                                status, st);
  if (rc != SEA_OK) return rc;
  // a pixel's keys are runs of differing lengths: the per-row kernels walk the CSR
  return launch_sparse_attn_rows(*shape, Q, K, V, rp_buf, col_idx, nullptr, O, P, st);
}

}  // extern "C"

namespace {
sea_status validate_decoder(const sea_shape* s, const sea_decoder* d) {
  if (d == nullptr) return SEA_ERR_INVALID_ARG;
  if (d->d_hidden < 1 || d->d_hidden > 1024 || d->c_s < 1 || d->c_h < 1) return SEA_ERR_INVALID_ARG;
  if (s->Kc % d->c_s != 0 || (!s->causal && s->T % d->c_s != 0)) return SEA_ERR_UNSUPPORTED;
  if (!d->W_mu || !d->b_mu || !d->W_nu1 || !d->b_nu1 || !d->W_nu2 || !d->b_nu2 || !d->conv1_w || !d->conv1_b || !d->conv2_w ||
      !d->conv2_b || !d->conv3_w || !d->conv3_b || !d->w_prob || !d->w_mix || (s->causal && !d->pos_emb))
    return SEA_ERR_INVALID_ARG;
  if ((long long)s->B * s->H * d->c_h * s->T * (s->Kc / d->c_s) > 2147483647ll * 4) return SEA_ERR_TOO_LARGE;
  return SEA_OK;
}
// the decoder's buffers follow the base layout
size_t decoder_ws_offset(const sea_shape& s) { return align_up(ws_layout(s).total, 256); }
}  // namespace

extern "C" {

sea_status sea_workspace_bytes_decoder(const sea_shape* shape, const sea_decoder* dec, size_t* bytes) {
  if (bytes == nullptr) return SEA_ERR_INVALID_ARG;
  sea_status rc = validate_shape(shape, true);
  if (rc != SEA_OK) return rc;
  if ((rc = validate_decoder(shape, dec)) != SEA_OK) return rc;
  *bytes = decoder_ws_offset(*shape) + decoder_layout(*shape, *dec).total;
  return SEA_OK;
}

sea_status sea_estimate_decoder(const sea_shape* shape, const sea_decoder* dec, const void* Q, const void* K, const void* V,
                                const float* omega, float* A_hat, float* Z, void* ws, size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  sea_status rc = validate_shape(shape, true);
  if (rc != SEA_OK) return rc;
  if ((rc = validate_decoder(shape, dec)) != SEA_OK) return rc;
  if (!Q || !K || !V || !omega || !A_hat || !ws) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(omega) || !aligned16(A_hat) || !aligned16(ws) ||
      (Z && !aligned16(Z)))
    return SEA_ERR_INVALID_ARG;
  const WsLayout L = ws_layout(*shape);
  const size_t doff = decoder_ws_offset(*shape);
  const DecoderLayout D = decoder_layout(*shape, *dec);
  if (ws_bytes < doff + D.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  float* z = Z ? Z : reinterpret_cast<float*>(w + doff + D.z);
  return launch_estimate_decoder(*shape, *dec, Q, K, V, omega, A_hat, z, w + doff, reinterpret_cast<float*>(w + L.est_state),
                                 w + L.est_split, reinterpret_cast<int32_t*>(w + L.status), static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_mix_output(const sea_shape* shape, const sea_decoder* dec, const float* Z, const float* A_hat, const void* V,
                          const int32_t* row_ptr, void* O, void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  sea_status rc = validate_shape(shape, true);
  if (rc != SEA_OK) return rc;
  if ((rc = validate_decoder(shape, dec)) != SEA_OK) return rc;
  if (!Z || !A_hat || !V || !O || !ws || (P && !row_ptr)) return SEA_ERR_INVALID_ARG;
  const size_t doff = decoder_ws_offset(*shape);
  if (ws_bytes < doff + decoder_layout(*shape, *dec).total) return SEA_ERR_WORKSPACE;
  return launch_mix_output(*shape, *dec, Z, A_hat, V, row_ptr, O, P, static_cast<char*>(ws) + doff,
                           static_cast<cudaStream_t>(cuda_stream));
}

sea_status sea_attention_decoder(const sea_shape* shape, const sea_decoder* dec, const void* Q, const void* K, const void* V,
                                 const float* omega, void* O, float* A_hat, int32_t* sel, int32_t* row_ptr, int32_t* col_idx,
                                 int64_t nnz_cap, void* P, void* ws, size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  sea_status rc = validate_shape(shape, true);
  if (rc != SEA_OK) return rc;
  if ((rc = validate_decoder(shape, dec)) != SEA_OK) return rc;
  if (!Q || !K || !V || !omega || !O || !ws) return SEA_ERR_INVALID_ARG;
  if (P && !col_idx) return SEA_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(ws) || !aligned16(omega) ||
      (A_hat && !aligned16(A_hat)) || (sel && !aligned16(sel)) || (row_ptr && !aligned16(row_ptr)) ||
      (col_idx && !aligned16(col_idx)) || (P && !aligned16(P)))
    return SEA_ERR_INVALID_ARG;
  if (col_idx && nnz_cap <= 0) return SEA_ERR_INVALID_ARG;
  if (nnz_cap > 2147483647ll) return SEA_ERR_TOO_LARGE;
  if (P && nnz_cap < mask_entries_bound(*shape, 0)) return SEA_ERR_TOO_LARGE;
  const WsLayout L = ws_layout(*shape);
  const size_t doff = decoder_ws_offset(*shape);
  const DecoderLayout D = decoder_layout(*shape, *dec);
  if (ws_bytes < doff + D.total) return SEA_ERR_WORKSPACE;
  char* w = static_cast<char*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t* status = reinterpret_cast<int32_t*>(w + L.status);
  float* a_buf = A_hat ? A_hat : reinterpret_cast<float*>(w + L.a_hat);
  float* z = reinterpret_cast<float*>(w + doff + D.z);
  rc = launch_estimate_decoder(*shape, *dec, Q, K, V, omega, a_buf, z, w + doff, reinterpret_cast<float*>(w + L.est_state),
                               w + L.est_split, status, st);
  if (rc != SEA_OK) return rc;
  int32_t* sel_buf = sel ? sel : reinterpret_cast<int32_t*>(w + L.sel);
  int32_t* rp_buf = row_ptr ? row_ptr : reinterpret_cast<int32_t*>(w + L.row_ptr);
  uint32_t* bits = reinterpret_cast<uint32_t*>(w + L.mask_bits);
  rc = launch_topk_mask(*shape, a_buf, sel_buf, rp_buf, col_idx, nnz_cap, reinterpret_cast<int32_t*>(w + L.row_counts),
                        reinterpret_cast<int32_t*>(w + L.tile_sums), bits, false, status, st);
  if (rc != SEA_OK) return rc;
  rc = launch_sparse_attn(*shape, Q, K, V, rp_buf, col_idx, sel_buf, O, P, bits, true, reinterpret_cast<float*>(w + L.p_scratch),
                          reinterpret_cast<uint32_t*>(w + L.tile_live), status, st);
  if (rc != SEA_OK) return rc;
  return launch_mix_output(*shape, *dec, z, a_buf, V, rp_buf, O, P, w + doff, st);
}

sea_status sea_workspace_host_bytes(const sea_shape* shape, size_t* bytes) {
  if (bytes == nullptr) return SEA_ERR_INVALID_ARG;
  const sea_status rc = validate_shape(shape, true);
  if (rc != SEA_OK) return rc;
  const size_t qkv = align_up((size_t)shape->B * shape->H * shape->T * kHeadDim * io_bytes(*shape), 256);
  const size_t om = align_up((size_t)shape->m * kHeadDim * sizeof(float), 256);
  const size_t wd = align_up((size_t)kHeadDim * shape->Kc * sizeof(float), 256);
  *bytes = ws_layout(*shape).total + 4 * qkv + om + wd;
  return SEA_OK;
}

sea_status sea_attention_host(const sea_shape* shape, const void* hQ, const void* hK, const void* hV,
                              const float* homega, const float* hW_dec, void* hO, void* ws,
                              size_t ws_bytes, void* cuda_stream) {
  Launch::count() = 0;
  size_t need = 0;
  sea_status rc = sea_workspace_host_bytes(shape, &need);
  if (rc != SEA_OK) return rc;
  if (!hQ || !hK || !hV || !homega || !hW_dec || !hO || !ws || !aligned16(ws)) return SEA_ERR_INVALID_ARG;
  if (ws_bytes < need) return SEA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t inner = ws_layout(*shape).total;
  const size_t qkv_b = (size_t)shape->B * shape->H * shape->T * kHeadDim * io_bytes(*shape);
  const size_t qkv = align_up(qkv_b, 256);
  const size_t om_b = (size_t)shape->m * kHeadDim * sizeof(float);
  const size_t wd_b = (size_t)kHeadDim * shape->Kc * sizeof(float);
  char* w = static_cast<char*>(ws);
  char* dQ = w + inner;
  char* dK = dQ + qkv;
  char* dV = dK + qkv;
  char* dO = dV + qkv;
  char* dOm = dO + qkv;
  char* dWd = dOm + align_up(om_b, 256);

  // The heads are independent, so the call runs as a pipeline over slices of them: while one slice
  // is computed on the caller's stream, the next one's Q, K, V come in on a second stream and the
  // previous one's O goes out on a third (the link carries both directions at once).  The two
  // copy streams and the events belong to the calling host thread, which creates them once.
  const int BH = shape->B * shape->H;
  int nslice = 1;
  for (int c = 8; c >= 2; c >>= 1)
    if (BH % c == 0 && BH / c >= 8) {
      nslice = c;
      break;
    }
  sea_shape sub = *shape;
  sub.B = 1;
  sub.H = BH / nslice;
  const size_t slice_b = qkv_b / nslice;

  HostPipe& pipe = host_pipe();
  rc = pipe.prepare() ? SEA_OK : SEA_ERR_CUDA;
  cudaStream_t s_in = pipe.s_in, s_out = pipe.s_out;
  cudaEvent_t ev_begin = pipe.ev_begin;
  cudaEvent_t* ev_in = pipe.ev_in;
  cudaEvent_t* ev_done = pipe.ev_done;
  int launches = 0;
  // the staging areas may still be read by work the caller enqueued earlier on `st`
  if (rc == SEA_OK && (cudaEventRecord(ev_begin, st) != cudaSuccess || cudaStreamWaitEvent(s_in, ev_begin, 0) != cudaSuccess ||
                       cudaStreamWaitEvent(s_out, ev_begin, 0) != cudaSuccess))
    rc = SEA_ERR_CUDA;
  if (rc == SEA_OK && (cudaMemcpyAsync(dOm, homega, om_b, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
                       cudaMemcpyAsync(dWd, hW_dec, wd_b, cudaMemcpyHostToDevice, s_in) != cudaSuccess))
    rc = SEA_ERR_CUDA;
  for (int c = 0; c < nslice && rc == SEA_OK; ++c) {
    const size_t off = (size_t)c * slice_b;
    if (cudaMemcpyAsync(dQ + off, static_cast<const char*>(hQ) + off, slice_b, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
        cudaMemcpyAsync(dK + off, static_cast<const char*>(hK) + off, slice_b, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
        cudaMemcpyAsync(dV + off, static_cast<const char*>(hV) + off, slice_b, cudaMemcpyHostToDevice, s_in) != cudaSuccess ||
        cudaEventRecord(ev_in[c], s_in) != cudaSuccess || cudaStreamWaitEvent(st, ev_in[c], 0) != cudaSuccess) {
      rc = SEA_ERR_CUDA;
      break;
    }
    rc = sea_attention(&sub, dQ + off, dK + off, dV + off, reinterpret_cast<const float*>(dOm),
                       reinterpret_cast<const float*>(dWd), nullptr, dO + off, nullptr, nullptr, nullptr, nullptr, 0,
                       nullptr, ws, inner, cuda_stream);
    launches += Launch::count();
    if (rc != SEA_OK) break;
    if (cudaEventRecord(ev_done[c], st) != cudaSuccess || cudaStreamWaitEvent(s_out, ev_done[c], 0) != cudaSuccess ||
        cudaMemcpyAsync(static_cast<char*>(hO) + off, dO + off, slice_b, cudaMemcpyDeviceToHost, s_out) != cudaSuccess)
      rc = SEA_ERR_CUDA;
  }
  // the call returns with all of its work finished, success or not
  if (s_in && cudaStreamSynchronize(s_in) != cudaSuccess && rc == SEA_OK) rc = SEA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess && rc == SEA_OK) rc = SEA_ERR_CUDA;
  if (s_out && cudaStreamSynchronize(s_out) != cudaSuccess && rc == SEA_OK) rc = SEA_ERR_CUDA;
  Launch::count() = launches;
  return rc;
}

sea_status sea_device_status(void* ws, int32_t* out, int32_t clear, void* cuda_stream) {
  if (!ws || !out) return SEA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(out, ws, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SEA_ERR_CUDA;
  if (clear && cudaMemsetAsync(ws, 0, sizeof(int32_t), st) != cudaSuccess) return SEA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SEA_ERR_CUDA;
  return SEA_OK;
}

int32_t sea_last_launch_count(void) { return Launch::count(); }

const char* sea_last_sparse_kernel(void) { return Launch::sparse_kernel(); }

double sea_last_sparse_flops(void) { return Launch::sparse_flops(); }

const char* sea_status_string(sea_status s) {
  switch (s) {
    case SEA_OK: return "ok";
    case SEA_ERR_INVALID_ARG: return "invalid argument";
    case SEA_ERR_UNSUPPORTED: return "unsupported shape";
    case SEA_ERR_WORKSPACE: return "workspace too small";
    case SEA_ERR_TOO_LARGE: return "size exceeds int32 indexing or nnz_cap";
    case SEA_ERR_CUDA: return "CUDA runtime error";
  }
  return "unknown status";
}

}  // extern "C"

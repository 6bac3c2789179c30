/*
 * libsea -- the deployed attention layer of SEA ("Sparse linear attention with
 * Estimated Attention mask"), as a C ABI over hand-written sm_100a kernels.
 *
 * The layer has the paper's two phases (Sec. 3.1): (1) a linear-cost estimate
 * A_hat [T x Kc] of the attention matrix from a kernel-based (FAVOR+) attention
 * followed by a decoder; (2) a per-row top-k_hat selection on A_hat that is
 * interpolated to a sparse T x T mask and drives a sparse attention
 * (scores at mask positions, row softmax, product with V).
 *
 * Conventions for every call
 *   - Pointers named Q, K, V, O, P, A_hat, sel, row_ptr, col_idx, omega, W_dec
 *     and ws are DEVICE pointers owned by the caller, 16-byte aligned, dense and
 *     row-major with the last index fastest.  The library never allocates or
 *     frees device memory.  State kept between calls: the contents of `ws`; the
 *     two copy streams and the events of sea_attention_host, which a host thread
 *     creates on its first call on a device and keeps until it exits; and the
 *     static scratch array of sea_topk_mask_static (see there).
 *   - Q, K, V, O are [B, H, T, d] in the dtype `shape->io`; d must be 64.
 *   - A "row" is one query: row = (b*H + h)*T + i, rows = B*H*T.
 *   - r = T / Kc keys are covered by one compressed column (T % Kc == 0; only
 *     sea_estimate, sea_sparse_attn without `sel` and the *_resized calls take
 *     other ratios).
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the default stream) and the call returns without synchronising.
 *   - Host-detectable errors (null pointer, bad shape, too small a workspace or
 *     nnz_cap, sizes beyond int32 indexing) return a code and launch nothing.
 *     Anomalies only visible on the device (a row longer than nnz_cap allows, a
 *     non-finite normaliser) set bits in a status word inside `ws`, the kernel
 *     finishes safely, and sea_device_status() reads the word back.
 *   - The sparse stage finds a row's entries of col_idx and P through row_ptr alone
 *     and never sees a capacity.  In sea_sparse_attn / sea_sparse_attn_masked the
 *     caller guarantees that col_idx and P hold row_ptr[rows] elements.  The fused
 *     calls return SEA_ERR_TOO_LARGE, launching nothing, when P is requested (or
 *     the sparse stage has to walk col_idx) and nnz_cap is below the largest mask
 *     the shape allows (rows*k_hat*r; capped calls: rows*k_hat*min(k_star, r)).
 *   - Inputs must be finite.
 *   - Calls that share a workspace must be ordered on one stream.
 */
#ifndef SEA_H_
#define SEA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SEA_OK = 0,
  SEA_ERR_INVALID_ARG = 1, /* null pointer, misaligned pointer, non-positive size */
  SEA_ERR_UNSUPPORTED = 2, /* d != 64, T % Kc != 0, m or Kc outside the built range */
  SEA_ERR_WORKSPACE = 3,   /* ws_bytes below sea_workspace_bytes() */
  SEA_ERR_TOO_LARGE = 4,   /* an index would not fit int32, or nnz_cap too small */
  SEA_ERR_CUDA = 5         /* a CUDA runtime call failed (launch, copy) */
} sea_status;

typedef enum { SEA_F32 = 0, SEA_BF16 = 1 } sea_dtype;

/* Bits of the device status word (sea_device_status). */
enum {
  SEA_DEV_ROW_OVERFLOW = 1, /* a CSR row did not fit below nnz_cap and was truncated */
  SEA_DEV_NONFINITE = 2,    /* the estimator met a zero or non-finite normaliser */
  SEA_DEV_TIMEOUT = 4       /* a bounded wait on an asynchronous copy or tensor-core product ran out: the output of that call is not valid */
};

typedef struct sea_shape {
  int32_t B, H, T, d; /* batch, heads, sequence length, head width (64) */
  int32_t m;          /* FAVOR+ random features, a multiple of 16 in [16, 128]; 0 when the estimator is not used */
  int32_t Kc;         /* width of the compressed estimate (the paper's K), 1 <= Kc <= 2048 */
  int32_t k_hat;      /* columns kept per row in the compressed space, 1 <= k_hat <= Kc */
  int32_t causal;     /* 0 or 1 */
  int32_t io;         /* sea_dtype of Q, K, V, O and P */
  float scale;        /* softmax scale applied to q.k; 0 selects 1/sqrt(d) */
} sea_shape;

/* Bytes of device workspace that are enough for any call with this shape.
 * The first 256 bytes of a workspace hold the device status word; the caller
 * zeroes them once (cudaMemset) before first use. */
sea_status sea_workspace_bytes(const sea_shape* shape, size_t* bytes);

/*
 * Attention estimation, Sec. 3.1 "Attention Matrix Estimation" with the FAVOR+
 * attention of Sec. 3 "Performer (FAVOR+)" and one linear head in place of the
 * trained MLP + CNN decoder of "CNN Decoder":
 *
 *   x = u * d^(-1/4),  phi_f(u) = exp(omega_f . x - |x|^2 / 2) / sqrt(m)
 *   C_i = sum_j phi(q_i).phi(k_j) v_j / sum_j phi(q_i).phi(k_j)
 *         (all j when causal == 0, j <= i when causal == 1)
 *   A_hat = C W_dec
 *
 * omega [m, d] fp32 and W_dec [d, Kc] fp32 are shared by all (b, h).
 * A_hat [B, H, T, Kc] fp32 is written in full.
 */
sea_status sea_estimate(const sea_shape* shape, const void* Q, const void* K, const void* V,
                        const float* omega, const float* W_dec, float* A_hat,
                        void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Mask generation, Sec. 3.1 "Grouped Top-k Selection" (per-query grouping) and
 * "Linear Sparse Attention Mask Generation" / App. "Sparse Interpolation".
 *
 * For every row the k_hat largest entries of A_hat[row, :] are selected; equal
 * values (including -0 and +0) go to the lower column.  sel [rows, k_hat] int32
 * receives the selected columns in ascending order (may be NULL).  Each selected
 * column c is up-sampled by nearest neighbour to the keys c*r .. c*r+r-1; causal
 * rows drop keys j > i.  The result is a flat CSR over all rows: row_ptr
 * [rows+1] int32, col_idx [row_ptr[rows]] int32 ascending within a row.
 * nnz_cap is the capacity of col_idx in elements; rows*k_hat*r always suffices.
 * col_idx may be NULL (only sel and row_ptr are produced).
 */
sea_status sea_topk_mask(const sea_shape* shape, const float* A_hat, int32_t* sel,
                         int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * sea_topk_mask without a workspace (the paper has no counterpart; this is an
 * interface variant of the call above, same kernels, same results).
 *
 * It is meant for callers that cannot allocate device memory and have no
 * workspace to pass: an engine plugin whose memory plan is frozen, or a serving
 * loop where cudaMalloc is off limits because it synchronises the device and can
 * fail under a fixed budget.  The call itself allocates and frees nothing: the
 * per-row counts and scan partials live in a static device array inside the
 * library (4.2 MB, held by every GPU that loads the library until the process
 * exits), which limits the call to rows = B*H*T <= 1 048 576; larger shapes
 * return SEA_ERR_TOO_LARGE.
 *
 * Differences from sea_topk_mask: `sel` is required (it is an output the caller
 * owns); when col_idx is given, nnz_cap must be at least rows*k_hat*r, otherwise
 * SEA_ERR_TOO_LARGE (there is no status word through which a truncated row could
 * be reported).  The first call on each device looks up the array's device
 * address (with that device current); make that first call before any stream
 * capture begins.  All calls on a device share the one array, which keeps the
 * previous call's contents (the call clears what has to start at zero): two
 * calls whose kernels overlap on the GPU race, so keep them on one stream or
 * order them with events.
 */
sea_status sea_topk_mask_static(const sea_shape* shape, const float* A_hat, int32_t* sel,
                                int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                void* cuda_stream);

/*
 * Sparse attention, Sec. 3.1.1 "Sparse Attention Mechanism": rho (q_i . k_j * scale
 * at the mask's positions), sigma (softmax over the non-zeros of each row, so that
 * every non-empty row of A* sums to 1) and C = A* V, fused.  The learned
 * re-scaling s_prob is not applied.
 *
 * The mask is the CSR (row_ptr, col_idx).  When `sel` is given (the output of
 * sea_topk_mask for the same shape) the kernel walks the selected runs of r keys
 * directly and col_idx may be NULL.  O [B, H, T, d] is written in full; a row
 * without entries gives O = 0.  P, when not NULL, receives the CSR probabilities
 * aligned with col_idx (P[row_ptr[row] + n] belongs to the row's n-th key), in
 * the io dtype, rounded once from fp32; O is accumulated from the unrounded
 * probabilities.
 */
sea_status sea_sparse_attn(const sea_shape* shape, const void* Q, const void* K, const void* V,
                           const int32_t* row_ptr, const int32_t* col_idx, const int32_t* sel,
                           void* O, void* P, void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The whole layer: sea_estimate -> sea_topk_mask -> sea_sparse_attn on one stream.
 * A_hat, sel, row_ptr, col_idx and P are optional outputs (NULL = kept inside the
 * workspace or not materialised).  When A_hat_in is not NULL the estimator stage
 * is skipped and that estimate is used (shape->m may then be 0 and omega, W_dec
 * may be NULL).
 */
sea_status sea_attention(const sea_shape* shape, const void* Q, const void* K, const void* V,
                         const float* omega, const float* W_dec, const float* A_hat_in,
                         void* O, float* A_hat, int32_t* sel, int32_t* row_ptr,
                         int32_t* col_idx, int64_t nnz_cap, void* P,
                         void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Causal-per-batch grouping, Sec. 3.1 "Grouped Top-k Selection" (the grouping the
 * paper recommends and measures with, App. "FlatCSR").  A_hat of a batch element is
 * viewed as [T, H, Kc]; for every query position t the H*k_hat largest of the H*Kc
 * entries A_hat[b, :, t, :] are selected, with no exchange along T.  Equal values
 * (including -0 and +0) go to the lower flattened index h*Kc + c.  A row (b, h, t)
 * therefore keeps between 0 and min(Kc, H*k_hat) columns, and every (b, t) keeps
 * exactly H*k_hat over its heads.  Requires Kc % 4 == 0 and H*(ceil(Kc/32) + 1) <=
 * 12288 (the position's bit strings in shared memory); positions of more than 32768
 * values are read several times instead of being kept in registers.
 *
 * mask_bits [rows, ceil(Kc/32)] uint32 receives the selection (bit c%32 of word
 * c/32 of a row is set when column c is kept; may be NULL).  The up-sampling and the
 * CSR are those of sea_topk_mask, with rows in the same flat order (b*H + h)*T + t:
 * where the paper stores one row per (b, t) over the flattened (head, key) axis and
 * transposes inside its kernels, the rows here are already per head.  nnz_cap
 * rows*k_hat*r always suffices.  col_idx may be NULL.
 */
sea_status sea_topk_mask_grouped(const sea_shape* shape, const float* A_hat, uint32_t* mask_bits,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                 void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * sea_sparse_attn for a mask given as bits (the output of sea_topk_mask_grouped, or
 * any selection of compressed columns in that layout) together with its row_ptr.
 * col_idx may be NULL when the shape allows the tile kernel (bf16, T % 128 == 0,
 * r = T/Kc a power of two >= 4, full workspace); otherwise it is required and
 * SEA_ERR_INVALID_ARG is returned without it.  When P is requested, no (b, t) may
 * keep more than H*k_hat columns over its heads: rows beyond that budget are
 * reported through SEA_DEV_ROW_OVERFLOW and their P entries are not written.
 */
sea_status sea_sparse_attn_masked(const sea_shape* shape, const void* Q, const void* K, const void* V,
                                  const int32_t* row_ptr, const int32_t* col_idx,
                                  const uint32_t* mask_bits, void* O, void* P,
                                  void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The whole layer with the causal-per-batch grouping:
 * sea_estimate -> sea_topk_mask_grouped -> sea_sparse_attn_masked on one stream.
 * Optional outputs and A_hat_in as for sea_attention.
 */
sea_status sea_attention_grouped(const sea_shape* shape, const void* Q, const void* K, const void* V,
                                 const float* omega, const float* W_dec, const float* A_hat_in,
                                 void* O, float* A_hat, uint32_t* mask_bits, int32_t* row_ptr,
                                 int32_t* col_idx, int64_t nnz_cap, void* P,
                                 void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Causal-aware per-query selection (causal shapes only; other shapes return
 * SEA_ERR_UNSUPPORTED).  The paper resizes every causal row of the estimate to the
 * row's own width (App. "Visualization of intermediate buffers"), so a row never
 * spends its budget on keys it may not see.  With the fixed interpolation ratio
 * used here that becomes: row i chooses its k_hat largest entries among the
 * compressed columns that hold a key j <= i (columns 0 .. floor(i / r)) and keeps
 * min(k_hat, floor(i / r) + 1) of them; no row is left without keys, and the first
 * k_hat*r rows of a head see every key up to their own.  Ties as in sea_topk_mask.
 * Outputs and the sparse stage as for sea_topk_mask_grouped / sea_sparse_attn_masked
 * (a row keeps at most k_hat columns, so the budget rule of the latter holds).
 */
sea_status sea_topk_mask_causal_aware(const sea_shape* shape, const float* A_hat, uint32_t* mask_bits,
                                      int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                      void* ws, size_t ws_bytes, void* cuda_stream);
sea_status sea_attention_causal_aware(const sea_shape* shape, const void* Q, const void* K, const void* V,
                                      const float* omega, const float* W_dec, const float* A_hat_in,
                                      void* O, float* A_hat, uint32_t* mask_bits, int32_t* row_ptr,
                                      int32_t* col_idx, int64_t nnz_cap, void* P,
                                      void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Capped replication for long sequences, App. "Sparse Interpolation": when
 * k*K/T < 1 the paper selects a single column per row (k_hat = 1) and limits its
 * replication to k* = min(k, ceil(T/K)) keys instead of the whole run of T/K,
 * sampled uniformly; the spacing is not given and is taken as the keys
 * c*r + floor(u*r/k_star), u = 0 .. k_star-1 (k_star >= r keeps the whole run).
 * Causal rows drop keys j > i.  Works for any k_hat; T % Kc == 0 is still
 * required.  col_idx is required (the sparse stage walks the CSR with the per-row
 * kernels); nnz_cap rows*k_hat*min(k_star, r) always suffices, and it is this
 * product, not the uncapped mask, that has to fit int32 (T = 131072, Kc = 128,
 * k_hat = 1, k_star = 64 with 32 heads is within range).  sea_workspace_bytes_capped
 * is sea_workspace_bytes under that limit.
 */
sea_status sea_workspace_bytes_capped(const sea_shape* shape, int32_t k_star, size_t* bytes);
sea_status sea_topk_mask_capped(const sea_shape* shape, int32_t k_star, const float* A_hat, int32_t* sel,
                                int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                void* ws, size_t ws_bytes, void* cuda_stream);
sea_status sea_attention_capped(const sea_shape* shape, int32_t k_star, const void* Q, const void* K,
                                const void* V, const float* omega, const float* W_dec,
                                const float* A_hat_in, void* O, float* A_hat, int32_t* sel,
                                int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* P,
                                void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * Nearest-neighbour resize of the compressed mask at any ratio, App. "Sparse
 * Interpolation" and App. "Visualization of intermediate buffers".  The selection
 * is that of sea_topk_mask (per query, k_hat of the Kc pixels of a row); the
 * up-sampling treats row i of the compressed mask as an image of Kc pixels that is
 * resized to W pixels: key j < W looks at pixel floor(j * Kc / W), so a selected
 * pixel c covers the keys ceil(c*W/Kc) .. ceil((c+1)*W/Kc) - 1.
 *   row_widths == 0: W = T for every row; T need not be a multiple of Kc (for
 *     T % Kc == 0 the result is that of sea_topk_mask); causal rows drop keys j > i.
 *   row_widths == 1 (causal shapes only): W = i + 1, the paper's handling of causal
 *     rows ("each row ... is resized with different target widths according to the
 *     token index"): a row's k_hat pixels spread over the keys it may see, so its
 *     length grows with i, and only rows narrower than Kc keys can lose pixels.
 * Outputs as for sea_topk_mask; nnz_cap rows*k_hat*ceil(T/Kc) always suffices and is
 * what sea_attention_resized requires (its sparse stage walks col_idx with the
 * per-row kernels, so col_idx is required there).  sea_workspace_bytes_resized is
 * sea_workspace_bytes without the T % Kc == 0 condition.
 */
sea_status sea_workspace_bytes_resized(const sea_shape* shape, size_t* bytes);
sea_status sea_topk_mask_resized(const sea_shape* shape, int32_t row_widths, const float* A_hat, int32_t* sel,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap,
                                 void* ws, size_t ws_bytes, void* cuda_stream);
sea_status sea_attention_resized(const sea_shape* shape, int32_t row_widths, const void* Q, const void* K,
                                 const void* V, const float* omega, const float* W_dec,
                                 const float* A_hat_in, void* O, float* A_hat, int32_t* sel,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* P,
                                 void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * The paper's estimator head and output mixing, with weights given by the caller (the
 * benchmark workloads use random-init ones; trained weights would come from the paper's
 * distillation, which is outside this library).
 *
 * Sec. 3.1 "Attention Matrix Estimation" / "CNN Decoder", App. "Attention Estimator CNN":
 *   V_cat = [V_I ; V], V_I the identity I_d resized by nearest neighbour to T rows (causal
 *   shapes: the positional embedding pos_emb [T, d] takes its place);
 *   C_perf = FAVOR+(Q, K, V_cat) [T, 2d];  Z = relu([C_perf ; V] W_mu + b_mu) [T, d_hidden];
 *   Z_hat = relu(Z W_nu1 + b_nu1) W_nu2 + b_nu2 [T, (Kc/c_s) c_h], reshaped over the heads to an
 *   image [H c_h, T, Kc/c_s] (entry j Kc/c_s + x of head h: channel h c_h + j, column x);
 *   conv 3x3 (C -> C, relu; not causal: stride c_s along T), conv 3x3 (C -> C, relu), nearest
 *   resize to [C, T, Kc], conv 3x3 (C -> H), softmax over Kc.  Causal shapes keep the height and
 *   pad every layer with two rows above and none below (row t sees rows t-2 .. t); the width is
 *   padded by one on both sides.  Where the paper gives no detail (activations, layer counts of the
 *   MLPs, paddings, the channel order) these are this library's readings.
 * Sec. 3.1.1: s_prob = sigmoid(Z . w_prob + b_prob) re-scales the sparse attention's
 *   probabilities and output; C_avg is, not causal, the V-average weighted by the column means
 *   of A_hat resized to T keys, and, causal, the running mean of V; s_mix = sigmoid(Z . w_mix +
 *   b_mix); C_sea = s_mix (s_prob C) + (1 - s_mix) C_avg.
 *
 * All weights are fp32 device arrays, row-major: W_mu [3d, d_hidden], W_nu1 [d_hidden, d_hidden],
 * W_nu2 [d_hidden, (Kc/c_s) c_h], conv1_w / conv2_w [C, C, 3, 3], conv3_w [H, C, 3, 3] with
 * C = H c_h, biases alongside, w_prob / w_mix [d_hidden]; pos_emb [T, d] has the io dtype.
 * Requires Kc % c_s == 0 and, for shapes that are not causal, T % c_s == 0.
 *
 * sea_estimate_decoder writes A_hat [B, H, T, Kc] (rows sum to one) and Z [B, H, T, d_hidden].
 * sea_mix_output turns O (the output C of sea_sparse_attn for a mask from that A_hat) into
 * C_sea in place and multiplies P (may be NULL) by s_prob.  sea_attention_decoder chains
 * sea_estimate_decoder -> sea_topk_mask -> sea_sparse_attn -> sea_mix_output; A_hat, sel,
 * row_ptr, col_idx, P are optional outputs as for sea_attention.  Workspace:
 * sea_workspace_bytes_decoder().  The arithmetic of the head is plain fp32.
 */
typedef struct sea_decoder {
  int32_t d_hidden;           /* d' of the paper, 1 .. 1024 */
  int32_t c_s, c_h;           /* width reduction and channel expansion (the paper uses 2 and 4) */
  const float *W_mu, *b_mu;
  const float *W_nu1, *b_nu1, *W_nu2, *b_nu2;
  const float *conv1_w, *conv1_b, *conv2_w, *conv2_b, *conv3_w, *conv3_b;
  const void* pos_emb;        /* causal shapes only */
  const float *w_prob, *w_mix;
  float b_prob, b_mix;
} sea_decoder;

sea_status sea_workspace_bytes_decoder(const sea_shape* shape, const sea_decoder* dec, size_t* bytes);
sea_status sea_estimate_decoder(const sea_shape* shape, const sea_decoder* dec, const void* Q, const void* K,
                                const void* V, const float* omega, float* A_hat, float* Z,
                                void* ws, size_t ws_bytes, void* cuda_stream);
sea_status sea_mix_output(const sea_shape* shape, const sea_decoder* dec, const float* Z, const float* A_hat,
                          const void* V, const int32_t* row_ptr, void* O, void* P,
                          void* ws, size_t ws_bytes, void* cuda_stream);
sea_status sea_attention_decoder(const sea_shape* shape, const sea_decoder* dec, const void* Q, const void* K,
                                 const void* V, const float* omega, void* O, float* A_hat, int32_t* sel,
                                 int32_t* row_ptr, int32_t* col_idx, int64_t nnz_cap, void* P,
                                 void* ws, size_t ws_bytes, void* cuda_stream);

/*
 * sea_attention for callers whose tensors live in HOST memory.  hQ, hK, hV,
 * homega, hW_dec are copied to staging areas inside `ws`, the layer runs, and O
 * is copied back to hO.  The heads are independent, so the call is a pipeline
 * over up to eight slices of them: a slice is computed on `cuda_stream` while
 * the next slice's inputs arrive and the previous slice's O leaves on two
 * streams of the library's own (created, with a few events, by a host thread's
 * first call on a device and kept by that thread); this overlap needs pinned
 * host memory, pageable memory gives the same result serially.
 * Bytes needed: sea_workspace_host_bytes().  The call returns after all its work
 * has finished, so hO is valid on return.  Not for use during stream capture.
 * The paper has no counterpart; this is the end-to-end form of the call above.
 */
sea_status sea_workspace_host_bytes(const sea_shape* shape, size_t* bytes);
sea_status sea_attention_host(const sea_shape* shape, const void* hQ, const void* hK,
                              const void* hV, const float* homega, const float* hW_dec,
                              void* hO, void* ws, size_t ws_bytes, void* cuda_stream);

/* Copies the device status word of `ws` to *out (host) and synchronises the
 * stream; with `clear` != 0 the word is reset to zero afterwards. */
sea_status sea_device_status(void* ws, int32_t* out, int32_t clear, void* cuda_stream);

/* Number of kernel launches the last call of each entry point enqueued from
 * this thread (for benchmark bookkeeping). */
int32_t sea_last_launch_count(void);

/* Name of the kernel that the sparse stage of this thread's last call launched
 * ("none" before the first one): the stage chooses among several kernels by shape,
 * dtype and workspace, and a benchmark has to know which one it timed. */
const char* sea_last_sparse_kernel(void);
/* Floating-point operations that launch executes when they follow from the shape alone (the
 * tile kernel visits every key tile a query tile may see, whatever the mask); 0 for the per-row
 * kernels, whose work is 4 * nnz * d. */
double sea_last_sparse_flops(void);

const char* sea_status_string(sea_status s);

#ifdef __cplusplus
}
#endif
#endif /* SEA_H_ */

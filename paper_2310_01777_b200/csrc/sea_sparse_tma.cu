// Sparse attention over runs of keys, staged by TMA (bf16, mask given as `sel`, r = 16, 32, 64, ...).
//
// Same arithmetic as the gather kernel in sea_sparse.cu (Sec. 3.1.1: scores at the mask's
// positions, row softmax, product with V; one warp per query row, tensor-core tiles with 16
// keys on the M side), but the selected runs are fetched as whole 16-key blocks (2 KB of K,
// 2 KB of V) by cp.async.bulk.tensor into a small per-warp ring of 128B-swizzled shared-memory
// slots and read back with ldmatrix, conflict-free.  This takes the gather off the load/store
// pipe, whose wavefront rate bounded the gather kernel (a fragment-shaped global load touches
// 2 to 4 lines per quarter-warp), and leaves one 128-byte wavefront per 128 bytes of K or V.
//
// The grid is persistent: every warp walks rows wg, wg + W, wg + 2W, ... (W = warps in the
// grid) and keeps ONE stream of block copies running across row boundaries - for each row all
// its K blocks, then all its V blocks - so the ring stays full while a row's softmax runs and
// while the next row starts.  The warp is its own producer: after a block has been read, lane 0
// issues the copy that is kSlots ahead in the stream; the row metadata that the producer needs
// (row_ptr pair, selected columns) is fetched one row early into registers.  Waits are bounded by
// a clock: when one runs out the warp sets SEA_DEV_TIMEOUT in the status word, waits (bounded again)
// for the copies it still has in flight, writes zeros to the output rows it leaves undone and stops.
#include <cuda.h>

#include "sea_common.cuh"
#include "sea_tc.cuh"

namespace sea {
namespace {

using namespace tc;

constexpr int kWarps = 8;
constexpr int kSlots = 4;              // ring depth per warp (power of two)
constexpr int kSlotBytes = 16 * 128;   // 16 keys x 64 bf16
constexpr int kMaxBlocks = 64;         // 16-key blocks per row (k_hat * r <= 1024, so k_hat <= 64)

struct alignas(1024) WarpRing {
  unsigned char slot[kSlots][kSlotBytes];
};

__device__ __forceinline__ float ex2(float x) {  // 2^x for x <= 0 (flushes denormal results to zero)
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Dynamic shared memory: kWarps rings (1024-byte aligned), then per warp the scores / packed
// probabilities (chunk floats) and the ring's barriers.
template <bool kWriteP>
__global__ void __launch_bounds__(kWarps * 32)
sparse_attn_blocks_tma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                              const __nv_bfloat16* __restrict__ Q, const int32_t* __restrict__ row_ptr,
                              const int32_t* __restrict__ sel, __nv_bfloat16* __restrict__ O,
                              __nv_bfloat16* __restrict__ P, int32_t* __restrict__ status, int rows, int seq_len,
                              int r, int k_hat, float scale_log2, int chunk) {
  extern __shared__ unsigned char smem_dyn[];
  // the swizzle pattern is a function of the shared-memory address: slots start on 1024-byte lines
  unsigned char* smem_raw = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = smem_u32(smem_raw) + warp * (uint32_t)sizeof(WarpRing);
  unsigned char* tail = smem_raw + sizeof(WarpRing) * kWarps;
  float* sc = reinterpret_cast<float*>(tail) + warp * chunk;
  const uint32_t bars = smem_u32(tail + sizeof(float) * kWarps * chunk) + warp * kSlots * 8;
  uint2* pairs = reinterpret_cast<uint2*>(sc);

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kSlots; ++s) mbar_init(bars + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();

  const int stride = gridDim.x * kWarps;
  const int wg = blockIdx.x * kWarps + warp;
  if (wg >= rows) return;
  const int g = lane >> 2, t = lane & 3;
  const int rb_shift = 31 - __clz(r >> 4);  // log2 of the 16-key blocks per selected column

  // ---- producer cursor: the next copy of this warp's stream ---------------------------------
  int p_row = wg - stride;     // row whose copies are being issued (none yet)
  int p_i = 0, p_nb = 0;       // next copy within the row: K blocks 0..nb-1, then V blocks
  uint32_t p_s = 0;            // copies issued so far
  int p_key0 = 0;              // first key row of the head in the [B*H*T][64] view
  int p_sel0 = 0, p_sel1 = 0;  // lane c holds sel[c] and sel[c+32] of p_row
  // metadata of the row after p_row, fetched early
  int nf_rp0 = 0, nf_rp1 = 0, nf_sel0 = 0, nf_sel1 = 0;
  auto fetch_meta = [&](int row) {
    if (row < rows) {
      nf_rp0 = __ldg(row_ptr + row);
      nf_rp1 = __ldg(row_ptr + row + 1);
      const int32_t* ms = sel + (size_t)row * k_hat;
      nf_sel0 = lane < k_hat ? __ldg(ms + lane) : 0;
      nf_sel1 = lane + 32 < k_hat ? __ldg(ms + lane + 32) : 0;
    }
  };
  fetch_meta(wg);
  uint32_t c_s = 0;  // copies consumed so far

  // Issues the next copy of the stream if the ring has a free slot.  Executed by all lanes
  // together; called once after every consumed block (and kSlots times to prime the ring).
  auto pump = [&]() {
    if (p_s - c_s >= (uint32_t)kSlots) return;
    while (p_i == 2 * p_nb) {  // next row of the stream (rows without keys are skipped)
      if (p_row >= rows - stride) { p_row = rows; p_nb = 0; p_i = 0; return; }
      p_row += stride;
      p_nb = (nf_rp1 - nf_rp0 + 15) >> 4;
      p_i = 0;
      p_sel0 = nf_sel0;
      p_sel1 = nf_sel1;
      p_key0 = (p_row / seq_len) * seq_len;
      fetch_meta(p_row + stride);
    }
    const bool is_k = p_i < p_nb;
    const int blk = is_k ? p_i : p_i - p_nb;
    const int c = blk >> rb_shift;
    const int col = __shfl_sync(0xffffffffu, c < 32 ? p_sel0 : p_sel1, c);
    if (lane == 0) {
      const uint32_t slot = p_s & (kSlots - 1);
      const uint32_t bar = bars + 8 * slot;
      mbar_expect_tx(bar, kSlotBytes);
      tma_load_2d(ring + slot * kSlotBytes, is_k ? &map_k : &map_v, 0, p_key0 + col * r + ((blk - (c << rb_shift)) << 4), bar);
    }
    ++p_i;
    ++p_s;
  };

  // ldmatrix lane roles.  K (plain): matrix mi -> rows 8*(mi&1).., chunk 2s + (mi>>1).
  // V (transposed): matrix mi -> rows 8*(mi>>1).., chunk 2i + (mi&1).  Offsets inside a slot:
  uint32_t k_off[4], v_off[4];
  {
    const int mi = lane >> 3, lr = lane & 7;
    const int k_row = lr + 8 * (mi & 1), v_row = lr + 8 * (mi >> 1);
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      k_off[s] = k_row * 128 + (((2 * s + (mi >> 1)) ^ (k_row & 7)) << 4);
      v_off[s] = v_row * 128 + (((2 * s + (mi & 1)) ^ (v_row & 7)) << 4);
    }
  }

  // consumer's own early fetch: row_ptr pair and q of the next row
  int n_rp0 = __ldg(row_ptr + wg), n_rp1 = __ldg(row_ptr + wg + 1);
  uint32_t n_qw[8];
  auto fetch_q = [&](int row) {
    const uint32_t* qp = reinterpret_cast<const uint32_t*>(Q + (size_t)row * kHeadDim) + t;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      n_qw[2 * s] = __ldg(qp + 8 * s);
      n_qw[2 * s + 1] = __ldg(qp + 8 * s + 4);
    }
  };
  fetch_q(wg);
#pragma unroll
  for (int i = 0; i < kSlots; ++i) pump();

  bool ok = true;
  int row = wg;
  for (; row < rows; row += stride) {
    const int base = n_rp0, n = n_rp1 - n_rp0;
    uint32_t qw[8];  // q as the B operand of every k-step: b0 = dims 16s+2t.., b1 = dims 16s+8+2t..
#pragma unroll
    for (int i = 0; i < 8; ++i) qw[i] = n_qw[i];
    if (row < rows - stride) {
      n_rp0 = __ldg(row_ptr + row + stride);
      n_rp1 = __ldg(row_ptr + row + stride + 1);
      fetch_q(row + stride);
    }
    __nv_bfloat16* out = O + (size_t)row * kHeadDim;
    if (n <= 0) {
      out[16 * t + g] = __float2bfloat16_rn(0.f);
      out[16 * t + 8 + g] = __float2bfloat16_rn(0.f);
      continue;
    }
    const int nb = (n + 15) >> 4;  // 16-key blocks of this row (only the last may be cut)
    const int cn16 = nb * 16;
    float mx = -INFINITY;
    for (int b = 0; b < nb; ++b) {
      const uint32_t slot = c_s & (kSlots - 1);
      ok = ok && mbar_wait_alone(bars + 8 * slot, (c_s / kSlots) & 1);
      const uint32_t sbase = ring + slot * kSlotBytes;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        uint32_t a[4];
        ldsm4(a, sbase + k_off[s]);
        mma16816(acc, a, qw[2 * s], qw[2 * s + 1]);
      }
      const int p0 = 16 * b;
      const float s0 = p0 + g < n ? acc[0] * scale_log2 : -INFINITY;
      const float s1 = p0 + g + 8 < n ? acc[2] * scale_log2 : -INFINITY;
      mx = fmaxf(mx, fmaxf(s0, s1));
      if (t == 0) {
        sc[p0 + g] = s0;
        sc[p0 + g + 8] = s1;
      }
      __syncwarp();
      ++c_s;
      pump();
    }
    ok = __all_sync(0xffffffffu, ok);  // a wait that ran out ends the warp's work after this row's K pass
    if (!ok) break;
    mx = warp_max(mx);

    float part = 0.f;
    for (int u = lane; u < cn16 / 2; u += 32) {
      float2 s = reinterpret_cast<float2*>(sc)[u];
      s.x = ex2(s.x - mx);
      s.y = ex2(s.y - mx);
      part += s.x + s.y;
      reinterpret_cast<float2*>(sc)[u] = s;
    }
    const float inv = 1.f / warp_sum(part);
    for (int u = lane; u < cn16 / 2; u += 32) {
      const float2 e = reinterpret_cast<float2*>(sc)[u];
      const float p0 = e.x * inv, p1 = e.y * inv;
      const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
      const uint32_t hw = *reinterpret_cast<const uint32_t*>(&h);
      const uint32_t lw = pack_bf16(p0 - __bfloat162float(h.x), p1 - __bfloat162float(h.y));
      pairs[u] = make_uint2(hw, lw);
      if (kWriteP) {
        __nv_bfloat16* pp = P + (size_t)base + 2 * u;
        if (2 * u < n) pp[0] = h.x;
        if (2 * u + 1 < n) pp[1] = h.y;
      }
    }
    __syncwarp();

    float acc_o[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc_o[i][e] = 0.f;
    for (int b = 0; b < nb; ++b) {
      const uint32_t slot = c_s & (kSlots - 1);
      ok = ok && mbar_wait_alone(bars + 8 * slot, (c_s / kSlots) & 1);
      const uint32_t sbase = ring + slot * kSlotBytes;
      const uint2 pa = pairs[8 * b + t];      // positions 16b+2t, 16b+2t+1
      const uint2 pb = pairs[8 * b + 4 + t];  // positions 16b+8+2t, 16b+9+2t
#pragma unroll
      for (int i = 0; i < 4; ++i) {  // tile i: rows g / g+8 = dims 16i+g / 16i+8+g
        uint32_t a[4];
        ldsm4_t(a, sbase + v_off[i]);
        mma16816(acc_o[i], a, pa.x, pb.x);
        mma16816(acc_o[i], a, pa.y, pb.y);
      }
      __syncwarp();
      ++c_s;
      pump();
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) break;
    // every lane of a quad holds the same sums; lane t writes tile t: dims 16t + g and 16t + 8 + g
    {
      float lo = acc_o[0][0], hi = acc_o[0][2];
      if (t == 1) { lo = acc_o[1][0]; hi = acc_o[1][2]; }
      if (t == 2) { lo = acc_o[2][0]; hi = acc_o[2][2]; }
      if (t == 3) { lo = acc_o[3][0]; hi = acc_o[3][2]; }
      out[16 * t + g] = __float2bfloat16_rn(lo);
      out[16 * t + 8 + g] = __float2bfloat16_rn(hi);
    }
  }
  if (!ok) {
    if (lane == 0) atomicOr(status, SEA_DEV_TIMEOUT);
    // copies already issued still land in this CTA's shared memory: wait for them before leaving
    for (; c_s != p_s; ++c_s) mbar_wait_drain(bars + 8 * (c_s & (kSlots - 1)), (c_s / kSlots) & 1);
    for (; row < rows; row += stride) {  // the rows this warp leaves undone read as zero
      __nv_bfloat16* out = O + (size_t)row * kHeadDim;
      out[2 * lane] = __float2bfloat16_rn(0.f);
      out[2 * lane + 1] = __float2bfloat16_rn(0.f);
    }
  }
}

template <bool kWriteP>
sea_status launch_tma(const sea_shape& s, const CUtensorMap& map_k, const CUtensorMap& map_v, const __nv_bfloat16* Q,
                      const int32_t* row_ptr, const int32_t* sel, __nv_bfloat16* O, __nv_bfloat16* P, int32_t* status,
                      cudaStream_t st) {
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
  const int chunk = (s.k_hat * r + 63) / 64 * 64;
  const size_t smem = 1024 + sizeof(WarpRing) * kWarps + sizeof(float) * kWarps * chunk + 8 * kWarps * kSlots;
  auto kern = sparse_attn_blocks_tma_kernel<kWriteP>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return SEA_ERR_CUDA;
  int dev = 0, sms = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kWarps * 32, smem) != cudaSuccess || per_sm < 1)
    return SEA_ERR_CUDA;
  const int want = (rows + kWarps - 1) / kWarps;
  const int grid = want < sms * per_sm ? want : sms * per_sm;  // persistent: one wave of CTAs
  const float scale = s.scale != 0.f ? s.scale : 0.125f;
  kern<<<grid, kWarps * 32, smem, st>>>(map_k, map_v, Q, row_ptr, sel, O, P, status, rows, s.T, r, s.k_hat,
                                        scale * 1.4426950408889634f, chunk);
  return check_launch();
}

}  // namespace

bool sparse_attn_tma_applicable(const sea_shape& s, const int32_t* sel, const int32_t* status) {
  const int r = s.T / s.Kc;
  return s.io == SEA_BF16 && sel != nullptr && status != nullptr && r % 16 == 0 && ((r >> 4) & ((r >> 4) - 1)) == 0 && s.k_hat <= kMaxBlocks &&
         (long long)s.k_hat * r <= 16 * kMaxBlocks && encode_fn() != nullptr;
}

sea_status launch_sparse_attn_tma(const sea_shape& s, const void* Q, const void* K, const void* V,
                                  const int32_t* row_ptr, const int32_t* sel, void* O, void* P,
                                  int32_t* status, cudaStream_t st) {
  using T = __nv_bfloat16;
  const unsigned long long rows = (unsigned long long)s.B * s.H * s.T;
  CUtensorMap map_k, map_v;
  if (!make_rows_map_bf16(&map_k, K, rows, 16) || !make_rows_map_bf16(&map_v, V, rows, 16)) return SEA_ERR_CUDA;
  Launch::sparse_kernel() = "sparse_attn_blocks_tma_kernel";
  Launch::sparse_flops() = 0.0;  // depends on the mask: 4 * nnz * d
  if (P) return launch_tma<true>(s, map_k, map_v, (const T*)Q, row_ptr, sel, (T*)O, (T*)P, status, st);
  return launch_tma<false>(s, map_k, map_v, (const T*)Q, row_ptr, sel, (T*)O, nullptr, status, st);
}

}  // namespace sea

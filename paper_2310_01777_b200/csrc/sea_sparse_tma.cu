// Sparse attention over runs of keys, staged by TMA (bf16, mask given as `sel`, r % 16 == 0).
//
// Same arithmetic as the gather kernel in sea_sparse.cu (Sec. 3.1.1: scores at the mask's
// positions, row softmax, product with V; one warp per query row, tensor-core tiles with 16
// keys on the M side), but the selected runs are fetched as whole 16-key blocks (2 KB of K,
// 2 KB of V) by cp.async.bulk.tensor into a small per-warp ring of 128B-swizzled shared-memory
// slots and read back with ldmatrix, conflict-free.  This takes the gather off the load/store
// pipe, whose wavefront rate bounded the gather kernel (a fragment-shaped global load touches
// 2 to 4 lines per quarter-warp), and leaves one 128-byte wavefront per 128 bytes of K or V.
//
// Each warp drives its own ring: lane 0 issues the copies, every lane waits on the slot's
// mbarrier, and a slot is refilled right after the warp has read it.  All K blocks of the row
// are consumed first (scores), then all V blocks, so V streams in during the softmax.  Waits
// are bounded: a wait that runs out sets SEA_DEV_TIMEOUT in the status word and the warp
// leaves its row zeroed.
#include <cuda.h>

#include "sea_common.cuh"

namespace sea {
namespace {

constexpr int kWarps = 8;
constexpr int kSlots = 4;              // ring depth per warp
constexpr int kSlotBytes = 16 * 128;   // 16 keys x 64 bf16
constexpr int kMaxBlocks = 64;         // 16-key blocks per row (k_hat * r <= 1024)
constexpr uint32_t kWaitPolls = 1u << 16;

struct alignas(1024) WarpRing {
  unsigned char slot[kSlots][kSlotBytes];
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait for the given phase parity; false when the poll budget ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const uint32_t a = smem_u32(bar);
  for (uint32_t i = 0; i < kWaitPolls; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(a), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
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

// Dynamic shared memory: kWarps rings (1024-byte aligned), then per warp: scores / packed
// probabilities (chunk floats), block starts (kMaxBlocks ints), barriers (kSlots).
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
  WarpRing& ring = reinterpret_cast<WarpRing*>(smem_raw)[warp];
  unsigned char* tail = smem_raw + sizeof(WarpRing) * kWarps;
  float* sc = reinterpret_cast<float*>(tail) + warp * chunk;
  int32_t* jstart = reinterpret_cast<int32_t*>(tail + sizeof(float) * kWarps * chunk) + warp * kMaxBlocks;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tail + sizeof(float) * kWarps * chunk + sizeof(int32_t) * kWarps * kMaxBlocks) +
                   warp * kSlots;
  uint2* pairs = reinterpret_cast<uint2*>(sc);

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kSlots; ++s) mbar_init(bars + s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();

  const int row = blockIdx.x * kWarps + warp;
  if (row >= rows) return;
  const int g = lane >> 2, t = lane & 3;
  const int bh = row / seq_len;
  const int base = __ldg(row_ptr + row);
  const int n = __ldg(row_ptr + row + 1) - base;
  __nv_bfloat16* out = O + (size_t)row * kHeadDim;
  auto zero_row = [&]() {
    if (t == 0) *reinterpret_cast<uint4*>(out + 8 * g) = make_uint4(0u, 0u, 0u, 0u);
  };
  if (n <= 0) {
    zero_row();
    return;
  }
  const int nb = (n + 15) >> 4;      // 16-key blocks of this row (only the last may be cut)
  const int total = 2 * nb;          // K blocks, then V blocks
  {
    const int rb = r >> 4;           // blocks per selected column
    const int32_t* my_sel = sel + (size_t)row * k_hat;
    for (int s = lane; s < nb; s += 32) {
      const int c = s / rb;
      jstart[s] = bh * seq_len + __ldg(my_sel + c) * r + (s - c * rb) * 16;
    }
  }
  __syncwarp();
  auto issue = [&](int i) {  // lane 0 only
    uint64_t* bar = bars + (i % kSlots);
    mbar_expect_tx(bar, kSlotBytes);
    const bool is_k = i < nb;
    tma_load_2d(ring.slot[i % kSlots], is_k ? &map_k : &map_v, 0, jstart[is_k ? i : i - nb], bar);
  };
  if (lane == 0) {
    for (int i = 0; i < min(kSlots, total); ++i) issue(i);
  }

  // q as the B operand of every k-step: b0 = dims 16s+2t.., b1 = dims 16s+8+2t..
  uint32_t qw[8];
  {
    const uint32_t* qp = reinterpret_cast<const uint32_t*>(Q + (size_t)row * kHeadDim) + t;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      qw[2 * s] = __ldg(qp + 8 * s);
      qw[2 * s + 1] = __ldg(qp + 8 * s + 4);
    }
  }

  const int cn16 = nb * 16;
  bool ok = true;
  float mx = -INFINITY;
  // ldmatrix lane roles.  K (plain): matrix mi -> rows 8*(mi&1).., chunk 2s + (mi>>1).
  // V (transposed): matrix mi -> rows 8*(mi>>1).., chunk 2i + (mi&1).
  const int mi = lane >> 3, lr = lane & 7;
  const int k_row = lr + 8 * (mi & 1), k_chk = mi >> 1;
  const int v_row = lr + 8 * (mi >> 1), v_chk = mi & 1;
  for (int b = 0; b < nb; ++b) {
    if (!__all_sync(0xffffffffu, mbar_wait(bars + (b % kSlots), (b / kSlots) & 1))) { ok = false; break; }
    const uint32_t sbase = smem_u32(ring.slot[b % kSlots]) + k_row * 128;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      uint32_t a[4];
      ldsm4(a, sbase + (((2 * s + k_chk) ^ (k_row & 7)) << 4));
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
    if (lane == 0 && b + kSlots < total) issue(b + kSlots);
  }
  if (!ok) {
    if (lane == 0) atomicOr(status, SEA_DEV_TIMEOUT);
    zero_row();
    return;
  }
  mx = warp_max(mx);

  float part = 0.f;
  for (int u = lane; u < cn16 / 2; u += 32) {
    float2 s = reinterpret_cast<float2*>(sc)[u];
    s.x = exp2f(s.x - mx);
    s.y = exp2f(s.y - mx);
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
    const int i_load = nb + b;
    if (!__all_sync(0xffffffffu, mbar_wait(bars + (i_load % kSlots), (i_load / kSlots) & 1))) { ok = false; break; }
    const uint32_t sbase = smem_u32(ring.slot[i_load % kSlots]) + v_row * 128;
    const uint2 pa = pairs[8 * b + t];      // positions 16b+2t, 16b+2t+1
    const uint2 pb = pairs[8 * b + 4 + t];  // positions 16b+8+2t, 16b+9+2t
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // tile i: rows g / g+8 = dims 16i+g / 16i+8+g
      uint32_t a[4];
      ldsm4_t(a, sbase + (((2 * i + v_chk) ^ (v_row & 7)) << 4));
      mma16816(acc_o[i], a, pa.x, pb.x);
      mma16816(acc_o[i], a, pa.y, pb.y);
    }
    __syncwarp();
    if (lane == 0 && i_load + kSlots < total) issue(i_load + kSlots);
  }
  if (!ok) {
    if (lane == 0) atomicOr(status, SEA_DEV_TIMEOUT);
    zero_row();
    return;
  }
  // every lane of a quad holds the same sums; lane t writes the two 8-dim groups 2t and 2t+1:
  // tile i = t (dims 16t + g and 16t + 8 + g)
  {
    float lo = acc_o[0][0], hi = acc_o[0][2];
    if (t == 1) { lo = acc_o[1][0]; hi = acc_o[1][2]; }
    if (t == 2) { lo = acc_o[2][0]; hi = acc_o[2][2]; }
    if (t == 3) { lo = acc_o[3][0]; hi = acc_o[3][2]; }
    out[16 * t + g] = __float2bfloat16_rn(lo);
    out[16 * t + 8 + g] = __float2bfloat16_rn(hi);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// [total_rows][64] bf16, boxes of 16 rows x 64 columns, 128-byte swizzle.
bool make_rows_map(CUtensorMap* map, const void* ptr, unsigned long long total_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {kHeadDim, total_rows};
  const cuuint64_t strides[1] = {kHeadDim * sizeof(__nv_bfloat16)};
  const cuuint32_t box[2] = {kHeadDim, 16};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool sparse_attn_tma_applicable(const sea_shape& s, const int32_t* sel, const int32_t* status) {
  const int r = s.T / s.Kc;
  return s.io == SEA_BF16 && sel != nullptr && status != nullptr && r % 16 == 0 &&
         (long long)s.k_hat * r <= 16 * kMaxBlocks && encode_fn() != nullptr;
}

sea_status launch_sparse_attn_tma(const sea_shape& s, const void* Q, const void* K, const void* V,
                                  const int32_t* row_ptr, const int32_t* sel, void* O, void* P,
                                  int32_t* status, cudaStream_t st) {
  using T = __nv_bfloat16;
  const int rows = s.B * s.H * s.T;
  const int r = s.T / s.Kc;
  CUtensorMap map_k, map_v;
  if (!make_rows_map(&map_k, K, (unsigned long long)rows) || !make_rows_map(&map_v, V, (unsigned long long)rows))
    return SEA_ERR_CUDA;
  const int chunk = (s.k_hat * r + 63) / 64 * 64;
  const size_t smem = 1024 + sizeof(WarpRing) * kWarps + sizeof(float) * kWarps * chunk + sizeof(int32_t) * kWarps * kMaxBlocks +
                      sizeof(uint64_t) * kWarps * kSlots;
  const float scale = s.scale != 0.f ? s.scale : 0.125f;
  const float scale_log2 = scale * 1.4426950408889634f;
  const int grid = (rows + kWarps - 1) / kWarps;
  if (P) {
    if (cudaFuncSetAttribute(sparse_attn_blocks_tma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SEA_ERR_CUDA;
    sparse_attn_blocks_tma_kernel<true><<<grid, kWarps * 32, smem, st>>>(map_k, map_v, (const T*)Q, row_ptr, sel, (T*)O, (T*)P,
                                                                         status, rows, s.T, r, s.k_hat, scale_log2, chunk);
  } else {
    if (cudaFuncSetAttribute(sparse_attn_blocks_tma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SEA_ERR_CUDA;
    sparse_attn_blocks_tma_kernel<false><<<grid, kWarps * 32, smem, st>>>(map_k, map_v, (const T*)Q, row_ptr, sel, (T*)O, nullptr,
                                                                          status, rows, s.T, r, s.k_hat, scale_log2, chunk);
  }
  return check_launch();
}

}  // namespace sea

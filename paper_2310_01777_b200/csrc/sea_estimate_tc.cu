// Attention estimation for bf16 inputs on the 5th-generation tensor cores (tcgen05, accumulators
// in tensor memory, operands staged by TMA).
//
//   x = u d^(-1/4);  phi_f(u) = exp(omega_f.x - |x|^2/2) / sqrt(m)          (Sec. 3 "Performer (FAVOR+)")
//   C_i = sum_j phi(q_i).phi(k_j) v_j / sum_j phi(q_i).phi(k_j);  A_hat = C W_dec   (Sec. 3.1, one
//   linear head in place of the trained decoder)
//
// The sequence is cut into chunks of 128 rows:
//   1. favor_state_tc_kernel:  S_c = phi(K_c)^T V_c  [m x 64]  and  z_c = phi(K_c)^T 1  [m], one CTA
//                              per (chunk, head), two CTAs per SM; causal: phi(K_c) is kept as
//                              ready-made operand tiles for kernel 3
//   2. favor_scan_tc_kernel:   exclusive prefix over the chunks of a head (causal) or the total,
//                              in a fixed order, written as bf16 head / remainder MMA operands
//   3. favor_output_tc_kernel: num = phi(Q_c) S + (phi(Q_c) phi(K_c)^T . tril) V_c, den likewise,
//                              C = num / den, A_hat = C W_dec; persistent CTAs that copy the next
//                              chunk's tiles in while the current one is computed, A_hat leaves
//                              through TMA stores
// Precision: the estimate has to agree with fp64 to 1e-3 and the feature map exponentiates a
// projection of magnitude ~10, so every fp32 operand is carried as a bf16 head plus a bf16
// remainder (2^-17 relative) and a product A B is evaluated as A_hi B_hi + A_hi B_lo + A_lo B_hi;
// Q, K and V are exact in bf16.  d^(-1/4) is folded into omega beforehand.
//
// Inside a CTA eight row warps own the 128 rows (a row and half of a tile's columns per thread:
// exponentials, masks, normalisers, splits) and one thread of a ninth warp issues the copies and
// the MMAs; the phases of a chunk follow one another through mbarriers.  Every wait is bounded; a
// wait that runs out sets SEA_DEV_TIMEOUT and the CTA drains and leaves.
#include "sea_common.cuh"
#include "sea_select.cuh"
#include "sea_tc.cuh"

namespace sea {
namespace {

using namespace tc;

constexpr int kRows = 128;                 // rows per chunk
constexpr int kTileBytes = kRows * 128;    // 128 rows x 64 bf16
constexpr int kParts = 2;                  // row warpgroups: each takes every kParts-th 32-column chunk of a tile
constexpr int kRowWarps = 4 * kParts;
constexpr int kThreads = 32 * (kRowWarps + 1);
// The output kernel has two more warpgroups: the control warp's (copies and MMAs; three warps idle)
// and one that selects the k_hat largest entries of every row of the A_hat tile while it is in
// tensor memory.  Registers per thread after the warpgroups re-balance: a warpgroup can only grow
// by what the others of the CTA have given back.
constexpr int kThreadsOut = 128 * (kParts + 2);
constexpr int kRegsOutLaunch = 65536 / kThreadsOut;
constexpr int kRegsOutRow = 168, kRegsOutCtl = 104, kRegsOutSel = 72;
static_assert(128 * (kParts * kRegsOutRow + kRegsOutCtl + kRegsOutSel) <= kRegsOutLaunch * kThreadsOut,
              "register re-balance exceeds the launch allocation");
constexpr int kWTile = 128;                // decoder columns per pass

// ---- operand preparation -----------------------------------------------------------------
// omega * d^(-1/4) as bf16 head / remainder [2][MP][64] (rows >= m zero) and W_dec as
// [2][64][KcP] (columns >= Kc zero).
__global__ void favor_prep_tc_kernel(const float* __restrict__ omega, const float* __restrict__ W_dec,
                                     __nv_bfloat16* __restrict__ om, __nv_bfloat16* __restrict__ wd, int m, int MP,
                                     int Kc, int KcP, float in_scale) {
  const int n_om = MP * kHeadDim, n_w = kHeadDim * KcP;
  for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < n_om + n_w; v += gridDim.x * blockDim.x) {
    float x;
    __nv_bfloat16 *hi, *lo;
    if (v < n_om) {
      x = (v / kHeadDim) < m ? omega[v] * in_scale : 0.f;
      hi = om + v;
      lo = om + n_om + v;
    } else {
      const int u = v - n_om, e = u / KcP, c = u - e * KcP;
      x = c < Kc ? W_dec[(size_t)e * Kc + c] : 0.f;
      hi = wd + u;
      lo = wd + n_w + u;
    }
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    *hi = h;
    *lo = __float2bfloat16_rn(x - __bfloat162float(h));
  }
}

// ---- pieces shared by the two chunk kernels ----------------------------------------------------
// |u|^2 / 16 = |x|^2 / 2 of row r of a [128][64] bf16 tile staged by a tiled copy with the
// 128-byte swizzle (16-byte piece j of row r sits at piece j ^ (r & 7) of the row's 128 bytes).
__device__ __forceinline__ float half_sq_norm_swizzled(const unsigned char* tile, int r) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint4 t = *reinterpret_cast<const uint4*>(tile + r * 128 + ((i ^ (r & 7)) << 4));
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
      s = fmaf(lo, lo, fmaf(hi, hi, s));
    }
  }
  return s * (1.f / 16.f);
}

// |u|^2 / 16 = |x|^2 / 2 of one row of a bf16 [.][64] matrix.
__device__ __forceinline__ float half_sq_norm(const __nv_bfloat16* row) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(row) + i);
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
      s = fmaf(lo, lo, fmaf(hi, hi, s));
    }
  }
  return s * (1.f / 16.f);
}

// Features of 32 projections (columns 32c .. 32c+31 of the row's projection tile):
// exp(e - |x|^2/2) / sqrt(m) = 2^(e log2(e) + bias) with the row's bias = -(|x|^2/2) log2(e) -
// log2(m)/2, or -inf for a row outside the sequence (2^-inf = 0); padded features give zero.
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float feature_bias(float half_sq, bool row_ok, int m) {
  return row_ok ? -half_sq * 1.4426950408889634f - 0.5f * log2f((float)m) : -INFINITY;
}
__device__ __forceinline__ void features32(const uint32_t (&e)[32], float (&phi)[32], float bias, int c, int m) {
  const float2 l2e = make_float2(1.4426950408889634f, 1.4426950408889634f), b2 = make_float2(bias, bias);
  if (32 * c + 32 <= m) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float2 x = __ffma2_rn(make_float2(__uint_as_float(e[2 * i]), __uint_as_float(e[2 * i + 1])), l2e, b2);
      phi[2 * i] = ex2f(x.x);
      phi[2 * i + 1] = ex2f(x.y);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i)
      phi[i] = 32 * c + i < m ? ex2f(fmaf(__uint_as_float(e[i]), 1.4426950408889634f, bias)) : 0.f;
  }
}
__device__ __forceinline__ void split32(const float (&x)[32], uint32_t (&hi)[16], uint32_t (&lo)[16]) {
#pragma unroll
  for (int i = 0; i < 16; ++i) split_pair(x[2 * i], x[2 * i + 1], hi[i], lo[i]);
}
// Writes 32 values of row `r` (columns 32c ..) of a [128][MP] operand kept as 64-column atoms of
// 128-byte rows with the 128-byte swizzle (atom stride 16 KB).
__device__ __forceinline__ void store_row32_swizzled(unsigned char* base, int r, int c, const uint32_t (&w)[16]) {
  unsigned char* row = base + (c >> 1) * kTileBytes + r * 128;
  const int q0 = (c & 1) * 4;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    *reinterpret_cast<uint4*>(row + (((q0 + j) ^ (r & 7)) << 4)) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
}
// Column offset (32-bit tensor-memory columns) of contraction step ks inside an operand written
// as [16 head words | 16 remainder words] per 32 values; the remainder sits 16 columns further on.
__device__ __forceinline__ uint32_t a_col(int ks) { return 32u * (ks >> 1) + 8u * (ks & 1); }

// AND of a predicate over the row threads (named barrier 1); also orders their memory accesses.
__device__ __forceinline__ bool rows_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.and.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(r) : "r"((uint32_t)ok), "n"(32 * kRowWarps) : "memory");
  return r != 0;
}
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
  fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];\n"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;\n" ::: "memory"); }
struct EstParams {
  const __nv_bfloat16 *Q, *K;   // for the rows' norms
  float* state_s;               // [BH][nchunk][MP][64]
  float* state_z;               // [BH][nchunk][MP]
  const float* z_prefix;        // [BH][nchunk][MP]
  float* A_hat;
  int32_t* status;
  int BH, T, m, Kc, nchunk, causal;
  int tma_store;                // A_hat leaves through TMA stores (its rows are 16-byte multiples)
  // selection inside the output kernel (Kc <= 128): null when the caller selects elsewhere
  int32_t* sel;                 // [BH * T][k_hat] ascending columns
  int32_t* row_counts;          // [BH * T] keys per row after up-sampling (null: not wanted)
  uint32_t* mask_bits;          // [BH * T][ceil(Kc / 32)] (null: not wanted)
  int k_hat, r;
};

template <int kRegs>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegs)); }
template <int kRegs>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegs)); }

// ---- kernel 1: chunk key states ---------------------------------------------------------------
enum { kS_Load = 0, kS_E, kS_Phi, kS_S, kS_Drain, kS_NumBars };

template <int MP>
__global__ void __launch_bounds__(kThreads, 2)
favor_state_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const __grid_constant__ CUtensorMap map_om, const __grid_constant__ CUtensorMap map_phi,
                      const EstParams p) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* sm = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  // phi(K) (head 32 KB, remainder 32 KB: [2 atoms][128 keys][64 f]) is written only after the
  // projections are complete, over the K tile and omega' that fed them: two CTAs fit an SM
  unsigned char* sPhi = sm;                            // 64 KB
  unsigned char* sK = sm;                              // 16 KB
  unsigned char* sOm = sK + kTileBytes;                // head 16 KB, remainder 16 KB ([MP][64])
  unsigned char* sV = sPhi + 4 * kTileBytes;           // 16 KB
  unsigned char* sOnes = sV + kTileBytes;              // 16 rows x 128 B of 1.0
  unsigned char* tail = sOnes + 2048;
  const uint32_t bars = smem_u32(tail);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kS_NumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8 * kS_NumBars + 4);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  constexpr uint32_t kColE = 0, kColS = 128, kColZ = 192, kCols = 256;

  const int chunk = blockIdx.x, bh = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    mbar_init(bar(kS_Load), 1);
    mbar_init(bar(kS_E), 1);
    mbar_init(bar(kS_Phi), kRowWarps);
    mbar_init(bar(kS_S), 1);
    mbar_init(bar(kS_Drain), 1);
    *abort_flag = 0;
    mbar_init_fence();
  }
  for (int i = tid; i < 2048 / 4; i += kThreads) reinterpret_cast<uint32_t*>(sOnes)[i] = 0x3f803f80u;
  fence_async_smem();
  if (warp == kRowWarps) tmem_alloc(smem_u32(tmem_slot), kCols);
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == kRowWarps) {
    {
      // ------------------------------------------------------------ copies and MMAs: the whole warp
      // walks the phases (so that descriptors stay in uniform registers), one elected lane issues
      const bool leader = elect_one();
      bool ok = true;
      if (leader) {
        mbar_expect_tx(bar(kS_Load), 2 * kTileBytes + 2 * MP * 128);
        tma_load_3d(smem_u32(sK), &map_k, 0, chunk * kRows, bh, bar(kS_Load));
        tma_load_3d(smem_u32(sV), &map_v, 0, chunk * kRows, bh, bar(kS_Load));
        tma_load_3d(smem_u32(sOm), &map_om, 0, 0, 0, bar(kS_Load));
        tma_load_3d(smem_u32(sOm) + kTileBytes, &map_om, 0, 0, 1, bar(kS_Load));
      }
      __syncwarp();
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kS_Load), 0, abort_flag));
      if (ok) {
        fence_after();
        // E = K omega'^T (head, then remainder of omega'), contraction over d in four steps
        const uint64_t dk = smem_desc(smem_u32(sK), 16, 1024);
        const uint64_t doh = smem_desc(smem_u32(sOm), 16, 1024), dol = smem_desc(smem_u32(sOm) + kTileBytes, 16, 1024);
        constexpr uint32_t idE = idesc_bf16(MP, false, false);
        if (leader) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_ss(tmem + kColE, dk + 2 * k, doh + 2 * k, idE, k > 0);
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_ss(tmem + kColE, dk + 2 * k, dol + 2 * k, idE, 1);
          mma_commit(bar(kS_E));
        }
        __syncwarp();
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kS_Phi), 0, abort_flag));
      }
      if (ok) {
        fence_after();
        if (p.causal && leader) {
          // the output kernel needs phi(K) of its own chunk again: keep the tiles (head atoms, remainder atoms)
          constexpr int kAtoms = MP > 64 ? 2 : 1;
          const int slice0 = (bh * p.nchunk + chunk) * 2 * kAtoms;
          for (int part = 0; part < 2; ++part)
            for (int a = 0; a < kAtoms; ++a)
              tma_store_3d(&map_phi, smem_u32(sPhi) + part * 2 * kTileBytes + a * kTileBytes, 0, 0, slice0 + part * kAtoms + a);
          bulk_commit();
        }
        // S = phi^T V and z = phi^T 1: A = phi read MN-major (features are its M index), B = V and a
        // tile of ones read MN-major; contraction over the 128 keys in eight steps
        constexpr uint32_t idS = idesc_bf16(64, true, true), idZ = idesc_bf16(16, true, true);
        const uint64_t dones = smem_desc(smem_u32(sOnes), 2048, 1024);
        const uint64_t ah0 = smem_desc(smem_u32(sPhi), kTileBytes, 1024), al0 = smem_desc(smem_u32(sPhi) + 2 * kTileBytes, kTileBytes, 1024);
        const uint64_t bv0 = smem_desc(smem_u32(sV), kTileBytes, 1024);
        if (leader) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {  // a step of 16 keys: 2048 bytes = 128 descriptor units
            mma_ss(tmem + kColS, ah0 + 128 * k, bv0 + 128 * k, idS, k > 0);
            mma_ss(tmem + kColS, al0 + 128 * k, bv0 + 128 * k, idS, 1);
            mma_ss(tmem + kColZ, ah0 + 128 * k, dones, idZ, k > 0);
            mma_ss(tmem + kColZ, al0 + 128 * k, dones, idZ, 1);
          }
          mma_commit(bar(kS_S));
        }
        __syncwarp();
      }
      if (leader) mma_commit(bar(kS_Drain));
      __syncwarp();
      mbar_wait(bar(kS_Drain), 0, abort_flag);
      mbar_wait_drain(bar(kS_Load), 0);  // the copies have landed before the CTA may leave
      if (leader) bulk_wait_all();       // and the stored tiles have left shared memory
      __syncwarp();
    }
  } else {
    // -------------------------------------------------------------- row warps
    const int quarter = warp & 3, part = warp >> 2, rt = quarter * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const int row = chunk * kRows + rt;
    const bool row_ok = row < p.T;
    const float bias = feature_bias(row_ok ? half_sq_norm(p.K + ((size_t)bh * p.T + row) * kHeadDim) : 0.f, row_ok, p.m);
    bool ok = __all_sync(0xffffffffu, mbar_wait(bar(kS_E), 0, abort_flag));
    if (ok) {
      fence_after();
      for (int c = part; c < MP / 32; c += kParts) {
        uint32_t e[32];
        tmem_ld32(lane_addr + kColE + 32 * c, e);
        tmem_ld_wait();
        float phi[32];
        features32(e, phi, bias, c, p.m);
        uint32_t hi[16], lo[16];
        split32(phi, hi, lo);
        store_row32_swizzled(sPhi, rt, c, hi);
        store_row32_swizzled(sPhi + 2 * kTileBytes, rt, c, lo);
      }
      fence_async_smem();
      warp_arrive(bar(kS_Phi), lane);
      ok = __all_sync(0xffffffffu, mbar_wait(bar(kS_S), 0, abort_flag));
    }
    if (ok) {
      fence_after();
      // tensor-memory lane = feature; parts 0 and 1 store 32 of the feature's 64 state columns
      // each, the last part also the normaliser
      constexpr int kZPart = kParts > 2 ? 2 : 0;
      uint32_t s[32], z[32];
      if (part < 2) tmem_ld32(lane_addr + kColS + 32 * part, s);
      if (part == kZPart) tmem_ld32(lane_addr + kColZ, z);
      tmem_ld_wait();
      if (rt < MP) {
        const size_t base = ((size_t)bh * p.nchunk + chunk) * MP + rt;
        if (part < 2) {
          float4* dst = reinterpret_cast<float4*>(p.state_s + base * kHeadDim + 32 * part);
#pragma unroll
          for (int i = 0; i < 8; ++i)
            dst[i] = make_float4(__uint_as_float(s[4 * i]), __uint_as_float(s[4 * i + 1]), __uint_as_float(s[4 * i + 2]),
                                 __uint_as_float(s[4 * i + 3]));
        }
        if (part == kZPart) p.state_z[base] = __uint_as_float(z[0]);
      }
    }
  }
  fence_before();
  __syncthreads();
  if (warp == kRowWarps) {
    __syncwarp();
    fence_after();
    tmem_dealloc(tmem, kCols);
  }
  if (tid == 0 && *abort_flag) atomicOr(p.status, SEA_DEV_TIMEOUT);
}

// ---- kernel 2: combination of the chunk states along the sequence ------------------------------
// One thread per (head, feature, pair of columns) - and per (head, feature) for z - walks the
// chunks in order: exclusive prefix when causal, the total (written for chunk 0 only) otherwise.
// Output per (head, chunk): bf16 head [MP][64], bf16 remainder [MP][64], and z as fp32 [MP].
__global__ void favor_scan_tc_kernel(const float* __restrict__ state_s, const float* __restrict__ state_z,
                                     __nv_bfloat16* __restrict__ s_split, float* __restrict__ z_prefix, int nchunk, int MP,
                                     long long total_threads, int causal) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (gid >= total_threads) return;
  const int per_head = MP * 33;  // 32 column pairs and one z slot per feature
  const long long bh = gid / per_head;
  const int v = (int)(gid - bh * per_head);
  const int f = v / 33, slot = v - f * 33;
  if (slot == 32) {
    const float* src = state_z + (size_t)bh * nchunk * MP + f;
    float* dst = z_prefix + (size_t)bh * nchunk * MP + f;
    float r = 0.f;
    for (int ch = 0; ch < nchunk; ++ch) {
      if (causal) dst[(size_t)ch * MP] = r;
      r += src[(size_t)ch * MP];
    }
    if (!causal) dst[0] = r;
    return;
  }
  const size_t per_chunk = (size_t)MP * kHeadDim;
  const float* src = state_s + (size_t)bh * nchunk * per_chunk + (size_t)f * kHeadDim + 2 * slot;
  __nv_bfloat16* dst = s_split + (size_t)bh * nchunk * 2 * per_chunk + (size_t)f * kHeadDim + 2 * slot;
  float r0 = 0.f, r1 = 0.f;
#pragma unroll 4
  for (int ch = 0; ch < nchunk; ++ch) {
    const float2 x = *reinterpret_cast<const float2*>(src + ch * per_chunk);
    if (causal) {
      uint32_t hi, lo;
      split_pair(r0, r1, hi, lo);
      *reinterpret_cast<uint32_t*>(dst + ch * 2 * per_chunk) = hi;
      *reinterpret_cast<uint32_t*>(dst + ch * 2 * per_chunk + per_chunk) = lo;
    }
    r0 += x.x;
    r1 += x.y;
  }
  if (!causal) {
    uint32_t hi, lo;
    split_pair(r0, r1, hi, lo);
    *reinterpret_cast<uint32_t*>(dst) = hi;
    *reinterpret_cast<uint32_t*>(dst + per_chunk) = lo;
  }
}

// ---- kernel 3: per-chunk output and decoder -----------------------------------------------------
// Persistent: a CTA walks the (head, chunk) items blockIdx.x, blockIdx.x + gridDim.x, ...; omega'
// is staged once, the next item's tiles are copied in as soon as the current item has stopped
// reading their places, and every barrier below completes once per item (or once per decoder pass).
enum {
  kO_Om = 0,               // omega' staged (once)
  kO_QK,                   // the item's Q tile
  kO_PhiK,                 // the item's phi(K) tiles (causal)
  kO_VS,                   // the item's V tile, prefix state and its normaliser
  kO_E,
  kO_Phi,                  // phi(Q): every row warp has written its first chunk of features ...
  kO_Phi2,                 // ... and all of them
  kO_A, kO_P, kO_Num, kO_C,
  kO_W,                    // [3] decoder columns staged (the third place only when a row of A_hat takes three passes or more)
  kO_WDone = kO_W + 3,     // [3] the MMAs that read them are complete
  kO_Ahat = kO_WDone + 3,  // [2] A_hat tile in tensor memory
  kO_AFree = kO_Ahat + 2,  // [2] rows have read it
  kO_Drain = kO_AFree + 2,
  kO_NumBars
};

// Named barrier `id` over the 128 threads of one column group of the row warps.
__device__ __forceinline__ void part_sync(int id) { asm volatile("bar.sync %0, 128;\n" ::"r"(id) : "memory"); }

template <int MP, int KSEL>
__global__ void __launch_bounds__(kThreadsOut, 1)
favor_output_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_om,
                       const __grid_constant__ CUtensorMap map_s, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_phi,
                       const EstParams p) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* sm = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  unsigned char* sQ = sm;                              // 16 KB
  unsigned char* sV = sQ + kTileBytes;                 // 16 KB
  unsigned char* sOm = sV + kTileBytes;                // head, remainder: 32 KB
  unsigned char* sS = sOm + 2 * kTileBytes;            // prefix state head, remainder [MP][64]: 32 KB
  unsigned char* sPhi = sS + 2 * kTileBytes;           // phi(K) head 32 KB, remainder 32 KB; later the decoder columns
  unsigned char* sOut = sPhi + 4 * kTileBytes;         // four boxes of 128 rows x 32 fp32 (a pass's column groups) bound for A_hat
  unsigned char* tail = sOut + 4 * kTileBytes;
  const uint32_t bars = smem_u32(tail);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kO_NumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8 * kO_NumBars + 4);
  constexpr int kTailHead = (8 * kO_NumBars + 8 + 127) / 128 * 128;  // barriers, slot, flag; z_s is a bulk-copy target (16-byte rule)
  float* z_s = reinterpret_cast<float*>(tail + kTailHead);           // [128]
  float* den_x = z_s + 128;                                            // [kParts][128]
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  // tensor memory: projections of Q -> phi(Q); projections of K -> in-chunk kernel matrix -> its
  // masked head / remainder; numerator; C.  A_hat tiles: with a single decoder pass per item (Kc <=
  // 128) the tile has columns of its own, so the next item's projections need not wait until the
  // rows have read it; with several passes the tiles alternate between the first two regions.
  constexpr uint32_t kColQ = 0, kColA = 128, kColNum = 256, kColC = 320, kColAh = 384, kCols = 512;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool causal = p.causal != 0;
  const int n_ct = (p.Kc + kWTile - 1) / kWTile;
  const bool single = n_ct == 1;
  const bool selecting = KSEL > 0 && p.sel != nullptr;  // the launcher only asks for it with a single pass
  const bool keep_a = p.A_hat != nullptr;               // without it the tile is only read by the selecting warps
  const int n_items = p.BH * p.nchunk;
  if (tid == 0) {
    for (int i = 0; i < kO_NumBars; ++i) {
      const bool from_rows = i == kO_Phi || i == kO_Phi2 || i == kO_P || i == kO_C;
      const bool tile_read = i >= kO_AFree && i < kO_AFree + 2;  // the rows, and the selecting warps
      mbar_init(bar(i), tile_read ? (keep_a ? kRowWarps : 0) + (selecting ? 4 : 0) : (from_rows ? kRowWarps : 1));
    }
    *abort_flag = 0;
    mbar_init_fence();
  }
  if (warp == kRowWarps) tmem_alloc(smem_u32(tmem_slot), kCols);
  fence_before();
  __syncthreads();
  fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp >= kRowWarps + 4) {
    // -------------------------------------------------------------- selection from the A_hat tile
    reg_dec<kRegsOutSel>();
    if constexpr (KSEL > 0) {
      if (selecting) {
        using namespace select;
        const int quarter = warp & 3, rt = quarter * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const int words = (p.Kc + 31) >> 5;
        uint32_t g = 0;
        for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++g) {
          const int bh = item / p.nchunk, chunk = item - bh * p.nchunk;
          const int row = chunk * kRows + rt;
          const bool row_ok = row < p.T;
          const size_t grow = (size_t)bh * p.T + row;
          const uint32_t b = g & 1;
          if (!__all_sync(0xffffffffu, mbar_wait_idle(bar(kO_Ahat + b), (g >> 1) & 1, abort_flag))) break;
          fence_after();
          // descending list of the KSEL largest values seen; +inf in the slots beyond k_hat keeps the
          // k_hat-th largest value of the row in the last slot, -inf stands for columns beyond Kc
          float top[KSEL];
#pragma unroll
          for (int q = 0; q < KSEL; ++q) top[q] = q < KSEL - p.k_hat ? INFINITY : -INFINITY;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (32 * c < p.Kc) {
              uint32_t e[32];
              tmem_ld32(lane_addr + kColAh + 32 * c, e);
              tmem_ld_wait();
#pragma unroll
              for (int h0 = 0; h0 < 32; h0 += KSEL) {
                float grp[KSEL];
#pragma unroll
                for (int j = 0; j < KSEL; ++j) grp[j] = 32 * c + h0 + j < p.Kc ? __uint_as_float(e[h0 + j]) : -INFINITY;
                merge_group<KSEL>(top, grp);
              }
            }
          }
          const float tau = top[KSEL - 1];
          int n_gt = 0;
#pragma unroll
          for (int q = 0; q < KSEL; ++q) n_gt += (top[q] != INFINITY && top[q] > tau);
          int ties_left = p.k_hat - n_gt;
          uint32_t gt[4] = {0u, 0u, 0u, 0u}, eq[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (32 * c < p.Kc) {
              uint32_t e[32];
              tmem_ld32(lane_addr + kColAh + 32 * c, e);
              tmem_ld_wait();
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float x = 32 * c + j < p.Kc ? __uint_as_float(e[j]) : -INFINITY;
                gt[c] |= (x > tau ? 1u : 0u) << j;
                eq[c] |= (x == tau ? 1u : 0u) << j;
              }
            }
          }
          warp_arrive(bar(kO_AFree + b), lane);
          if (row_ok) {
            int32_t* my_sel = p.sel + grow * p.k_hat;
            int out = 0, cnt = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if (32 * c < p.Kc)
                emit_columns(gt[c], eq[c], 32 * c, ties_left, my_sel, out, cnt,
                             p.mask_bits != nullptr ? p.mask_bits + grow * words + c : nullptr, row, p.r, p.causal);
            if (p.row_counts != nullptr) p.row_counts[grow] = cnt;
          }
        }
      }
    }
  } else if (warp >= kRowWarps) {
    reg_dec<kRegsOutCtl>();
    if (warp == kRowWarps) {
      // ------------------------------------------------------------ copies and MMAs: the whole warp
      // walks the phases (so that descriptors and counters stay in uniform registers), one elected
      // lane issues the copies, the MMAs and their commits
      const bool leader = elect_one();
      bool ok = true;
      uint32_t it = 0;          // items done: parity of the per-item barriers
      uint32_t g = 0;           // decoder passes issued so far: pass g uses buffers g & 1
      // Places for the decoder's column tiles: the two halves of phi(K)'s area, and - when a row of
      // A_hat takes three passes or more - omega's, which is free between an item's projections and
      // the next item's: the passes ct = om_ct (mod 3) read from there, the last of them is pass
      // n_ct - 2, and omega' is copied in again once that pass's products are complete.  With three
      // places a tile is asked for two passes before its turn instead of one.
      const bool three = n_ct >= 3;
      const int om_ct = three ? (n_ct - 2) % 3 : -1;
      auto slot_of = [&](int ct, uint32_t pass) -> int {  // pass: the running number of the pass (for the two-place rotation)
        if (!three) return (int)(pass & 1u);
        const int q = (ct - om_ct + 3) % 3;
        return q == 0 ? 2 : q - 1;
      };
      uint32_t w_loads[3] = {0u, 0u, 0u};  // tiles requested per place
      uint32_t w_uses[3] = {0u, 0u, 0u};   // passes issued per place
      uint32_t w_next = 0;                 // decoder passes whose columns have been requested
      uint32_t om_loads = 1;               // copies of omega' requested
      uint32_t afree_next = 0;  // decoder passes whose tile the rows are known to have read
      auto load_qk = [&](int item) {
        if (!leader) return;
        const int bh = item / p.nchunk, chunk = item - bh * p.nchunk;
        mbar_expect_tx(bar(kO_QK), kTileBytes);
        tma_load_3d(smem_u32(sQ), &map_q, 0, chunk * kRows, bh, bar(kO_QK));
      };
      // phi(K) of the item's chunk, as the state kernel left it: head atoms, remainder atoms
      constexpr int kAtoms = MP > 64 ? 2 : 1;
      auto load_phik = [&](int item) {
        if (!leader) return;
        mbar_expect_tx(bar(kO_PhiK), 2 * kAtoms * kTileBytes);
        for (int part = 0; part < 2; ++part)
          for (int a = 0; a < kAtoms; ++a)
            tma_load_3d(smem_u32(sPhi) + part * 2 * kTileBytes + a * kTileBytes, &map_phi, 0, 0,
                        item * 2 * kAtoms + part * kAtoms + a, bar(kO_PhiK));
      };
      auto load_vs = [&](int item) {
        if (!leader) return;
        const int bh = item / p.nchunk, chunk = item - bh * p.nchunk;
        const bool prefix = !causal || chunk > 0;
        const int state_idx = (bh * p.nchunk + (causal ? chunk : 0)) * 2;
        mbar_expect_tx(bar(kO_VS), (causal ? kTileBytes : 0) + (prefix ? 2 * MP * 128 + MP * 4 : 0));
        if (causal) tma_load_3d(smem_u32(sV), &map_v, 0, chunk * kRows, bh, bar(kO_VS));
        if (prefix) {
          tma_load_3d(smem_u32(sS), &map_s, 0, 0, state_idx, bar(kO_VS));
          tma_load_3d(smem_u32(sS) + kTileBytes, &map_s, 0, 0, state_idx + 1, bar(kO_VS));
          bulk_load(smem_u32(z_s), p.z_prefix + (size_t)(state_idx / 2) * MP, MP * 4, bar(kO_VS));
        }
      };
      // decoder columns of column tile ct of the current item into their place
      auto load_w = [&](int ct) {
        const int sl = slot_of(ct, w_next);
        const uint32_t dst = sl < 2 ? smem_u32(sPhi) + sl * 2 * kTileBytes : smem_u32(sOm);
        if (leader) {
          mbar_expect_tx(bar(kO_W + sl), 4 * 8192);
          for (int part = 0; part < 2; ++part)
            for (int atom = 0; atom < 2; ++atom)
              tma_load_3d(dst + part * kTileBytes + atom * 8192, &map_w, ct * kWTile + 64 * atom, 0, part, bar(kO_W + sl));
        }
        ++w_loads[sl];
        ++w_next;
      };
      auto load_om = [&]() {
        if (leader) {
          mbar_expect_tx(bar(kO_Om), 2 * MP * 128);
          tma_load_3d(smem_u32(sOm), &map_om, 0, 0, 0, bar(kO_Om));
          tma_load_3d(smem_u32(sOm) + kTileBytes, &map_om, 0, 0, 1, bar(kO_Om));
        }
      };
      auto wait_afree_upto = [&](uint32_t upto) {  // the rows have read the tiles of passes 0 .. upto-1
        while (ok && afree_next < upto) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_AFree + (afree_next & 1)), (afree_next >> 1) & 1, abort_flag));
          ++afree_next;
        }
      };
      const int first = blockIdx.x;
      if (first < n_items) {
        load_om();
        load_qk(first);
        load_vs(first);
        __syncwarp();
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_Om), 0, abort_flag));
      }
      const uint64_t doh = smem_desc(smem_u32(sOm), 16, 1024), dol = smem_desc(smem_u32(sOm) + kTileBytes, 16, 1024);
      for (int item = first; item < n_items && ok; item += gridDim.x, ++it) {
        const int chunk = item % p.nchunk;
        const bool has_prefix = !causal || chunk > 0;
        const int next = item + gridDim.x;
        const uint32_t par = it & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_QK), par, abort_flag));
        // the projections go where the previous item's A_hat tiles were, and phi(K) where its decoder
        // columns were: the rows have read the former (which also means the MMAs that read the
        // latter are complete); with a tile region of its own only the MMAs matter
        if (!single) wait_afree_upto(g);
        else if (ok && g > 0) {
          const int ps = (int)((g - 1) & 1u);
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_WDone + ps), (w_uses[ps] - 1) & 1, abort_flag));
        }
        // omega' is back (it made room for decoder columns during the previous item's passes)
        if (ok && three) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_Om), (om_loads - 1) & 1, abort_flag));
        if (!ok) break;
        fence_after();
        if (causal) load_phik(item);
        {
          constexpr uint32_t idE = idesc_bf16(MP, false, false);
          const uint64_t dq = smem_desc(smem_u32(sQ), 16, 1024);
          if (leader) {
#pragma unroll
            for (int k = 0; k < 4; ++k) mma_ss(tmem + kColQ, dq + 2 * k, doh + 2 * k, idE, k > 0);
#pragma unroll
            for (int k = 0; k < 4; ++k) mma_ss(tmem + kColQ, dq + 2 * k, dol + 2 * k, idE, 1);
            mma_commit(bar(kO_E));
          }
          __syncwarp();
        }
        // The contractions over the features start once every row warp has written its first chunk
        // (features 0 .. 32 kParts - 1: steps 0 .. kStep1 - 1) and go on when all are there.
        constexpr int kSteps = MP / 16, kStep1 = kSteps < 2 * kParts ? kSteps : 2 * kParts;
        constexpr uint32_t idA = idesc_bf16(128, false, false);
        constexpr uint32_t idS = idesc_bf16(64, false, true);
        const uint64_t bh0 = smem_desc(smem_u32(sPhi), 16, 1024), bl0 = smem_desc(smem_u32(sPhi) + 2 * kTileBytes, 16, 1024);
        const uint64_t sh0 = smem_desc(smem_u32(sS), kTileBytes, 1024), sl0 = smem_desc(smem_u32(sS) + kTileBytes, kTileBytes, 1024);
        // in-chunk kernel matrix phi(Q) phi(K)^T: A = phi(Q) in tensor memory, B = phi(K) K-major
        auto mma_kernel_matrix = [&](int k_lo, int k_hi) {
          if (!leader) return;
#pragma unroll
          for (int k = k_lo; k < k_hi; ++k) {
            constexpr int kUnitsPerTile = kTileBytes / 16;
            const uint32_t off = (k >> 2) * kUnitsPerTile + (k & 3) * 2;  // descriptor units of 16 bytes
            const uint32_t a = tmem + kColQ + a_col(k);
            mma_ts(tmem + kColA, a, bh0 + off, idA, k > 0);
            mma_ts(tmem + kColA, a, bl0 + off, idA, 1);
            mma_ts(tmem + kColA, a + 16, bh0 + off, idA, 1);
          }
        };
        // phi(Q) S: B = the state read MN-major (16 features = 2048 bytes = 128 descriptor units per step)
        auto mma_prefix = [&](int k_lo, int k_hi) {
          if (!leader) return;
#pragma unroll
          for (int k = k_lo; k < k_hi; ++k) {
            const uint32_t a = tmem + kColQ + a_col(k);
            mma_ts(tmem + kColNum, a, sh0 + 128 * k, idS, k > 0);
            mma_ts(tmem + kColNum, a, sl0 + 128 * k, idS, 1);
            mma_ts(tmem + kColNum, a + 16, sh0 + 128 * k, idS, 1);
          }
        };
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_Phi), par, abort_flag));
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(causal ? kO_PhiK : kO_VS), par, abort_flag));
        if (!ok) break;
        fence_after();
        if (causal) mma_kernel_matrix(0, kStep1);
        else mma_prefix(0, kStep1);  // not causal: every item has a prefix (the total)
        __syncwarp();
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_Phi2), par, abort_flag));
        if (!ok) break;
        fence_after();
        // the rows have read the projections (and the Q tile, for their norms): it is free for the next item
        if (next < n_items) load_qk(next);
        if (causal) {
          mma_kernel_matrix(kStep1, kSteps);
          if (leader) mma_commit(bar(kO_A));
          __syncwarp();
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_VS), par, abort_flag));
          if (!ok) break;
          fence_after();
          if (has_prefix) mma_prefix(0, kSteps);
        } else {
          mma_prefix(kStep1, kSteps);
        }
        __syncwarp();
        if (causal) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_P), par, abort_flag));
          if (!ok) break;
          fence_after();
        }
        // phi(K) is no longer read (the rows waited for the kernel matrix): its place takes the
        // decoder columns of this item's first passes
        load_w(0);
        if (n_ct > 1) load_w(1);
        if (three) load_w(2);  // omega's place: the projections were complete before the rows wrote phi(Q)
        if (causal) {
          constexpr uint32_t idN = idesc_bf16(64, false, true);
          const uint64_t bv0 = smem_desc(smem_u32(sV), kTileBytes, 1024);
          if (leader) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const uint32_t a = tmem + kColA + a_col(k);
              mma_ts(tmem + kColNum, a, bv0 + 128 * k, idN, (has_prefix || k > 0) ? 1u : 0u);
              mma_ts(tmem + kColNum, a + 16, bv0 + 128 * k, idN, 1);
            }
          }
          __syncwarp();
        }
        if (leader) mma_commit(bar(kO_Num));
        __syncwarp();
        ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_C), par, abort_flag));
        if (!ok) break;
        fence_after();
        // numerator complete and read: V, the state and its normaliser are free for the next item
        if (next < n_items) load_vs(next);
        // A_hat tile = C W: A = C in tensor memory (64 values: four steps), B = decoder columns MN-major
        constexpr uint32_t idW = idesc_bf16(kWTile, false, true);
        for (int ct = 0; ct < n_ct && ok; ++ct, ++g) {
          const uint32_t b = g & 1;
          const int sl = slot_of(ct, g);
          ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_W + sl), w_uses[sl] & 1, abort_flag));
          // the rows have read the tile that was in this buffer
          if (single) wait_afree_upto(g);
          else if (g >= 2) wait_afree_upto(g - 1);
          if (!ok) break;
          fence_after();
          const uint32_t wbase = sl < 2 ? smem_u32(sPhi) + sl * 2 * kTileBytes : smem_u32(sOm);
          const uint32_t d = tmem + (single ? kColAh : (b ? kColA : kColQ));
          const uint64_t wh0 = smem_desc(wbase, 8192, 1024), wl0 = smem_desc(wbase + kTileBytes, 8192, 1024);
          if (leader) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const uint32_t a = tmem + kColC + a_col(k);
              mma_ts(d, a, wh0 + 128 * k, idW, k > 0);
              mma_ts(d, a, wl0 + 128 * k, idW, 1);
              mma_ts(d, a + 16, wh0 + 128 * k, idW, 1);
            }
            mma_commit(bar(kO_Ahat + b));
            mma_commit(bar(kO_WDone + sl));
          }
          ++w_uses[sl];
          __syncwarp();
          if (ct >= 1 && (three || ct + 1 < n_ct)) {
            // the place the previous pass read from takes the columns of the pass that comes
            // round to it next (one pass on with two places, two with three), or omega' again
            const int ps = slot_of(ct - 1, g - 1);
            const int ct_new = ct + (three ? 2 : 1);
            if (ct_new < n_ct || (ps == 2 && next < n_items)) {
              ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_WDone + ps), (w_uses[ps] - 1) & 1, abort_flag));
              if (ok) {
                if (ct_new < n_ct) {
                  load_w(ct_new);
                } else {
                  load_om();
                  ++om_loads;
                }
              }
            }
          }
        }
      }
      if (leader) mma_commit(bar(kO_Drain));
      __syncwarp();
      mbar_wait(bar(kO_Drain), 0, abort_flag);
      // copies still in flight must land before the CTA may leave (only after a wait ran out can
      // any be outstanding here: every armed phase is waited for in the loop above)
      if (!ok) {
        mbar_wait_drain(bar(kO_Om), (om_loads - 1) & 1);
        mbar_wait_drain(bar(kO_QK), it & 1);
        mbar_wait_drain(bar(kO_VS), it & 1);
        if (causal) mbar_wait_drain(bar(kO_PhiK), it & 1);
        for (int sl = 0; sl < 3; ++sl)
          if (w_loads[sl] > 0) mbar_wait_drain(bar(kO_W + sl), (w_loads[sl] - 1) & 1);
      }
    }
  } else {
    // -------------------------------------------------------------- row warps
    reg_inc<kRegsOutRow>();
    const int quarter = warp & 3, part = warp >> 2, rt = quarter * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const bool elected = quarter == 0 && lane == 0;  // issues this column group's stores
    unsigned char* my_boxes = sOut + part * (4 / kParts) * kTileBytes;  // one box per column group of a pass
    uint32_t it = 0, g = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
      const int bh = item / p.nchunk, chunk = item - bh * p.nchunk;
      const bool has_prefix = !causal || chunk > 0;
      const uint32_t par = it & 1;
      const int row = chunk * kRows + rt;
      const bool row_ok = row < p.T;
      const size_t grow = (size_t)bh * p.T + row;
      // the row's norm from the staged Q tile (the control warp refills it only after every row
      // warp has arrived at kO_Phi below); rows past T are zero-filled by the copy
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_QK), par, abort_flag));
      const float bias_q = feature_bias(ok ? half_sq_norm_swizzled(sQ, rt) : 0.f, row_ok, p.m);
      float den = 0.f;
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_E), par, abort_flag));
      if (ok && has_prefix) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_VS), par, abort_flag));  // z has landed
      if (ok) {
        fence_after();
        bool first_chunk = true;
        for (int c = part; c < MP / 32; c += kParts) {
          uint32_t e[32];
          float phi[32];
          uint32_t hi[16], lo[16];
          tmem_ld32(lane_addr + kColQ + 32 * c, e);
          tmem_ld_wait();
          features32(e, phi, bias_q, c, p.m);
          if (has_prefix) {
            float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 32; ++i) d4[i & 3] = fmaf(phi[i], z_s[32 * c + i], d4[i & 3]);
            den += (d4[0] + d4[1]) + (d4[2] + d4[3]);
          }
          split32(phi, hi, lo);
          tmem_st16(lane_addr + kColQ + 32 * c, hi);
          tmem_st16(lane_addr + kColQ + 32 * c + 16, lo);
          if (first_chunk) {  // the contractions may start on the first 32 kParts features
            tmem_st_wait();
            warp_arrive(bar(kO_Phi), lane);
            first_chunk = false;
          }
        }
        if (first_chunk) warp_arrive(bar(kO_Phi), lane);  // no chunk of its own
        tmem_st_wait();
        warp_arrive(bar(kO_Phi2), lane);
        if (causal) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_A), par, abort_flag));
      }
      if (ok && causal) {
        fence_after();
        // keep keys j <= i of the chunk; rows of the normaliser; head / remainder in place
        for (int c = part; c < 4; c += kParts) {
          uint32_t e[32];
          float a[32];
          uint32_t hi[16], lo[16];
          tmem_ld32(lane_addr + kColA + 32 * c, e);
          tmem_ld_wait();
          float d4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            a[i] = (32 * c + i <= rt) ? __uint_as_float(e[i]) : 0.f;
            d4[i & 3] += a[i];
          }
          den += (d4[0] + d4[1]) + (d4[2] + d4[3]);
          split32(a, hi, lo);
          tmem_st16(lane_addr + kColA + 32 * c, hi);
          tmem_st16(lane_addr + kColA + 32 * c + 16, lo);
        }
        tmem_st_wait();
        warp_arrive(bar(kO_P), lane);
      }
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_Num), par, abort_flag));
      den_x[part * kRows + rt] = den;
      ok = rows_all(ok);
      if (ok) {
        fence_after();
        den = 0.f;
#pragma unroll
        for (int q = 0; q < kParts; ++q) den += den_x[q * kRows + rt];
        if (row_ok && !(den > 0.f && den < INFINITY)) atomicOr(p.status, SEA_DEV_NONFINITE);
        const float inv = 1.f / den;
        if (part < 2) {  // C has 64 columns: two chunks
          uint32_t e[32];
          float cv[32];
          uint32_t hi[16], lo[16];
          tmem_ld32(lane_addr + kColNum + 32 * part, e);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) cv[i] = row_ok ? __uint_as_float(e[i]) * inv : 0.f;
          split32(cv, hi, lo);
          tmem_st16(lane_addr + kColC + 32 * part, hi);
          tmem_st16(lane_addr + kColC + 32 * part + 16, lo);
          tmem_st_wait();
        }
        warp_arrive(bar(kO_C), lane);
      }
      // ---- decoder passes: tile out of tensor memory, then to A_hat (when the caller keeps it)
      float* out = p.A_hat + grow * p.Kc;
      for (int ct = 0; ct < n_ct && keep_a; ++ct, ++g) {
        const uint32_t b = g & 1;
        constexpr int kMine = 4 / kParts;  // chunks of the 128-column tile per thread
        uint32_t e[kMine][32];
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(kO_Ahat + b), (g >> 1) & 1, abort_flag));
        if (ok) {
          fence_after();
#pragma unroll
          for (int cc = 0; cc < kMine; ++cc)
            tmem_ld32(lane_addr + (single ? kColAh : (b ? kColA : kColQ)) + 32 * (part + kParts * cc), e[cc]);
          tmem_ld_wait();
          warp_arrive(bar(kO_AFree + b), lane);
        }
        if (p.tma_store) {
          // the column groups' boxes: wait until their previous stores have been read out, fill them
          // (128-byte rows, swizzled like the copy expects), hand them to the copy engine
          if (elected) bulk_wait_read();
          part_sync(2 + part);
          if (ok) {
#pragma unroll
            for (int cc = 0; cc < kMine; ++cc)
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(my_boxes + cc * kTileBytes + rt * 128 + ((j ^ (rt & 7)) << 4)) =
                    make_uint4(e[cc][4 * j], e[cc][4 * j + 1], e[cc][4 * j + 2], e[cc][4 * j + 3]);
          }
          fence_async_smem();
          part_sync(2 + part);
          if (elected && ok) {
#pragma unroll
            for (int cc = 0; cc < kMine; ++cc) {
              const int col0 = ct * kWTile + 32 * (part + kParts * cc);
              if (col0 < p.Kc) tma_store_3d(&map_a, smem_u32(my_boxes + cc * kTileBytes), col0, chunk * kRows, bh);
            }
            bulk_commit();
          }
        } else if (ok && row_ok) {
#pragma unroll
          for (int cc = 0; cc < kMine; ++cc) {
            const int col0 = ct * kWTile + 32 * (part + kParts * cc);
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (col0 + i < p.Kc) out[col0 + i] = __uint_as_float(e[cc][i]);
          }
        }
      }
    }
    if (elected) bulk_wait_all();
  }
  fence_before();
  __syncthreads();
  if (warp == kRowWarps) {
    __syncwarp();
    fence_after();
    tmem_dealloc(tmem, kCols);
  }
  if (tid == 0 && *abort_flag) atomicOr(p.status, SEA_DEV_TIMEOUT);
}

int padded_features(int m) { return m <= 32 ? 32 : (m <= 64 ? 64 : 128); }
size_t padded_kc(const sea_shape& s) { return ((size_t)s.Kc + 63) / 64 * 64; }  // whole 64-column copy boxes

template <int MP>
sea_status launch_mp(const sea_shape& s, const __nv_bfloat16* Q, const __nv_bfloat16* K, const __nv_bfloat16* V,
                     const float* omega, const float* W_dec, float* A_hat, float* state, unsigned char* scratch,
                     const SelectOut* so, int32_t* status, cudaStream_t st) {
  const int BH = s.B * s.H;
  const int nchunk = (s.T + kRows - 1) / kRows;
  const size_t KcP = padded_kc(s);
  // carve-up of the scratch area (estimate_tc_split_bytes)
  __nv_bfloat16* om = reinterpret_cast<__nv_bfloat16*>(scratch);                       // [2][MP][64]
  __nv_bfloat16* wd = om + 2 * 128 * kHeadDim;                                         // [2][64][KcP]
  __nv_bfloat16* s_split = wd + 2 * kHeadDim * KcP;                                    // [BH][nchunk][2][MP][64]
  float* z_prefix = reinterpret_cast<float*>(s_split + (size_t)BH * nchunk * 2 * MP * kHeadDim);  // [BH][nchunk][MP]
  __nv_bfloat16* phik = reinterpret_cast<__nv_bfloat16*>(z_prefix + (size_t)BH * nchunk * MP);  // [BH][nchunk][2][atoms][128][64]
  float* state_s = state;                                                              // [BH][nchunk][MP][64]
  float* state_z = state + (size_t)BH * nchunk * MP * kHeadDim;                        // [BH][nchunk][MP]

  CUtensorMap mq, mk, mv, mom, ms, mw, ma, mphi;
  if (!make_map_bf16_3d(&mq, Q, kHeadDim, s.T, BH, kHeadDim, kRows) ||
      !make_map_bf16_3d(&mk, K, kHeadDim, s.T, BH, kHeadDim, kRows) ||
      !make_map_bf16_3d(&mv, V, kHeadDim, s.T, BH, kHeadDim, kRows) ||
      !make_map_bf16_3d(&mom, om, kHeadDim, MP, 2, kHeadDim, MP) ||
      !make_map_bf16_3d(&ms, s_split, kHeadDim, MP, (unsigned long long)BH * nchunk * 2, kHeadDim, MP) ||
      !make_map_bf16_3d(&mw, wd, KcP, kHeadDim, 2, 64, kHeadDim) ||
      !make_map_bf16_3d(&mphi, phik, kHeadDim, kRows, (unsigned long long)BH * nchunk * 2 * (MP > 64 ? 2 : 1), kHeadDim, kRows))
    return SEA_ERR_CUDA;

  const int n_prep = MP * kHeadDim + kHeadDim * (int)KcP;
  favor_prep_tc_kernel<<<(n_prep + 255) / 256, 256, 0, st>>>(omega, W_dec, om, wd, s.m, MP, s.Kc, (int)KcP,
                                                             0.35355339059327373f);
  sea_status rc = check_launch();
  if (rc != SEA_OK) return rc;

  EstParams prm{};
  prm.Q = Q;
  prm.K = K;
  prm.state_s = state_s;
  prm.state_z = state_z;
  prm.z_prefix = z_prefix;
  prm.A_hat = A_hat;
  prm.status = status;
  prm.BH = BH;
  prm.T = s.T;
  prm.m = s.m;
  prm.Kc = s.Kc;
  prm.nchunk = nchunk;
  prm.causal = s.causal;
  // A_hat [BH][T][Kc] fp32 in boxes of 128 rows x 32 columns; without a map (rows that are no
  // multiple of 16 bytes) the rows store their values themselves
  prm.tma_store = (A_hat != nullptr && s.Kc % 4 == 0 &&
                   make_map_3d(&ma, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, A_hat, s.Kc, s.T, BH, 32, kRows)) ? 1 : 0;
  if (!prm.tma_store) ma = mq;  // a valid map that is never used
  const bool selecting = so != nullptr && so->sel != nullptr && estimate_tc_selects(s);
  if (A_hat == nullptr && !selecting) return SEA_ERR_INVALID_ARG;  // the estimate would go nowhere
  if (selecting) {
    prm.sel = so->sel;
    prm.row_counts = so->row_counts;
    prm.mask_bits = so->mask_bits;
    prm.k_hat = s.k_hat;
    prm.r = s.T / s.Kc;
  }

  const size_t smem1 = 1024 + 5 * kTileBytes + 2048 + 8 * kS_NumBars + 16;
  const size_t smem3 = 1024 + (10 + 4) * kTileBytes + (8 * kO_NumBars + 8 + 127) / 128 * 128 + (1 + kParts) * 128 * 4;
  if (cudaFuncSetAttribute(favor_state_tc_kernel<MP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess)
    return SEA_ERR_CUDA;
  const dim3 grid(nchunk, BH);
  favor_state_tc_kernel<MP><<<grid, kThreads, smem1, st>>>(mk, mv, mom, mphi, prm);
  if ((rc = check_launch()) != SEA_OK) return rc;
  // a causal sequence of one chunk has no prefix to form
  if (!(s.causal && nchunk == 1)) {
    const long long total = (long long)BH * MP * 33;
    favor_scan_tc_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(state_s, state_z, s_split, z_prefix, nchunk, MP,
                                                                          total, s.causal);
    if ((rc = check_launch()) != SEA_OK) return rc;
  }
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SEA_ERR_CUDA;
  const int n_items = BH * nchunk;
  const int grid3 = n_items < sms ? n_items : sms;
#define SEA_OUT(KS)                                                                                                       \
  do {                                                                                                                    \
    if (cudaFuncSetAttribute(favor_output_tc_kernel<MP, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem3) != \
        cudaSuccess)                                                                                                      \
      return SEA_ERR_CUDA;                                                                                                \
    favor_output_tc_kernel<MP, KS><<<grid3, kThreadsOut, smem3, st>>>(mq, mv, mom, ms, mw, ma, mphi, prm);               \
  } while (0)
  if (!selecting) SEA_OUT(0);
  else if (s.k_hat <= 16) SEA_OUT(16);
  else SEA_OUT(32);
#undef SEA_OUT
  return check_launch();
}

}  // namespace

// fp32 chunk states [BH][nchunk][MP][65] of the tensor-core estimator.
size_t estimate_tc_state_bytes(const sea_shape& s) {
  if (s.m <= 0) return 0;
  const size_t nchunk = ((size_t)s.T + kRows - 1) / kRows;
  return (size_t)s.B * s.H * nchunk * padded_features(s.m) * (kHeadDim + 1) * sizeof(float);
}
// bf16 operands: omega' and W_dec (head / remainder) and the scanned states with their normalisers.
size_t estimate_tc_split_bytes(const sea_shape& s) {
  if (s.m <= 0) return 0;
  const size_t nchunk = ((size_t)s.T + kRows - 1) / kRows;
  const size_t MP = padded_features(s.m);
  const size_t elems = 2 * (size_t)128 * kHeadDim + 2 * (size_t)kHeadDim * padded_kc(s) +
                       (size_t)s.B * s.H * nchunk * (2 * MP * kHeadDim + 2 * MP) +
                       (size_t)s.B * s.H * nchunk * 2 * (MP > 64 ? 2 : 1) * kRows * kHeadDim;  // phi(K) tiles
  return elems * sizeof(__nv_bfloat16) + 256;
}
bool estimate_tc_applicable(const sea_shape& s) {
  return s.io == SEA_BF16 && s.m >= 16 && s.m <= 128 && encode_fn() != nullptr;
}
// The output kernel can select a row's k_hat largest entries itself while the row's whole A_hat is
// one tile in tensor memory.
bool estimate_tc_selects(const sea_shape& s) { return estimate_tc_applicable(s) && s.Kc <= kWTile && s.k_hat <= 32; }

sea_status launch_estimate_tc(const sea_shape& s, const void* Q, const void* K, const void* V, const float* omega,
                              const float* W_dec, float* A_hat, float* est_state, void* split_buf, const SelectOut* so,
                              int32_t* status, cudaStream_t st) {
  using T = __nv_bfloat16;
  unsigned char* scratch = static_cast<unsigned char*>(split_buf);
  switch (padded_features(s.m)) {
    case 32:
      return launch_mp<32>(s, (const T*)Q, (const T*)K, (const T*)V, omega, W_dec, A_hat, est_state, scratch, so, status, st);
    case 64:
      return launch_mp<64>(s, (const T*)Q, (const T*)K, (const T*)V, omega, W_dec, A_hat, est_state, scratch, so, status, st);
    default:
      return launch_mp<128>(s, (const T*)Q, (const T*)K, (const T*)V, omega, W_dec, A_hat, est_state, scratch, so, status, st);
  }
}

}  // namespace sea

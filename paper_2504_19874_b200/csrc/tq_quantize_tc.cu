// Tensor-core quantisation path (sm_100a): the rotation y = Pi u and the QJL projection
// z = S' e as tcgen05 GEMMs fed by TMA, with the nearest-centroid search, bit packing,
// residual and sign extraction fused into the epilogue that reads the accumulators from TMEM.
//
// fp32 fidelity on bf16 tensor cores: every fp32 operand is split into two bf16 limbs
// (v = hi + lo + O(2^-17 |v|)), and each product is formed as hi*hi + hi*lo + lo*hi with fp32
// accumulation (3 MMA passes).  The dropped terms are ~2^-17 relative per product, i.e.
// ~1e-7 on a rotated coordinate of a unit vector at d = 1536 -- far inside the 1e-5 window in
// which a nearest-centroid decision may legitimately differ from exact arithmetic.
//
// Two forms of the GEMM kernel: one CTA per 128 x 256 tile, and (the usual one at d > 128) a pair of CTAs of one
// cluster per 256 x 256 tile (tcgen05 cta_group::2), which halves what every SM reads of B from shared memory.
#include <atomic>
#include <cstdlib>
#include <algorithm>
#include <mutex>

#include "tq_quantize_tc.h"
#include "tq_tc.cuh"

namespace tq {
namespace tc {

namespace {

constexpr int BM = 128;          // rows of X per tile = TMEM lanes
constexpr int BK = 64;           // bf16 elements per 128-byte swizzled row
constexpr int UMMA_K = 16;
constexpr int EPS = 4;           // epilogue warps per TMEM lane group: each takes 1/EPS of the tile's columns
constexpr int NSPLIT = 2;        // warps that prepare the next block's operand limbs beside the GEMM (see SplitTask)
constexpr int NTHREADS = 32 * (2 + 4 * EPS + NSPLIT);   // warp 0: TMA, warp 1: MMA + TMEM owner, the epilogue warps, the split warps

// CTAS = 2: two CTAs of a cluster share one 256-row tile (tcgen05 cta_group::2).  Each loads its own 128 rows of A and
// its own half of B's rows, so a k-block costs each SM 64 KB of shared-memory writes instead of 96 and its MMAs read
// half of B from the partner: the shared-memory bandwidth that caps the one-CTA kernel (158 bytes per clock wanted,
// 128 available) drops to 104.
template <int BN, int CTAS>
struct Cfg {
  static constexpr int kBRows = BN / CTAS;                                  // rows of B this CTA loads
  static constexpr int kStageBytes = 2 * BM * BK * 2 + 2 * kBRows * BK * 2; // A hi/lo + B hi/lo
  static constexpr int kStages = CTAS == 2 ? 3 : ((BN == 256) ? 2 : (BN == 128 ? 3 : 4));
  static constexpr int kTmemCols = 2 * BN;                                  // two accumulators
  static constexpr int kStoreBytes = 4 * EPS * 2048;   // MODE 1: one [32 rows x 64 B] box per epilogue warp, staged for a TMA store
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 512 /*barriers, centroids*/ + kStoreBytes;
};

struct GemmArgs {
  int64_t M;             // valid rows
  int N, K;              // = d, d
  int tiles_m, tiles_n;
  Codebook cb;
  uint8_t* out;          // packed idx (MODE 0/1) or qjl (MODE 2) rows
  size_t out_rb;
  __nv_bfloat16* E1;     // MODE 1: residual limbs, pitch ldE
  __nv_bfloat16* E2;
  const CUtensorMap* store_e1;   // host pointers to the TMA store maps of E1 / E2 (box 32 rows x 32 columns, 64-byte swizzle);
  const CUtensorMap* store_e2;   // the launcher passes them on as kernel arguments
  int64_t ldE;
  float* gpart;          // MODE 1: [EPS * tiles_n][Mpad] partial sums of e^2 (one per epilogue warp's columns)
  int64_t Mpad;
  const float* nu;       // MODE 1: per-row norm (row with nu == 0 has residual 0); nullable
  // TQ_LAYOUT_NIBBLE (BITS = 3 with MODE 1, and MODE 2): the codes of 32 coordinates are four words of the combined
  // row [idx row | qjl row], nibble = index | sign << 3.  MODE 1 writes them with the sign bits clear, MODE 2 ORs
  // the sign bits in.
  int nibble;
  // Operand preparation of the NEXT block of rows (nu = ||x||, u = x / nu, bf16 limbs of u), done by NSPLIT spare
  // warps of every CTA while this launch's GEMM runs: the GEMM is bound by the tensor pipe and shared memory, the
  // preparation by HBM and a little issue bandwidth, so it hides completely.  Only the project launch (MODE 2)
  // carries one: its own A operand is the residual, so the limb buffers of X are free to be rewritten.
  struct SplitTask {
    const void* X;       // first row of the next block
    int64_t ldx, rows;   // rows == 0: nothing to do
    int d, dpad, is_f32, normalize;
    __nv_bfloat16* L1;
    __nv_bfloat16* L2;
    float* norms;        // nullable
  } split;
  uint8_t* nib_idx;      // idx rows (stride nib_idx_rb) and qjl rows (stride nib_qjl_rb) of this block of rows
  uint8_t* nib_qjl;
  size_t nib_idx_rb, nib_qjl_rb;
  int* status;
};

// Bit i of the low byte of x at bit 4 i + 3.
__device__ __forceinline__ uint32_t spread_to_nibble_tops(uint32_t x) {
  x &= 0xffu;
  x = (x | (x << 12)) & 0x000f000fu;
  x = (x | (x << 6)) & 0x03030303u;
  x = (x | (x << 3)) & 0x11111111u;
  return x << 3;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// fp32 rows, 16-byte aligned, of at most 2048 NV / 16 elements per segment: a segment is held in registers (NV x 16
// bytes per lane, all loads in flight at once); a row of one segment is read once, longer rows a second time (from L2)
// after the norm is known.  NV follows d, so that short rows do not pay for sixteen mostly empty rounds (at d = 200 the
// kernel was bound by the issue of predicated-off instructions, 2.6 TB/s).  The sums are those of NV = 16: the rounds
// left out added fma(0, 0, s) = s.
template <bool NORMALIZE, int NV>
__device__ __forceinline__ void split_rows_vec(const float* __restrict__ X, int64_t ldx, int64_t n, int d, int dpad,
                                               __nv_bfloat16* __restrict__ L1, __nv_bfloat16* __restrict__ L2,
                                               float* __restrict__ norms, int64_t warp, int64_t nwarps, int lane) {
  const int nseg = (d + 128 * NV - 1) / (128 * NV);
  if (NV < 16) {
    // short rows (one segment): 16 / NV rows of a warp are in flight at once -- a single row of 800 bytes per warp
    // does not keep enough bytes in flight to fill the memory pipe
    constexpr int RB = 16 / NV;
    for (int64_t r0 = warp * RB; r0 < n; r0 += nwarps * RB) {
      float4 v[RB][NV];
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const float4* row4 = reinterpret_cast<const float4*>(X + min(r0 + k, n - 1) * ldx);
#pragma unroll
        for (int i = 0; i < NV; ++i) {
          const int c = lane + 32 * i;
          v[k][i] = (4 * c < d) ? __ldg(row4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int64_t r = r0 + k;
        if (r >= n) break;
        float inv = 1.f;
        if (NORMALIZE) {
          float s = 0.f;
#pragma unroll
          for (int i = 0; i < NV; ++i)
            s = fmaf(v[k][i].x, v[k][i].x, fmaf(v[k][i].y, v[k][i].y, fmaf(v[k][i].z, v[k][i].z, fmaf(v[k][i].w, v[k][i].w, s))));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          const float nu = sqrtf(s);
          inv = (nu > 0.f) ? 1.f / nu : 0.f;
          if (lane == 0 && norms != nullptr) norms[r] = nu;
        }
#pragma unroll
        for (int i = 0; i < NV; ++i) {
          const int c = lane + 32 * i;
          if (4 * c >= d) continue;
          const float u0 = v[k][i].x * inv, u1 = v[k][i].y * inv, u2 = v[k][i].z * inv, u3 = v[k][i].w * inv;
          const float h0 = __bfloat162float(__float2bfloat16_rn(u0)), h1 = __bfloat162float(__float2bfloat16_rn(u1));
          const float h2 = __bfloat162float(__float2bfloat16_rn(u2)), h3 = __bfloat162float(__float2bfloat16_rn(u3));
          *reinterpret_cast<uint2*>(L1 + r * dpad + 4 * c) = make_uint2(pack_bf16x2(h0, h1), pack_bf16x2(h2, h3));
          *reinterpret_cast<uint2*>(L2 + r * dpad + 4 * c) = make_uint2(pack_bf16x2(u0 - h0, u1 - h1), pack_bf16x2(u2 - h2, u3 - h3));
        }
      }
    }
    return;
  }
  for (int64_t r = warp; r < n; r += nwarps) {
    const float4* row4 = reinterpret_cast<const float4*>(X + r * ldx);
    float4 v[NV];
    auto load_seg = [&](int seg) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int c = seg * 32 * NV + lane + 32 * i;
        v[i] = (4 * c < d) ? __ldg(row4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    float inv = 1.f;
    load_seg(0);
    if (NORMALIZE) {
      float s = 0.f;
      for (int seg = 0; seg < nseg; ++seg) {
        if (seg > 0) load_seg(seg);
#pragma unroll
        for (int i = 0; i < NV; ++i) s = fmaf(v[i].x, v[i].x, fmaf(v[i].y, v[i].y, fmaf(v[i].z, v[i].z, fmaf(v[i].w, v[i].w, s))));
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const float nu = sqrtf(s);
      inv = (nu > 0.f) ? 1.f / nu : 0.f;
      if (lane == 0 && norms != nullptr) norms[r] = nu;
    }
    for (int seg = 0; seg < nseg; ++seg) {
      if (nseg > 1 && (seg > 0 || NORMALIZE)) load_seg(seg);   // registers hold the last segment read
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int c = seg * 32 * NV + lane + 32 * i;
        if (4 * c >= d) continue;
        const float u0 = v[i].x * inv, u1 = v[i].y * inv, u2 = v[i].z * inv, u3 = v[i].w * inv;
        const float h0 = __bfloat162float(__float2bfloat16_rn(u0)), h1 = __bfloat162float(__float2bfloat16_rn(u1));
        const float h2 = __bfloat162float(__float2bfloat16_rn(u2)), h3 = __bfloat162float(__float2bfloat16_rn(u3));
        *reinterpret_cast<uint2*>(L1 + r * dpad + 4 * c) = make_uint2(pack_bf16x2(h0, h1), pack_bf16x2(h2, h3));
        *reinterpret_cast<uint2*>(L2 + r * dpad + 4 * c) = make_uint2(pack_bf16x2(u0 - h0, u1 - h1), pack_bf16x2(u2 - h2, u3 - h3));
      }
    }
  }
}

// One warp per row: nu = ||x|| (optional), u = x / nu, u = hi + lo in bf16.  Rows warp, warp + nwarps, ...
template <typename T, bool NORMALIZE>
__device__ __forceinline__ void split_rows(const T* __restrict__ X, int64_t ldx, int64_t n, int d, int dpad,
                                           __nv_bfloat16* __restrict__ L1, __nv_bfloat16* __restrict__ L2,
                                           float* __restrict__ norms, int64_t warp, int64_t nwarps, int lane) {
  if constexpr (sizeof(T) == 4) {
    if ((d & 3) == 0 && (ldx & 3) == 0 && (reinterpret_cast<uintptr_t>(X) & 15) == 0 && dpad == d) {
      if (d <= 256) split_rows_vec<NORMALIZE, 2>(X, ldx, n, d, dpad, L1, L2, norms, warp, nwarps, lane);
      else if (d <= 512) split_rows_vec<NORMALIZE, 4>(X, ldx, n, d, dpad, L1, L2, norms, warp, nwarps, lane);
      else if (d <= 1024) split_rows_vec<NORMALIZE, 8>(X, ldx, n, d, dpad, L1, L2, norms, warp, nwarps, lane);
      else split_rows_vec<NORMALIZE, 16>(X, ldx, n, d, dpad, L1, L2, norms, warp, nwarps, lane);
      return;
    }
  }
  for (int64_t r = warp; r < n; r += nwarps) {
    const T* row = X + r * ldx;
    float inv = 1.f;
    if (NORMALIZE) {
      float s = 0.f;
      for (int j = lane; j < d; j += 32) {
        float v;
        if constexpr (sizeof(T) == 4) v = row[j]; else v = __bfloat162float(row[j]);
        s = fmaf(v, v, s);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const float nu = sqrtf(s);
      inv = (nu > 0.f) ? 1.f / nu : 0.f;
      if (lane == 0 && norms != nullptr) norms[r] = nu;
    }
    for (int j0 = lane * 8; j0 < dpad; j0 += 256) {
      uint32_t h[4], l[4];
#pragma unroll
      for (int p = 0; p < 4; ++p) {
        float u[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int j = j0 + 2 * p + q;
          float v = 0.f;
          if (j < d) {
            if constexpr (sizeof(T) == 4) v = row[j]; else v = __bfloat162float(row[j]);
          }
          u[q] = v * inv;
        }
        const float h0 = __bfloat162float(__float2bfloat16_rn(u[0]));
        const float h1 = __bfloat162float(__float2bfloat16_rn(u[1]));
        h[p] = pack_bf16x2(h0, h1);
        l[p] = pack_bf16x2(u[0] - h0, u[1] - h1);
      }
      *reinterpret_cast<uint4*>(L1 + r * dpad + j0) = make_uint4(h[0], h[1], h[2], h[3]);
      *reinterpret_cast<uint4*>(L2 + r * dpad + j0) = make_uint4(l[0], l[1], l[2], l[3]);
    }
  }
}

template <typename T, bool NORMALIZE>
__global__ void __launch_bounds__(256) split_rows_kernel(const T* __restrict__ X, int64_t ldx, int64_t n, int d, int dpad,
                                                         __nv_bfloat16* __restrict__ L1, __nv_bfloat16* __restrict__ L2,
                                                         float* __restrict__ norms) {
  split_rows<T, NORMALIZE>(X, ldx, n, d, dpad, L1, L2, norms, (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5),
                           (int64_t)gridDim.x * (blockDim.x >> 5), threadIdx.x & 31);
}

// MODE 0: idx.  MODE 1: idx + residual limbs + partial ||e||^2.  MODE 2: sign bits.
template <int BN, int MODE, int BITS, int CTAS>
__global__ void __launch_bounds__(NTHREADS, 1)
quantize_gemm_kernel(const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmA2,
                     const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                     const __grid_constant__ CUtensorMap tmE1, const __grid_constant__ CUtensorMap tmE2, GemmArgs a) {
  using C = Cfg<BN, CTAS>;
  const int rank = CTAS == 2 ? (int)cluster_ctarank() : 0;   // CTA of the pair; rank 0 issues the MMAs
  const int64_t unit = blockIdx.x / CTAS, nunits = gridDim.x / CTAS;   // a unit = one CTA or one pair
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::kStages * C::kStageBytes);
  uint64_t* full = bars;                    // [kStages]  TMA -> MMA
  uint64_t* empty = bars + C::kStages;      // [kStages]  MMA -> TMA
  uint64_t* tfull = bars + 2 * C::kStages;  // [2]        MMA -> epilogue
  uint64_t* tempty = tfull + 2;             // [2]        epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // the centroids in shared memory: indexed by the code they are one wavefront per load, where the same index into
  // the kernel's constant arguments is replayed once per distinct code of the warp
  float* cs = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(bars) + 128);   // [16]
  unsigned char* stg = reinterpret_cast<unsigned char*>(bars) + 512;                    // [4 EPS][2048], 512-byte aligned
  if (MODE == 1 && threadIdx.x < 16) cs[threadIdx.x] = a.cb.c[threadIdx.x];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (a.K + BK - 1) / BK;
  const int64_t num_tiles = (int64_t)a.tiles_m * a.tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&tfull[i], 1);
      mbar_init(&tempty[i], 4 * EPS * CTAS);   // the leader's: the epilogue warps of both CTAs arrive
    }
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmA1);
    tma_prefetch_desc(&tmA2);
    tma_prefetch_desc(&tmB1);
    tma_prefetch_desc(&tmB2);
  }
  if (warp == 1) {
    if (CTAS == 2) tmem_alloc_pair(tmem_slot, C::kTmemCols);
    else tmem_alloc(tmem_slot, C::kTmemCols);
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync();   // the partner's barriers exist before anything arrives on them
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t t = unit; t < num_tiles && ok; t += nunits) {
        const int m0 = ((int)(t / a.tiles_n) * CTAS + rank) * BM, n0 = (int)(t % a.tiles_n) * BN + rank * C::kBRows;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(&empty[stage], phase ^ 1u, abort_flag, a.status))) break;
          unsigned char* sa = smem + stage * C::kStageBytes;
          if (CTAS == 2) {
            // both CTAs' bytes are counted on the leader's barrier, which the leader arms for both
            if (rank == 0) mbar_arrive_expect_tx(&full[stage], 2 * C::kStageBytes);
            tma_load_2d_pair(sa, &tmA1, &full[stage], kb * BK, m0);
            tma_load_2d_pair(sa + BM * BK * 2, &tmA2, &full[stage], kb * BK, m0);
            tma_load_2d_pair(sa + 2 * BM * BK * 2, &tmB1, &full[stage], kb * BK, n0);
            tma_load_2d_pair(sa + 2 * BM * BK * 2 + C::kBRows * BK * 2, &tmB2, &full[stage], kb * BK, n0);
          } else {
            mbar_arrive_expect_tx(&full[stage], C::kStageBytes);
            tma_load_2d(sa, &tmA1, &full[stage], kb * BK, m0);
            tma_load_2d(sa + BM * BK * 2, &tmA2, &full[stage], kb * BK, m0);
            tma_load_2d(sa + 2 * BM * BK * 2, &tmB1, &full[stage], kb * BK, n0);
            tma_load_2d(sa + 2 * BM * BK * 2 + BN * BK * 2, &tmB2, &full[stage], kb * BK, n0);
          }
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        // let copies already in flight land before the CTA's shared memory is given up
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(BM * CTAS, BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int64_t it = 0;
      for (int64_t t = unit; t < num_tiles && ok; t += nunits, ++it) {
        const uint32_t acc = (uint32_t)(it & 1), acc_phase = (uint32_t)((it >> 1) & 1);
        if (!(ok = mbar_wait(&tempty[acc], acc_phase ^ 1u, abort_flag, a.status))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!(ok = mbar_wait(&full[stage], phase, abort_flag, a.status))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * C::kStageBytes);
          const uint64_t a1 = smem_desc_sw128(sa), a2 = smem_desc_sw128(sa + BM * BK * 2);
          const uint64_t b1 = smem_desc_sw128(sa + 2 * BM * BK * 2);
          const uint64_t b2 = smem_desc_sw128(sa + 2 * BM * BK * 2 + C::kBRows * BK * 2);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t off = (uint64_t)((k * UMMA_K * 2) >> 4);   // 32 bytes per K step
            if (CTAS == 2) {
              umma_bf16_pair(d_tmem, a1 + off, b2 + off, idesc, (kb | k) != 0 ? 1u : 0u);   // hi * lo
              umma_bf16_pair(d_tmem, a2 + off, b1 + off, idesc, 1u);                        // lo * hi
              umma_bf16_pair(d_tmem, a1 + off, b1 + off, idesc, 1u);                        // hi * hi
            } else {
              umma_bf16(d_tmem, a1 + off, b2 + off, idesc, (kb | k) != 0 ? 1u : 0u);
              umma_bf16(d_tmem, a2 + off, b1 + off, idesc, 1u);
              umma_bf16(d_tmem, a1 + off, b1 + off, idesc, 1u);
            }
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (CTAS == 2) umma_commit_pair(&empty[stage]);
          else umma_commit(&empty[stage]);
          if (++stage == C::kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (ok) {
          if (CTAS == 2) umma_commit_pair(&tfull[acc]);
          else umma_commit(&tfull[acc]);
        }
      }
    }
    __syncwarp();
  } else if (warp >= 2 + 4 * EPS) {
    // ------------------------------------------------------------ operand limbs of the next block of rows
    const GemmArgs::SplitTask& t = a.split;
    if (t.rows > 0) {
      const int64_t sw = (int64_t)blockIdx.x * NSPLIT + (warp - 2 - 4 * EPS), nsw = (int64_t)gridDim.x * NSPLIT;
      if (t.is_f32) {
        const float* X = static_cast<const float*>(t.X);
        if (t.normalize) split_rows<float, true>(X, t.ldx, t.rows, t.d, t.dpad, t.L1, t.L2, t.norms, sw, nsw, lane);
        else split_rows<float, false>(X, t.ldx, t.rows, t.d, t.dpad, t.L1, t.L2, t.norms, sw, nsw, lane);
      } else {
        const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(t.X);
        if (t.normalize) split_rows<__nv_bfloat16, true>(X, t.ldx, t.rows, t.d, t.dpad, t.L1, t.L2, t.norms, sw, nsw, lane);
        else split_rows<__nv_bfloat16, false>(X, t.ldx, t.rows, t.d, t.dpad, t.L1, t.L2, t.norms, sw, nsw, lane);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (4 x EPS warps: 4 TMEM lane groups x EPS column parts)
    const int lg = warp & 3;   // TMEM lane group this warp may read
    const int half = (warp - 2) >> 2;   // which part (of EPS) of the tile's columns this warp takes
    bool ok = true;
    int64_t it = 0;
    for (int64_t t = unit; t < num_tiles && ok; t += nunits, ++it) {
      const uint32_t acc = (uint32_t)(it & 1), acc_phase = (uint32_t)((it >> 1) & 1);
      const int tm = (int)(t / a.tiles_n), tn = (int)(t % a.tiles_n);
      const int64_t row = (int64_t)(tm * CTAS + rank) * BM + lg * 32 + lane;
      const int n0 = tn * BN;
      if (!(ok = mbar_wait(&tfull[acc], acc_phase, abort_flag, a.status))) break;
      tc_fence_after();
      const bool row_ok = row < a.M;
      bool zero_row = false;
      if (MODE == 1 && a.nu != nullptr && row_ok) zero_row = (__ldg(a.nu + row) == 0.f);
      float gsum = 0.f;
      uint32_t* out_row = reinterpret_cast<uint32_t*>(a.out + (size_t)(row_ok ? row : 0) * a.out_rb);
      const size_t row_words = a.out_rb / 4;
#pragma unroll 1
      for (int c = half * (BN / 32 / EPS); c < (half + 1) * (BN / 32 / EPS); ++c) {
        const int col0 = n0 + c * 32;
        if (col0 >= a.N) break;   // uniform across the CTA: nothing but zero padding beyond
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(lg * 32) << 16) + acc * BN + c * 32, v);
        tmem_ld_wait();
        if (MODE == 2) {
          uint32_t word = 0;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const bool bit = (__uint_as_float(v[i]) >= 0.f) && (col0 + i < a.N);
            word |= (bit ? 1u : 0u) << i;
          }
          const size_t w = (size_t)(col0 >> 5);
          if (a.nibble) {
            const size_t off = 16 * w;   // the group's four words of the combined row
            if (row_ok && off < a.nib_idx_rb + a.nib_qjl_rb) {
              uint4* dst = reinterpret_cast<uint4*>(off < a.nib_idx_rb ? a.nib_idx + (size_t)row * a.nib_idx_rb + off
                                                                       : a.nib_qjl + (size_t)row * a.nib_qjl_rb + (off - a.nib_idx_rb));
              uint4 cur = *dst;   // written by the rotate launch of the same block of rows
              cur.x |= spread_to_nibble_tops(word);
              cur.y |= spread_to_nibble_tops(word >> 8);
              cur.z |= spread_to_nibble_tops(word >> 16);
              cur.w |= spread_to_nibble_tops(word >> 24);
              *dst = cur;
            }
          } else if (row_ok && w < row_words) {
            out_row[w] = word;
          }
        } else {
          constexpr int NB = (1 << BITS) - 1;
          unsigned long long bitbuf = 0;
          int nb = 0, nw = 0;
          uint32_t words[BITS > 0 ? BITS : 1];
          uint32_t nibw[4] = {0u, 0u, 0u, 0u};
          uint32_t e1[16], e2[16];
#pragma unroll
          for (int i2 = 0; i2 < 16; ++i2) {
            float ehi[2] = {0.f, 0.f}, elo[2] = {0.f, 0.f};
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int i = 2 * i2 + q;
              const float y = __uint_as_float(v[i]);
              const bool col_ok = (col0 + i < a.N);
              int code = 0;
#pragma unroll
              for (int tix = 0; tix < NB; ++tix) code += (y > a.cb.t[tix]) ? 1 : 0;
              if (!col_ok) code = 0;
              if (BITS == 3 && MODE == 1) nibw[i >> 3] |= (uint32_t)code << (4 * (i & 7));
              if (BITS > 0) {
                bitbuf |= (unsigned long long)code << nb;
                nb += BITS;
                if (nb >= 32) {
                  words[nw++] = (uint32_t)bitbuf;
                  bitbuf >>= 32;
                  nb -= 32;
                }
              }
              if (MODE == 1) {
                const float e = (col_ok && !zero_row) ? (y - cs[code]) : 0.f;
                gsum = fmaf(e, e, gsum);
                ehi[q] = __bfloat162float(__float2bfloat16_rn(e));
                elo[q] = e - ehi[q];
              }
            }
            if (MODE == 1) {
              e1[i2] = pack_bf16x2(ehi[0], ehi[1]);
              e2[i2] = pack_bf16x2(elo[0], elo[1]);
            }
          }
          if (BITS == 3 && MODE == 1 && a.nibble) {
            const size_t off = 16 * (size_t)(col0 >> 5);
            if (row_ok && off < a.nib_idx_rb + a.nib_qjl_rb) {
              uint4* dst = reinterpret_cast<uint4*>(off < a.nib_idx_rb ? a.nib_idx + (size_t)row * a.nib_idx_rb + off
                                                                       : a.nib_qjl + (size_t)row * a.nib_qjl_rb + (off - a.nib_idx_rb));
              *dst = make_uint4(nibw[0], nibw[1], nibw[2], nibw[3]);
            }
          } else if (BITS > 0 && row_ok) {
            const size_t w0 = (size_t)(col0 >> 5) * BITS;
#pragma unroll
            for (int q = 0; q < BITS; ++q)
              if (w0 + q < row_words) out_row[w0 + q] = words[q];
          }
          if (MODE == 1) {
            // The warp's 32 rows x 32 columns of each residual limb go out as one TMA store: a row per thread, staged in
            // shared memory in the 64-byte swizzle (16-byte piece q of row r at q ^ ((r >> 1) & 3): four wavefronts per
            // instruction, the minimum for 512 bytes).  Stores straight from the registers were 16 bytes per lane at the
            // matrix's row stride, 32 lines per instruction, and cost a tenth of the whole quantiser.  Rows past M and
            // columns past N hold zeros or scratch inside the buffer's padding; the map clips columns past ldE.
            unsigned char* buf = stg + (warp - 2) * 2048;
            const int64_t row0 = row - lane;
            {   // (the map is Mpad rows high: a tile that overhangs the buffer is clipped by the store itself)
              const uint32_t sw = (uint32_t)((lane >> 1) & 3);
#pragma unroll
              for (int limb = 0; limb < 2; ++limb) {
                if (lane == 0) tma_store_wait_read();   // the previous box has left the buffer
                __syncwarp();
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const uint32_t* e = limb == 0 ? e1 : e2;
                  *reinterpret_cast<uint4*>(buf + lane * 64 + ((q ^ sw) << 4)) = make_uint4(e[4 * q], e[4 * q + 1], e[4 * q + 2], e[4 * q + 3]);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) {
                  tma_store_2d(limb == 0 ? &tmE1 : &tmE2, buf, col0, (int)row0);
                  tma_store_commit();
                }
              }
            }
          }
        }
      }
      // accumulator fully read: hand the TMEM buffer back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2) mbar_arrive_leader(&tempty[acc]);
        else mbar_arrive(&tempty[acc]);
      }
      if (MODE == 1 && row_ok && TQ_DEVICE_CHECK(row < a.Mpad && tn < a.tiles_n, a.status))
        a.gpart[(int64_t)(EPS * tn + half) * a.Mpad + row] = gsum;
      // pad words past the last tile's columns (rows whose stride exceeds the tiles' coverage)
      if (a.nibble && tn == a.tiles_n - 1 && half == EPS - 1 && row_ok) {
        if (MODE == 1) {   // words of the combined row that no group of 32 coordinates owns
          const size_t wi = a.nib_idx_rb / 4, wq = a.nib_qjl_rb / 4;
          for (size_t w = (size_t)((a.N + 31) >> 5) * 4; w < wi + wq; ++w)
            (w < wi ? reinterpret_cast<uint32_t*>(a.nib_idx + (size_t)row * a.nib_idx_rb)[w]
                    : reinterpret_cast<uint32_t*>(a.nib_qjl + (size_t)row * a.nib_qjl_rb)[w - wi]) = 0u;
        }
      } else if (tn == a.tiles_n - 1 && half == EPS - 1 && row_ok) {
        constexpr int kBitsPerCoord = (MODE == 2) ? 1 : BITS;
        if (kBitsPerCoord > 0) {
          const size_t covered = (size_t)((a.N + 31) >> 5) * kBitsPerCoord;
          for (size_t w = covered; w < row_words; ++w) out_row[w] = 0u;
        }
      }
    }
    if (MODE == 1) {   // the residual stores of this warp have completed before the CTA gives up its shared memory
      if (lane == 0) tma_store_wait_all();
      __syncwarp();
    }
  }

  tc_fence_before();
  if (CTAS == 2) cluster_sync();   // neither CTA leaves while the partner may still arrive on its barriers or read its rows
  else __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, C::kTmemCols);
    else tmem_dealloc(tmem_base, C::kTmemCols);
  }
}

// ---------------------------------------------------------------- operand splitting
// gamma = sqrt(sum over column tiles of the partial sums), in tile order (deterministic).
__global__ void gamma_finish_kernel(const float* __restrict__ gpart, int64_t Mpad, int tiles_n, int64_t rows,
                                    float* __restrict__ gamma) {
  const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  float s = 0.f;
  for (int t = 0; t < tiles_n; ++t) s += gpart[(int64_t)t * Mpad + r];
  gamma[r] = sqrtf(s);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// bf16 matrix [rows, cols] with row pitch `pitch` elements; box = 64 columns x box_rows, 128B swizzle.
bool make_map(CUtensorMap* map, const __nv_bfloat16* base, int64_t rows, int cols, int64_t pitch, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 matrix [rows, cols] with row pitch `pitch` elements, for TMA stores of [32 rows x 32 columns] boxes staged in
// shared memory in the 64-byte swizzle.
bool make_store_map(CUtensorMap* map, __nv_bfloat16* base, int64_t rows, int64_t cols, int64_t pitch) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Byte matrix [rows, row_bytes] with row pitch `pitch` bytes; box = box_bytes x box_rows; `swizzle` = 0 (plain
// rows in shared memory) or 32 / 64 / 128 (that swizzle span; box_bytes must not exceed it).
bool make_byte_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t row_bytes, uint64_t pitch,
                   uint32_t box_bytes, uint32_t box_rows, int swizzle) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)pitch};
  const cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = swizzle == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : swizzle == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                : CU_TENSOR_MAP_SWIZZLE_NONE;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static std::atomic<int> cached{0};   // all devices of a process are taken to be alike
  int sms = cached.load(std::memory_order_relaxed);
  if (sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cached.store(sms, std::memory_order_relaxed);
  }
  return sms;
}

namespace {

template <int BN, int MODE, int BITS, int CTAS>
cudaError_t launch_gemm_t(const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap& b1, const CUtensorMap& b2,
                          const GemmArgs& args, cudaStream_t st) {
  auto kern = quantize_gemm_kernel<BN, MODE, BITS, CTAS>;
  using C = Cfg<BN, CTAS>;
  // function attributes are per device: remember the devices this launcher has prepared
  static std::atomic<unsigned long long> attr_devices{0};   // written by any thread that launches
  int attr_dev = 0;
  if (cudaGetDevice(&attr_dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (attr_dev >= 64 || !((attr_devices.load(std::memory_order_relaxed) >> attr_dev) & 1ull)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    if (attr_dev < 64) attr_devices.fetch_or(1ull << attr_dev, std::memory_order_relaxed);
  }
  const int64_t tiles = (int64_t)args.tiles_m * args.tiles_n;   // tiles_m counts rows of BM * CTAS
  const int units = (int)std::min<int64_t>(tiles, sm_count() / CTAS);
  count_launches(1);
  // the store maps of the residual limbs (MODE 1); any valid map otherwise
  const CUtensorMap& e1 = args.store_e1 ? *args.store_e1 : a1;
  const CUtensorMap& e2 = args.store_e2 ? *args.store_e2 : a2;
  if (CTAS == 1) {
    kern<<<units, NTHREADS, C::kSmemBytes, st>>>(a1, a2, b1, b2, e1, e2, args);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(units * CTAS));
  cfg.blockDim = dim3(NTHREADS);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, a1, a2, b1, b2, e1, e2, args);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <int BN, int MODE, int CTAS>
cudaError_t launch_gemm_bits(int bits, const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap& b1,
                             const CUtensorMap& b2, const GemmArgs& args, cudaStream_t st) {
  if constexpr (MODE == 2) {
    return launch_gemm_t<BN, 2, 1, CTAS>(a1, a2, b1, b2, args, st);
  } else {
    switch (bits) {
      case 0: return launch_gemm_t<BN, MODE, 0, CTAS>(a1, a2, b1, b2, args, st);
      case 1: return launch_gemm_t<BN, MODE, 1, CTAS>(a1, a2, b1, b2, args, st);
      case 2: return launch_gemm_t<BN, MODE, 2, CTAS>(a1, a2, b1, b2, args, st);
      case 3: return launch_gemm_t<BN, MODE, 3, CTAS>(a1, a2, b1, b2, args, st);
      default: return launch_gemm_t<BN, MODE, 4, CTAS>(a1, a2, b1, b2, args, st);
    }
  }
}

// ctas = 2: CTA pairs (only with 256-column tiles); b1, b2 are then the maps with half-height boxes.
template <int MODE>
cudaError_t launch_gemm(int bn, int ctas, int bits, const CUtensorMap& a1, const CUtensorMap& a2, const CUtensorMap& b1,
                        const CUtensorMap& b2, const GemmArgs& args, cudaStream_t st) {
  if (bn == 256 && ctas == 2) return launch_gemm_bits<256, MODE, 2>(bits, a1, a2, b1, b2, args, st);
  if (bn == 256) return launch_gemm_bits<256, MODE, 1>(bits, a1, a2, b1, b2, args, st);
  return launch_gemm_bits<128, MODE, 1>(bits, a1, a2, b1, b2, args, st);
}

}  // namespace

int pick_bn(int d) { return d > 128 ? 256 : 128; }

bool supported(int d) { return d >= 128 && encode_fn() != nullptr; }

cudaError_t build_matrix_limbs(const float* dM, int rows, int d, int dpad, int bn, MatrixLimbs* out) {
  out->hi = out->lo = nullptr;
  const size_t bytes = (size_t)rows * dpad * sizeof(__nv_bfloat16);
  cudaError_t e = cudaMalloc(&out->hi, bytes);
  if (e != cudaSuccess) return e;
  e = cudaMalloc(&out->lo, bytes);
  if (e != cudaSuccess) return e;
  const int blocks = std::min((rows + 7) / 8, 148 * 8);
  split_rows_kernel<float, false><<<blocks, 256>>>(dM, d, rows, d, dpad, out->hi, out->lo, nullptr);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (!make_map(&out->map_hi, out->hi, rows, d, dpad, bn) || !make_map(&out->map_lo, out->lo, rows, d, dpad, bn) ||
      !make_map(&out->map_hi_half, out->hi, rows, d, dpad, bn / 2) || !make_map(&out->map_lo_half, out->lo, rows, d, dpad, bn / 2))
    return cudaErrorInvalidValue;
  return cudaSuccess;
}

void free_matrix_limbs(MatrixLimbs* m) {
  cudaFree(m->hi);
  cudaFree(m->lo);
  m->hi = m->lo = nullptr;
}

// CTA pairs can be switched off (TQ_GEMM_PAIRS=0) to compare the two kernels on one machine.
bool pair_tiles_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("TQ_GEMM_PAIRS");
    return e == nullptr || e[0] != '0';
  }();
  return on;
}

size_t scratch_bytes_per_row(const tq_plan* plan) {
  const int tiles_n = (plan->d + plan->tc_bn - 1) / plan->tc_bn;
  size_t per = (size_t)plan->dpad * 2 * 2 + sizeof(float);                            // X limbs + nu
  if (plan->mode == TQ_PROD) per += (size_t)plan->dpad * 2 * 2 + (size_t)tiles_n * 4 * EPS;  // E limbs + partial sums (EPS per column tile)
  return per;
}

int quantize(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx, uint8_t* idx, uint8_t* qjl,
             float* gamma, float* norms, void* scratch, size_t scratch_bytes, cudaStream_t st, const char* who) {
  const int d = plan->d, dpad = plan->dpad, bn = plan->tc_bn;
  const int tiles_n = (d + bn - 1) / bn;
  const bool prod = plan->mode == TQ_PROD;
  const size_t per_row = scratch_bytes_per_row(plan);
  int64_t R = (int64_t)(scratch_bytes / per_row) / BM * BM;
  R = std::min<int64_t>(R, round_up64(n, BM));
  TQ_REQUIRE(R >= BM, TQ_ERR_WORKSPACE, "%s: scratch of %zu bytes cannot hold one block of %d rows", who, scratch_bytes, BM);
  // The operand limbs of block i + 1 are prepared by spare warps of a GEMM launch of block i.  TQ_PROD: the project
  // launch (its A operand is the residual, the limbs of X are free by then), one set of limb buffers.  TQ_MSE: the
  // rotate launch itself, so the scratch is used as two half-size sets written and read in turn (when the data
  // spans more than one block and each half still holds a tile).
  // Two warps per CTA keep up only while the GEMM gives them time: its work per row grows with d^2, theirs with d.
  // Measured per 10^6 rows with the CTA-pair GEMMs: TQ_MSE d = 1536 10.1 ms with them against 10.6 without; TQ_PROD
  // loses (d = 1536: 22.1 against 21.5 ms, d = 3072 alike), so its project launch carries no such task any more; at
  // d = 1024 and below the spare warps are the critical path for both.
  const bool overlap = !prod && d >= 1536;
  const bool pingpong = overlap && !prod && n > R / 2 / BM * BM && R / 2 >= BM;
  const int64_t Rbuf = R;   // rows the carved buffers hold in all
  if (pingpong) R = R / 2 / BM * BM;
  // carve the scratch (every part is a multiple of 256 bytes because Rbuf is a multiple of 128)
  char* p = static_cast<char*>(scratch);
  __nv_bfloat16* XL1 = reinterpret_cast<__nv_bfloat16*>(p); p += (size_t)Rbuf * dpad * 2;
  __nv_bfloat16* XL2 = reinterpret_cast<__nv_bfloat16*>(p); p += (size_t)Rbuf * dpad * 2;
  __nv_bfloat16 *EL1 = nullptr, *EL2 = nullptr;
  float* gpart = nullptr;
  if (prod) {
    EL1 = reinterpret_cast<__nv_bfloat16*>(p); p += (size_t)Rbuf * dpad * 2;
    EL2 = reinterpret_cast<__nv_bfloat16*>(p); p += (size_t)Rbuf * dpad * 2;
    gpart = reinterpret_cast<float*>(p); p += (size_t)Rbuf * tiles_n * 4 * EPS;
  }
  // limb buffers of block number b
  auto limbs1 = [&](int64_t b) { return XL1 + (pingpong && (b & 1) ? (size_t)R * dpad : 0); };
  auto limbs2 = [&](int64_t b) { return XL2 + (pingpong && (b & 1) ? (size_t)R * dpad : 0); };
  const size_t xsz = (x_dtype == TQ_F32) ? 4 : 2;
  auto launch_split = [&](int64_t r0, cudaStream_t s) -> cudaError_t {
    const int64_t rows = std::min(R, n - r0);
    const void* Xc = static_cast<const char*>(X) + (size_t)r0 * ldx * xsz;
    float* nu_out = norms ? norms + r0 : nullptr;
    const int blocks = (int)std::min<int64_t>((rows + 7) / 8, (int64_t)sm_count() * 8);
    __nv_bfloat16 *L1 = limbs1(r0 / R), *L2 = limbs2(r0 / R);
    if (norms) {
      if (x_dtype == TQ_F32)
        split_rows_kernel<float, true><<<blocks, 256, 0, s>>>(static_cast<const float*>(Xc), ldx, rows, d, dpad, L1, L2, nu_out);
      else
        split_rows_kernel<__nv_bfloat16, true><<<blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(Xc), ldx, rows, d, dpad, L1, L2, nu_out);
    } else {
      if (x_dtype == TQ_F32)
        split_rows_kernel<float, false><<<blocks, 256, 0, s>>>(static_cast<const float*>(Xc), ldx, rows, d, dpad, L1, L2, nullptr);
      else
        split_rows_kernel<__nv_bfloat16, false><<<blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(Xc), ldx, rows, d, dpad, L1, L2, nullptr);
    }
    count_launches(1);
    return cudaGetLastError();
  };
  for (int64_t r0 = 0; r0 < n; r0 += R) {
    const int64_t rows = std::min(R, n - r0);
    float* nu_out = norms ? norms + r0 : nullptr;
    // 1. nu, u = x / nu, bf16 limbs of u: by a launch of its own for the first block (and for TQ_MSE plans), by the
    //    spare warps of the previous block's project launch otherwise
    if (r0 == 0 || !overlap || (!prod && !pingpong)) TQ_CHECK_CUDA(launch_split(r0, st), who);
    __nv_bfloat16 *XLc1 = limbs1(r0 / R), *XLc2 = limbs2(r0 / R);
    auto next_block_task = [&](GemmArgs& ga) {
      ga.split.X = static_cast<const char*>(X) + (size_t)(r0 + R) * ldx * xsz;
      ga.split.ldx = ldx;
      ga.split.rows = std::min(R, n - (r0 + R));
      ga.split.d = d;
      ga.split.dpad = dpad;
      ga.split.is_f32 = x_dtype == TQ_F32 ? 1 : 0;
      ga.split.normalize = norms ? 1 : 0;
      ga.split.L1 = limbs1(r0 / R + 1);
      ga.split.L2 = limbs2(r0 / R + 1);
      ga.split.norms = norms ? norms + r0 + R : nullptr;
    };

    CUtensorMap mA1, mA2;
    TQ_REQUIRE(make_map(&mA1, XLc1, rows, d, dpad, BM) && make_map(&mA2, XLc2, rows, d, dpad, BM), TQ_ERR_CUDA,
               "%s: cuTensorMapEncodeTiled failed", who);
    GemmArgs g;
    g.M = rows;
    g.N = d;
    g.K = d;
    // CTA pairs on 256-row tiles where the tile is 256 columns wide and the block has more rows than one CTA's tile
    const int ctas = (bn == 256 && pair_tiles_enabled() && rows > BM) ? 2 : 1;
    g.tiles_m = (int)((rows + BM * ctas - 1) / (BM * ctas));
    g.tiles_n = tiles_n;
    g.cb = plan->cb;
    g.out = idx ? idx + (size_t)r0 * plan->idx_row_bytes : nullptr;
    g.out_rb = plan->idx_row_bytes;
    g.E1 = EL1;
    g.E2 = EL2;
    g.ldE = dpad;
    CUtensorMap sE1, sE2;
    g.store_e1 = g.store_e2 = nullptr;
    if (prod) {
      TQ_REQUIRE(make_store_map(&sE1, EL1, R, dpad, dpad) && make_store_map(&sE2, EL2, R, dpad, dpad), TQ_ERR_CUDA,
                 "%s: cuTensorMapEncodeTiled failed (residual stores)", who);
      g.store_e1 = &sE1;
      g.store_e2 = &sE2;
    }
    g.gpart = gpart;
    g.Mpad = R;
    g.nu = nu_out;
    g.split.rows = 0;
    g.nibble = (plan->layout == TQ_LAYOUT_NIBBLE) ? 1 : 0;
    g.nib_idx = idx ? idx + (size_t)r0 * plan->idx_row_bytes : nullptr;
    g.nib_qjl = qjl ? qjl + (size_t)r0 * plan->qjl_row_bytes : nullptr;
    g.nib_idx_rb = plan->idx_row_bytes;
    g.nib_qjl_rb = plan->qjl_row_bytes;
    g.status = plan->d_status;
    // 2. y = Pi u, idx (+ residual limbs and partial norms)
    if (!prod) {
      if (pingpong && r0 + R < n) next_block_task(g);
      TQ_CHECK_CUDA(launch_gemm<0>(bn, ctas, plan->mse_bits, mA1, mA2, ctas == 2 ? plan->pi_limbs.map_hi_half : plan->pi_limbs.map_hi,
                                   ctas == 2 ? plan->pi_limbs.map_lo_half : plan->pi_limbs.map_lo, g, st), who);
      continue;
    }
    TQ_CHECK_CUDA(launch_gemm<1>(bn, ctas, plan->mse_bits, mA1, mA2, ctas == 2 ? plan->pi_limbs.map_hi_half : plan->pi_limbs.map_hi,
                                 ctas == 2 ? plan->pi_limbs.map_lo_half : plan->pi_limbs.map_lo, g, st), who);
    // 3. gamma = ||e||
    gamma_finish_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(gpart, R, EPS * tiles_n, rows, gamma + r0);
    count_launches(1);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
    // 4. qjl = sign(S' e)
    CUtensorMap mE1, mE2;
    TQ_REQUIRE(make_map(&mE1, EL1, rows, d, dpad, BM) && make_map(&mE2, EL2, rows, d, dpad, BM), TQ_ERR_CUDA,
               "%s: cuTensorMapEncodeTiled failed", who);
    g.out = qjl + (size_t)r0 * plan->qjl_row_bytes;
    g.out_rb = plan->qjl_row_bytes;
    if (overlap && r0 + R < n) next_block_task(g);   // the limbs of X are free by now
    TQ_CHECK_CUDA(launch_gemm<2>(bn, ctas, 1, mE1, mE2, ctas == 2 ? plan->sp_limbs.map_hi_half : plan->sp_limbs.map_hi,
                                 ctas == 2 ? plan->sp_limbs.map_lo_half : plan->sp_limbs.map_lo, g, st), who);
  }
  return TQ_OK;
}

}  // namespace tc
}  // namespace tq

// C ABI of libtq: argument checking, plan set-up and kernel dispatch.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "tq_attend_simt.cuh"
#include "tq_gemm_simt.cuh"
#include "tq_internal.h"
#include "tq_quantize_tc.h"
#include "tq_scan_mma.h"
#include "tq_scan_nib.h"
#include "tq_scan_simt.cuh"
#include "tq_scan_tc.h"
#include "tq_tc.cuh"

using namespace tq;

namespace {

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// S' = S Pi^T in fp64 (set-up, once per plan): out[i][j] = sum_k S[i][k] Pi[j][k].
__global__ void sprime_kernel(const float* __restrict__ S, const float* __restrict__ Pi, float* __restrict__ out, int d) {
  __shared__ double sa[16][17], sb[16][17];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int i = blockIdx.y * 16 + ty, j = blockIdx.x * 16 + tx;
  double acc = 0.0;
  for (int k0 = 0; k0 < d; k0 += 16) {
    const int ia = blockIdx.y * 16 + ty, jb = blockIdx.x * 16 + ty;
    sa[ty][tx] = (ia < d && k0 + tx < d) ? (double)S[(size_t)ia * d + k0 + tx] : 0.0;
    sb[ty][tx] = (jb < d && k0 + tx < d) ? (double)Pi[(size_t)jb * d + k0 + tx] : 0.0;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) acc += sa[ty][k] * sb[tx][k];
    __syncthreads();
  }
  if (i < d && j < d) out[(size_t)i * d + j] = (float)acc;
}

int check_plan(const tq_plan* plan, const char* who) {
  TQ_REQUIRE(plan != nullptr, TQ_ERR_INVALID_ARG, "%s: plan is NULL", who);
  int dev = -1;
  TQ_CHECK_CUDA(cudaGetDevice(&dev), who);
  TQ_REQUIRE(dev == plan->device, TQ_ERR_INVALID_ARG, "%s: plan was created on device %d, current device is %d", who,
             plan->device, dev);
  return TQ_OK;
}

int check_rows(const char* who, const char* name, const void* p, int dtype, int64_t rows, int64_t ld, int d) {
  TQ_REQUIRE(dtype == TQ_F32 || dtype == TQ_BF16, TQ_ERR_UNSUPPORTED, "%s: unknown dtype %d for %s", who, dtype, name);
  TQ_REQUIRE(p != nullptr, TQ_ERR_INVALID_ARG, "%s: %s is NULL", who, name);
  TQ_REQUIRE(ld >= d, TQ_ERR_INVALID_ARG, "%s: row stride of %s (%lld) is smaller than d (%d)", who, name, (long long)ld, d);
  TQ_REQUIRE(aligned(p, 16), TQ_ERR_ALIGNMENT, "%s: %s is not 16-byte aligned", who, name);
  (void)rows;
  return TQ_OK;
}

int check_codes(const tq_plan* plan, const char* who, const uint8_t* idx, const uint8_t* qjl, const float* gamma) {
  if (plan->mse_bits > 0) {
    TQ_REQUIRE(idx != nullptr, TQ_ERR_INVALID_ARG, "%s: idx is NULL", who);
    TQ_REQUIRE(aligned(idx, 16), TQ_ERR_ALIGNMENT, "%s: idx is not 16-byte aligned", who);
  }
  if (plan->mode == TQ_PROD) {
    TQ_REQUIRE(qjl != nullptr && gamma != nullptr, TQ_ERR_INVALID_ARG, "%s: qjl / gamma is NULL for a TQ_PROD plan", who);
    TQ_REQUIRE(aligned(qjl, 16) && aligned(gamma, 4), TQ_ERR_ALIGNMENT, "%s: qjl / gamma is misaligned", who);
  }
  return TQ_OK;
}

simt::Codes make_codes(const tq_plan* plan, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma) {
  simt::Codes c;
  c.idx = idx;
  c.idx_rb = plan->idx_row_bytes;
  c.qjl = (plan->mode == TQ_PROD) ? qjl : nullptr;
  c.qjl_rb = plan->qjl_row_bytes;
  c.gamma = gamma;
  c.cb = plan->cb;
  c.d = plan->d;
  c.dpad = plan->dpad;
  c.coef = plan->coef;
  c.rows = n;
  c.nibble = plan->layout == TQ_LAYOUT_NIBBLE;
  return c;
}

size_t qcat_bytes(const tq_plan* plan, int nq) {
  return align_up((size_t)nq * plan->ncat * plan->dpad * sizeof(float), 256);
}

constexpr int64_t kTensorChunk = 65536;    // rows per launch the tensor-core quantiser asks scratch for
constexpr int64_t kResidualChunk = 16384;  // rows of E kept in flight by tq_quantize_prod (L2-sized)
constexpr int64_t kTopkBlockMin = 4096, kTopkBlockPref = 65536;
constexpr int kFewQueries = 16;  // up to this many queries the code scan is bandwidth-bound
// top-k on the tensor-path scan: candidate pairs kept per query, queries per pass, dense-buffer rows
constexpr int kCandCap = 32768;
constexpr int64_t kFilterMinN = 65536;
constexpr int64_t kDenseRowsMin = 4096;
constexpr int kGroupQueries = tscan::kQueriesPerPass * tscan::kPassesPerGroup;

// The two engines behind the bit-plane scan: register-fed integer MMA (2 or 4 queries per pass) for few
// queries, tcgen05 (32 queries per pass, 64 in calls of more than 32 queries) from 7 queries on (measured at d = 1536, b = 4, n = 10^6: a short
// tcgen05 pass 0.69 ms, register-fed passes 0.24 ms for 1-2 queries and 0.37 ms for 3-4, so 4 + 3 queries
// already cost more).
struct ScanEngine {
  const tq_plan* plan;
  bool tc;
  bool nib;                 // register-fed table-lookup scan of the nibble layout (2 or 8 queries per pass)
  int qpp;                  // queries per pass
  int64_t dense_rows_pref;  // rows of the dense score buffer that keep the rescue pass to a few launches
  size_t ws_bytes;          // engine workspace (constants + B operand)
};

ScanEngine pick_engine(const tq_plan* plan, int nq) {
  ScanEngine e;
  e.plan = plan;
  e.nib = plan->layout == TQ_LAYOUT_NIBBLE;
  // nibble layout (measured at n = 10^6): at d = 1536 a tcgen05 pass costs 0.53 ms against 0.28 ms per pass of the
  // eight-query register-fed shape, so it wins from 15 queries on; where that shape does not fit shared memory
  // (d = 3072: 0.84 ms against 0.35 ms per two-query pass) from five queries on
  const int tc_from = !e.nib ? 7 : nscan::queries_per_pass(plan, 8) == 8 ? 15 : 5;
  e.tc = nq >= tc_from && tscan::available(plan);
  e.nib = e.nib && !e.tc;
  e.qpp = e.tc ? tscan::queries_per_pass(nq) : e.nib ? nscan::queries_per_pass(plan, nq) : mscan::queries_per_pass(plan, nq);
  e.dense_rows_pref = 1 << 20;   // n = 10^6: the guarded rescue is one scan + one selection launch per pass
  e.ws_bytes = e.tc ? tscan::workspace_bytes(plan) : e.nib ? nscan::workspace_bytes(plan) : mscan::workspace_bytes(plan);
  return e;
}

// Prepares what the pass starting at query q0 needs (the tcgen05 engine builds 256 queries at a time).
int engine_prepare(const ScanEngine& e, const float* Qcat, int q0, int nq, void* ws, cudaStream_t st, const char* who) {
  const int ncols = e.plan->ncat * e.plan->dpad;
  if (e.nib) return nscan::prepare(e.plan, Qcat + (size_t)q0 * ncols, std::min(e.qpp, nq - q0), ws, st, who);
  if (e.tc) {
    if (q0 % kGroupQueries != 0) return TQ_OK;
    return tscan::prepare_group(e.plan, Qcat + (size_t)q0 * ncols, std::min(kGroupQueries, nq - q0), ws, st, who);
  }
  return mscan::prepare(e.plan, Qcat + (size_t)q0 * ncols, std::min(e.qpp, nq - q0), ws, st, who);
}

int engine_run(const ScanEngine& e, int q0, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
               const float* norms, float* scores, int64_t lds, const mscan::Filter* filter, const int* run_if, const void* ws,
               cudaStream_t st, const char* who) {
  if (e.nib) return nscan::run(e.plan, nqp, n, idx, qjl, gamma, norms, scores, lds, filter, run_if, ws, true, st, who);
  if (e.tc)
    return tscan::run_pass(e.plan, (q0 % kGroupQueries) / tscan::kQueriesPerPass, nqp, n, idx, qjl, gamma, norms, scores, lds,
                           filter, run_if, ws, st, who);
  return mscan::run(e.plan, nqp, n, idx, qjl, gamma, norms, scores, lds, filter, run_if, ws, st, who);
}

size_t ms_score_fixed(const tq_plan* plan, int nq) { return qcat_bytes(plan, nq) + align_up(pick_engine(plan, nq).ws_bytes, 256); }
size_t ms_topk_fixed(const tq_plan* plan, int nq) {
  return ms_score_fixed(plan, nq) + 1024 /* tau, count, overflow */ + (size_t)pick_engine(plan, nq).qpp * kCandCap * 8;
}

template <typename T>
cudaError_t launch_row_norm(const T* X, int64_t ld, int64_t n, int d, float* out, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  const int64_t blocks = std::min<int64_t>((n + 7) / 8, 148 * 16);
  scan::row_norm_kernel<T><<<(unsigned)blocks, 256, 0, st>>>(X, ld, n, d, out);
  count_launches(1);
  return cudaGetLastError();
}

// Stage-1 GEMM of both quantisers: Y = X Pi^T with the nearest-centroid epilogue.
template <int BITS, int MODE>
cudaError_t launch_rotate_quantize(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx,
                                   const float* nu, uint8_t* idx, float* E, int64_t ldE, cudaStream_t st) {
  simt::EpQuantize<BITS, MODE> ep;
  ep.cb = plan->cb;
  ep.nu = nu;
  ep.out = idx;
  ep.out_rb = plan->idx_row_bytes;
  ep.E = E;
  ep.ldE = ldE;
  ep.d = plan->d;
  simt::RowsF32 B{plan->dPi, plan->d, plan->d, plan->d};
  if (x_dtype == TQ_F32) {
    simt::RowsF32 A{static_cast<const float*>(X), ldx, n, plan->d};
    return simt::launch_gemm(A, B, ep, n, (int64_t)plan->d, plan->d, st);
  }
  simt::RowsBF16 A{static_cast<const __nv_bfloat16*>(X), ldx, n, plan->d};
  return simt::launch_gemm(A, B, ep, n, (int64_t)plan->d, plan->d, st);
}

template <int MODE>
cudaError_t dispatch_rotate_quantize(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx,
                                     const float* nu, uint8_t* idx, float* E, int64_t ldE, cudaStream_t st) {
  switch (plan->mse_bits) {
    case 0: return launch_rotate_quantize<0, MODE>(plan, X, x_dtype, n, ldx, nu, idx, E, ldE, st);
    case 1: return launch_rotate_quantize<1, MODE>(plan, X, x_dtype, n, ldx, nu, idx, E, ldE, st);
    case 2: return launch_rotate_quantize<2, MODE>(plan, X, x_dtype, n, ldx, nu, idx, E, ldE, st);
    case 3: return launch_rotate_quantize<3, MODE>(plan, X, x_dtype, n, ldx, nu, idx, E, ldE, st);
    default: return launch_rotate_quantize<4, MODE>(plan, X, x_dtype, n, ldx, nu, idx, E, ldE, st);
  }
}

cudaError_t compute_norms(const void* X, int x_dtype, int64_t n, int64_t ldx, int d, float* norms, cudaStream_t st) {
  if (x_dtype == TQ_F32) return launch_row_norm(static_cast<const float*>(X), ldx, n, d, norms, st);
  return launch_row_norm(static_cast<const __nv_bfloat16*>(X), ldx, n, d, norms, st);
}

// True when the packed rows have bytes that no 32-coordinate group writes.
bool has_pad_words(int d, int bits, size_t row_bytes) {
  return bits > 0 && (size_t)((d + 31) / 32) * bits * 4 < row_bytes;
}

// Few queries: one warp per output column j forms <Rot[j, :], q> for up to 8 queries at a time.  The
// warp's slice of the matrix row goes to registers first, so that its latency overlaps the staging
// of the queries in shared memory; each lane sums its products in fp32, the 32 partial sums are
// added in fp64.  The matrix is read once per 8 queries.
constexpr int kRotQ = 8, kRotChunk = 2048;   // 64 KB of queries per chunk (dynamic shared memory)
constexpr int kRotQPerBlock = 64;            // queries per CTA (grid.y covers the rest)

template <typename T>
__global__ void __launch_bounds__(256) rotate_queries_kernel(const float* __restrict__ Rot, int nrows, int d,
                                                             const T* __restrict__ Q, int64_t ldq, int nq,
                                                             float* __restrict__ Qcat, int64_t ldo) {
  extern __shared__ __align__(16) float qs_raw[];
  float (*qs)[kRotChunk] = reinterpret_cast<float (*)[kRotChunk]>(qs_raw);
  // a successor launched as a programmatic dependent may be scheduled while this grid drains (it waits for
  // this grid's completion before it reads Qcat)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * 8 + warp;
  const float* row = Rot + (size_t)min(j, nrows - 1) * d;
  const bool vec = (d & 3) == 0;   // rows are 16-byte aligned
  const int q_begin = blockIdx.y * kRotQPerBlock, q_end = min(nq, q_begin + kRotQPerBlock);
  for (int q0 = q_begin; q0 < q_end; q0 += kRotQ) {
    float acc[kRotQ];
#pragma unroll
    for (int qq = 0; qq < kRotQ; ++qq) acc[qq] = 0.f;
    const int nact = min(kRotQ, q_end - q0);   // queries of this round: the others are neither staged nor summed
    for (int c0 = 0; c0 < d; c0 += kRotChunk) {
      const int len = min(kRotChunk, d - c0);
      float4 r[kRotChunk / 128];
      if (vec) {
        const float4* row4 = reinterpret_cast<const float4*>(row + c0);
#pragma unroll
        for (int i = 0; i < kRotChunk / 128; ++i) {
          const int c4 = lane + 32 * i;
          r[i] = (4 * c4 < len) ? __ldg(row4 + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
      __syncthreads();
      for (int e = threadIdx.x; e < nact * (kRotChunk / 4); e += blockDim.x) {
        const int qq = e / (kRotChunk / 4), c = 4 * (e % (kRotChunk / 4));
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        if (q0 + qq < q_end && c < len) {
          const T* src = Q + (int64_t)(q0 + qq) * ldq + c0 + c;
#pragma unroll
          for (int t = 0; t < 4; ++t)
            if (c + t < len) v[t] = scan::to_f32<T>(src[t]);
        }
        *reinterpret_cast<float4*>(&qs[qq][c]) = make_float4(v[0], v[1], v[2], v[3]);
      }
      __syncthreads();
      if (vec) {
#pragma unroll
        for (int i = 0; i < kRotChunk / 128; ++i) {
          const int c4 = lane + 32 * i;
          if (4 * c4 < len) {
#pragma unroll
            for (int qq = 0; qq < kRotQ; ++qq) {
              if (qq < nact) {
                const float4 v = *reinterpret_cast<const float4*>(&qs[qq][4 * c4]);
                acc[qq] = fmaf(r[i].x, v.x, fmaf(r[i].y, v.y, fmaf(r[i].z, v.z, fmaf(r[i].w, v.w, acc[qq]))));
              }
            }
          }
        }
      } else {
        for (int c = lane; c < len; c += 32) {
          const float rv = __ldg(row + c0 + c);
#pragma unroll
          for (int qq = 0; qq < kRotQ; ++qq)
            if (qq < nact) acc[qq] = fmaf(rv, qs[qq][c], acc[qq]);
        }
      }
    }
#pragma unroll
    for (int qq = 0; qq < kRotQ; ++qq) {
      if (qq >= nact) break;
      double v = (double)acc[qq];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && j < nrows && q0 + qq < q_end) Qcat[(int64_t)(q0 + qq) * ldo + j] = (float)v;
    }
  }
}

// Many queries: the same sums in the same order (a lane adds its products over ascending columns 4 lane + 128 i in
// fp32, the 32 partial sums are added in fp64 by the same butterfly), so a query's rotated form does not depend on
// which kernel formed it -- but a warp holds eight matrix rows against the eight staged queries (64 FMAs per pair of
// 16-byte loads), a CTA of four warps 32 rows, and the queries are read once per 32 output columns instead of once
// per 8.  Three CTAs per SM hide each other's staging.
constexpr int kRmRows = 8, kRmWarps = 4, kRmRowsPerBlock = kRmWarps * kRmRows;
constexpr int kRotManyFrom = 64;   // queries from which the blocked kernel is used (d a multiple of 4)

template <typename T>
__global__ void __launch_bounds__(32 * kRmWarps) rotate_many_kernel(const float* __restrict__ Rot, int nrows, int d,
                                                                    const T* __restrict__ Q, int64_t ldq, int nq,
                                                                    float* __restrict__ Qcat, int64_t ldo) {
  extern __shared__ __align__(16) float qs_raw[];
  float (*qs)[kRotChunk] = reinterpret_cast<float (*)[kRotChunk]>(qs_raw);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * kRmRowsPerBlock + warp * kRmRows;
  const int q_begin = blockIdx.y * kRotQPerBlock, q_end = min(nq, q_begin + kRotQPerBlock);
  for (int q0 = q_begin; q0 < q_end; q0 += kRotQ) {
    float acc[kRmRows][kRotQ];
#pragma unroll
    for (int rr = 0; rr < kRmRows; ++rr)
#pragma unroll
      for (int qq = 0; qq < kRotQ; ++qq) acc[rr][qq] = 0.f;
    const int nact = min(kRotQ, q_end - q0);
    for (int c0 = 0; c0 < d; c0 += kRotChunk) {
      const int len = min(kRotChunk, d - c0);
      __syncthreads();
      for (int e = threadIdx.x; e < nact * (kRotChunk / 4); e += blockDim.x) {
        const int qq = e / (kRotChunk / 4), c = 4 * (e % (kRotChunk / 4));
        if (c >= len) continue;   // columns past the chunk's end are not read below
        const T* src = Q + (int64_t)(q0 + qq) * ldq + c0 + c;
        float v[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) v[t] = scan::to_f32<T>(src[t]);   // d is a multiple of 4: whole groups of four
        *reinterpret_cast<float4*>(&qs[qq][c]) = make_float4(v[0], v[1], v[2], v[3]);
      }
      __syncthreads();
#pragma unroll 2
      for (int i = 0; i < kRotChunk / 128; ++i) {
        const int c4 = lane + 32 * i;
        if (4 * c4 >= len) break;
        float4 r[kRmRows];
#pragma unroll
        for (int rr = 0; rr < kRmRows; ++rr)
          r[rr] = __ldg(reinterpret_cast<const float4*>(Rot + (size_t)min(j0 + rr, nrows - 1) * d + c0) + c4);
#pragma unroll
        for (int qq = 0; qq < kRotQ; ++qq) {
          if (qq < nact) {
            const float4 v = *reinterpret_cast<const float4*>(&qs[qq][4 * c4]);
#pragma unroll
            for (int rr = 0; rr < kRmRows; ++rr)
              acc[rr][qq] = fmaf(r[rr].x, v.x, fmaf(r[rr].y, v.y, fmaf(r[rr].z, v.z, fmaf(r[rr].w, v.w, acc[rr][qq]))));
          }
        }
      }
    }
    // The 32 partial sums of each of the warp's 64 outputs are added in fp64 along the tree of the xor butterfly
    // (lanes l and l ^ 16, then ^ 8, 4, 2, 1: every lane of the butterfly ends with the same bits, additions being
    // commutative), but transposed: at each level a lane keeps half of its values and hands the other half to its
    // partner, so that 62 fp64 additions per lane do what 320 would; lane l ends with outputs 2 l and 2 l + 1.
    static_assert(kRmRows * kRotQ == 64, "the transposed reduction is written for 64 outputs per warp");
    const bool b4 = (lane & 16) != 0, b3 = (lane & 8) != 0, b2 = (lane & 4) != 0, b1 = (lane & 2) != 0, b0 = (lane & 1) != 0;
    double w1[32], w2[16], w3[8], w4[4], w5[2];
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      const float lo = acc[k / kRotQ][k % kRotQ], hi = acc[(k + 32) / kRotQ][k % kRotQ];
      const float got = __shfl_xor_sync(0xffffffffu, b4 ? lo : hi, 16);
      w1[k] = (double)(b4 ? hi : lo) + (double)got;
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) w2[k] = (b3 ? w1[k + 16] : w1[k]) + __shfl_xor_sync(0xffffffffu, b3 ? w1[k] : w1[k + 16], 8);
#pragma unroll
    for (int k = 0; k < 8; ++k) w3[k] = (b2 ? w2[k + 8] : w2[k]) + __shfl_xor_sync(0xffffffffu, b2 ? w2[k] : w2[k + 8], 4);
#pragma unroll
    for (int k = 0; k < 4; ++k) w4[k] = (b1 ? w3[k + 4] : w3[k]) + __shfl_xor_sync(0xffffffffu, b1 ? w3[k] : w3[k + 4], 2);
#pragma unroll
    for (int k = 0; k < 2; ++k) w5[k] = (b0 ? w4[k + 2] : w4[k]) + __shfl_xor_sync(0xffffffffu, b0 ? w4[k] : w4[k + 2], 1);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int idx = 2 * lane + k, rr = idx / kRotQ, qq = idx % kRotQ;
      if (qq < nact && j0 + rr < nrows) Qcat[(int64_t)(q0 + qq) * ldo + j0 + rr] = (float)w5[k];
    }
  }
}

template <typename T>
cudaError_t launch_rotate_queries(const tq_plan* plan, const T* Q, int64_t ldq, int nq, float* Qcat, cudaStream_t st) {
  const int ncols = plan->ncat * plan->dpad;
  constexpr int smem = kRotQ * kRotChunk * (int)sizeof(float);
  // function attributes are per device: remember the devices this launcher has prepared
  static std::atomic<unsigned long long> attr_devices{0};   // written by any thread that launches
  int attr_dev = 0;
  if (cudaGetDevice(&attr_dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (attr_dev >= 64 || !((attr_devices.load(std::memory_order_relaxed) >> attr_dev) & 1ull)) {
    cudaError_t e = cudaFuncSetAttribute(rotate_queries_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (attr_dev < 64) attr_devices.fetch_or(1ull << attr_dev, std::memory_order_relaxed);
  }
  if (nq >= kRotManyFrom && (plan->d & 3) == 0) {
    static std::atomic<unsigned long long> many_devices{0};
    if (attr_dev >= 64 || !((many_devices.load(std::memory_order_relaxed) >> attr_dev) & 1ull)) {
      cudaError_t e = cudaFuncSetAttribute(rotate_many_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
      if (attr_dev < 64) many_devices.fetch_or(1ull << attr_dev, std::memory_order_relaxed);
    }
    const dim3 grid((unsigned)((ncols + kRmRowsPerBlock - 1) / kRmRowsPerBlock), (unsigned)((nq + kRotQPerBlock - 1) / kRotQPerBlock));
    rotate_many_kernel<T><<<grid, 32 * kRmWarps, smem, st>>>(plan->dRotCat, ncols, plan->d, Q, ldq, nq, Qcat, ncols);
    count_launches(1);
    return cudaGetLastError();
  }
  const dim3 grid((unsigned)((ncols + 7) / 8), (unsigned)((nq + kRotQPerBlock - 1) / kRotQPerBlock));
  rotate_queries_kernel<T><<<grid, 256, smem, st>>>(plan->dRotCat, ncols, plan->d, Q, ldq, nq, Qcat, ncols);
  count_launches(1);
  return cudaGetLastError();
}

// Q' = Q Pi^T and Q'' = Q S^T side by side: Qcat[nq, ncat*dpad].
cudaError_t prepare_queries(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, float* Qcat,
                            cudaStream_t st) {
  const int ncols = plan->ncat * plan->dpad;
  (void)ncols;
  // Both kernels add the same products in the same order, so that a query's rotated form (and hence its
  // estimates) does not depend on how many other queries came with it.
  if (q_dtype == TQ_F32) return launch_rotate_queries(plan, static_cast<const float*>(Q), ldq, nq, Qcat, st);
  return launch_rotate_queries(plan, static_cast<const __nv_bfloat16*>(Q), ldq, nq, Qcat, st);
}

template <int BITS, bool PROD>
cudaError_t launch_scan_few(const scan::ScanArgs& base, int nq, cudaStream_t st) {
  const size_t per_query = (size_t)(PROD ? 2 : 1) * 32 * base.groups * sizeof(float);
  int tile = 8;
  while (tile > 1 && per_query * tile > 200 * 1024) tile >>= 1;
  if (per_query * tile > 220 * 1024) return cudaErrorInvalidConfiguration;
  const int64_t blocks = std::min<int64_t>((base.n + 255) / 256, 148 * 2);
  for (int q0 = 0; q0 < nq; q0 += tile) {
    scan::ScanArgs a = base;
    a.q0 = q0;
    a.nq_tile = std::min(tile, nq - q0);
    cudaError_t e = cudaSuccess;
    const size_t smem = per_query * tile;
#define TQ_SCAN_LAUNCH(NQ)                                                                                  \
  e = cudaFuncSetAttribute(scan::scan_few_kernel<BITS, NQ, PROD>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                           (int)smem);                                                                      \
  if (e == cudaSuccess) scan::scan_few_kernel<BITS, NQ, PROD><<<(unsigned)blocks, 256, smem, st>>>(a);
    switch (tile) {
      case 8: TQ_SCAN_LAUNCH(8) break;
      case 4: TQ_SCAN_LAUNCH(4) break;
      case 2: TQ_SCAN_LAUNCH(2) break;
      default: TQ_SCAN_LAUNCH(1) break;
    }
#undef TQ_SCAN_LAUNCH
    if (e != cudaSuccess) return e;
    count_launches(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Scores of queries (already prepared in Qcat) against vectors [v0, v0 + cn).
cudaError_t score_block(const tq_plan* plan, const float* Qcat, int nq, int64_t v0, int64_t cn, const uint8_t* idx,
                        const uint8_t* qjl, const float* gamma, const float* norms, float* scores, int64_t lds,
                        cudaStream_t st) {
  const uint8_t* idx_b = idx ? idx + (size_t)v0 * plan->idx_row_bytes : nullptr;
  const uint8_t* qjl_b = qjl ? qjl + (size_t)v0 * plan->qjl_row_bytes : nullptr;
  const float* gamma_b = gamma ? gamma + v0 : nullptr;
  const float* norms_b = norms ? norms + v0 : nullptr;
  const int ncols = plan->ncat * plan->dpad;
  if (nq <= kFewQueries) {
    scan::ScanArgs a;
    a.idx = idx_b;
    a.idx_rb = plan->idx_row_bytes;
    a.qjl = (plan->mode == TQ_PROD) ? qjl_b : nullptr;
    a.qjl_rb = plan->qjl_row_bytes;
    a.gamma = gamma_b;
    a.norms = norms_b;
    a.cb = plan->cb;
    a.d = plan->d;
    a.groups = (plan->d + 31) / 32;
    a.coef = plan->coef;
    a.n = cn;
    a.Qcat = Qcat;
    a.ldq = ncols;
    a.dpad = plan->dpad;
    a.q0 = 0;
    a.nq_tile = 0;
    a.scores = scores;
    a.lds = lds;
    const bool prod = plan->mode == TQ_PROD;
    switch (plan->mse_bits) {
      case 0: return launch_scan_few<0, true>(a, nq, st);
      case 1: return prod ? launch_scan_few<1, true>(a, nq, st) : launch_scan_few<1, false>(a, nq, st);
      case 2: return prod ? launch_scan_few<2, true>(a, nq, st) : launch_scan_few<2, false>(a, nq, st);
      case 3: return prod ? launch_scan_few<3, true>(a, nq, st) : launch_scan_few<3, false>(a, nq, st);
      default: return prod ? launch_scan_few<4, true>(a, nq, st) : launch_scan_few<4, false>(a, nq, st);
    }
  }
  simt::RowsF32 A{Qcat, ncols, nq, ncols};
  simt::Codes B = make_codes(plan, cn, idx_b, qjl_b, gamma_b);
  simt::EpStore ep{scores, lds, nullptr, norms_b};
  return simt::launch_gemm(A, B, ep, (int64_t)nq, cn, ncols, st);
}

}  // namespace

// ======================================================================================
extern "C" int tq_plan_create(int d, int bits, int mode, const float* Pi, const float* S, const float* centroids,
                              tq_plan** out) {
  const char* who = "tq_plan_create";
  TQ_RANGE(who);
  TQ_REQUIRE(out != nullptr, TQ_ERR_INVALID_ARG, "%s: out is NULL", who);
  *out = nullptr;
  TQ_REQUIRE(mode == TQ_MSE || mode == TQ_PROD, TQ_ERR_INVALID_ARG, "%s: unknown mode %d", who, mode);
  TQ_REQUIRE(d >= 2 && d <= TQ_MAX_D, TQ_ERR_UNSUPPORTED, "%s: d=%d outside 2..%d", who, d, TQ_MAX_D);
  const int mse_bits = (mode == TQ_PROD) ? bits - 1 : bits;
  TQ_REQUIRE(bits >= 1 && mse_bits <= 4, TQ_ERR_UNSUPPORTED, "%s: bits=%d unsupported for this mode", who, bits);
  TQ_REQUIRE(Pi != nullptr && centroids != nullptr, TQ_ERR_INVALID_ARG, "%s: Pi / centroids is NULL", who);
  TQ_REQUIRE(mode == TQ_MSE || S != nullptr, TQ_ERR_INVALID_ARG, "%s: S is NULL for a TQ_PROD plan", who);
  const int levels = 1 << mse_bits;
  for (int i = 0; i < levels; ++i) {
    TQ_REQUIRE(std::isfinite(centroids[i]), TQ_ERR_INVALID_ARG, "%s: centroid %d is not finite", who, i);
    TQ_REQUIRE(i == 0 || centroids[i] > centroids[i - 1], TQ_ERR_INVALID_ARG, "%s: centroids must be strictly ascending", who);
  }

  tq_plan* p = new (std::nothrow) tq_plan();
  TQ_REQUIRE(p != nullptr, TQ_ERR_INVALID_ARG, "%s: out of host memory", who);
  std::memset(p, 0, sizeof(*p));
  p->d = d;
  p->dpad = round_up(d, 8);
  p->bits = bits;
  p->mode = mode;
  p->mse_bits = mse_bits;
  p->ncat = (mode == TQ_PROD) ? 2 : 1;
  p->coef = (float)(std::sqrt(M_PI / 2.0) / d);
  p->idx_row_bytes = tq_idx_row_bytes(d, mse_bits);
  p->qjl_row_bytes = tq_qjl_row_bytes(d);
  p->cb.bits = mse_bits;
  for (int i = 0; i < 16; ++i) p->cb.c[i] = (i < levels) ? centroids[i] : 0.f;
  for (int i = 0; i < 15; ++i) p->cb.t[i] = (i + 1 < levels) ? 0.5f * (centroids[i] + centroids[i + 1]) : INFINITY;

  const size_t dd = (size_t)d * d;
  const int ncols = p->ncat * p->dpad;
  auto fail = [&](int code) {
    tq_plan_destroy(p);
    return code;
  };
#define PLAN_CUDA(call, what)                                        \
  do {                                                               \
    cudaError_t e_ = (call);                                         \
    if (e_ != cudaSuccess) {                                         \
      set_error("%s: %s: %s", who, what, cudaGetErrorString(e_));    \
      return fail(TQ_ERR_CUDA);                                      \
    }                                                                \
  } while (0)
  PLAN_CUDA(cudaGetDevice(&p->device), "cudaGetDevice");
  PLAN_CUDA(cudaMalloc(&p->dPi, dd * sizeof(float)), "cudaMalloc Pi");
  PLAN_CUDA(cudaMemcpy(p->dPi, Pi, dd * sizeof(float), cudaMemcpyHostToDevice), "copy Pi");
  std::vector<float> rot((size_t)ncols * d, 0.f), back((size_t)d * ncols, 0.f);
  for (int i = 0; i < d; ++i) {
    std::memcpy(&rot[(size_t)i * d], Pi + (size_t)i * d, d * sizeof(float));
    for (int j = 0; j < d; ++j) back[(size_t)j * ncols + i] = Pi[(size_t)i * d + j];
  }
  float* dS = nullptr;
  if (mode == TQ_PROD) {
    for (int i = 0; i < d; ++i) {
      std::memcpy(&rot[(size_t)(p->dpad + i) * d], S + (size_t)i * d, d * sizeof(float));
      for (int j = 0; j < d; ++j) back[(size_t)j * ncols + p->dpad + i] = S[(size_t)i * d + j];
    }
    PLAN_CUDA(cudaMalloc(&dS, dd * sizeof(float)), "cudaMalloc S");
    cudaError_t e = cudaMemcpy(dS, S, dd * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMalloc(&p->dSp, dd * sizeof(float));
    if (e == cudaSuccess) {
      dim3 grid((d + 15) / 16, (d + 15) / 16), block(16, 16);
      sprime_kernel<<<grid, block>>>(dS, p->dPi, p->dSp, d);
      e = cudaGetLastError();
      if (e == cudaSuccess) e = cudaDeviceSynchronize();
    }
    cudaFree(dS);
    PLAN_CUDA(e, "S' = S Pi^T");
  }
  PLAN_CUDA(cudaMalloc(&p->dRotCat, rot.size() * sizeof(float)), "cudaMalloc RotCat");
  PLAN_CUDA(cudaMemcpy(p->dRotCat, rot.data(), rot.size() * sizeof(float), cudaMemcpyHostToDevice), "copy RotCat");
  PLAN_CUDA(cudaMalloc(&p->dBackT, back.size() * sizeof(float)), "cudaMalloc BackT");
  PLAN_CUDA(cudaMemcpy(p->dBackT, back.data(), back.size() * sizeof(float), cudaMemcpyHostToDevice), "copy BackT");
  PLAN_CUDA(cudaMalloc(&p->d_status, sizeof(int)), "cudaMalloc status");
  PLAN_CUDA(cudaMemset(p->d_status, 0, sizeof(int)), "clear status");
  if (tc::supported(d)) {
    p->tc_bn = tc::pick_bn(d);
    PLAN_CUDA(tc::build_matrix_limbs(p->dPi, d, d, p->dpad, p->tc_bn, &p->pi_limbs), "bf16 limbs of Pi");
    if (mode == TQ_PROD)
      PLAN_CUDA(tc::build_matrix_limbs(p->dSp, d, d, p->dpad, p->tc_bn, &p->sp_limbs), "bf16 limbs of S'");
    p->tc_ok = 1;
  }
  mscan::plan_init(p);
  nscan::plan_init(p);
  PLAN_CUDA(cudaDeviceSynchronize(), "synchronize");
#undef PLAN_CUDA
  *out = p;
  return TQ_OK;
}

extern "C" int tq_plan_destroy(tq_plan* plan) {
  if (!plan) return TQ_OK;
  cudaFree(plan->dPi);
  cudaFree(plan->dSp);
  cudaFree(plan->dRotCat);
  cudaFree(plan->dBackT);
  cudaFree(plan->d_status);
  tc::free_matrix_limbs(&plan->pi_limbs);
  tc::free_matrix_limbs(&plan->sp_limbs);
  delete plan;
  return TQ_OK;
}

extern "C" int tq_plan_set_layout(tq_plan* plan, int layout) {
  const char* who = "tq_plan_set_layout";
  TQ_REQUIRE(plan != nullptr, TQ_ERR_INVALID_ARG, "%s: plan is NULL", who);
  TQ_REQUIRE(layout == TQ_LAYOUT_CANONICAL || layout == TQ_LAYOUT_NIBBLE, TQ_ERR_INVALID_ARG, "%s: unknown layout %d", who, layout);
  TQ_REQUIRE(layout == TQ_LAYOUT_CANONICAL || plan->nb.ok, TQ_ERR_UNSUPPORTED,
             "%s: the nibble layout needs a TQ_PROD plan with b = 4, d >= 128 (d=%d, b=%d, mode=%d)", who, plan->d, plan->bits,
             plan->mode);
  plan->layout = layout;
  return TQ_OK;
}

extern "C" int tq_plan_layout(const tq_plan* plan) { return plan ? plan->layout : -1; }

extern "C" int tq_convert_layout(const tq_plan* plan, int64_t n, uint8_t* idx, uint8_t* qjl, int from, int to, void* stream) {
  const char* who = "tq_convert_layout";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(n >= 0, TQ_ERR_INVALID_ARG, "%s: n is negative", who);
  for (int l : {from, to})
    TQ_REQUIRE(l == TQ_LAYOUT_CANONICAL || l == TQ_LAYOUT_NIBBLE, TQ_ERR_INVALID_ARG, "%s: unknown layout %d", who, l);
  TQ_REQUIRE(plan->nb.ok, TQ_ERR_UNSUPPORTED, "%s: this plan has no nibble layout (TQ_PROD, b = 4, d >= 128 only)", who);
  if (n == 0 || from == to) return TQ_OK;
  TQ_REQUIRE(idx != nullptr && qjl != nullptr, TQ_ERR_INVALID_ARG, "%s: idx / qjl is NULL", who);
  TQ_REQUIRE(aligned(idx, 16) && aligned(qjl, 16), TQ_ERR_ALIGNMENT, "%s: idx / qjl is not 16-byte aligned", who);
  return nscan::convert(plan, n, idx, qjl, to, static_cast<cudaStream_t>(stream), who);
}

// A one-warp kernel whose barrier nobody arrives at: the bounded wait must give up after `limit` cycles, raise the
// CTA's abort flag and record TQ_ERR_TIMEOUT in the plan's status word.  Nothing traps, nothing spins past the limit.
__global__ void wait_timeout_selftest_kernel(int* status, long long limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    tc::mbar_init(&bar, 1);
    abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool ok = tc::mbar_wait_slow(&bar, 0u, &abort_flag, status, limit);
    if (ok || abort_flag != 1) atomicExch(status, TQ_ERR_CUDA);   // anything but "gave up and said so" is a different error
  }
}

extern "C" int tq_selftest_wait_timeout(tq_plan* plan, long long limit_cycles, void* stream) {
  const char* who = "tq_selftest_wait_timeout";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(limit_cycles >= 1 && limit_cycles <= 100000000LL, TQ_ERR_INVALID_ARG, "%s: limit outside 1..1e8 cycles", who);
  wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(plan->d_status, limit_cycles);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

extern "C" int tq_plan_status(tq_plan* plan) {
  const char* who = "tq_plan_status";
  TQ_RANGE(who);
  TQ_REQUIRE(plan != nullptr, TQ_ERR_INVALID_ARG, "%s: plan is NULL", who);
  TQ_CHECK_CUDA(cudaDeviceSynchronize(), who);
  int st = 0;
  TQ_CHECK_CUDA(cudaMemcpy(&st, plan->d_status, sizeof(int), cudaMemcpyDeviceToHost), who);
  if (st != 0) {
    cudaMemset(plan->d_status, 0, sizeof(int));
    if (st == TQ_ERR_BOUNDS) {
      set_error("%s: a device-side index check of the TQ_DEBUG build failed (the access was skipped)", who);
      return TQ_ERR_BOUNDS;
    }
    if (st != TQ_ERR_TIMEOUT) {
      set_error("%s: a kernel recorded the unexpected status %d", who, st);
      return TQ_ERR_CUDA;
    }
    set_error("%s: a kernel gave up a bounded wait (pipeline stall); results of that call are invalid", who);
    return TQ_ERR_TIMEOUT;
  }
  return TQ_OK;
}

extern "C" size_t tq_workspace_bytes(const tq_plan* plan, int op, int64_t n, int nq, int k) {
  if (!plan || n < 0 || nq < 0) return 0;
  (void)k;
  switch (op) {
    case TQ_OP_QUANTIZE:
      if (n == 0) return 0;
      if (plan->tc_ok)
      {
        // rows per launch: 65,536 at d = 1536 and more for short rows (same scratch bytes), so that a launch of the
        // persistent GEMM stays long against its prologue and the launch sequence
        const int64_t chunk = std::min<int64_t>(kTensorChunk * std::max(1, 1536 / plan->dpad), 8 * kTensorChunk);
        // (half as many rows again when n exceeds the chunk: fewer, longer launches measured faster than 65,536-row
        // ones, also than 65,536-row ones whose operand split ran beside the previous block's GEMMs)
        return align_up((size_t)std::min<int64_t>(round_up64(n, 128), n > chunk ? chunk + chunk / 2 : chunk) *
                            tc::scratch_bytes_per_row(plan),
                        256);
      }
      if (plan->mode != TQ_PROD) return 0;
      return align_up((size_t)std::min<int64_t>(n, kResidualChunk) * plan->dpad * sizeof(float), 256);
    case TQ_OP_SCORE:
      return plan->ms.ok ? ms_score_fixed(plan, nq) : qcat_bytes(plan, nq);
    case TQ_OP_TOPK:
      if (plan->ms.ok)
        return ms_topk_fixed(plan, nq) +
               align_up((size_t)pick_engine(plan, nq).qpp *
                            std::max<int64_t>(std::min<int64_t>(n, pick_engine(plan, nq).dense_rows_pref), kDenseRowsMin) * sizeof(float),
                        256);
      return qcat_bytes(plan, nq) + align_up((size_t)nq * std::min<int64_t>(n, kTopkBlockPref) * sizeof(float), 256);
    case TQ_OP_WSUM: {
      const size_t ncols = (size_t)plan->ncat * plan->dpad;
      const size_t chunks = (size_t)((n + attend::WS_TOK - 1) / attend::WS_TOK);
      return align_up((size_t)nq * ncols * sizeof(float), 256) +
             align_up(chunks * std::min(nq, attend::WS_NW) * ncols * sizeof(float), 256);
    }
    default:
      return 0;
  }
}

extern "C" int tq_quantize_mse(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx, uint8_t* idx,
                               float* norms, void* scratch, size_t scratch_bytes, void* stream) {
  const char* who = "tq_quantize_mse";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(plan->mode == TQ_MSE, TQ_ERR_INVALID_ARG, "%s: plan was created for TQ_PROD", who);
  TQ_REQUIRE(n >= 0, TQ_ERR_INVALID_ARG, "%s: n is negative", who);
  if (n == 0) return TQ_OK;
  if ((rc = check_rows(who, "X", X, x_dtype, n, ldx, plan->d))) return rc;
  TQ_REQUIRE(idx != nullptr, TQ_ERR_INVALID_ARG, "%s: idx is NULL", who);
  TQ_REQUIRE(aligned(idx, 16) && aligned(norms, 4), TQ_ERR_ALIGNMENT, "%s: idx / norms is misaligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (plan->tc_ok) {
    const size_t need = tq_workspace_bytes(plan, TQ_OP_QUANTIZE, std::min<int64_t>(n, 128), 0, 0);
    TQ_REQUIRE(scratch != nullptr && scratch_bytes >= need, TQ_ERR_WORKSPACE, "%s: scratch of %zu bytes, at least %zu needed",
               who, scratch_bytes, need);
    TQ_REQUIRE(aligned(scratch, 256), TQ_ERR_ALIGNMENT, "%s: scratch is not 256-byte aligned", who);
    return tc::quantize(plan, X, x_dtype, n, ldx, idx, nullptr, nullptr, norms, scratch, scratch_bytes, st, who);
  }
  if (norms) TQ_CHECK_CUDA(compute_norms(X, x_dtype, n, ldx, plan->d, norms, st), who);
  if (has_pad_words(plan->d, plan->mse_bits, plan->idx_row_bytes))
    TQ_CHECK_CUDA(cudaMemsetAsync(idx, 0, (size_t)n * plan->idx_row_bytes, st), who);
  TQ_CHECK_CUDA(dispatch_rotate_quantize<0>(plan, X, x_dtype, n, ldx, norms, idx, nullptr, 0, st), who);
  return TQ_OK;
}

extern "C" int tq_quantize_prod(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx, uint8_t* idx,
                                uint8_t* qjl, float* gamma, float* norms, void* scratch, size_t scratch_bytes,
                                void* stream) {
  const char* who = "tq_quantize_prod";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(plan->mode == TQ_PROD, TQ_ERR_INVALID_ARG, "%s: plan was created for TQ_MSE", who);
  TQ_REQUIRE(n >= 0, TQ_ERR_INVALID_ARG, "%s: n is negative", who);
  if (n == 0) return TQ_OK;
  if ((rc = check_rows(who, "X", X, x_dtype, n, ldx, plan->d))) return rc;
  if ((rc = check_codes(plan, who, idx, qjl, gamma))) return rc;
  TQ_REQUIRE(aligned(norms, 4), TQ_ERR_ALIGNMENT, "%s: norms is misaligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (plan->tc_ok) {
    const size_t least = tq_workspace_bytes(plan, TQ_OP_QUANTIZE, std::min<int64_t>(n, 128), 0, 0);
    TQ_REQUIRE(scratch != nullptr && scratch_bytes >= least, TQ_ERR_WORKSPACE,
               "%s: scratch of %zu bytes, at least %zu needed", who, scratch_bytes, least);
    TQ_REQUIRE(aligned(scratch, 256), TQ_ERR_ALIGNMENT, "%s: scratch is not 256-byte aligned", who);
    // (the GEMM epilogues write whichever layout the plan has)
    return tc::quantize(plan, X, x_dtype, n, ldx, idx, qjl, gamma, norms, scratch, scratch_bytes, st, who);
  }
  const size_t need = tq_workspace_bytes(plan, TQ_OP_QUANTIZE, n, 0, 0);
  TQ_REQUIRE(scratch != nullptr && scratch_bytes >= need, TQ_ERR_WORKSPACE, "%s: scratch of %zu bytes, %zu needed", who,
             scratch_bytes, need);
  TQ_REQUIRE(aligned(scratch, 16), TQ_ERR_ALIGNMENT, "%s: scratch is not 16-byte aligned", who);
  const int d = plan->d;
  const int64_t ldE = plan->dpad;
  float* E = static_cast<float*>(scratch);
  int64_t chunk = (int64_t)(scratch_bytes / ((size_t)ldE * sizeof(float)));
  if (chunk < n) chunk = chunk / simt::BM * simt::BM;
  chunk = std::min(chunk, n);
  TQ_REQUIRE(chunk > 0, TQ_ERR_WORKSPACE, "%s: scratch too small for one block of rows", who);

  if (norms) TQ_CHECK_CUDA(compute_norms(X, x_dtype, n, ldx, d, norms, st), who);
  if (has_pad_words(d, plan->mse_bits, plan->idx_row_bytes))
    TQ_CHECK_CUDA(cudaMemsetAsync(idx, 0, (size_t)n * plan->idx_row_bytes, st), who);
  if (has_pad_words(d, 1, plan->qjl_row_bytes))
    TQ_CHECK_CUDA(cudaMemsetAsync(qjl, 0, (size_t)n * plan->qjl_row_bytes, st), who);
  const size_t xsz = (x_dtype == TQ_F32) ? 4 : 2;
  for (int64_t r0 = 0; r0 < n; r0 += chunk) {
    const int64_t rows = std::min(chunk, n - r0);
    const void* Xc = static_cast<const char*>(X) + (size_t)r0 * ldx * xsz;
    uint8_t* idx_c = idx ? idx + (size_t)r0 * plan->idx_row_bytes : nullptr;
    // Stage 1: y = Pi x, idx, rotated residual e = y/nu - c[idx]   (Algorithm 2, steps idx and r)
    TQ_CHECK_CUDA(dispatch_rotate_quantize<1>(plan, Xc, x_dtype, rows, ldx, norms ? norms + r0 : nullptr, idx_c, E, ldE, st), who);
    // gamma = ||r|| = ||e||
    TQ_CHECK_CUDA(launch_row_norm(E, ldE, rows, d, gamma + r0, st), who);
    // Stage 2: qjl = sign(S r) = sign(S' e)
    simt::EpQuantize<1, 2> ep;
    ep.cb = plan->cb;
    ep.nu = nullptr;
    ep.out = qjl + (size_t)r0 * plan->qjl_row_bytes;
    ep.out_rb = plan->qjl_row_bytes;
    ep.E = nullptr;
    ep.ldE = 0;
    ep.d = d;
    simt::RowsF32 A{E, ldE, rows, d};
    simt::RowsF32 B{plan->dSp, d, d, d};
    TQ_CHECK_CUDA(simt::launch_gemm(A, B, ep, rows, (int64_t)d, d, st), who);
  }
  return TQ_OK;
}

extern "C" int tq_dequantize(const tq_plan* plan, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
                             const float* norms, float* Xhat, int64_t ldxh, void* stream) {
  const char* who = "tq_dequantize";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(n >= 0, TQ_ERR_INVALID_ARG, "%s: n is negative", who);
  if (n == 0) return TQ_OK;
  if ((rc = check_codes(plan, who, idx, qjl, gamma))) return rc;
  TQ_REQUIRE(Xhat != nullptr, TQ_ERR_INVALID_ARG, "%s: Xhat is NULL", who);
  TQ_REQUIRE(ldxh >= plan->d, TQ_ERR_INVALID_ARG, "%s: ldxh < d", who);
  TQ_REQUIRE(aligned(Xhat, 16), TQ_ERR_ALIGNMENT, "%s: Xhat is not 16-byte aligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int ncols = plan->ncat * plan->dpad;
  simt::Codes A = make_codes(plan, n, idx, qjl, gamma);
  simt::RowsF32 B{plan->dBackT, ncols, plan->d, ncols};
  simt::EpStore ep{Xhat, ldxh, norms, nullptr};
  TQ_CHECK_CUDA(simt::launch_gemm(A, B, ep, n, (int64_t)plan->d, ncols, st), who);
  return TQ_OK;
}

// Engine for a score call whose workspace holds `avail` bytes behind the rotated queries: the preferred one, or,
// when the many-query engine's operand does not fit, the few-query engine (same estimates, more passes).
static bool engine_that_fits(const tq_plan* plan, int nq, size_t avail, ScanEngine* out) {
  *out = pick_engine(plan, nq);
  if (align_up(out->ws_bytes, 256) <= avail) return true;
  if (!out->tc) return false;
  *out = pick_engine(plan, std::min(nq, 6));
  return align_up(out->ws_bytes, 256) <= avail;
}

// tq_score on a workspace that is known to be large enough: rotated queries first, then the engine's operand.
static int score_on_workspace(const tq_plan* plan, const ScanEngine* eng, const void* Q, int q_dtype, int nq, int64_t ldq,
                              int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms,
                              float* scores, int64_t lds, void* workspace, cudaStream_t st, const char* who) {
  int rc;
  float* Qcat = static_cast<float*>(workspace);
  TQ_CHECK_CUDA(prepare_queries(plan, Q, q_dtype, nq, ldq, Qcat, st), who);
  if (plan->ms.ok) {
    void* msw = static_cast<char*>(workspace) + qcat_bytes(plan, nq);
    for (int q0 = 0; q0 < nq; q0 += eng->qpp) {
      const int nqp = std::min(eng->qpp, nq - q0);
      if ((rc = engine_prepare(*eng, Qcat, q0, nq, msw, st, who))) return rc;
      if ((rc = engine_run(*eng, q0, nqp, n, idx, qjl, gamma, norms, scores + (int64_t)q0 * lds, lds, nullptr, nullptr, msw, st, who)))
        return rc;
    }
    return TQ_OK;
  }
  TQ_CHECK_CUDA(score_block(plan, Qcat, nq, 0, n, idx, qjl, gamma, norms, scores, lds, st), who);
  return TQ_OK;
}

static int check_score_args(const tq_plan* plan, const char* who, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
                            const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* scores, int64_t lds) {
  int rc;
  if ((rc = check_rows(who, "Q", Q, q_dtype, nq, ldq, plan->d))) return rc;
  if ((rc = check_codes(plan, who, idx, qjl, gamma))) return rc;
  TQ_REQUIRE(scores != nullptr && lds >= n, TQ_ERR_INVALID_ARG, "%s: scores is NULL or lds < n", who);
  TQ_REQUIRE(aligned(scores, 16), TQ_ERR_ALIGNMENT, "%s: scores is not 16-byte aligned", who);
  return TQ_OK;
}

extern "C" int tq_score(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
                        const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms, float* scores,
                        int64_t lds, void* workspace, size_t workspace_bytes, void* stream) {
  const char* who = "tq_score";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(n >= 0 && nq >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (n == 0 || nq == 0) return TQ_OK;
  if ((rc = check_score_args(plan, who, Q, q_dtype, nq, ldq, n, idx, qjl, gamma, scores, lds))) return rc;
  const size_t need = tq_workspace_bytes(plan, TQ_OP_SCORE, n, nq, 0);
  TQ_REQUIRE(workspace != nullptr && workspace_bytes >= need, TQ_ERR_WORKSPACE, "%s: workspace of %zu bytes, %zu needed",
             who, workspace_bytes, need);
  TQ_REQUIRE(aligned(workspace, 16), TQ_ERR_ALIGNMENT, "%s: workspace is not 16-byte aligned", who);
  ScanEngine eng{};
  if (plan->ms.ok) eng = pick_engine(plan, nq);
  return score_on_workspace(plan, &eng, Q, q_dtype, nq, ldq, n, idx, qjl, gamma, norms, scores, lds, workspace,
                            static_cast<cudaStream_t>(stream), who);
}

// ---- prepared queries: rotation and operand set-up once, any number of scans afterwards
// Buffer: rotated queries, then one engine workspace per pass (per group of 256 queries on the tcgen05 engine).
static size_t prepared_slots(const ScanEngine& e, int nq) {
  const int per = e.tc ? kGroupQueries : e.qpp;
  return (size_t)((nq + per - 1) / per);
}

extern "C" size_t tq_query_bytes(const tq_plan* plan, int nq) {
  if (!plan || nq <= 0) return 0;
  size_t b = qcat_bytes(plan, nq);
  if (plan->ms.ok) {
    const ScanEngine e = pick_engine(plan, nq);
    b += prepared_slots(e, nq) * align_up(e.ws_bytes, 256);
  }
  return b;
}

extern "C" int tq_query_prepare(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, void* prepared,
                                size_t prepared_bytes, void* stream) {
  const char* who = "tq_query_prepare";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(nq >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (nq == 0) return TQ_OK;
  if ((rc = check_rows(who, "Q", Q, q_dtype, nq, ldq, plan->d))) return rc;
  const size_t need = tq_query_bytes(plan, nq);
  TQ_REQUIRE(prepared != nullptr && prepared_bytes >= need, TQ_ERR_WORKSPACE, "%s: buffer of %zu bytes, %zu needed", who,
             prepared_bytes, need);
  TQ_REQUIRE(aligned(prepared, 256), TQ_ERR_ALIGNMENT, "%s: buffer is not 256-byte aligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* Qcat = static_cast<float*>(prepared);
  TQ_CHECK_CUDA(prepare_queries(plan, Q, q_dtype, nq, ldq, Qcat, st), who);
  if (!plan->ms.ok) return TQ_OK;
  const ScanEngine eng = pick_engine(plan, nq);
  const size_t slot = align_up(eng.ws_bytes, 256);
  char* base = static_cast<char*>(prepared) + qcat_bytes(plan, nq);
  const int per = eng.tc ? kGroupQueries : eng.qpp;
  for (int q0 = 0; q0 < nq; q0 += per)
    if ((rc = engine_prepare(eng, Qcat, q0, nq, base + (size_t)(q0 / per) * slot, st, who))) return rc;
  return TQ_OK;
}

extern "C" int tq_score_prepared(const tq_plan* plan, const void* prepared, int nq, int64_t n, const uint8_t* idx,
                                 const uint8_t* qjl, const float* gamma, const float* norms, float* scores, int64_t lds,
                                 void* stream) {
  const char* who = "tq_score_prepared";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(n >= 0 && nq >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (n == 0 || nq == 0) return TQ_OK;
  TQ_REQUIRE(prepared != nullptr && aligned(prepared, 256), TQ_ERR_INVALID_ARG, "%s: prepared buffer is NULL or misaligned", who);
  if ((rc = check_codes(plan, who, idx, qjl, gamma))) return rc;
  TQ_REQUIRE(scores != nullptr && lds >= n, TQ_ERR_INVALID_ARG, "%s: scores is NULL or lds < n", who);
  TQ_REQUIRE(aligned(scores, 16), TQ_ERR_ALIGNMENT, "%s: scores is not 16-byte aligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const float* Qcat = static_cast<const float*>(prepared);
  if (!plan->ms.ok) {
    TQ_CHECK_CUDA(score_block(plan, Qcat, nq, 0, n, idx, qjl, gamma, norms, scores, lds, st), who);
    return TQ_OK;
  }
  const ScanEngine eng = pick_engine(plan, nq);
  const size_t slot = align_up(eng.ws_bytes, 256);
  const char* base = static_cast<const char*>(prepared) + qcat_bytes(plan, nq);
  const int per = eng.tc ? kGroupQueries : eng.qpp;
  for (int q0 = 0; q0 < nq; q0 += eng.qpp) {
    const int nqp = std::min(eng.qpp, nq - q0);
    const void* ws = base + (size_t)(q0 / per) * slot;
    // the codes may have been written by the kernel just ahead in the stream: no early start of the scan here
    if (eng.nib) rc = nscan::run(plan, nqp, n, idx, qjl, gamma, norms, scores + (int64_t)q0 * lds, lds, nullptr, nullptr, ws, false, st, who);
    else rc = engine_run(eng, q0, nqp, n, idx, qjl, gamma, norms, scores + (int64_t)q0 * lds, lds, nullptr, nullptr, ws, st, who);
    if (rc) return rc;
  }
  return TQ_OK;
}

// Top-k through the tensor-path scan.  Large n: a pilot pass over the first rows gives, per query,
// the k-th best score among them -- a lower bound on the final k-th score -- and the full pass
// keeps only (score, id) pairs at or above it; a final selection sorts the survivors.  Should a
// candidate list overflow (massive ties, adversarial order) a device-side flag switches on a
// dense block-by-block rescue pass that is otherwise launched as a no-op.
static int topk_ms(const tq_plan* plan, const float* Qcat, int nq, int64_t n, const uint8_t* idx, const uint8_t* qjl,
                   const float* gamma, const float* norms, int k, float* top_scores, int32_t* top_ids, char* ws,
                   size_t ws_bytes, cudaStream_t st, const char* who) {
  int rc;
  const ScanEngine eng = pick_engine(plan, nq);
  void* msw = ws;
  char* p = ws + align_up(eng.ws_bytes, 256);
  float* tau = reinterpret_cast<float*>(p);          // [qpp] (qpp <= 64: 256 bytes)
  int* count = reinterpret_cast<int*>(p + 256);      // [qpp], then the overflow flag
  int* overflow = count + eng.qpp;
  p += 1024;
  float* cand_s = reinterpret_cast<float*>(p);
  int* cand_i = reinterpret_cast<int*>(p + (size_t)eng.qpp * kCandCap * 4);
  p += (size_t)eng.qpp * kCandCap * 8;
  float* dense = reinterpret_cast<float*>(p);
  const int64_t dense_floats = (int64_t)((ws + ws_bytes - p) / sizeof(float));
  const int qpp = eng.qpp;
  const size_t xrb = plan->idx_row_bytes, qrb = plan->qjl_row_bytes;
  for (int q0 = 0; q0 < nq; q0 += qpp) {
    const int nqp = std::min(qpp, nq - q0);
    float* ts = top_scores + (size_t)q0 * k;
    int32_t* ti = top_ids + (size_t)q0 * k;
    if ((rc = engine_prepare(eng, Qcat, q0, nq, msw, st, who))) return rc;
    const int64_t dense_rows = dense_floats / qpp;
    const bool use_filter = n >= kFilterMinN && dense_rows >= std::min<int64_t>(n, eng.dense_rows_pref);
    const int* guard = nullptr;
    if (use_filter) {
      int64_t m = std::max<int64_t>(round_up64(n / 64, 256), round_up64(std::max(k, 4096), 256));
      m = std::min<int64_t>(m, std::min<int64_t>(dense_rows / 256 * 256, n));
      if ((rc = engine_run(eng, q0, nqp, m, idx, qjl, gamma, norms, dense, m, nullptr, nullptr, msw, st, who))) return rc;
      TQ_CHECK_CUDA(mscan::select_topk(dense, nullptr, nullptr, (int)m, (int)m, 0, nqp, k, 0, ts, ti, tau, nullptr, nullptr, st), who);
      TQ_CHECK_CUDA(cudaMemsetAsync(count, 0, (size_t)(qpp + 1) * sizeof(int), st), who);   // counters and the overflow flag
      mscan::Filter f{tau, count, cand_s, cand_i, kCandCap};
      if ((rc = engine_run(eng, q0, nqp, n, idx, qjl, gamma, norms, nullptr, 0, &f, nullptr, msw, st, who))) return rc;
      TQ_CHECK_CUDA(mscan::select_topk(cand_s, cand_i, count, kCandCap, 0, 0, nqp, k, 0, ts, ti, nullptr, overflow, nullptr, st), who);
      guard = overflow;
    }
    // dense block flow: the whole job for small n, the guarded rescue otherwise
    int64_t block = std::min<int64_t>(dense_rows, n);
    if (block < n) block = block / 256 * 256;
    for (int64_t v0 = 0; v0 < n; v0 += block) {
      const int64_t cn = std::min(block, n - v0);
      if ((rc = engine_run(eng, q0, nqp, cn, idx ? idx + (size_t)v0 * xrb : nullptr, qjl ? qjl + (size_t)v0 * qrb : nullptr,
                           gamma ? gamma + v0 : nullptr, norms ? norms + v0 : nullptr, dense, block, nullptr, guard, msw, st, who)))
        return rc;
      TQ_CHECK_CUDA(mscan::select_topk(dense, nullptr, nullptr, (int)block, (int)cn, (int)v0, nqp, k, v0 > 0 ? 1 : 0, ts, ti,
                                       nullptr, nullptr, guard, st), who);
    }
  }
  return TQ_OK;
}

extern "C" int tq_topk(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
                       const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms, int k,
                       float* top_scores, int32_t* top_ids, void* workspace, size_t workspace_bytes, void* stream) {
  const char* who = "tq_topk";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(n >= 0 && nq >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (nq == 0) return TQ_OK;
  TQ_REQUIRE(n <= 0x7fffffffLL, TQ_ERR_UNSUPPORTED, "%s: ids are int32, n too large", who);
  TQ_REQUIRE(k >= 1 && k <= TQ_MAX_K && k <= n, TQ_ERR_UNSUPPORTED, "%s: k=%d outside 1..min(n, %d)", who, k, TQ_MAX_K);
  if ((rc = check_rows(who, "Q", Q, q_dtype, nq, ldq, plan->d))) return rc;
  if ((rc = check_codes(plan, who, idx, qjl, gamma))) return rc;
  TQ_REQUIRE(top_scores != nullptr && top_ids != nullptr, TQ_ERR_INVALID_ARG, "%s: output is NULL", who);
  const size_t qb = qcat_bytes(plan, nq);
  const size_t need = plan->ms.ok ? ms_topk_fixed(plan, nq) + (size_t)pick_engine(plan, nq).qpp * kDenseRowsMin * sizeof(float)
                                  : qb + align_up((size_t)nq * std::min<int64_t>(n, kTopkBlockMin) * sizeof(float), 256);
  TQ_REQUIRE(workspace != nullptr && workspace_bytes >= need, TQ_ERR_WORKSPACE, "%s: workspace of %zu bytes, %zu needed",
             who, workspace_bytes, need);
  TQ_REQUIRE(aligned(workspace, 256), TQ_ERR_ALIGNMENT, "%s: workspace is not 256-byte aligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* Qcat = static_cast<float*>(workspace);
  if (plan->ms.ok) {
    TQ_CHECK_CUDA(prepare_queries(plan, Q, q_dtype, nq, ldq, Qcat, st), who);
    return topk_ms(plan, Qcat, nq, n, idx, qjl, gamma, norms, k, top_scores, top_ids, static_cast<char*>(workspace) + qb,
                   workspace_bytes - qb, st, who);
  }
  float* blockbuf = reinterpret_cast<float*>(static_cast<char*>(workspace) + qb);
  int64_t block = (int64_t)((workspace_bytes - qb) / ((size_t)nq * sizeof(float)));
  block = std::min(block, n);
  if (block < n) block = block / 256 * 256;
  TQ_CHECK_CUDA(prepare_queries(plan, Q, q_dtype, nq, ldq, Qcat, st), who);
  for (int64_t v0 = 0; v0 < n; v0 += block) {
    const int64_t cn = std::min(block, n - v0);
    TQ_CHECK_CUDA(score_block(plan, Qcat, nq, v0, cn, idx, qjl, gamma, norms, blockbuf, block, st), who);
    scan::topk_merge_kernel<<<nq, 256, 0, st>>>(blockbuf, block, v0, cn, k, v0 == 0 ? 1 : 0, top_scores, top_ids);
    count_launches(1);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
  }
  return TQ_OK;
}

template <int BITS>
static cudaError_t launch_wsum_partial(const tq_plan* plan, const attend::WsumArgs& a, dim3 grid, cudaStream_t st) {
  if (plan->mode == TQ_PROD) attend::wsum_partial_kernel<BITS, true><<<grid, 128, 0, st>>>(a);
  else attend::wsum_partial_kernel<BITS, false><<<grid, 128, 0, st>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

extern "C" int tq_wsum(const tq_plan* plan, const float* W, int nw, int64_t ldw, int64_t n, const uint8_t* idx,
                       const uint8_t* qjl, const float* gamma, const float* norms, float* out, int64_t ldo,
                       void* workspace, size_t workspace_bytes, void* stream) {
  const char* who = "tq_wsum";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);
  if (rc) return rc;
  TQ_REQUIRE(n >= 0 && nw >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (nw == 0) return TQ_OK;
  TQ_REQUIRE(out != nullptr && ldo >= plan->d, TQ_ERR_INVALID_ARG, "%s: out is NULL or ldo < d", who);
  TQ_REQUIRE(aligned(out, 16), TQ_ERR_ALIGNMENT, "%s: out is not 16-byte aligned", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (n == 0) {
    TQ_CHECK_CUDA(cudaMemset2DAsync(out, (size_t)ldo * sizeof(float), 0, (size_t)plan->d * sizeof(float), nw, st), who);
    return TQ_OK;
  }
  TQ_REQUIRE(W != nullptr && ldw >= n, TQ_ERR_INVALID_ARG, "%s: W is NULL or ldw < n", who);
  if ((rc = check_codes(plan, who, idx, qjl, gamma))) return rc;
  const size_t need = tq_workspace_bytes(plan, TQ_OP_WSUM, n, nw, 0);
  TQ_REQUIRE(workspace != nullptr && workspace_bytes >= need, TQ_ERR_WORKSPACE, "%s: workspace of %zu bytes, %zu needed",
             who, workspace_bytes, need);
  TQ_REQUIRE(aligned(workspace, 16), TQ_ERR_ALIGNMENT, "%s: workspace is not 16-byte aligned", who);
  const int ncols = plan->ncat * plan->dpad;
  float* oprime = static_cast<float*>(workspace);
  float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + align_up((size_t)nw * ncols * sizeof(float), 256));
  const int nchunks = (int)((n + attend::WS_TOK - 1) / attend::WS_TOK);
  for (int w0 = 0; w0 < nw; w0 += attend::WS_NW) {
    attend::WsumArgs a;
    a.W = W + (int64_t)w0 * ldw;
    a.ldw = ldw;
    a.nw = std::min(attend::WS_NW, nw - w0);
    a.n = n;
    a.idx = idx;
    a.idx_rb = plan->idx_row_bytes;
    a.qjl = qjl;
    a.qjl_rb = plan->qjl_row_bytes;
    a.gamma = gamma;
    a.norms = norms;
    a.cb = plan->cb;
    a.d = plan->d;
    a.dpad = plan->dpad;
    a.ncols = ncols;
    a.coef = plan->coef;
    a.nibble = plan->layout == TQ_LAYOUT_NIBBLE;
    a.partial = partial;
    const dim3 grid((unsigned)nchunks, (unsigned)((plan->d + 127) / 128));
    // columns the partial kernel never writes (pad coordinates) must read as zero
    TQ_CHECK_CUDA(cudaMemsetAsync(partial, 0, (size_t)nchunks * a.nw * ncols * sizeof(float), st), who);
    cudaError_t e;
    switch (plan->mse_bits) {
      case 0: e = launch_wsum_partial<0>(plan, a, grid, st); break;
      case 1: e = launch_wsum_partial<1>(plan, a, grid, st); break;
      case 2: e = launch_wsum_partial<2>(plan, a, grid, st); break;
      case 3: e = launch_wsum_partial<3>(plan, a, grid, st); break;
      default: e = launch_wsum_partial<4>(plan, a, grid, st); break;
    }
    TQ_CHECK_CUDA(e, who);
    attend::wsum_reduce_kernel<<<(unsigned)((a.nw * ncols + 255) / 256), 256, 0, st>>>(partial, nchunks, a.nw, ncols,
                                                                                        oprime + (size_t)w0 * ncols);
    count_launches(1);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
  }
  // out = o' [Pi ; S]
  simt::RowsF32 A{oprime, ncols, nw, ncols};
  simt::RowsF32 B{plan->dBackT, ncols, plan->d, ncols};
  simt::EpStore ep{out, ldo, nullptr, nullptr};
  TQ_CHECK_CUDA(simt::launch_gemm(A, B, ep, (int64_t)nw, (int64_t)plan->d, ncols, st), who);
  return TQ_OK;
}

extern "C" int tq_select_topk(const float* cand_scores, const int32_t* cand_ids, int nq, int64_t m, int64_t ld, int k,
                              float* top_scores, int32_t* top_ids, void* stream) {
  const char* who = "tq_select_topk";
  TQ_RANGE(who);
  TQ_REQUIRE(nq >= 0 && m >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  TQ_REQUIRE(k >= 1 && k <= TQ_MAX_K, TQ_ERR_UNSUPPORTED, "%s: k=%d outside 1..%d", who, k, TQ_MAX_K);
  TQ_REQUIRE(m <= 0x7fffffffLL && ld <= 0x7fffffffLL, TQ_ERR_UNSUPPORTED, "%s: m / ld too large", who);
  if (nq == 0) return TQ_OK;
  TQ_REQUIRE(top_scores != nullptr && top_ids != nullptr, TQ_ERR_INVALID_ARG, "%s: output is NULL", who);
  TQ_REQUIRE(m == 0 || (cand_scores != nullptr && cand_ids != nullptr && ld >= m), TQ_ERR_INVALID_ARG,
             "%s: candidates are NULL or ld < m", who);
  TQ_CHECK_CUDA(mscan::select_pairs(cand_scores, cand_ids, (int)ld, (int)m, nq, k, top_scores, top_ids,
                                    static_cast<cudaStream_t>(stream)), who);
  return TQ_OK;
}

extern "C" int tq_softmax(const float* s1, const float* s2, int nw, int64_t n, int64_t lds, float scale, float* W,
                          int64_t ldw, void* stream) {
  const char* who = "tq_softmax";
  TQ_RANGE(who);
  TQ_REQUIRE(nw >= 0 && n >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (nw == 0 || n == 0) return TQ_OK;
  TQ_REQUIRE(s1 != nullptr && W != nullptr, TQ_ERR_INVALID_ARG, "%s: s1 / W is NULL", who);
  TQ_REQUIRE(lds >= n && ldw >= n, TQ_ERR_INVALID_ARG, "%s: row stride smaller than n", who);
  attend::softmax_rows_kernel<<<nw, 1024, 0, static_cast<cudaStream_t>(stream)>>>(s1, s2, lds, n, scale, W, ldw);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

// ======================================================================================
// tq_score_static: tq_score for callers that cannot allocate.  The rotated-query workspace is
// this file-scope device array instead of a caller buffer.  In host code the array's name is
// only a handle for the runtime, not a device address, so the address is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernels get.
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[TQ_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// Device address of the static scratch on the current device (looked up on first use).
int static_scratch(const char* who, int device, void** out) {
  TQ_REQUIRE(device >= 0 && device < kMaxDevices, TQ_ERR_UNSUPPORTED, "%s: device ordinal %d not supported", who, device);
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[device] == nullptr) {
    void* p = nullptr;
    TQ_CHECK_CUDA(cudaGetSymbolAddress(&p, g_static_scratch), who);
    TQ_REQUIRE(p != nullptr && aligned(p, 256), TQ_ERR_CUDA, "%s: static scratch has no usable device address", who);
    g_static_ptr[device] = p;
  }
  *out = g_static_ptr[device];
  return TQ_OK;
}

}  // namespace

// Largest nq tq_score_static accepts for this plan (0 if even one query does not fit).
extern "C" int tq_score_static_max_queries(const tq_plan* plan) {
  if (!plan) return 0;
  int lo = 0, hi = 1 << 16;
  while (lo < hi) {   // the need grows with nq
    const int mid = lo + (hi - lo + 1) / 2;
    const size_t qb = qcat_bytes(plan, mid);
    ScanEngine e{};
    const bool ok = qb <= (size_t)TQ_STATIC_SCRATCH_BYTES &&
                    (!plan->ms.ok || engine_that_fits(plan, mid, (size_t)TQ_STATIC_SCRATCH_BYTES - qb, &e));
    if (ok) lo = mid; else hi = mid - 1;
  }
  return lo;
}

extern "C" int tq_score_static(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
                               const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms,
                               float* scores, int64_t lds, void* stream) {
  const char* who = "tq_score_static";
  TQ_RANGE(who);
  int rc = check_plan(plan, who);   // also makes sure the plan's device is the current one
  if (rc) return rc;
  TQ_REQUIRE(n >= 0 && nq >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  if (n == 0 || nq == 0) return TQ_OK;
  if ((rc = check_score_args(plan, who, Q, q_dtype, nq, ldq, n, idx, qjl, gamma, scores, lds))) return rc;
  const size_t qb = qcat_bytes(plan, nq);
  ScanEngine eng{};
  const bool fits = qb <= (size_t)TQ_STATIC_SCRATCH_BYTES &&
                    (!plan->ms.ok || engine_that_fits(plan, nq, (size_t)TQ_STATIC_SCRATCH_BYTES - qb, &eng));
  TQ_REQUIRE(fits, TQ_ERR_WORKSPACE,
             "%s: %d queries at d=%d need more scratch than the built-in array holds (%u bytes; at most %d queries "
             "for this plan); use tq_score with a caller workspace or fewer queries per call",
             who, nq, plan->d, (unsigned)TQ_STATIC_SCRATCH_BYTES, tq_score_static_max_queries(plan));
  void* ws = nullptr;
  if ((rc = static_scratch(who, plan->device, &ws))) return rc;
  // Every byte the kernels read from the array (rotated queries, then the scan engine's constants and operand)
  // is written by this call before it is read, so the previous call's leftovers never show.
  return score_on_workspace(plan, &eng, Q, q_dtype, nq, ldq, n, idx, qjl, gamma, norms, scores, lds, ws,
                            static_cast<cudaStream_t>(stream), who);
}

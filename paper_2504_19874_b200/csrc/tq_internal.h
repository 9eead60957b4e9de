// Internal declarations shared by the translation units of libtq (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <nvtx3/nvToolsExt.h>

#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "tq.h"

namespace tq {

void set_error(const char* fmt, ...);
void count_launches(int k);   // kernels enqueued by this library (diagnostic counter)
int lloyd_max(int d, int bits, double* c_out);

// Every API call that enqueues device work opens an NVTX range with its own name (visible in Nsight Systems /
// Compute timelines; a no-op without a profiler attached) and, when the environment variable TQ_LOG is set to a
// non-empty value other than 0, writes one line to stderr.
bool log_enabled();
struct CallRange {
  explicit CallRange(const char* name) {
    nvtxRangePushA(name);
    if (log_enabled()) std::fprintf(stderr, "[tq] %s\n", name);
  }
  ~CallRange() { nvtxRangePop(); }
  CallRange(const CallRange&) = delete;
  CallRange& operator=(const CallRange&) = delete;
};
#define TQ_RANGE(name) tq::CallRange tq_call_range_(name)

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
inline int64_t round_up64(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

// Codebook and thresholds by value, so kernels get them through the parameter space.
struct Codebook {
  float c[16];   // centroids, ascending
  float t[15];   // boundaries fl32(0.5f * (c_i + c_{i+1}))
  int bits;      // b_m
};

// A d x d fp32 matrix split into two bf16 limbs (M = hi + lo + O(2^-17)), rows padded to dpad,
// with the TMA descriptors the tensor-core GEMM uses for it as the B operand.
// Device-side index checks of the TQ_DEBUG build: `if (TQ_DEVICE_CHECK(row < n, status)) out[row] = v;`.  In a release
// build the condition is not evaluated.  A failed check records TQ_ERR_BOUNDS in the plan's status word (reported by
// tq_plan_status) and the access is skipped.
#ifdef __CUDACC__
#ifdef TQ_DEBUG
__device__ __forceinline__ bool device_check_failed(int* status) {
  if (status != nullptr) atomicExch(status, TQ_ERR_BOUNDS);
  return false;
}
#define TQ_DEVICE_CHECK(cond, status) ((cond) ? true : ::tq::device_check_failed(status))
#else
#define TQ_DEVICE_CHECK(cond, status) (true)
#endif
#endif

struct MatrixLimbs {
  __nv_bfloat16* hi;
  __nv_bfloat16* lo;
  alignas(64) CUtensorMap map_hi;
  alignas(64) CUtensorMap map_lo;
  alignas(64) CUtensorMap map_hi_half;   // boxes of half as many rows: what one CTA of a pair loads
  alignas(64) CUtensorMap map_lo_half;
};

}  // namespace tq

// Per-(d, b, mode) device state: the "global parameters" of Algorithms 1 and 2.
struct tq_plan {
  int d;          // dimension
  int dpad;       // d rounded up to a multiple of 8 (virtual K extent of one code half)
  int bits;       // total bits b
  int mode;       // TQ_MSE / TQ_PROD
  int mse_bits;   // b_m
  int device;
  float coef;     // sqrt(pi/2) / d
  size_t idx_row_bytes, qjl_row_bytes;
  tq::Codebook cb;
  float* dPi;      // [d, d]            y = Pi x            (rows of Pi)
  float* dSp;      // [d, d]            S' = S Pi^T         (TQ_PROD)
  float* dRotCat;  // [ncat*dpad, d]    rows: Pi (padded to dpad rows) then S     (query preparation)
  float* dBackT;   // [d, ncat*dpad]    row j: [ Pi[:, j] | S[:, j] ]             (dequantisation)
  int ncat;        // 1 (mse) or 2 (prod): halves of the virtual K axis [ c[idx] | coef*gamma*z ]
  // tensor-core quantisation path (d >= 128)
  int tc_ok;       // 1 when the limbs / TMA descriptors below are built
  int tc_bn;       // N extent of its MMA tile
  tq::MatrixLimbs pi_limbs;   // Pi
  tq::MatrixLimbs sp_limbs;   // S' (TQ_PROD)
  // bit-plane scan on the integer tensor path (d >= 128, antisymmetric codebook)
  struct {
    int ok;            // 1 when this plan can use it
    int R;             // ranges of 512 coordinates per row
    double alpha[8];   // odd Walsh coefficients of the codebook: index bits 0..3, then the 3-bit parities
    double amax;       // max |alpha|
    double csum;       // mean term minus the sum of alpha: constant part of sum_j q'_j c[idx_j]
  } ms;
  // nibble layout of the codes and the table-lookup scan (TQ_PROD with a 3-bit MSE stage)
  int layout;      // TQ_LAYOUT_*: arrangement of the idx / qjl rows this plan writes and reads
  struct {
    int ok;                            // 1 when this plan may be switched to TQ_LAYOUT_NIBBLE
    int nbi, nbq;                      // 64-byte blocks of an idx row / a qjl row
    uint32_t hi_a, hi_b, lo_a, lo_b;   // 16-bit centroid table t_i = 256 h_i + l_i as bytes: h of entries 0..3, 4..7, l alike
    double delta;                      // c_i ~ delta * t_i
  } nb;
  int* d_status;   // device word: set to TQ_ERR_TIMEOUT by a kernel whose bounded wait ran out
};

#define TQ_CHECK_CUDA(call, what)                                                        \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      tq::set_error("%s: %s", what, cudaGetErrorString(e_));                             \
      return TQ_ERR_CUDA;                                                                \
    }                                                                                    \
  } while (0)

#define TQ_REQUIRE(cond, code, ...)                                                      \
  do {                                                                                   \
    if (!(cond)) {                                                                       \
      tq::set_error(__VA_ARGS__);                                                        \
      return code;                                                                       \
    }                                                                                    \
  } while (0)

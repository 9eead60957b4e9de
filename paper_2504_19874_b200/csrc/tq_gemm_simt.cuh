// CUDA-core fp32 GEMM  C[M,N] = A[M,K] * B[N,K]^T  with pluggable operand loaders and
// epilogues.  It serves the shapes where the rotation is not tensor-bound (small d), the
// set-up products (query preparation) and dequantisation, where exact fp32 FMAs are wanted.
// A loader hands out 8 consecutive k of one row as floats; an epilogue consumes the 8x8
// accumulator block each thread owns.
#pragma once

#include "tq_internal.h"

namespace tq {
namespace simt {

constexpr int BM = 128, BN = 128, BK = 16, NT = 256;
constexpr int LDS_A = BM + 4, LDS_B = BN + 4;
constexpr int STAGE_LD = BN + 4;  // byte stride of the code staging tile

__device__ __forceinline__ bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// ---------------------------------------------------------------- operand loaders
struct RowsF32 {
  const float* p;
  int64_t ld;
  int64_t rows;
  int K;
  __device__ __forceinline__ void load(int64_t r, int k0, float (&v)[8]) const {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
    if (r >= rows || k0 >= K) return;
    const float* s = p + r * ld + k0;
    if (k0 + 8 <= K && aligned16(s)) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(s));
      const float4 b = __ldg(reinterpret_cast<const float4*>(s) + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
      v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (k0 + i < K) v[i] = __ldg(s + i);
    }
  }
};

struct RowsBF16 {
  const __nv_bfloat16* p;
  int64_t ld;
  int64_t rows;
  int K;
  __device__ __forceinline__ void load(int64_t r, int k0, float (&v)[8]) const {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
    if (r >= rows || k0 >= K) return;
    const __nv_bfloat16* s = p + r * ld + k0;
    if (k0 + 8 <= K && aligned16(s)) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(s));
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (k0 + i < K) v[i] = __bfloat162float(s[i]);
    }
  }
};

// Virtual operand decoded from packed codes: columns [0, dpad) are c[idx_j], columns
// [dpad, 2*dpad) are coef * gamma * z_j (present when qjl != nullptr).
struct Codes {
  const uint8_t* idx;
  size_t idx_rb;
  const uint8_t* qjl;
  size_t qjl_rb;
  const float* gamma;
  Codebook cb;
  int d, dpad;
  float coef;
  int64_t rows;
  bool nibble;   // TQ_LAYOUT_NIBBLE: nibble j of the combined row [idx row | qjl row] = index | sign << 3
  __device__ __forceinline__ void load(int64_t r, int k0, float (&v)[8]) const {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = 0.f;
    if (r >= rows) return;
    if (nibble) {   // k0 is a multiple of 8: one 32-bit word of the combined row holds the eight coordinates
      const int j0 = k0 < dpad ? k0 : k0 - dpad;
      if (j0 >= d) return;
      const size_t byte = (size_t)j0 >> 1;
      const uint8_t* s = byte < idx_rb ? idx + (size_t)r * idx_rb + byte : qjl + (size_t)r * qjl_rb + (byte - idx_rb);
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(s));
      const float g = k0 < dpad ? 0.f : coef * __ldg(gamma + r);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (j0 + i >= d) break;
        const uint32_t nib = (w >> (4 * i)) & 15u;
        v[i] = k0 < dpad ? cb.c[nib & 7u] : ((nib & 8u) ? g : -g);
      }
      return;
    }
    if (k0 < dpad) {
      const int bits = cb.bits;
      if (bits == 0 || k0 >= d) return;
      const size_t off = ((size_t)k0 * bits) >> 3;
      const uint8_t* s = idx + (size_t)r * idx_rb + off;
      uint32_t w = 0;
      for (int i = 0; i < bits; ++i)
        if (off + i < idx_rb) w |= (uint32_t)__ldg(s + i) << (8 * i);
      const uint32_t mask = (1u << bits) - 1u;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (k0 + i < d) v[i] = cb.c[(w >> (i * bits)) & mask];
    } else if (qjl != nullptr) {
      const int j0 = k0 - dpad;
      if (j0 >= d) return;
      const uint32_t byte = __ldg(qjl + (size_t)r * qjl_rb + (j0 >> 3));
      const float g = coef * __ldg(gamma + r);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (j0 + i < d) v[i] = ((byte >> i) & 1u) ? g : -g;
    }
  }
};

// ---------------------------------------------------------------- epilogues
// Thread (tx, ty) of the 16x16 layout owns rows {ty*4+i, 64+ty*4+i} and columns
// {tx*4+j, 64+tx*4+j}, i, j in 0..3.
__device__ __forceinline__ int tile_row(int ty, int i) { return (i < 4) ? ty * 4 + i : 64 + ty * 4 + (i - 4); }
__device__ __forceinline__ int tile_col(int tx, int j) { return (j < 4) ? tx * 4 + j : 64 + tx * 4 + (j - 4); }

struct EpStore {
  float* C;
  int64_t ldc;
  const float* row_scale;  // multiplies row m (nullable)
  const float* col_scale;  // multiplies column n (nullable)
  __device__ __forceinline__ void run(float (&acc)[8][8], int64_t m0, int64_t n0, int64_t M, int64_t N,
                                      int tid, unsigned char* smem) const {
    const int tx = tid % 16, ty = tid / 16;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int64_t r = m0 + tile_row(ty, i);
      if (r >= M) continue;
      const float rs = row_scale ? __ldg(row_scale + r) : 1.f;
#pragma unroll
      for (int jh = 0; jh < 2; ++jh) {
        const int64_t c = n0 + tile_col(tx, jh * 4);
        float o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float cs = (col_scale && c + j < N) ? __ldg(col_scale + c + j) : 1.f;
          o[j] = acc[i][jh * 4 + j] * rs * cs;
        }
        float* dst = C + r * ldc + c;
        if (c + 4 <= N && aligned16(dst)) {
          *reinterpret_cast<float4*>(dst) = make_float4(o[0], o[1], o[2], o[3]);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (c + j < N) dst[j] = o[j];
        }
      }
    }
  }
};

// MODE 0: nearest-centroid index (Algorithm 1, idx_j) -> packed idx.
// MODE 1: the same plus the rotated residual e = y/nu - c[idx] written to E (Algorithm 2).
// MODE 2: sign bits of the accumulator (qjl = sign(S r)) -> packed, BITS must be 1.
template <int BITS, int MODE>
struct EpQuantize {
  Codebook cb;
  const float* nu;   // per-row norm; nullptr = 1
  uint8_t* out;      // packed rows (idx or qjl)
  size_t out_rb;
  float* E;          // MODE 1
  int64_t ldE;
  int d;
  __device__ __forceinline__ void run(float (&acc)[8][8], int64_t m0, int64_t n0, int64_t M, int64_t N,
                                      int tid, unsigned char* stage) const {
    const int tx = tid % 16, ty = tid / 16;
    constexpr int NB = (1 << BITS) - 1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int rl = tile_row(ty, i);
      const int64_t r = m0 + rl;
      float v = 1.f;
      if (MODE != 2 && nu != nullptr && r < M) v = __ldg(nu + r);
      const float vcmp = (v > 0.f) ? v : 1.f;
      const float inv = (v > 0.f) ? 1.f / v : 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int cl = tile_col(tx, j);
        const float y = acc[i][j];
        int code = 0;
        if (MODE == 2) {
          code = (y >= 0.f) ? 1 : 0;
        } else {
#pragma unroll
          for (int t = 0; t < NB; ++t) code += (y > cb.t[t] * vcmp) ? 1 : 0;
        }
        if (MODE == 1) {
          const int64_t c = n0 + cl;
          if (r < M && c < d) E[r * ldE + c] = (v > 0.f) ? (y * inv - cb.c[code]) : 0.f;
        }
        if (BITS > 0) stage[rl * STAGE_LD + cl] = (unsigned char)code;
      }
    }
    if (BITS == 0) return;
    __syncthreads();
    // Pack: a group of 32 coordinates makes exactly BITS 32-bit words of the row's bit stream.
    for (int task = tid; task < BM * (BN / 32); task += NT) {
      const int rl = task / (BN / 32), g = task % (BN / 32);
      const int64_t r = m0 + rl;
      const int64_t cbase = n0 + g * 32;
      if (r >= M || cbase >= d) continue;
      const uint32_t* src = reinterpret_cast<const uint32_t*>(stage + rl * STAGE_LD + g * 32);
      unsigned long long bitbuf = 0;
      int nb = 0, widx = 0;
      uint32_t* dst = reinterpret_cast<uint32_t*>(out + (size_t)r * out_rb);
      const size_t word0 = (size_t)(cbase / 32) * BITS;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const uint32_t four = src[q];
#pragma unroll
        for (int s = 0; s < 4; ++s) {
          const int col = q * 4 + s;
          uint32_t code = (four >> (8 * s)) & 0xffu;
          if (cbase + col >= d) code = 0;
          bitbuf |= (unsigned long long)code << nb;
          nb += BITS;
          if (nb >= 32) {
            if ((word0 + widx + 1) * 4 <= out_rb) dst[word0 + widx] = (uint32_t)bitbuf;
            bitbuf >>= 32;
            nb -= 32;
            ++widx;
          }
        }
      }
    }
  }
};

// ---------------------------------------------------------------- kernel
template <class AL, class BL, class EP>
__global__ void __launch_bounds__(NT) gemm_tn_kernel(AL A, BL B, EP ep, int64_t M, int64_t N, int K, int64_t tiles_n) {
  __shared__ __align__(16) float As[2][BK][LDS_A];
  __shared__ __align__(16) float Bs[2][BK][LDS_B];
  static_assert(sizeof(As) >= BM * STAGE_LD, "staging tile must fit in the A buffers");
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  const int64_t bid = blockIdx.x;
  const int64_t n0 = (bid % tiles_n) * BN, m0 = (bid / tiles_n) * BM;
  const int lrow = tid % 128, lk = (tid / 128) * 8;

  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  float ra[8], rb[8];
  A.load(m0 + lrow, lk, ra);
  B.load(n0 + lrow, lk, rb);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    As[0][lk + i][lrow] = ra[i];
    Bs[0][lk + i][lrow] = rb[i];
  }
  __syncthreads();
  const int ktiles = (K + BK - 1) / BK;
  for (int kt = 0; kt < ktiles; ++kt) {
    const int cur = kt & 1;
    if (kt + 1 < ktiles) {
      A.load(m0 + lrow, (kt + 1) * BK + lk, ra);
      B.load(n0 + lrow, (kt + 1) * BK + lk, rb);
    }
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[cur][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[cur][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[cur][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[cur][k][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (kt + 1 < ktiles) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        As[cur ^ 1][lk + i][lrow] = ra[i];
        Bs[cur ^ 1][lk + i][lrow] = rb[i];
      }
    }
    __syncthreads();
  }
  ep.run(acc, m0, n0, M, N, tid, reinterpret_cast<unsigned char*>(&As[0][0][0]));
}

template <class AL, class BL, class EP>
inline cudaError_t launch_gemm(const AL& A, const BL& B, const EP& ep, int64_t M, int64_t N, int K, cudaStream_t st) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  const int64_t tiles_n = (N + BN - 1) / BN, tiles_m = (M + BM - 1) / BM;
  const int64_t blocks = tiles_n * tiles_m;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  gemm_tn_kernel<AL, BL, EP><<<(unsigned)blocks, NT, 0, st>>>(A, B, ep, M, N, K, tiles_n);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace simt
}  // namespace tq

// CUDA-core kernels of the scan side: row norms, the few-query packed-code scan
// (estimator of Section 3.2 on the codes) and the running top-k merge.
#pragma once

#include <cfloat>

#include "tq_internal.h"

namespace tq {
namespace scan {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---------------------------------------------------------------- row L2 norms (Section 1.3)
template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__global__ void __launch_bounds__(256) row_norm_kernel(const T* __restrict__ X, int64_t ld, int64_t n, int d,
                                                        float* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t r = warp; r < n; r += nwarps) {
    const T* row = X + r * ld;
    float s = 0.f;
    for (int j = lane; j < d; j += 32) {
      const float v = to_f32<T>(row[j]);
      s = fmaf(v, v, s);
    }
    s = warp_sum(s);
    if (lane == 0) out[r] = sqrtf(s);
  }
}

// ---------------------------------------------------------------- few-query scan
struct ScanArgs {
  const uint8_t* idx;
  size_t idx_rb;
  const uint8_t* qjl;   // nullptr for TQ_MSE
  size_t qjl_rb;
  const float* gamma;
  const float* norms;   // nullptr = 1
  Codebook cb;
  int d, groups;        // groups = ceil(d / 32)
  float coef;
  int64_t n;
  const float* Qcat;    // [nq, ldq]: (Pi q | S q), each half dpad wide
  int64_t ldq;
  int dpad;
  int q0, nq_tile;      // queries [q0, q0 + nq_tile) are served by this launch
  float* scores;        // [nq, lds]
  int64_t lds;
};

// One warp walks 32 consecutive vectors; lane g decodes the g-th group of 32 coordinates
// (BITS words of idx, one word of qjl).  Queries sit in shared memory, permuted so that
// lanes reading coordinate i of their own group hit consecutive banks.
template <int BITS, int NQ, bool PROD>
__global__ void __launch_bounds__(256) scan_few_kernel(ScanArgs a) {
  extern __shared__ float qs[];  // [NQ][PROD ? 2 : 1][32 * groups]
  __shared__ float cbs[16];
  const int G = a.groups;
  const int half = 32 * G;
  constexpr int NH = PROD ? 2 : 1;
  for (int e = threadIdx.x; e < NQ * NH * half; e += blockDim.x) {
    const int q = e / (NH * half), rem = e % (NH * half);
    const int h = rem / half, pos = rem % half;
    const int i = pos / G, g = pos % G;
    const int j = g * 32 + i;
    float v = 0.f;
    if (q < a.nq_tile && j < a.d) v = a.Qcat[(int64_t)(a.q0 + q) * a.ldq + h * a.dpad + j];
    qs[e] = v;
  }
  if (threadIdx.x < 16) cbs[threadIdx.x] = a.cb.c[threadIdx.x];
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int64_t nblocks = (a.n + 31) / 32;
  const size_t idx_words = a.idx_rb / 4;
  constexpr uint32_t MASK = (1u << BITS) - 1u;

  for (int64_t blk = warp; blk < nblocks; blk += nwarps) {
    const int64_t v0 = blk * 32;
    float res[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) res[q] = 0.f;
    const int nv = (int)min((int64_t)32, a.n - v0);
    for (int vv = 0; vv < nv; ++vv) {
      const int64_t v = v0 + vv;
      float am[NQ], as[NQ];
#pragma unroll
      for (int q = 0; q < NQ; ++q) { am[q] = 0.f; as[q] = 0.f; }
      for (int g = lane; g < G; g += 32) {
        if (BITS > 0) {
          const uint32_t* row = reinterpret_cast<const uint32_t*>(a.idx + (size_t)v * a.idx_rb);
          uint32_t w[BITS > 0 ? BITS : 1];
#pragma unroll
          for (int t = 0; t < BITS; ++t) {
            const size_t wi = (size_t)g * BITS + t;
            w[t] = (wi < idx_words) ? __ldg(row + wi) : 0u;
          }
          unsigned long long buf = 0;
          int nb = 0, nw = 0;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            if (nb < BITS) {
              buf |= (unsigned long long)w[nw] << nb;
              nb += 32;
              ++nw;
            }
            const float c = cbs[(uint32_t)buf & MASK];
            buf >>= BITS;
            nb -= BITS;
#pragma unroll
            for (int q = 0; q < NQ; ++q) am[q] = fmaf(c, qs[(q * NH) * half + i * G + g], am[q]);
          }
        }
        if (PROD) {
          const uint32_t* row = reinterpret_cast<const uint32_t*>(a.qjl + (size_t)v * a.qjl_rb);
          const uint32_t w = ((size_t)g * 4 < a.qjl_rb) ? __ldg(row + g) : 0u;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const uint32_t flip = (~(w >> i) & 1u) << 31;  // bit 0 -> z = -1
#pragma unroll
            for (int q = 0; q < NQ; ++q)
              as[q] += __uint_as_float(__float_as_uint(qs[(q * NH + 1) * half + i * G + g]) ^ flip);
          }
        }
      }
      const float nu = a.norms ? __ldg(a.norms + v) : 1.f;
      const float gm = PROD ? a.coef * __ldg(a.gamma + v) : 0.f;
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        const float m = warp_sum(am[q]);
        const float s = PROD ? warp_sum(as[q]) : 0.f;
        const float est = nu * (m + gm * s);
        if (lane == vv) res[q] = est;
      }
    }
    if (lane < nv) {
#pragma unroll
      for (int q = 0; q < NQ; ++q)
        if (q < a.nq_tile) a.scores[(int64_t)(a.q0 + q) * a.lds + v0 + lane] = res[q];
    }
  }
}

// ---------------------------------------------------------------- running top-k
// One CTA per query keeps the best k (score desc, id asc) seen so far in top_s/top_i and
// merges a block of scores for vectors [v0, v0 + cn).  Candidates above the current k-th
// score are buffered and merged by a bitonic sort of (list + buffer).
constexpr int TOPK_CAP = 1024;

__device__ __forceinline__ bool better(float s1, int i1, float s2, int i2) {
  return (s1 > s2) || (s1 == s2 && i1 < i2);
}

__device__ inline void bitonic_sort_desc(float* s, int* id, int n /* power of two */) {
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = threadIdx.x; t < n; t += blockDim.x) {
        const int p = t ^ j;
        if (p > t) {
          const bool up = ((t & k) == 0);  // this pair sorts "best first" when up
          const bool t_better = better(s[t], id[t], s[p], id[p]);
          if (up ? !t_better : t_better) {
            const float fs = s[t]; s[t] = s[p]; s[p] = fs;
            const int fi = id[t]; id[t] = id[p]; id[p] = fi;
          }
        }
      }
      __syncthreads();
    }
  }
}

__global__ void __launch_bounds__(256) topk_merge_kernel(const float* __restrict__ scores, int64_t lds, int64_t v0,
                                                         int64_t cn, int k, int first, float* __restrict__ top_s,
                                                         int* __restrict__ top_i) {
  __shared__ float ss[2 * TOPK_CAP];
  __shared__ int si[2 * TOPK_CAP];
  __shared__ int count;
  __shared__ float thr;
  const int q = blockIdx.x;
  const float* row = scores + (int64_t)q * lds;
  for (int t = threadIdx.x; t < 2 * TOPK_CAP; t += blockDim.x) {
    float s = -INFINITY;
    int id = 0x7fffffff;
    if (t < k && !first) {
      s = top_s[(int64_t)q * k + t];
      id = top_i[(int64_t)q * k + t];
    }
    ss[t] = s;
    si[t] = id;
  }
  if (threadIdx.x == 0) count = 0;
  __syncthreads();
  if (threadIdx.x == 0) thr = ss[k - 1];
  __syncthreads();
  for (int64_t base = 0; base < cn; base += blockDim.x) {
    const int64_t p = base + threadIdx.x;
    if (p < cn) {
      const float s = row[p];
      if (s > thr) {
        const int slot = atomicAdd(&count, 1);
        ss[TOPK_CAP + slot] = s;
        si[TOPK_CAP + slot] = (int)(v0 + p);
      }
    }
    __syncthreads();
    const bool last = base + blockDim.x >= cn;
    if (count > TOPK_CAP - (int)blockDim.x || (last && count > 0)) {
      bitonic_sort_desc(ss, si, 2 * TOPK_CAP);
      for (int t = TOPK_CAP + threadIdx.x; t < 2 * TOPK_CAP; t += blockDim.x) {
        ss[t] = -INFINITY;
        si[t] = 0x7fffffff;
      }
      if (threadIdx.x == 0) {
        count = 0;
        thr = ss[k - 1];
      }
      __syncthreads();
    }
  }
  for (int t = threadIdx.x; t < k; t += blockDim.x) {
    top_s[(int64_t)q * k + t] = ss[t];
    top_i[(int64_t)q * k + t] = si[t];
  }
}

}  // namespace scan
}  // namespace tq

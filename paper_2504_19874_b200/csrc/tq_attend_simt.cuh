// CUDA-core kernels of the attention tail over a compressed KV cache: softmax of the (summed)
// score rows, and the weighted sum of dequantised vectors taken in the code domain,
//   sum_t w_t x~_t = Pi^T (sum_t w_t nu_t c[idx_t]) + S^T (coef sum_t w_t nu_t gamma_t z_t),
// so that the d x d products are applied once per output row instead of once per token.
#pragma once

#include <cfloat>

#include "tq_internal.h"

namespace tq {
namespace attend {

constexpr int WS_TOK = 128;   // tokens per partial sum
constexpr int WS_NW = 8;      // weight rows per launch

// W[w, t] = softmax_t( scale * (s1[w, t] + s2[w, t]) ); s2 may be null.  One CTA per row.
__global__ void __launch_bounds__(1024) softmax_rows_kernel(const float* __restrict__ s1, const float* __restrict__ s2,
                                                            int64_t lds, int64_t n, float scale, float* __restrict__ W,
                                                            int64_t ldw) {
  __shared__ float red[32];
  __shared__ float bcast;
  const int64_t base = (int64_t)blockIdx.x * lds;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  auto logit = [&](int64_t t) { return scale * (s1[base + t] + (s2 ? s2[base + t] : 0.f)); };
  float mx = -FLT_MAX;
  for (int64_t t = threadIdx.x; t < n; t += blockDim.x) mx = fmaxf(mx, logit(t));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = red[0];
    for (int w = 1; w < nwarps; ++w) m = fmaxf(m, red[w]);
    bcast = m;
  }
  __syncthreads();
  mx = bcast;
  __syncthreads();
  // sum of exponentials: per-thread partial sums in fp32, combined in a fixed order in fp64
  float sm = 0.f;
  for (int64_t t = threadIdx.x; t < n; t += blockDim.x) sm += __expf(logit(t) - mx);
  double ds = (double)sm;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ds += __shfl_xor_sync(0xffffffffu, ds, o);
  __shared__ double dred[32];
  if (lane == 0) dred[warp] = ds;
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot = 0.0;
    for (int w = 0; w < nwarps; ++w) tot += dred[w];
    bcast = (float)(1.0 / tot);
  }
  __syncthreads();
  const float inv = bcast;
  for (int64_t t = threadIdx.x; t < n; t += blockDim.x) W[(int64_t)blockIdx.x * ldw + t] = __expf(logit(t) - mx) * inv;
}

struct WsumArgs {
  const float* W;       // [nw, ldw]
  int64_t ldw;
  int nw;               // <= WS_NW
  int64_t n;
  const uint8_t* idx;
  size_t idx_rb;
  const uint8_t* qjl;
  size_t qjl_rb;
  const float* gamma;
  const float* norms;   // nullable
  Codebook cb;
  int d, dpad, ncols;
  float coef;
  bool nibble;          // TQ_LAYOUT_NIBBLE (BITS = 3, PROD): nibble j of [idx row | qjl row] = index | sign << 3
  float* partial;       // [nchunks, nw, ncols]
};

// Thread j owns coordinate j; the CTA walks WS_TOK tokens with the (scaled) weights in shared memory.
template <int BITS, bool PROD>
__global__ void __launch_bounds__(128) wsum_partial_kernel(WsumArgs a) {
  __shared__ float wn[WS_NW][WS_TOK];
  __shared__ float wg[PROD ? WS_NW : 1][WS_TOK];
  const int64_t t0 = (int64_t)blockIdx.x * WS_TOK;
  const int ntok = (int)min((int64_t)WS_TOK, a.n - t0);
  for (int e = threadIdx.x; e < WS_NW * WS_TOK; e += blockDim.x) {
    const int w = e / WS_TOK, tt = e % WS_TOK;
    float v = 0.f, g = 0.f;
    if (w < a.nw && tt < ntok) {
      const int64_t t = t0 + tt;
      v = a.W[(int64_t)w * a.ldw + t] * (a.norms ? a.norms[t] : 1.f);
      if (PROD) g = v * a.coef * a.gamma[t];
    }
    wn[w][tt] = v;
    if (PROD) wg[w][tt] = g;
  }
  __syncthreads();
  const int j = blockIdx.y * blockDim.x + threadIdx.x;
  if (j >= a.d) return;
  float acc[WS_NW], accs[WS_NW];
#pragma unroll
  for (int w = 0; w < WS_NW; ++w) acc[w] = accs[w] = 0.f;
  constexpr uint32_t MASK = (1u << BITS) - 1u;
  const int bitpos = j * BITS, byte0 = bitpos >> 3, sh = bitpos & 7;
  for (int tt = 0; tt < ntok; ++tt) {
    const int64_t t = t0 + tt;
    if (a.nibble) {
      const size_t byte = (size_t)j >> 1;
      const uint32_t x = byte < a.idx_rb ? a.idx[(size_t)t * a.idx_rb + byte] : a.qjl[(size_t)t * a.qjl_rb + (byte - a.idx_rb)];
      const uint32_t nib = (x >> (4 * (j & 1))) & 15u;
      const float c = a.cb.c[nib & 7u];
#pragma unroll
      for (int w = 0; w < WS_NW; ++w) {
        acc[w] = fmaf(wn[w][tt], c, acc[w]);
        if (PROD) accs[w] += (nib & 8u) ? wg[w][tt] : -wg[w][tt];
      }
      continue;
    }
    if (BITS > 0) {
      const uint8_t* row = a.idx + (size_t)t * a.idx_rb;
      uint32_t v = row[byte0];
      if (sh + BITS > 8) v |= (uint32_t)row[byte0 + 1] << 8;
      const float c = a.cb.c[(v >> sh) & MASK];
#pragma unroll
      for (int w = 0; w < WS_NW; ++w) acc[w] = fmaf(wn[w][tt], c, acc[w]);
    }
    if (PROD) {
      const uint32_t bit = (a.qjl[(size_t)t * a.qjl_rb + (j >> 3)] >> (j & 7)) & 1u;
#pragma unroll
      for (int w = 0; w < WS_NW; ++w) accs[w] += bit ? wg[w][tt] : -wg[w][tt];
    }
  }
  for (int w = 0; w < a.nw; ++w) {
    float* p = a.partial + ((size_t)blockIdx.x * a.nw + w) * a.ncols;
    p[j] = acc[w];
    if (PROD) p[a.dpad + j] = accs[w];
  }
}

// o'[w, col] = sum over chunks, in chunk order (deterministic).
__global__ void __launch_bounds__(256) wsum_reduce_kernel(const float* __restrict__ partial, int nchunks, int nw, int ncols,
                                                          float* __restrict__ out) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= nw * ncols) return;
  float s = 0.f;
  for (int c = 0; c < nchunks; ++c) s += partial[(size_t)c * nw * ncols + e];
  out[e] = s;
}

}  // namespace attend
}  // namespace tq

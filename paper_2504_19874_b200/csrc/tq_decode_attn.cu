// Decode attention over a compressed KV cache in three launches: scores of the Section 3.2 estimator on the packed K
// codes, softmax over the tokens, and the weighted sum of the dequantised V vectors taken in the code domain
// (Section 4.3 use of the quantisers), for all KV heads and channel groups of a layer at once.
//
// Two sets of kernels.  Antisymmetric codebooks (every Lloyd-Max codebook of the even coordinate density) take the
// integer tensor path of tq_decode_mma.cuh: prepare_mma_kernel, partial_mma_kernel.  Any other codebook takes the
// table-lookup kernels of this file:
//
//   prepare_kernel   per (head, group): gathers the group's channels of the head's queries and forms
//                    q' = Pi q, q'' = S q.
//   partial_kernel   per (head, slice of 256 tokens), flash-decode style:
//                    A) thread = token.  The MSE term sum_c q'_c c[idx_c] and the QJL term
//                       sum_i q''_i z_i are sums of table entries: four index bits (4, 2 or 1
//                       coordinates; one coordinate for 3-bit indices) select one float4 holding the
//                       partial sums of up to four queries, built per CTA from q', q'' and the codebook.
//                       logit = scale * sum_groups nu (mse + coef gamma qjl).
//                    B) slice maximum, p = exp(logit - max), sum of p.
//                    C) thread = output coordinate: acc[c] = sum_t p_t nu^V_t c_V[idx^V_{t,c}], walked
//                       in a fixed order, so results do not depend on timing.
//
// Both are followed by
//   merge_kernel     per (head, group): combines the slices (max / sum rescaling), divides by the sum and
//                    applies x~ = Pi_V^T y' per group, scattering to the group's channels.
//
// The table-lookup kernel spends ~120 warp instructions per token and head on CUDA cores; the unfused path (tq_score,
// tq_softmax, tq_wsum per head and group) is two orders of magnitude slower at 32k tokens because each of its 88
// launches serves one head.
#include <atomic>
#include <algorithm>
#include <cfloat>
#include <cstring>

#include "tq_internal.h"

namespace tq {
namespace kvdec {

constexpr int MAXG = TQ_MAX_KV_GROUPS;
constexpr int MAXQ = 4;          // queries per KV head (one float4 of partial sums)
constexpr int MAXD = 128;        // channels per group
constexpr int SLICE = 256;       // tokens per CTA
constexpr int NT = 256;          // threads per CTA

struct GroupDev {
  const uint8_t* k_idx;
  const uint8_t* k_qjl;
  const float* k_gamma;
  const float* k_norms;
  const uint8_t* v_idx;
  const float* v_norms;
  const int32_t* k_channels;
  const int32_t* v_channels;
  const float* k_backt;    // [d, ncat*dpad]: column o = row o of [Pi ; S]
  const float* v_pi;       // [d, d]
  float k_cent[16], v_cent[16];
  int k_bits, v_bits, k_prod;
  int k_idx_rb, k_qjl_rb, v_idx_rb;
  int k_dpad;
  float coef;
  int lut_mse_off, lut_qjl_off;   // float4 offsets of this group's tables in shared memory
  int vunit0;   // first of this group's units (runs of coordinates sharing bytes of the value row)
  int k_idx_soff, k_qjl_soff, v_idx_soff;   // byte offsets of the staged code rows inside their shared-memory buffers
};

struct Args {
  GroupDev g[MAXG];
  int ngroups, heads, qpk, d, nslices;
  int64_t tokens;
  int64_t head_stride;   // rows between consecutive heads in the code arrays (>= tokens)
  float scale;
  float* qrot;      // [heads, ngroups, MAXQ, 2*MAXD]
  float* part_ml;   // [heads, nslices, 2, MAXQ]      slice maximum, slice sum of exponentials
  float* part_acc;  // [heads, nslices, ngroups*d, MAXQ]
  int lut_float4;   // float4 entries of all tables
  int vunits, region0;   // units of all groups; float4 entries of the first shared-memory region
  int kbuf_bytes, vbuf_bytes;   // shared-memory room for the slice's K and V code rows
  int* status;      // the plans' device status word (bounded waits; index checks of the TQ_DEBUG build)
  int64_t ldq_dbg, ldo_dbg;   // row lengths of Q and out that a channel index must stay inside
};

__host__ __device__ inline int mse_lookups(int d, int bits) {   // table rows of the MSE term
  return bits == 0 ? 0 : bits == 1 ? d / 4 : bits == 2 ? d / 2 : d;
}
__host__ __device__ inline int mse_entries(int bits) { return bits == 3 ? 8 : 16; }

// ------------------------------------------------------------------ query preparation
template <typename T>
__global__ void __launch_bounds__(128) prepare_kernel(Args a, const T* __restrict__ Q, int64_t ldq) {
  __shared__ float qs[MAXQ][MAXD];
  const int h = blockIdx.x / a.ngroups, gi = blockIdx.x % a.ngroups;
  const GroupDev& g = a.g[gi];
  const int d = a.d;
  for (int e = threadIdx.x; e < MAXQ * d; e += blockDim.x) {
    const int j = e / d, c = e % d;
    float v = 0.f;
    if (j < a.qpk) {
      const int ch = g.k_channels[h * d + c];
      if (TQ_DEVICE_CHECK(ch >= 0 && ch < a.ldq_dbg, a.status)) v = (float)Q[(int64_t)(h * a.qpk + j) * ldq + ch];
    }
    qs[j][c] = v;
  }
  __syncthreads();
  float* out = a.qrot + (size_t)(h * a.ngroups + gi) * MAXQ * 2 * MAXD;
  const int nrows = (g.k_prod ? 2 : 1) * g.k_dpad;
  for (int o = threadIdx.x; o < nrows; o += blockDim.x) {
    const int half = o / g.k_dpad, r = o % g.k_dpad;
    float acc[MAXQ] = {0.f, 0.f, 0.f, 0.f};
    if (r < d) {
      const float* col = g.k_backt + o;   // consecutive threads read consecutive addresses
#pragma unroll 8
      for (int c = 0; c < d; ++c) {
        const float m = col[(size_t)c * nrows];
#pragma unroll
        for (int j = 0; j < MAXQ; ++j) acc[j] = fmaf(m, qs[j][c], acc[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < MAXQ; ++j) out[(size_t)j * 2 * MAXD + half * MAXD + r] = acc[j];
  }
}

// ------------------------------------------------------------------ per-slice scores, weights, V sums
__device__ __forceinline__ void add4(float4& a, const float4 b) {
  a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
}
// A table of E entries keeps the (x, y) halves of its float4 entries in one array of float2 and the (z, w) halves
// in a second one behind it: lanes that read different entries of one table row then hit different banks
// (16-byte entries collide pairwise), at the price of two loads per lookup.
__device__ __forceinline__ void add_entry(float4& a, const float2* __restrict__ t2, int entries, int e) {
  const float2 lo = t2[e], hi = t2[entries + e];
  a.x += lo.x; a.y += lo.y; a.z += hi.x; a.w += hi.y;
}
__device__ __forceinline__ void put_entry(float2* t2, int entries, int e, float x, float y, float z, float w) {
  t2[e] = make_float2(x, y);
  t2[entries + e] = make_float2(z, w);
}

// Asynchronous copy of a contiguous run of code rows into shared memory (the whole CTA takes part).
// Rows are 4-byte aligned; 16-byte pieces are used where the source allows.
__device__ __forceinline__ void stage_rows(unsigned char* dst, const unsigned char* src, int bytes) {
  const uint32_t d0 = (uint32_t)__cvta_generic_to_shared(dst);
  int done = 0;
  if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
    done = bytes & ~15;
    for (int i = threadIdx.x * 16; i < done; i += NT * 16)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d0 + i), "l"(src + i) : "memory");
  }
  for (int i = done + threadIdx.x * 4; i < bytes; i += NT * 4)
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(d0 + i), "l"(src + i) : "memory");
}

__host__ __device__ inline int vunits_of(int d, int bits) { return (bits == 1 || bits == 3) ? d / 8 : d / 4; }

// Value sums of one unit: BV-bit indices of CU consecutive coordinates sit in NB bytes of the row.
template <int BV>
__device__ __forceinline__ void vsum_unit(const unsigned char* vb, int rb, const float4* __restrict__ wg,
                                          const float* __restrict__ ct, int ph, int nrep, int ntok, float4* dst) {
  constexpr int CU = (BV == 1 || BV == 3) ? 8 : 4;
  constexpr int NB = BV == 3 ? 3 : (BV == 4 ? 2 : 1);
  float4 acc[CU];
#pragma unroll
  for (int u = 0; u < CU; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
  for (int tl = ph; tl < ntok; tl += nrep) {
    const unsigned char* p = vb + (size_t)tl * rb;
    uint32_t x = p[0];
    if (NB > 1) x |= (uint32_t)p[1] << 8;
    if (NB > 2) x |= (uint32_t)p[2] << 16;
    const float4 w = wg[tl];
#pragma unroll
    for (int u = 0; u < CU; ++u) {
      const float cv = ct[(x >> (BV * u)) & ((1u << BV) - 1u)];
      acc[u].x = fmaf(w.x, cv, acc[u].x); acc[u].y = fmaf(w.y, cv, acc[u].y);
      acc[u].z = fmaf(w.z, cv, acc[u].z); acc[u].w = fmaf(w.w, cv, acc[u].w);
    }
  }
#pragma unroll
  for (int u = 0; u < CU; ++u) dst[u] = acc[u];
}

__global__ void __launch_bounds__(NT) partial_kernel(Args a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float4* lut = reinterpret_cast<float4*>(smem_raw);                       // [lut_float4]
  float4* lg = lut + a.lut_float4;                                         // [SLICE] logits, then p
  // region0 (float4) >= tables + logits and >= the per-phase sums of phase C, which reuse that room
  float4* wvg = lut + a.region0;                                           // [ngroups][SLICE] p * nu^V of the group
  float* qs = reinterpret_cast<float*>(wvg);                               // rotated queries while the tables are built
  unsigned char* kbuf = reinterpret_cast<unsigned char*>(wvg + a.ngroups * SLICE);
  unsigned char* vbuf = kbuf + a.kbuf_bytes;
  float* vcent = reinterpret_cast<float*>(vbuf + a.vbuf_bytes);            // [MAXG][16]
  float* red = vcent + MAXG * 16;                                          // [NT/32][MAXQ] + [MAXQ]
  const int h = blockIdx.x / a.nslices, sl = blockIdx.x % a.nslices;
  const int64_t t0 = (int64_t)sl * SLICE;
  const int ntok = (int)min((int64_t)SLICE, a.tokens - t0);
  const int64_t row0 = (int64_t)h * a.head_stride + t0;
  const int d = a.d, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // ---- the slice's code rows travel to shared memory while the tables are built: every row is touched once,
  //      and a thread that waited for its own row would see one DRAM latency per token
  for (int gi = 0; gi < a.ngroups; ++gi) {
    const GroupDev& g = a.g[gi];
    if (g.k_bits > 0) stage_rows(kbuf + g.k_idx_soff, g.k_idx + (size_t)row0 * g.k_idx_rb, ntok * g.k_idx_rb);
    if (g.k_prod) stage_rows(kbuf + g.k_qjl_soff, g.k_qjl + (size_t)row0 * g.k_qjl_rb, ntok * g.k_qjl_rb);
    stage_rows(vbuf + g.v_idx_soff, g.v_idx + (size_t)row0 * g.v_idx_rb, ntok * g.v_idx_rb);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  {
    const float* q = a.qrot + (size_t)h * a.ngroups * MAXQ * 2 * MAXD;
    for (int e = tid; e < a.ngroups * MAXQ * 2 * MAXD; e += NT) qs[e] = q[e];
  }
  __syncthreads();

  // ---- tables: entry (lookup L, value v) = sum over the coordinates the L-th field covers
  for (int gi = 0; gi < a.ngroups; ++gi) {
    const GroupDev& g = a.g[gi];
    const float* q = qs + (size_t)gi * MAXQ * 2 * MAXD;
    const int nl = mse_lookups(d, g.k_bits), ne = mse_entries(g.k_bits);
    const int cpl = g.k_bits == 1 ? 4 : g.k_bits == 2 ? 2 : 1;   // coordinates per lookup
    for (int e = tid; e < nl * ne; e += NT) {
      const int L = e / ne, v = e % ne;
      float s[MAXQ] = {0.f, 0.f, 0.f, 0.f};
      for (int u = 0; u < cpl; ++u) {
        const int c = L * cpl + u;
        const float cent = g.k_cent[(v >> (u * g.k_bits)) & ((1 << g.k_bits) - 1)];
#pragma unroll
        for (int j = 0; j < MAXQ; ++j) s[j] = fmaf(q[j * 2 * MAXD + c], cent, s[j]);
      }
      put_entry(reinterpret_cast<float2*>(lut + g.lut_mse_off), nl * ne, e, s[0], s[1], s[2], s[3]);
    }
    if (g.k_prod) {
      for (int e = tid; e < (d / 4) * 16; e += NT) {
        const int L = e >> 4, v = e & 15;
        float s[MAXQ] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float sg = ((v >> u) & 1) ? 1.f : -1.f;
#pragma unroll
          for (int j = 0; j < MAXQ; ++j) s[j] = fmaf(sg, q[j * 2 * MAXD + MAXD + 4 * L + u], s[j]);
        }
        put_entry(reinterpret_cast<float2*>(lut + g.lut_qjl_off), (d / 4) * 16, e, s[0], s[1], s[2], s[3]);
      }
    }
    if (tid < 16) vcent[gi * 16 + tid] = g.v_cent[tid];
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- A: logits of this slice's tokens (thread = token)
  float mx[MAXQ] = {-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX};
  for (int tl = tid; tl < ntok; tl += NT) {
    const int64_t row = row0 + tl;
    float4 score = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int gi = 0; gi < a.ngroups; ++gi) {
      const GroupDev& g = a.g[gi];
      const float nu = g.k_norms ? __ldg(g.k_norms + row) : 1.f;
      const float cg = g.k_prod ? g.coef * __ldg(g.k_gamma + row) : 0.f;
      float4 am = make_float4(0.f, 0.f, 0.f, 0.f), aq = make_float4(0.f, 0.f, 0.f, 0.f);
      if (g.k_bits == 3) {          // 8 coordinates per 3 bytes
        const uint8_t* p = kbuf + g.k_idx_soff + (size_t)tl * g.k_idx_rb;
        const float2* tb = reinterpret_cast<const float2*>(lut + g.lut_mse_off);
        const int ent = d * 8;
        for (int c8 = 0; c8 < d / 8; ++c8) {
          const uint32_t x = (uint32_t)p[3 * c8] | ((uint32_t)p[3 * c8 + 1] << 8) | ((uint32_t)p[3 * c8 + 2] << 16);
#pragma unroll
          for (int u = 0; u < 8; ++u) add_entry(am, tb, ent, (c8 * 8 + u) * 8 + (int)((x >> (3 * u)) & 7u));
        }
      } else if (g.k_bits > 0) {    // nibbles never straddle a word
        const uint32_t* p = reinterpret_cast<const uint32_t*>(kbuf + g.k_idx_soff + (size_t)tl * g.k_idx_rb);
        const float2* tb = reinterpret_cast<const float2*>(lut + g.lut_mse_off);
        const int nw = d * g.k_bits / 32, ent = nw * 8 * 16;
        auto word = [&](int w, uint32_t x) {
#pragma unroll
          for (int u = 0; u < 8; ++u) add_entry(am, tb, ent, (w * 8 + u) * 16 + (int)((x >> (4 * u)) & 15u));
        };
        int w = 0;
        if ((g.k_idx_rb & 7) == 0)   // 8-byte loads where the rows allow (4-byte loads at a 16-byte row stride collide 4-way)
          for (; w + 1 < nw; w += 2) {
            const uint2 xx = *reinterpret_cast<const uint2*>(p + w);
            word(w, xx.x);
            word(w + 1, xx.y);
          }
        for (; w < nw; ++w) word(w, p[w]);
      }
      if (g.k_prod) {
        const uint32_t* p = reinterpret_cast<const uint32_t*>(kbuf + g.k_qjl_soff + (size_t)tl * g.k_qjl_rb);
        const float2* tb = reinterpret_cast<const float2*>(lut + g.lut_qjl_off);
        const int ent = (d / 4) * 16;
        auto word = [&](int w, uint32_t x) {
#pragma unroll
          for (int u = 0; u < 8; ++u) add_entry(aq, tb, ent, (w * 8 + u) * 16 + (int)((x >> (4 * u)) & 15u));
        };
        int w = 0;
        if ((g.k_qjl_rb & 7) == 0)
          for (; w + 1 < d / 32; w += 2) {
            const uint2 xx = *reinterpret_cast<const uint2*>(p + w);
            word(w, xx.x);
            word(w + 1, xx.y);
          }
        for (; w < d / 32; ++w) word(w, p[w]);
      }
      score.x += nu * fmaf(cg, aq.x, am.x);
      score.y += nu * fmaf(cg, aq.y, am.y);
      score.z += nu * fmaf(cg, aq.z, am.z);
      score.w += nu * fmaf(cg, aq.w, am.w);
    }
    const float4 l4 = make_float4(a.scale * score.x, a.scale * score.y, a.scale * score.z, a.scale * score.w);
    lg[tl] = l4;
    mx[0] = fmaxf(mx[0], l4.x); mx[1] = fmaxf(mx[1], l4.y); mx[2] = fmaxf(mx[2], l4.z); mx[3] = fmaxf(mx[3], l4.w);
  }

  // ---- B: slice maximum, exponentials, their sum (fixed reduction order)
#pragma unroll
  for (int j = 0; j < MAXQ; ++j) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx[j] = fmaxf(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], o));
    if (lane == 0) red[warp * MAXQ + j] = mx[j];
  }
  __syncthreads();
  if (tid < MAXQ) {
    float m = red[tid];
    for (int w = 1; w < NT / 32; ++w) m = fmaxf(m, red[w * MAXQ + tid]);
    red[(NT / 32) * MAXQ + tid] = m;
  }
  __syncthreads();
  float smax[MAXQ], sum[MAXQ] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int j = 0; j < MAXQ; ++j) smax[j] = red[(NT / 32) * MAXQ + j];
  __syncthreads();
  for (int tl = tid; tl < ntok; tl += NT) {
    const float4 l4 = lg[tl];
    const float4 p = make_float4(expf(l4.x - smax[0]), expf(l4.y - smax[1]), expf(l4.z - smax[2]), expf(l4.w - smax[3]));
    sum[0] += p.x; sum[1] += p.y; sum[2] += p.z; sum[3] += p.w;
    for (int gi = 0; gi < a.ngroups; ++gi) {
      const float nv = a.g[gi].v_norms ? __ldg(a.g[gi].v_norms + row0 + tl) : 1.f;
      wvg[gi * SLICE + tl] = make_float4(p.x * nv, p.y * nv, p.z * nv, p.w * nv);
    }
  }
#pragma unroll
  for (int j = 0; j < MAXQ; ++j) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum[j] += __shfl_xor_sync(0xffffffffu, sum[j], o);
    if (lane == 0) red[warp * MAXQ + j] = sum[j];
  }
  __syncthreads();
  float* ml = a.part_ml + (size_t)(h * a.nslices + sl) * 2 * MAXQ;
  if (tid < MAXQ) {
    float s = 0.f;
    for (int w = 0; w < NT / 32; ++w) s += red[w * MAXQ + tid];
    ml[tid] = smax[tid];
    ml[MAXQ + tid] = s;
  }

  // ---- C: acc[oc] = sum_t p_t nu^V_t c_V[idx^V_{t,c}].  A thread owns the 4 or 8 coordinates that share 1-3 bytes
  //      of the value row (so that one load and one weight fetch serve all of them) and one of nrep token phases;
  //      the phases are added in a fixed order afterwards.  The tables and logits are dead by now: their room
  //      holds the per-phase sums.
  const int ncoord = a.ngroups * d;
  const int nrep = max(1, NT / a.vunits);
  float4* rbuf = lut;   // [nrep][ncoord]
  if (tid < nrep * a.vunits) {
    int gi = 0;
    while (gi + 1 < a.ngroups && tid >= nrep * a.g[gi + 1].vunit0) ++gi;
    const GroupDev& g = a.g[gi];
    const int local = tid - nrep * g.vunit0, nu_g = vunits_of(d, g.v_bits);
    const int ph = local / nu_g, u = local % nu_g;
    const float* ct = vcent + gi * 16;
    const float4* wg = wvg + gi * SLICE;
    const unsigned char* vb = vbuf + g.v_idx_soff;
    float4* dst = rbuf + (size_t)ph * ncoord + gi * d;
    switch (g.v_bits) {
      case 1: vsum_unit<1>(vb + u, g.v_idx_rb, wg, ct, ph, nrep, ntok, dst + u * 8); break;
      case 2: vsum_unit<2>(vb + u, g.v_idx_rb, wg, ct, ph, nrep, ntok, dst + u * 4); break;
      case 3: vsum_unit<3>(vb + 3 * u, g.v_idx_rb, wg, ct, ph, nrep, ntok, dst + u * 8); break;
      default: vsum_unit<4>(vb + 2 * u, g.v_idx_rb, wg, ct, ph, nrep, ntok, dst + u * 4); break;
    }
  }
  __syncthreads();
  float4* out = reinterpret_cast<float4*>(a.part_acc) + (size_t)(h * a.nslices + sl) * ncoord;
  for (int oc = tid; oc < ncoord; oc += NT) {
    float4 sacc = rbuf[oc];
    for (int r = 1; r < nrep; ++r) add4(sacc, rbuf[(size_t)r * ncoord + oc]);
    out[oc] = sacc;
  }
}

#include "tq_decode_mma.cuh"

// ------------------------------------------------------------------ merge of the slices + inverse rotation
// One CTA per (head, group), all queries of the head at once: slice weights exp(m_s - M) / L, the weighted sum of the
// slices' partial value sums (float4 = the four queries of a coordinate), then x~ = Pi_V^T y' scattered to the group's
// channels.  Every sum runs in a fixed order.  The kernel is a chain of memory latencies, so Pi_V (an input of the
// call) is fetched into shared memory before the wait for the kernel ahead, and the threads are many enough that
// every load of a step is in flight at once.
constexpr int MERGE_NT = 512;
constexpr int MERGE_PF = 2;    // partial sums a merge thread requests ahead (more would take the registers that let the CTA start beside the partial kernel)
__global__ void __launch_bounds__(MERGE_NT, 2) merge_kernel(Args a, float* __restrict__ out, int64_t ldo) {
  extern __shared__ __align__(16) float pis[];   // [d][d] Pi_V
  __shared__ float4 wsl[MERGE_NT];
  __shared__ float4 yp[MERGE_NT];
  __shared__ float ys[MAXQ][MAXD];
  __shared__ float redm[MERGE_NT / 32][MAXQ];
  __shared__ double redl[MERGE_NT / 32][MAXQ];
  __shared__ float stat[2][MAXQ];
  __shared__ int chan[MAXD];
  const int h = blockIdx.x / a.ngroups, gi = blockIdx.x % a.ngroups;
  const int ncoord = a.ngroups * a.d, d = a.d, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const GroupDev& g = a.g[gi];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  {
    const float4* src = reinterpret_cast<const float4*>(g.v_pi);
    float4* dst = reinterpret_cast<float4*>(pis);
    for (int i = tid; i < d * d / 4; i += MERGE_NT) dst[i] = __ldg(src + i);
    if (tid < d) chan[tid] = g.v_channels[h * d + tid];
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the slices' partial results come from the kernel before
  const float4* ml4 = reinterpret_cast<const float4*>(a.part_ml + (size_t)h * a.nslices * 2 * MAXQ);   // [slice][max, sum]
  // Everything this thread needs from the partial kernel for the first MERGE_NT slices is requested at once -- its
  // slice's maximum and sum, and the first MERGE_PF partial sums of its coordinate -- so that the reductions below
  // run while the loads are in flight, instead of one round trip to L2 per phase.  Sums and their order are unchanged.
  const int nph = MERGE_NT / d, c = tid % d, ph = tid / d;   // thread = (coordinate c of the group, slice phase ph)
  const float4* acc4 = reinterpret_cast<const float4*>(a.part_acc) + (size_t)h * a.nslices * ncoord + gi * d + c;
  const int ns_first = min(MERGE_NT, a.nslices);
  float4 m_own = make_float4(-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX), l_own = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid < ns_first) {
    m_own = ml4[2 * tid];
    l_own = ml4[2 * tid + 1];
  }
  float4 vpre[MERGE_PF];
#pragma unroll
  for (int i = 0; i < MERGE_PF; ++i) {
    const int s = ph + i * nph;
    vpre[i] = (ph < nph && s < ns_first) ? acc4[(size_t)s * ncoord] : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  {   // global maximum and sum per query
    float M[MAXQ] = {-FLT_MAX, -FLT_MAX, -FLT_MAX, -FLT_MAX};
    for (int s = tid; s < a.nslices; s += MERGE_NT) {
      const float4 m = (s == tid) ? m_own : ml4[2 * s];
      M[0] = fmaxf(M[0], m.x); M[1] = fmaxf(M[1], m.y); M[2] = fmaxf(M[2], m.z); M[3] = fmaxf(M[3], m.w);
    }
#pragma unroll
    for (int j = 0; j < MAXQ; ++j) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) M[j] = fmaxf(M[j], __shfl_xor_sync(0xffffffffu, M[j], o));
      if (lane == 0) redm[warp][j] = M[j];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < MAXQ; ++j) {
      M[j] = redm[0][j];
      for (int w = 1; w < MERGE_NT / 32; ++w) M[j] = fmaxf(M[j], redm[w][j]);
    }
    double L[MAXQ] = {0.0, 0.0, 0.0, 0.0};
    for (int s = tid; s < a.nslices; s += MERGE_NT) {
      const float4 m = (s == tid) ? m_own : ml4[2 * s], l = (s == tid) ? l_own : ml4[2 * s + 1];
      L[0] += (double)l.x * (double)expf(m.x - M[0]); L[1] += (double)l.y * (double)expf(m.y - M[1]);
      L[2] += (double)l.z * (double)expf(m.z - M[2]); L[3] += (double)l.w * (double)expf(m.w - M[3]);
    }
#pragma unroll
    for (int j = 0; j < MAXQ; ++j) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) L[j] += __shfl_xor_sync(0xffffffffu, L[j], o);
      if (lane == 0) redl[warp][j] = L[j];
    }
    __syncthreads();
    if (tid < MAXQ) {
      double Ls = 0.0;
      for (int w = 0; w < MERGE_NT / 32; ++w) Ls += redl[w][tid];
      stat[0][tid] = M[tid];
      stat[1][tid] = (float)(1.0 / Ls);
    }
    __syncthreads();
  }
  const float4 Mv = make_float4(stat[0][0], stat[0][1], stat[0][2], stat[0][3]);
  const float4 inv = make_float4(stat[1][0], stat[1][1], stat[1][2], stat[1][3]);
  float4 y = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s0 = 0; s0 < a.nslices; s0 += MERGE_NT) {
    const int ns = min(MERGE_NT, a.nslices - s0);
    __syncthreads();
    if (tid < ns) {
      const float4 m = (s0 == 0) ? m_own : ml4[2 * (s0 + tid)];
      wsl[tid] = make_float4(expf(m.x - Mv.x) * inv.x, expf(m.y - Mv.y) * inv.y, expf(m.z - Mv.z) * inv.z, expf(m.w - Mv.w) * inv.w);
    }
    __syncthreads();
    if (ph < nph) {
      int s = ph;
      if (s0 == 0) {   // the partial sums already in registers
#pragma unroll
        for (int i = 0; i < MERGE_PF; ++i, s += nph) {
          if (s < ns) {
            const float4 v = vpre[i], w = wsl[s];
            y.x = fmaf(w.x, v.x, y.x); y.y = fmaf(w.y, v.y, y.y); y.z = fmaf(w.z, v.z, y.z); y.w = fmaf(w.w, v.w, y.w);
          }
        }
      }
#pragma unroll 8
      for (; s < ns; s += nph) {
        const float4 v = acc4[(size_t)(s0 + s) * ncoord], w = wsl[s];
        y.x = fmaf(w.x, v.x, y.x); y.y = fmaf(w.y, v.y, y.y); y.z = fmaf(w.z, v.z, y.z); y.w = fmaf(w.w, v.w, y.w);
      }
    }
  }
  yp[tid] = y;
  __syncthreads();
  if (tid < d) {
    float4 sum = yp[tid];
    for (int p = 1; p < nph; ++p) add4(sum, yp[p * d + tid]);
    ys[0][tid] = sum.x; ys[1][tid] = sum.y; ys[2][tid] = sum.z; ys[3][tid] = sum.w;
  }
  __syncthreads();
  // x~_k = sum_c Pi[c][k] y'_c, scattered to the group's channels of this head
  for (int it = tid; it < d * a.qpk; it += MERGE_NT) {
    const int k = it % d, j = it / d;
    float v = 0.f;
#pragma unroll 8
    for (int cc = 0; cc < d; ++cc) v = fmaf(pis[cc * d + k], ys[j][cc], v);
    if (TQ_DEVICE_CHECK(chan[k] >= 0 && chan[k] < a.ldo_dbg, a.status)) out[(int64_t)(h * a.qpk + j) * ldo + chan[k]] = v;
  }
}


// ------------------------------------------------------------------ append of one token per head
struct AppendGroup {
  uint8_t* k_idx; uint8_t* k_qjl; float* k_gamma; float* k_norms;
  uint8_t* v_idx; float* v_norms;
  const int32_t* k_channels; const int32_t* v_channels;
  const float* k_backt; const float* k_sp; const float* v_backt;   // [d, ncat*dpad] (column j = row j of Pi), S' [d, d]
  Codebook k_cb, v_cb;
  int k_prod, k_idx_rb, k_qjl_rb, v_idx_rb, k_ncols, v_ncols;
};
struct AppendArgs {
  AppendGroup g[MAXG];
  int ngroups, heads, d;
  int64_t head_stride, position;
};

// Quant_mse / Quant_prod (Algorithms 1, 2) of one d-vector by one CTA, thread j = rotated coordinate j, with the
// comparisons the batch quantiser makes: y = Pi x, idx_j = #{i : y_j > t_i nu}, e = y / nu - c[idx],
// z = sign(S' e), gamma = ||e||.
template <typename T>
__global__ void __launch_bounds__(MAXD) append_kernel(AppendArgs a, const T* __restrict__ K, int64_t ldk,
                                                      const T* __restrict__ V, int64_t ldv) {
  __shared__ float xs[MAXD], es[MAXD], red[4];
  __shared__ uint32_t words[MAXD * 4 / 32 + 1];
  const int h = blockIdx.x / a.ngroups, gi = blockIdx.x % a.ngroups, isv = blockIdx.y;
  const AppendGroup& g = a.g[gi];
  const int d = a.d, j = threadIdx.x, lane = j & 31, warp = j >> 5;
  const int64_t row = (int64_t)h * a.head_stride + a.position;
  const Codebook& cb = isv ? g.v_cb : g.k_cb;
  const bool prod = !isv && g.k_prod;
  const int bm = cb.bits;
  auto block_sum = [&](float v) -> float {   // fixed order: lanes by shuffles, then the warps in turn
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float s = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w];
    return s;
  };
  float x = 0.f;
  if (j < d) {
    const int ch = (isv ? g.v_channels : g.k_channels)[h * d + j];
    x = isv ? (float)V[(int64_t)h * ldv + ch] : (float)K[(int64_t)h * ldk + ch];
  }
  xs[j] = x;
  if (j < (int)(sizeof(words) / sizeof(words[0]))) words[j] = 0u;
  float nu = sqrtf(block_sum(x * x));   // the sync inside also publishes xs and words
  // no norms array: the row is taken as already unit-norm and quantised as it is, like tq_quantize_*
  if ((isv ? g.v_norms : g.k_norms) == nullptr) nu = 1.f;
  const float inv = nu > 0.f ? 1.f / nu : 0.f, vcmp = nu > 0.f ? nu : 1.f;
  const float* bt = isv ? g.v_backt : g.k_backt;
  const int ncols = isv ? g.v_ncols : g.k_ncols;
  float y = 0.f;
  if (j < d)
    for (int c = 0; c < d; ++c) y = fmaf(bt[(size_t)c * ncols + j], xs[c], y);
  int code = 0;
  for (int t = 0; t < (1 << bm) - 1; ++t) code += (y > cb.t[t] * vcmp) ? 1 : 0;
  if (j < d && bm > 0) {
    const int bit = j * bm;
    atomicOr(&words[bit >> 5], (uint32_t)code << (bit & 31));
    if ((bit & 31) + bm > 32) atomicOr(&words[(bit >> 5) + 1], (uint32_t)code >> (32 - (bit & 31)));
  }
  const float e = (j < d && nu > 0.f) ? y * inv - cb.c[code] : 0.f;
  es[j] = e;
  float gamma = 0.f;
  if (prod) gamma = sqrtf(block_sum(e * e)); else __syncthreads();
  uint8_t* idx_row = (isv ? g.v_idx + (size_t)row * g.v_idx_rb : g.k_idx + (size_t)row * g.k_idx_rb);
  const int idx_rb = isv ? g.v_idx_rb : g.k_idx_rb;
  if (bm > 0 && j < idx_rb / 4) reinterpret_cast<uint32_t*>(idx_row)[j] = (j < (d * bm + 31) / 32) ? words[j] : 0u;
  float* norms = isv ? g.v_norms : g.k_norms;
  if (j == 0 && norms) norms[row] = nu;
  if (prod) {
    if (j == 0) g.k_gamma[row] = gamma;
    float sp = 0.f;
    if (j < d) {
      const float* srow = g.k_sp + (size_t)j * d;
      for (int c = 0; c < d; ++c) sp = fmaf(srow[c], es[c], sp);
    }
    const uint32_t bits = __ballot_sync(0xffffffffu, j < d && sp >= 0.f);
    uint32_t* qrow = reinterpret_cast<uint32_t*>(g.k_qjl + (size_t)row * g.k_qjl_rb);
    if (lane == 0 && warp < g.k_qjl_rb / 4) qrow[warp] = bits;
  }
}

// B fragments of the tensor path: at most 8 plane words and one sign word per 32 coordinates and group
size_t bfrag_bytes(int ngroups, int heads, int d) { return (size_t)heads * ngroups * (d / 32) * 9 * 32 * sizeof(uint4); }

size_t workspace_bytes(int ngroups, int heads, int64_t tokens, int d) {
  const int64_t nslices = std::max<int64_t>(1, (tokens + SLICE - 1) / SLICE);
  size_t b = (size_t)heads * ngroups * MAXQ * 2 * MAXD * sizeof(float);
  b += (size_t)heads * nslices * 2 * MAXQ * sizeof(float);
  b = (b + 255) / 256 * 256;
  b += (size_t)heads * nslices * ngroups * d * MAXQ * sizeof(float);
  b = (b + 255) / 256 * 256;
  b += bfrag_bytes(ngroups, heads, d);
  b += (size_t)heads * ngroups * MAXQ * 2 * sizeof(KConst);
  return (b + 255) / 256 * 256;
}


// Launch with the programmatic-stream-serialisation attribute.
template <typename... KArgs, typename... LArgs>
cudaError_t launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, LArgs... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, args...);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Walsh coefficients of an antisymmetric codebook of 2^bits entries (see tq_decode_mma.cuh); false if it is not one.
bool walsh_coefficients(const float* c, int bits, float* alpha) {
  for (int i = 0; i < 8; ++i) alpha[i] = 0.f;
  if (bits == 0) return true;
  const int n = 1 << bits;
  for (int i = 0; i < n / 2; ++i)
    if (c[i] != -c[n - 1 - i]) return false;
  auto coef = [&](unsigned subset) {
    double s = 0.0;
    for (int idx = 0; idx < n; ++idx) {
      int sign = 1;
      for (int i = 0; i < bits; ++i)
        if (((subset >> i) & 1u) && !((idx >> i) & 1)) sign = -sign;
      s += sign * (double)c[idx];
    }
    return (float)(s / n);
  };
  for (int o = 0; o < bits; ++o) alpha[o] = coef(1u << o);
  if (bits == 3) alpha[3] = coef(7u);
  if (bits == 4)
    for (int o = 0; o < 4; ++o) alpha[4 + o] = coef(15u & ~(1u << o));
  return true;
}

// Layout of the tensor path for this call; false if it cannot run (codebook shape, shared memory).
bool plan_mma(int ngroups, int d, const Args& a, char* workspace, size_t off, int heads, MmaArgs* out, size_t* smem_out) {
  MmaArgs& ma = *out;
  std::memset(&ma, 0, sizeof(ma));
  int kw = 0, vw = 0, r0 = 0;
  auto take = [&](int bytes) {
    const int at = r0;
    r0 += (bytes + 15) / 16 * 16;
    return at;
  };
  for (int gi = 0; gi < ngroups; ++gi) {
    const GroupDev& g = a.g[gi];
    MmaGroup& m = ma.m[gi];
    if (!walsh_coefficients(g.k_cent, g.k_bits, m.k_alpha) || !walsh_coefficients(g.v_cent, g.v_bits, m.v_alpha)) return false;
    m.k_w0 = kw;
    m.k_mse_nw = plane_words(d, g.k_bits);
    m.k_raw_nw = raw_words(d, g.k_bits);
    m.k_qjl_nw = g.k_prod ? d / 32 : 0;
    if (g.k_bits > 0 && g.k_idx_rb < 4 * m.k_raw_nw) return false;
    if (g.k_prod && g.k_qjl_rb < 4 * m.k_qjl_nw) return false;
    m.k_idx_rb = g.k_bits > 0 ? g.k_idx_rb : 0;
    m.k_qjl_rb = g.k_prod ? g.k_qjl_rb : 0;
    m.k_der_rb = 4 * (m.k_mse_nw - m.k_raw_nw);
    m.k_idx_off = take(SLICE * m.k_idx_rb);
    m.k_qjl_off = take(SLICE * m.k_qjl_rb);
    m.k_der_off = take(SLICE * m.k_der_rb);
    kw += m.k_mse_nw + m.k_qjl_nw;
    m.v_w0 = vw;
    m.v_nw = plane_words(d, g.v_bits);
    m.v_raw_nw = raw_words(d, g.v_bits);
    if (g.v_idx_rb < 4 * m.v_raw_nw) return false;
    m.v_rb = g.v_idx_rb;
    m.v_raw_off = take(SLICE * m.v_rb);
    m.v_pos0 = 32 * vw;
    vw += m.v_nw;
  }
  if (kw == 0) return false;
  ma.kw = kw;
  ma.vw = vw;
  ma.qstride16 = vw | 1;
  ma.vpos = 32 * vw;
  ma.dstride = (ma.vpos + 8 * ngroups + 31) / 32 * 32 + 8;
  ma.bs_off = take(16 * kw * 32);
  ma.knu_off = take(2 * ngroups * SLICE * 4);
  const int vnu_off_rel = 16 * (SLICE / 4) * ma.qstride16 + ngroups * WT_ROWS * WT_STRIDE;   // behind region 0
  ma.region0 = std::max(r0, WT_ROWS * ma.dstride * 4);
  ma.region0 = (ma.region0 + 15) / 16 * 16;
  for (int gi = 0; gi < ngroups; ++gi) {   // the copies of the slice's rows and scalars
    const GroupDev& g = a.g[gi];
    const MmaGroup& m = ma.m[gi];
    auto add = [&](const void* src, int rb, int dst_off) {
      CopyJob& j = ma.job[ma.njobs++];
      j.src = static_cast<const unsigned char*>(src);
      j.row_bytes = rb;
      j.dst_off = dst_off;
    };
    add(g.v_idx, g.v_idx_rb, m.v_raw_off);
    if (g.k_bits > 0) add(g.k_idx, g.k_idx_rb, m.k_idx_off);
    if (g.k_prod) {
      add(g.k_qjl, g.k_qjl_rb, m.k_qjl_off);
      add(g.k_gamma, 4, ma.knu_off + (ngroups + gi) * SLICE * 4);
    }
    if (g.k_norms) add(g.k_norms, 4, ma.knu_off + gi * SLICE * 4);
    if (g.v_norms) add(g.v_norms, 4, ma.region0 + vnu_off_rel + gi * SLICE * 4);
  }
  const size_t smem = (size_t)ma.region0 + (size_t)16 * (SLICE / 4) * ma.qstride16 + (size_t)ngroups * WT_ROWS * WT_STRIDE +
                      (size_t)ngroups * SLICE * 4 + (size_t)ngroups * MAXQ * 2 * sizeof(KConst) + 2 * (NT / 32) * MAXQ * 4 + MAXG * 4;
  if (smem > 200 * 1024) return false;
  if ((size_t)kw * 32 * sizeof(uint4) * heads > bfrag_bytes(ngroups, heads, d)) return false;
  ma.bfrag = reinterpret_cast<uint4*>(workspace + off);
  ma.kconst = reinterpret_cast<KConst*>(workspace + off + bfrag_bytes(ngroups, heads, d));
  *smem_out = smem;
  return true;
}
}  // namespace kvdec
}  // namespace tq

namespace tq {
namespace kvdec {
struct ZeroArgs {
  const int32_t* v_channels[MAXG];
  int ngroups, d, q_per_kv;
};
// Row r = h * q_per_kv + j of `out`: zeros in the columns that receive the groups' coordinates for KV head h.
__global__ void zero_channels_kernel(ZeroArgs z, float* __restrict__ out, int64_t ldo) {
  const int r = blockIdx.x, h = r / z.q_per_kv;
  for (int gi = 0; gi < z.ngroups; ++gi)
    for (int c = threadIdx.x; c < z.d; c += blockDim.x) out[(int64_t)r * ldo + z.v_channels[gi][h * z.d + c]] = 0.f;
}
}  // namespace kvdec
}  // namespace tq

extern "C" size_t tq_attend_decode_workspace_bytes(int ngroups, int heads, int64_t tokens, int d) {
  if (ngroups <= 0 || heads <= 0 || tokens < 0 || d <= 0) return 0;
  return tq::kvdec::workspace_bytes(ngroups, heads, tokens, d);
}

extern "C" int tq_attend_decode(const tq_kv_group* groups, int ngroups, int heads, int64_t tokens, int64_t head_stride, int q_per_kv,
                                const void* Q, int q_dtype, int64_t ldq, float scale, float* out, int64_t ldo,
                                void* workspace, size_t workspace_bytes, void* stream) {
  using namespace tq;
  using namespace tq::kvdec;
  const char* who = "tq_attend_decode";
  TQ_RANGE(who);
  TQ_REQUIRE(groups != nullptr && ngroups >= 1 && ngroups <= MAXG, TQ_ERR_INVALID_ARG, "%s: 1..%d channel groups", who, MAXG);
  TQ_REQUIRE(heads >= 0 && tokens >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  TQ_REQUIRE(head_stride >= tokens, TQ_ERR_INVALID_ARG, "%s: head_stride %lld is smaller than tokens %lld", who,
             (long long)head_stride, (long long)tokens);
  TQ_REQUIRE(q_per_kv >= 1 && q_per_kv <= MAXQ, TQ_ERR_UNSUPPORTED, "%s: 1..%d queries per KV head", who, MAXQ);
  TQ_REQUIRE(q_dtype == TQ_F32 || q_dtype == TQ_BF16, TQ_ERR_UNSUPPORTED, "%s: unknown query dtype %d", who, q_dtype);
  if (heads == 0) return TQ_OK;
  TQ_REQUIRE(out != nullptr && Q != nullptr, TQ_ERR_INVALID_ARG, "%s: Q or out is NULL", who);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  Args a;
  std::memset(&a, 0, sizeof(a));
  const int d = groups[0].plan_k ? groups[0].plan_k->d : 0;
  TQ_REQUIRE(d >= 32 && d <= MAXD && d % 32 == 0, TQ_ERR_UNSUPPORTED, "%s: group dimension %d (multiples of 32 up to %d)", who, d, MAXD);
  TQ_REQUIRE(ldq >= 1 && ldo >= 1, TQ_ERR_INVALID_ARG, "%s: bad row stride", who);
  int lut = 0, kbytes = 0, vbytes = 0, vunits = 0;
  for (int gi = 0; gi < ngroups; ++gi) {
    const tq_kv_group& s = groups[gi];
    TQ_REQUIRE(s.plan_k && s.plan_v, TQ_ERR_INVALID_ARG, "%s: group %d has no plan", who, gi);
    TQ_REQUIRE(s.plan_k->d == d && s.plan_v->d == d, TQ_ERR_UNSUPPORTED, "%s: all groups must share one dimension", who);
    TQ_REQUIRE(s.plan_k->layout == TQ_LAYOUT_CANONICAL && s.plan_v->layout == TQ_LAYOUT_CANONICAL, TQ_ERR_UNSUPPORTED,
               "%s: group %d: plans must use the canonical code layout", who, gi);
    TQ_REQUIRE(s.plan_v->mode == TQ_MSE && s.plan_v->mse_bits >= 1, TQ_ERR_UNSUPPORTED,
               "%s: values must be quantised with TurboQuant_mse", who);
    TQ_REQUIRE(s.plan_k->device == s.plan_v->device, TQ_ERR_INVALID_ARG, "%s: plans of different devices", who);
    const bool prod = s.plan_k->mode == TQ_PROD;
    TQ_REQUIRE(s.k_channels && s.v_channels && s.v_idx, TQ_ERR_INVALID_ARG, "%s: group %d: NULL channel list or codes", who, gi);
    TQ_REQUIRE(s.plan_k->mse_bits == 0 || s.k_idx, TQ_ERR_INVALID_ARG, "%s: group %d: k_idx is NULL", who, gi);
    TQ_REQUIRE(!prod || (s.k_qjl && s.k_gamma), TQ_ERR_INVALID_ARG, "%s: group %d: k_qjl / k_gamma is NULL", who, gi);
    TQ_REQUIRE(((reinterpret_cast<uintptr_t>(s.k_idx) | reinterpret_cast<uintptr_t>(s.k_qjl) | reinterpret_cast<uintptr_t>(s.v_idx)) & 3) == 0,
               TQ_ERR_ALIGNMENT, "%s: group %d: codes are not 4-byte aligned", who, gi);
    GroupDev& g = a.g[gi];
    g.k_idx = s.k_idx; g.k_qjl = s.k_qjl; g.k_gamma = s.k_gamma; g.k_norms = s.k_norms;
    g.v_idx = s.v_idx; g.v_norms = s.v_norms;
    g.k_channels = s.k_channels; g.v_channels = s.v_channels;
    g.k_backt = s.plan_k->dBackT; g.v_pi = s.plan_v->dPi;
    for (int i = 0; i < 16; ++i) { g.k_cent[i] = s.plan_k->cb.c[i]; g.v_cent[i] = s.plan_v->cb.c[i]; }
    g.k_bits = s.plan_k->mse_bits; g.v_bits = s.plan_v->mse_bits; g.k_prod = prod ? 1 : 0;
    g.k_idx_rb = (int)s.plan_k->idx_row_bytes; g.k_qjl_rb = (int)s.plan_k->qjl_row_bytes; g.v_idx_rb = (int)s.plan_v->idx_row_bytes;
    g.k_dpad = s.plan_k->dpad;
    g.coef = s.plan_k->coef;
    g.lut_mse_off = lut;
    lut += mse_lookups(d, g.k_bits) * mse_entries(g.k_bits);
    g.lut_qjl_off = lut;
    if (prod) lut += (d / 4) * 16;
    g.k_idx_soff = kbytes;
    kbytes += (g.k_bits > 0 ? SLICE * g.k_idx_rb + 15 : 0) / 16 * 16;
    g.k_qjl_soff = kbytes;
    kbytes += (prod ? SLICE * g.k_qjl_rb + 15 : 0) / 16 * 16;
    g.vunit0 = vunits;
    vunits += vunits_of(d, g.v_bits);
    g.v_idx_soff = vbytes;
    vbytes += (SLICE * g.v_idx_rb + 15) / 16 * 16;
  }
  if (tokens == 0) {   // no tokens: the columns named by v_channels are zero
    ZeroArgs z;
    for (int gi = 0; gi < ngroups; ++gi) z.v_channels[gi] = groups[gi].v_channels;
    z.ngroups = ngroups; z.d = d; z.q_per_kv = q_per_kv;
    zero_channels_kernel<<<heads * q_per_kv, 128, 0, st>>>(z, out, ldo);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
    count_launches(1);
    return TQ_OK;
  }
  const int64_t nslices = (tokens + SLICE - 1) / SLICE;
  TQ_REQUIRE((int64_t)heads * nslices < (1 << 30), TQ_ERR_UNSUPPORTED, "%s: too many (head, slice) pairs", who);
  const size_t need = kvdec::workspace_bytes(ngroups, heads, tokens, d);
  TQ_REQUIRE(workspace != nullptr && workspace_bytes >= need, TQ_ERR_WORKSPACE, "%s: workspace of %zu bytes, %zu needed", who,
             workspace_bytes, need);
  TQ_REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 255) == 0, TQ_ERR_ALIGNMENT, "%s: workspace is not 256-byte aligned", who);
  a.ngroups = ngroups; a.heads = heads; a.qpk = q_per_kv; a.d = d; a.nslices = (int)nslices;
  a.tokens = tokens; a.head_stride = head_stride; a.scale = scale; a.lut_float4 = lut;
  a.kbuf_bytes = kbytes; a.vbuf_bytes = vbytes;
  a.status = groups[0].plan_k->d_status; a.ldq_dbg = ldq; a.ldo_dbg = ldo;
  a.vunits = vunits;
  a.region0 = std::max(lut + SLICE, std::max(1, NT / vunits) * ngroups * d);
  char* w = static_cast<char*>(workspace);
  a.qrot = reinterpret_cast<float*>(w);
  size_t off = (size_t)heads * ngroups * MAXQ * 2 * MAXD * sizeof(float);
  a.part_ml = reinterpret_cast<float*>(w + off);
  off += (size_t)heads * nslices * 2 * MAXQ * sizeof(float);
  off = (off + 255) / 256 * 256;
  a.part_acc = reinterpret_cast<float*>(w + off);
  off += (size_t)heads * nslices * ngroups * d * MAXQ * sizeof(float);
  off = (off + 255) / 256 * 256;

  int dev = 0;
  TQ_CHECK_CUDA(cudaGetDevice(&dev), who);
  TQ_REQUIRE(dev == groups[0].plan_k->device, TQ_ERR_INVALID_ARG, "%s: the plans belong to device %d, current device is %d", who,
             groups[0].plan_k->device, dev);
  const size_t merge_smem = (size_t)d * d * sizeof(float);
  static std::atomic<size_t> merge_smem_set[16];
  if (dev >= 16 || merge_smem > merge_smem_set[dev].load(std::memory_order_relaxed)) {
    TQ_CHECK_CUDA(cudaFuncSetAttribute(merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)merge_smem), who);
    if (dev < 16) merge_smem_set[dev].store(merge_smem, std::memory_order_relaxed);
  }
  // ---- the tensor path: antisymmetric codebooks (every Lloyd-Max codebook of the library is) and a slice that fits
  //      in shared memory; otherwise the table-lookup kernel
  MmaArgs ma;
  size_t mma_smem = 0;
  if (plan_mma(ngroups, d, a, static_cast<char*>(workspace), off, heads, &ma, &mma_smem)) {
    // all three launches may be scheduled while their predecessor in the stream drains; each orders itself with
    // griddepcontrol.wait before it reads or writes global memory that another kernel touches
    if (q_dtype == TQ_F32)
      TQ_CHECK_CUDA(launch_after(prepare_mma_kernel<float>, dim3((unsigned)(heads * ngroups)), dim3(256), 0, st, a, ma,
                                 static_cast<const float*>(Q), ldq), who);
    else
      TQ_CHECK_CUDA(launch_after(prepare_mma_kernel<__nv_bfloat16>, dim3((unsigned)(heads * ngroups)), dim3(256), 0, st, a, ma,
                                 static_cast<const __nv_bfloat16*>(Q), ldq), who);
    static std::atomic<size_t> mma_smem_set[16];
    if (dev >= 16 || mma_smem > mma_smem_set[dev].load(std::memory_order_relaxed)) {
      TQ_CHECK_CUDA(cudaFuncSetAttribute(partial_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mma_smem), who);
      // several CTAs per SM hide the latencies of the kernel's short phases: ask for the largest shared-memory carve-out
      TQ_CHECK_CUDA(cudaFuncSetAttribute(partial_mma_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared), who);
      if (dev < 16) mma_smem_set[dev].store(mma_smem, std::memory_order_relaxed);
    }
    TQ_CHECK_CUDA(launch_after(partial_mma_kernel, dim3((unsigned)(heads * nslices)), dim3(NT), mma_smem, st, a, ma), who);
    TQ_CHECK_CUDA(launch_after(merge_kernel, dim3((unsigned)(heads * ngroups)), dim3(MERGE_NT), merge_smem, st, a, out, ldo), who);
    count_launches(3);
    return TQ_OK;
  }
  if (q_dtype == TQ_F32)
    prepare_kernel<float><<<heads * ngroups, 128, 0, st>>>(a, static_cast<const float*>(Q), ldq);
  else
    prepare_kernel<__nv_bfloat16><<<heads * ngroups, 128, 0, st>>>(a, static_cast<const __nv_bfloat16*>(Q), ldq);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  const size_t smem = (size_t)a.region0 * sizeof(float4) + (size_t)ngroups * SLICE * sizeof(float4) + kbytes + vbytes +
                      MAXG * 16 * sizeof(float) + (NT / 32 + 1) * MAXQ * sizeof(float);
  TQ_REQUIRE(smem <= 220 * 1024, TQ_ERR_UNSUPPORTED, "%s: %zu bytes of shared memory needed (too many wide groups)", who, smem);
  static std::atomic<size_t> smem_set[16];   // zero-initialised; written by any thread that launches
  if (dev >= 16 || smem > smem_set[dev].load(std::memory_order_relaxed)) {
    TQ_CHECK_CUDA(cudaFuncSetAttribute(partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem), who);
    if (dev < 16) smem_set[dev].store(smem, std::memory_order_relaxed);
  }
  partial_kernel<<<(unsigned)(heads * nslices), NT, smem, st>>>(a);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  merge_kernel<<<heads * ngroups, MERGE_NT, merge_smem, st>>>(a, out, ldo);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  count_launches(3);
  return TQ_OK;
}

extern "C" int tq_kv_append(const tq_kv_group* groups, int ngroups, int heads, int64_t head_stride, int64_t position,
                            const void* K, const void* V, int kv_dtype, int64_t ldk, int64_t ldv, void* stream) {
  using namespace tq;
  using namespace tq::kvdec;
  const char* who = "tq_kv_append";
  TQ_RANGE(who);
  TQ_REQUIRE(groups != nullptr && ngroups >= 1 && ngroups <= MAXG, TQ_ERR_INVALID_ARG, "%s: 1..%d channel groups", who, MAXG);
  TQ_REQUIRE(heads >= 0, TQ_ERR_INVALID_ARG, "%s: negative size", who);
  TQ_REQUIRE(position >= 0 && position < head_stride, TQ_ERR_INVALID_ARG, "%s: position %lld outside [0, head_stride %lld)", who,
             (long long)position, (long long)head_stride);
  TQ_REQUIRE(kv_dtype == TQ_F32 || kv_dtype == TQ_BF16, TQ_ERR_UNSUPPORTED, "%s: unknown dtype %d", who, kv_dtype);
  if (heads == 0) return TQ_OK;
  TQ_REQUIRE(K != nullptr && V != nullptr, TQ_ERR_INVALID_ARG, "%s: K or V is NULL", who);
  AppendArgs a;
  std::memset(&a, 0, sizeof(a));
  const int d = groups[0].plan_k ? groups[0].plan_k->d : 0;
  TQ_REQUIRE(d >= 32 && d <= MAXD && d % 32 == 0, TQ_ERR_UNSUPPORTED, "%s: group dimension %d (multiples of 32 up to %d)", who, d, MAXD);
  for (int gi = 0; gi < ngroups; ++gi) {
    const tq_kv_group& s = groups[gi];
    TQ_REQUIRE(s.plan_k && s.plan_v, TQ_ERR_INVALID_ARG, "%s: group %d has no plan", who, gi);
    TQ_REQUIRE(s.plan_k->d == d && s.plan_v->d == d, TQ_ERR_UNSUPPORTED, "%s: all groups must share one dimension", who);
    TQ_REQUIRE(s.plan_k->layout == TQ_LAYOUT_CANONICAL && s.plan_v->layout == TQ_LAYOUT_CANONICAL, TQ_ERR_UNSUPPORTED,
               "%s: group %d: plans must use the canonical code layout", who, gi);
    TQ_REQUIRE(s.plan_v->mode == TQ_MSE && s.plan_v->mse_bits >= 1, TQ_ERR_UNSUPPORTED,
               "%s: values must be quantised with TurboQuant_mse", who);
    const bool prod = s.plan_k->mode == TQ_PROD;
    TQ_REQUIRE(s.k_channels && s.v_channels && s.v_idx, TQ_ERR_INVALID_ARG, "%s: group %d: NULL channel list or codes", who, gi);
    TQ_REQUIRE(s.plan_k->mse_bits == 0 || s.k_idx, TQ_ERR_INVALID_ARG, "%s: group %d: k_idx is NULL", who, gi);
    TQ_REQUIRE(!prod || (s.k_qjl && s.k_gamma), TQ_ERR_INVALID_ARG, "%s: group %d: k_qjl / k_gamma is NULL", who, gi);
    TQ_REQUIRE(((reinterpret_cast<uintptr_t>(s.k_idx) | reinterpret_cast<uintptr_t>(s.k_qjl) | reinterpret_cast<uintptr_t>(s.v_idx)) & 3) == 0,
               TQ_ERR_ALIGNMENT, "%s: group %d: codes are not 4-byte aligned", who, gi);
    AppendGroup& g = a.g[gi];
    g.k_idx = s.k_idx; g.k_qjl = s.k_qjl; g.k_gamma = s.k_gamma; g.k_norms = s.k_norms;
    g.v_idx = s.v_idx; g.v_norms = s.v_norms;
    g.k_channels = s.k_channels; g.v_channels = s.v_channels;
    g.k_backt = s.plan_k->dBackT; g.k_sp = s.plan_k->dSp; g.v_backt = s.plan_v->dBackT;
    g.k_cb = s.plan_k->cb; g.v_cb = s.plan_v->cb;
    g.k_prod = prod ? 1 : 0;
    g.k_idx_rb = (int)s.plan_k->idx_row_bytes; g.k_qjl_rb = (int)s.plan_k->qjl_row_bytes; g.v_idx_rb = (int)s.plan_v->idx_row_bytes;
    g.k_ncols = s.plan_k->ncat * s.plan_k->dpad; g.v_ncols = s.plan_v->ncat * s.plan_v->dpad;
  }
  a.ngroups = ngroups; a.heads = heads; a.d = d; a.head_stride = head_stride; a.position = position;
  int dev = -1;
  TQ_CHECK_CUDA(cudaGetDevice(&dev), who);
  for (int gi = 0; gi < ngroups; ++gi)
    TQ_REQUIRE(groups[gi].plan_k->device == dev && groups[gi].plan_v->device == dev, TQ_ERR_INVALID_ARG,
               "%s: group %d: the plans belong to another device than the current one (%d)", who, gi, dev);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid((unsigned)(heads * ngroups), 2);
  if (kv_dtype == TQ_F32)
    append_kernel<float><<<grid, MAXD, 0, st>>>(a, static_cast<const float*>(K), ldk, static_cast<const float*>(V), ldv);
  else
    append_kernel<__nv_bfloat16><<<grid, MAXD, 0, st>>>(a, static_cast<const __nv_bfloat16*>(K), ldk,
                                                         static_cast<const __nv_bfloat16*>(V), ldv);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  count_launches(1);
  return TQ_OK;
}

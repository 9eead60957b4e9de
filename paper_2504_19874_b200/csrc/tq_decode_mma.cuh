// Decode attention over a compressed KV cache on the integer tensor path (mma.sync.m16n8k32, u8 x s8 / u8 x u8 -> s32).
// Included by tq_decode_attn.cu inside namespace tq::kvdec, after Args and GroupDev.
//
// Bit-plane form.  A Lloyd-Max codebook of the even coordinate density (Section 3.1) is antisymmetric, i.e. an odd
// function of the index bits: c[idx] = sum_T alpha_T s_T over the subsets T of odd size, s_T = prod_{i in T} (2 bit_i - 1)
// = 2 parity_T - 1.  A code row therefore becomes a row of "plane bits" (the index bits themselves, plus for 3-bit
// indices the parity of the three bits, for 4-bit indices the four 3-subset parities) and
//     sum_c q_c c[idx_c]          = sum_pos alpha(pos) q_{c(pos)} (2 bit(pos) - 1)      (Section 3.2 estimator, MSE term)
//     sum_t w_t c[idx_{t,c}]      = sum_{pos in c} alpha(pos) sum_t w_t (2 bit_t(pos) - 1)   (value sums, Section 4.3)
// are 0/1 matrices times fixed-point integer matrices.  `word & (0x01010101 << k)` turns plane bits k, k + 8, k + 16,
// k + 24 of a word into the four bytes (0 or 2^k) of an operand register; the factor 2^k is divided out of the other
// operand (scores) or of the result (value sums, exactly).  int32 accumulation is exact, so neither term depends on the
// order of the tokens or on which warp took which tile.
//
//   prepare_mma_kernel   per (head, group): q' = Pi q, q'' = S q of the head's queries, then the B operand of the scores
//                        (four balanced radix-256 digits of round(2 alpha q 2^f / 2^k) per plane bit and query) and the
//                        per-query constants.
//   partial_mma_kernel   per (head, slice of 256 tokens):
//                        0) code rows -> shared memory (cp.async): key planes as [token][word], value planes as
//                           [4 tokens][word][token of the four], then transposed in place to [4 tokens][word][byte]
//                           so that a register holds one byte of four consecutive tokens; derived planes, scalars
//                        A) scores: A = plane bits of 16 tokens, B = query digits (columns = 4 queries x 4 digits)
//                        B) slice maximum, p = exp(logit - max), sum of p; w = p nu^V as three u8 digits per (group,
//                           query, token)
//                        C) value sums: A = weight digits (rows = 4 queries x 4 digit slots, K = tokens), B = value
//                           plane bits (columns = plane bits) and one column of ones (sum_t w); per digit 2 X - sum_t w
//                           is a small exact integer; the plane bits of a coordinate are added in a fixed order
//   merge_kernel         combines the slices.

struct MmaGroup {
  int k_w0;                                 // first B-fragment word (k-step) of the group: MSE planes, then sign words
  int k_mse_nw, k_raw_nw, k_qjl_nw;         // words of the MSE planes (the first k_raw_nw are the index bits themselves), sign words
  int k_idx_off, k_qjl_off, k_der_off;      // byte offsets in region 0: staged index rows, sign rows, derived plane words
  int k_idx_rb, k_qjl_rb, k_der_rb;         // bytes per staged row / per token of derived words
  int v_w0, v_nw, v_raw_nw;                 // words of the value planes in a token quad's row of the transposed planes
  int v_raw_off, v_rb;                      // staged value rows
  int v_pos0;                               // first plane-bit position of the group among all V positions
  float k_alpha[8], v_alpha[8];             // Walsh coefficients: single bits o = 0..3, then (b = 3) the parity of all
                                            // three bits at [3], (b = 4) the parity of the bits other than o at [4 + o]
};

struct KConst {
  int wd[4];        // per balanced digit: sum over the plane bits of 2^k digit(pos), k = pos % 8
  float scale;      // 2^-(f + 1)
  float pad[3];
};

struct CopyJob {
  const unsigned char* src;   // first row of head 0
  int row_bytes;              // bytes per token in global memory
  int dst_off;                // byte offset in shared memory
};

struct MmaArgs {
  MmaGroup m[MAXG];
  CopyJob job[6 * MAXG];  // the slice's code rows and per-token scalars: one contiguous run of global memory each
  int njobs;
  int kw;                 // B-fragment words of all groups
  int vw;                 // words per token of the value planes
  int qstride16;          // 16-byte units between consecutive token quads of the value planes (odd, >= vw)
  int vpos;               // plane-bit positions of all groups' values = 32 * vw
  int dstride;            // ints between digit rows of the value sums (>= vpos + 8 * ngroups, = 8 mod 32)
  int bs_off, knu_off;    // byte offsets in region 0 of the B fragments and of the key scalars (nu, then gamma)
  int region0;            // bytes of the region that holds what the scores need, later the value sums
  uint4* bfrag;           // [heads][kw][32]  B fragments of the scores
  KConst* kconst;         // [heads][ngroups][MAXQ][2]  constants of the MSE and sign terms
};

constexpr int WT_STRIDE = SLICE + 16;   // bytes between digit rows of the weights (bank-conflict-free fragment loads)
constexpr int WT_ROWS = 12;             // rows 3 j + dg: three digits of four queries
constexpr int MAXPW = 9 * (MAXD / 32);  // plane words of one group's keys: at most 8 per 32 coordinates + the sign word

// shared-memory accesses by 32-bit address (the hot loops keep their address arithmetic in 32 bits)
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts64(uint32_t a, int x, int y) {
  asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(a), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t prmt_b(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
// 2^e as a float, e in [-126, 127]
__device__ __forceinline__ float pow2f(int e) { return __int_as_float((e + 127) << 23); }

// Words of the plane row of a d-coordinate code row with `bits` index bits per coordinate.
__host__ __device__ inline int plane_words(int d, int bits) {
  return bits == 0 ? 0 : bits <= 2 ? d * bits / 32 : bits == 3 ? d * 4 / 32 : d * 8 / 32;
}
__host__ __device__ inline int raw_words(int d, int bits) { return d * bits / 32; }

// Plane-bit position -> coordinate and Walsh coefficient.
__device__ __forceinline__ void plane_pos(int d, int bits, int pos, const float* __restrict__ alpha, int& c, float& a) {
  if (bits == 1) {
    c = pos; a = alpha[0];
  } else if (bits == 2) {
    c = pos >> 1; a = alpha[pos & 1];
  } else if (bits == 3) {
    if (pos < 3 * d) {
      c = pos / 3; a = alpha[pos % 3];
    } else {   // parity word j, bit p: taken from word 3 j + p % 3 of the stream, same bit
      const int q = pos - 3 * d, j = q >> 5, p = q & 31;
      c = (96 * j + 32 * (p % 3) + p) / 3; a = alpha[3];
    }
  } else {
    if (pos < 4 * d) {
      c = pos >> 2; a = alpha[pos & 3];
    } else {
      const int q = pos - 4 * d;
      c = q >> 2; a = alpha[4 + (q & 3)];
    }
  }
}

// Derived plane words of one code row: from its raw index words to `der` (3-bit indices: one parity word per three
// raw words; 4-bit indices: one word of 3-subset parities per raw word).
__device__ __forceinline__ void derive_planes(const uint32_t* raw, uint32_t* der, int d, int bits) {
  if (bits == 3) {
    const int nw = 3 * d / 32;
    for (int j = 0; j < nw / 3; ++j) {
      uint32_t z = 0u;
#pragma unroll
      for (int r = 0; r < 3; ++r) {
        const int i = 3 * j + r;
        const uint32_t x = raw[i], nx = i + 1 < nw ? raw[i + 1] : 0u;
        const uint32_t y = x ^ __funnelshift_r(x, nx, 1) ^ __funnelshift_r(x, nx, 2);
        z |= y & (0x49249249u << r);   // bits p with p % 3 == r
      }
      der[j] = z;
    }
  } else if (bits == 4) {
    const int nw = d / 8;
    for (int i = 0; i < nw; ++i) {
      const uint32_t x = raw[i];
      const uint32_t t = (x ^ (x >> 1) ^ (x >> 2) ^ (x >> 3)) & 0x11111111u;   // parity of each nibble
      der[i] = x ^ (t * 15u);                                                  // bit o: parity of the other three bits
    }
  }
}

// ------------------------------------------------------------------ query preparation for the tensor path
template <typename T>
__global__ void __launch_bounds__(256) prepare_mma_kernel(Args a, MmaArgs ma, const T* __restrict__ Q, int64_t ldq) {
  __shared__ float qs[MAXQ][MAXD];
  __shared__ float qr[MAXQ][2 * MAXD];           // q' then q''
  __shared__ int wmax[2][MAXQ];                  // bit patterns of the largest |weight| per term and query
  __shared__ int wdsum[2][MAXQ][4];
  __shared__ uint32_t wdig[MAXPW * 32][MAXQ];    // the four digit bytes of every (plane bit, query)
  const int h = blockIdx.x / a.ngroups, gi = blockIdx.x % a.ngroups;
  const GroupDev& g = a.g[gi];
  const MmaGroup& m = ma.m[gi];
  const int d = a.d, tid = threadIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the slices' code rows may start to travel
  // this kernel may itself have been scheduled while the kernel ahead in the stream drains (it may produce Q)
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (int e = tid; e < MAXQ * d; e += blockDim.x) {
    const int j = e / d, c = e % d;
    float v = 0.f;
    if (j < a.qpk) {
      const int ch = g.k_channels[h * d + c];
      if (TQ_DEVICE_CHECK(ch >= 0 && ch < a.ldq_dbg, a.status)) v = (float)Q[(int64_t)(h * a.qpk + j) * ldq + ch];
    }
    qs[j][c] = v;
  }
  if (tid < 2 * MAXQ) wmax[tid / MAXQ][tid % MAXQ] = 0;
  if (tid < 2 * MAXQ * 4) (&wdsum[0][0][0])[tid] = 0;
  __syncthreads();
  const int nrows = (g.k_prod ? 2 : 1) * g.k_dpad;
  for (int o = tid; o < 2 * MAXD; o += blockDim.x) {
    const int half = o / MAXD, r = o % MAXD;
    float acc[MAXQ] = {0.f, 0.f, 0.f, 0.f};
    if (r < d && (half == 0 || g.k_prod)) {
      const float* col = g.k_backt + half * g.k_dpad + r;
#pragma unroll 32
      for (int c = 0; c < d; ++c) {   // independent loads: unrolled deep, the kernel is latency-bound
        const float mm = __ldg(col + (size_t)c * nrows);
#pragma unroll
        for (int j = 0; j < MAXQ; ++j) acc[j] = fmaf(mm, qs[j][c], acc[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < MAXQ; ++j) qr[j][o] = acc[j];
  }
  __syncthreads();

  // weight of plane bit `pos` (group-local: MSE planes, then sign bits) for query j: 2 alpha q'_c, 2 q''_i
  const int npos_mse = 32 * m.k_mse_nw, npos = npos_mse + 32 * m.k_qjl_nw;
  auto weight = [&](int pos, int j) -> float {
    if (pos < npos_mse) {
      int c; float al;
      plane_pos(d, g.k_bits, pos, m.k_alpha, c, al);
      return 2.f * al * qr[j][c];
    }
    return 2.f * qr[j][MAXD + pos - npos_mse];
  };
  // (item = tid + 256 i: a thread keeps its query j = tid % 4; lanes of equal j are combined before the atomics)
  const int j = tid & 3;
  {
    float mx[2] = {0.f, 0.f};
    for (int pos = tid >> 2; pos < npos; pos += blockDim.x / 4) {
      const float w = fabsf(weight(pos, j));
      if (pos < npos_mse) mx[0] = fmaxf(mx[0], w); else mx[1] = fmaxf(mx[1], w);
    }
#pragma unroll
    for (int term = 0; term < 2; ++term) {
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) mx[term] = fmaxf(mx[term], __shfl_xor_sync(0xffffffffu, mx[term], o));
      if ((tid & 31) < 4) atomicMax(&wmax[term][j], __float_as_int(mx[term]));
    }
  }
  __syncthreads();
  // exponent f with |w| 2^f < 2^30 (clamped: weights below 2^-90 of the scale do not matter)
  auto fexp = [&](int term, int jj) -> int {
    const int bits = wmax[term][jj];
    if (bits == 0) return 0;
    const int e = ((bits >> 23) & 255) - 126;   // |w| < 2^e
    return max(-90, min(110, 30 - e));
  };
  {
    const int fe[2] = {fexp(0, j), fexp(1, j)};
    int sums[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
    for (int pos = tid >> 2; pos < npos; pos += blockDim.x / 4) {
      const int term = pos < npos_mse ? 0 : 1, k = pos & 7;
      int W = __float2int_rn(weight(pos, j) * pow2f(fe[term] - k));
      uint32_t packed = 0u;
#pragma unroll
      for (int dg = 0; dg < 4; ++dg) {   // balanced radix-256 digits, the top one takes what is left
        const int lo = dg == 3 ? W : ((W + 128) & 255) - 128;
        W = (W - lo) >> 8;
        packed |= (uint32_t)(lo & 255) << (8 * dg);
        if (term == 0) sums[0][dg] += lo * (1 << k); else sums[1][dg] += lo * (1 << k);
      }
      wdig[pos][j] = packed;
    }
#pragma unroll
    for (int term = 0; term < 2; ++term)
#pragma unroll
      for (int dg = 0; dg < 4; ++dg) {
        int v = sums[term][dg];
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if ((tid & 31) < 4) atomicAdd(&wdsum[term][j][dg], v);
      }
  }
  __syncthreads();
  // B fragments: word w, lane (n, kq): registers (tile 0, K half 0), (tile 0, half 1), (tile 1, half 0), (tile 1, half 1);
  // byte i of K half r: plane bit 32 w + 8 i + kq + 4 r; column n of tile tt: query n / 2, digit 2 tt + (n & 1)
  uint4* bf = ma.bfrag + ((size_t)h * ma.kw + m.k_w0) * 32;
  for (int it = tid; it < (npos >> 5) * 32; it += blockDim.x) {
    const int w = it >> 5, lane = it & 31, n = lane >> 2, kq = lane & 3, jq = n >> 1;
    uint32_t reg[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int r = 0; r < 2; ++r)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t pk = wdig[32 * w + 8 * i + kq + 4 * r][jq] >> (8 * (n & 1));
        reg[r] |= (pk & 255u) << (8 * i);
        reg[2 + r] |= ((pk >> 16) & 255u) << (8 * i);
      }
    bf[(size_t)w * 32 + lane] = make_uint4(reg[0], reg[1], reg[2], reg[3]);
  }
  if (tid < 2 * MAXQ) {
    const int term = tid / MAXQ, jc = tid % MAXQ;
    KConst c;
#pragma unroll
    for (int dg = 0; dg < 4; ++dg) c.wd[dg] = wdsum[term][jc][dg];
    c.scale = pow2f(-(fexp(term, jc) + 1));
    c.pad[0] = c.pad[1] = c.pad[2] = 0.f;
    ma.kconst[((size_t)(h * a.ngroups + gi) * MAXQ + jc) * 2 + term] = c;
  }
}

// ------------------------------------------------------------------ per-slice scores, weights, value sums
template <int BYTES>
__device__ __forceinline__ void cp_async_piece(uint32_t dst, const void* src) {
  if (BYTES == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// Scores of two 16-token tiles against `nw` plane words: rows r0 (tile 0, token g8), r0 + skip8 (token g8 + 8),
// r1, r1 + skip8 (tile 1); bfr = this lane's B fragment of the first word, 512 bytes per word.
__device__ __forceinline__ void score_words(int (&acc)[2][2][4], uint32_t r0, uint32_t r1, uint32_t skip8, int nw, uint32_t bfr,
                                            uint32_t m0, uint32_t m1) {
#pragma unroll 2
  for (int w = 0; w < nw; ++w) {
    const uint32_t x0 = lds32(r0 + 4 * w), x1 = lds32(r0 + skip8 + 4 * w);
    const uint32_t y0 = lds32(r1 + 4 * w), y1 = lds32(r1 + skip8 + 4 * w);
    const uint4 b = lds128(bfr + 512 * w);
    mma_u8s8(acc[0][0], x0 & m0, x1 & m0, x0 & m1, x1 & m1, b.x, b.y);
    mma_u8s8(acc[0][1], x0 & m0, x1 & m0, x0 & m1, x1 & m1, b.z, b.w);
    mma_u8s8(acc[1][0], y0 & m0, y1 & m0, y0 & m1, y1 & m1, b.x, b.y);
    mma_u8s8(acc[1][1], y0 & m0, y1 & m0, y0 & m1, y1 & m1, b.z, b.w);
  }
}

// Value sums of N units (half plane words) of one group over all k-steps of the slice; digit rows to shared memory.
// wa_lo / wa_hi: this lane's weight rows g8 and g8 + 8 (K offset 4 kq applied); b0[u]: this lane's first token quad of
// unit u; dd[u]: where the unit's first tile goes in digit row g8 (columns 2 kq, 2 kq + 1).
template <int N>
__device__ __forceinline__ void vsum_chunk(uint32_t wa_lo, uint32_t wa_hi, const uint32_t (&b0)[3], const uint32_t (&dd)[3],
                                           uint32_t qrow4, uint32_t mn, bool hi_rows, uint32_t hi_skip, bool with_ones, uint32_t dd_ones) {
  constexpr int NKS = SLICE / 32;
  int acc[N > 0 ? N : 1][2][4], acc1[4] = {0, 0, 0, 0};
#pragma unroll
  for (int u = 0; u < N; ++u)
#pragma unroll
    for (int tt = 0; tt < 2; ++tt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[u][tt][e] = 0;
#pragma unroll
  for (int ks = 0; ks < NKS; ++ks) {
    const uint32_t a0 = lds32(wa_lo + 32 * ks), a1 = lds32(wa_hi + 32 * ks);
    const uint32_t a2 = lds32(wa_lo + 32 * ks + 16), a3 = lds32(wa_hi + 32 * ks + 16);
    if (with_ones) mma_u8u8(acc1, a0, a1, a2, a3, 0x01010101u, 0x01010101u);
#pragma unroll
    for (int u = 0; u < N; ++u) {
      const uint2 x0 = lds64(b0[u] + 2 * ks * qrow4), x1 = lds64(b0[u] + (2 * ks + 1) * qrow4);
      mma_u8u8(acc[u][0], a0, a1, a2, a3, x0.x & mn, x1.x & mn);
      mma_u8u8(acc[u][1], a0, a1, a2, a3, x0.y & mn, x1.y & mn);
    }
  }
  if (with_ones) {
    sts64(dd_ones, acc1[0], acc1[1]);
    if (hi_rows) sts64(dd_ones + hi_skip, acc1[2], acc1[3]);
  }
#pragma unroll
  for (int u = 0; u < N; ++u)
#pragma unroll
    for (int tt = 0; tt < 2; ++tt) {
      sts64(dd[u] + 32 * tt, acc[u][tt][0], acc[u][tt][1]);
      if (hi_rows) sts64(dd[u] + 32 * tt + hi_skip, acc[u][tt][2], acc[u][tt][3]);
    }
}

__global__ void __launch_bounds__(NT, 4) partial_mma_kernel(Args a, MmaArgs ma) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int ng = a.ngroups, d = a.d;
  // region 0: what the scores need (staged code rows, B fragments, key scalars); later the digit rows of the value sums
  float* knu = reinterpret_cast<float*>(smem_raw + ma.knu_off);                  // [ng][SLICE]
  float* kgm = knu + ng * SLICE;                                                 // [ng][SLICE]
  uint32_t* vq = reinterpret_cast<uint32_t*>(smem_raw + ma.region0);             // [SLICE / 4][qstride16][4]
  unsigned char* wt = reinterpret_cast<unsigned char*>(vq + (SLICE / 4) * ma.qstride16 * 4);   // [ng][WT_ROWS][WT_STRIDE]
  float* vnu = reinterpret_cast<float*>(wt + ng * WT_ROWS * WT_STRIDE);          // [ng][SLICE]
  KConst* kc = reinterpret_cast<KConst*>(vnu + ng * SLICE);                      // [ng][MAXQ][2]
  float* red = reinterpret_cast<float*>(kc + ng * MAXQ * 2);                     // [2][NT / 32][MAXQ]
  int* vmax = reinterpret_cast<int*>(red + 2 * (NT / 32) * MAXQ);                // [MAXG] bit patterns of max nu^V
  const uint32_t s_base = (uint32_t)__cvta_generic_to_shared(smem_raw);

  const int h = blockIdx.x / a.nslices, sl = blockIdx.x % a.nslices;
  const int64_t t0 = (int64_t)sl * SLICE;
  const int ntok = (int)min((int64_t)SLICE, a.tokens - t0);
  const int64_t row0 = (int64_t)h * a.head_stride + t0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g8 = lane >> 2, kq = lane & 3;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- 0) the slice's code rows and scalars are contiguous in global memory: one flat copy each, dealt to the warps.
  //         They are inputs of the call; the wait for the kernel ahead (the query-side operand) comes only after the
  //         value planes are in place, so that the first wave of CTAs works while that kernel runs.
  for (int jb = warp; jb < ma.njobs; jb += NT / 32) {
    const CopyJob job = ma.job[jb];
    const unsigned char* src = job.src + (size_t)row0 * job.row_bytes;
    const uint32_t dst = s_base + job.dst_off;
    const int bytes = ntok * job.row_bytes;
    int done = 0;
    if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
      done = bytes & ~15;
      for (int i = lane * 16; i < done; i += 32 * 16) cp_async_piece<16>(dst + i, src + i);
    }
    for (int i = done + lane * 4; i < bytes; i += 32 * 4) cp_async_piece<4>(dst + i, src + i);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  if (tid < MAXG) vmax[tid] = 0;
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- thread = token: derived planes, defaults of absent scalars, largest value norm of the slice; the value
  //      planes go to [token quad][word][byte]: the four lanes of a quad hold word w of their tokens and exchange
  //      bytes, so that lane s ends with byte s of the four tokens
  {
    const uint32_t sel1 = (lane & 1) ? 0x3715u : 0x6240u, sel2 = (lane & 2) ? 0x3276u : 0x5410u;
    uint32_t* vslot = vq + (tid >> 2) * ma.qstride16 * 4 + (tid & 3);   // [quad][word 0][lane of the quad]; words are 4 apart
    auto transpose_store = [&](uint32_t* slot, uint32_t x) {
      const uint32_t u = prmt_b(x, __shfl_xor_sync(0xffffffffu, x, 1), sel1);
      *slot = prmt_b(u, __shfl_xor_sync(0xffffffffu, u, 2), sel2);
    };
    const bool live = tid < ntok;
    for (int gi = 0; gi < ng; ++gi) {
      const GroupDev& g = a.g[gi];
      const MmaGroup& m = ma.m[gi];
      float vm = 0.f;
      if (live) {
        if (g.k_bits >= 3)
          derive_planes(reinterpret_cast<const uint32_t*>(smem_raw + m.k_idx_off + tid * m.k_idx_rb),
                        reinterpret_cast<uint32_t*>(smem_raw + m.k_der_off + tid * m.k_der_rb), d, g.k_bits);
        if (!g.k_norms) knu[gi * SLICE + tid] = 1.f;
        if (!g.k_prod) kgm[gi * SLICE + tid] = 0.f;
        if (!g.v_norms) vnu[gi * SLICE + tid] = 1.f;
        vm = fmaxf(vnu[gi * SLICE + tid], 0.f);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, o));
      if (lane == 0) atomicMax(&vmax[gi], __float_as_int(vm));
      const uint32_t* rv = reinterpret_cast<const uint32_t*>(smem_raw + m.v_raw_off + tid * m.v_rb);
      uint32_t* v0 = vslot + 4 * m.v_w0;
      const int nw = m.v_raw_nw;
      if (g.v_bits <= 2) {
        for (int w = 0; w < nw; ++w) transpose_store(v0 + 4 * w, live ? rv[w] : 0u);
      } else if (g.v_bits == 3) {
        for (int j = 0; j < nw / 3; ++j) {
          uint32_t x[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) x[r] = (live && 3 * j + r < nw) ? rv[3 * j + r] : 0u;
          uint32_t z = 0u;
#pragma unroll
          for (int r = 0; r < 3; ++r) {
            const uint32_t y = x[r] ^ __funnelshift_r(x[r], x[r + 1], 1) ^ __funnelshift_r(x[r], x[r + 1], 2);
            z |= y & (0x49249249u << r);
            transpose_store(v0 + 4 * (3 * j + r), x[r]);
          }
          transpose_store(v0 + 4 * (nw + j), z);
        }
      } else {
        for (int w = 0; w < nw; ++w) {
          const uint32_t x = live ? rv[w] : 0u;
          const uint32_t t = (x ^ (x >> 1) ^ (x >> 2) ^ (x >> 3)) & 0x11111111u;
          transpose_store(v0 + 4 * w, x);
          transpose_store(v0 + 4 * (nw + w), x ^ (t * 15u));
        }
      }
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the query-side operand is the previous kernel's output
  {
    const uint4* src = ma.bfrag + (size_t)h * ma.kw * 32;
    uint4* bs = reinterpret_cast<uint4*>(smem_raw + ma.bs_off);
    for (int i = tid; i < ma.kw * 32; i += NT) bs[i] = __ldg(src + i);
    const uint4* cs = reinterpret_cast<const uint4*>(ma.kconst + (size_t)h * ng * MAXQ * 2);
    for (int i = tid; i < ng * MAXQ * 2 * 2; i += NT) reinterpret_cast<uint4*>(kc)[i] = __ldg(cs + i);
  }
  __syncthreads();

  // ---- A) scores.  Thread (g8, kq) of a warp: tokens g8 and g8 + 8 of the warp's two 16-token tiles, query kq.
  constexpr int MT = SLICE / 16 / (NT / 32);
  static_assert(MT == 2, "two tiles per warp");
  const uint32_t m0 = 0x01010101u << kq, m1 = m0 << 4;
  const int tok0 = 16 * warp + g8, tok1 = 16 * (warp + NT / 32) + g8;   // rows g8 of the two tiles
  float logit[MT][2];
  {
    float score[MT][2] = {{0.f, 0.f}, {0.f, 0.f}};
    for (int gi = 0; gi < ng; ++gi) {
      const MmaGroup& m = ma.m[gi];
      const uint32_t bfr = s_base + ma.bs_off + (m.k_w0 * 32 + lane) * 16;
      float term[2][MT][2];   // [mse, sign][tile][row]
#pragma unroll
      for (int tm = 0; tm < 2; ++tm) {
        int acc[MT][2][4];
#pragma unroll
        for (int i = 0; i < MT; ++i)
#pragma unroll
          for (int tt = 0; tt < 2; ++tt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][tt][e] = 0;
        if (tm == 0) {
          score_words(acc, s_base + m.k_idx_off + tok0 * m.k_idx_rb, s_base + m.k_idx_off + tok1 * m.k_idx_rb, 8 * m.k_idx_rb,
                      m.k_raw_nw, bfr, m0, m1);
          if (m.k_mse_nw > m.k_raw_nw)
            score_words(acc, s_base + m.k_der_off + tok0 * m.k_der_rb, s_base + m.k_der_off + tok1 * m.k_der_rb, 8 * m.k_der_rb,
                        m.k_mse_nw - m.k_raw_nw, bfr + 512 * m.k_raw_nw, m0, m1);
        } else {
          score_words(acc, s_base + m.k_qjl_off + tok0 * m.k_qjl_rb, s_base + m.k_qjl_off + tok1 * m.k_qjl_rb, 8 * m.k_qjl_rb,
                      m.k_qjl_nw, bfr + 512 * m.k_mse_nw, m0, m1);
        }
        // sum_pos W (2 bit - 1), digit by digit (each difference is a small exact integer), then Horner in fp32
        const KConst c = kc[(gi * MAXQ + kq) * 2 + tm];
#pragma unroll
        for (int i = 0; i < MT; ++i)
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const float d0 = (float)(2 * acc[i][0][2 * hh] - c.wd[0]), d1 = (float)(2 * acc[i][0][2 * hh + 1] - c.wd[1]);
            const float d2 = (float)(2 * acc[i][1][2 * hh] - c.wd[2]), d3 = (float)(2 * acc[i][1][2 * hh + 1] - c.wd[3]);
            term[tm][i][hh] = fmaf(256.f, fmaf(256.f, fmaf(256.f, d3, d2), d1), d0) * c.scale;
          }
      }
      const float coef = a.g[gi].coef;
#pragma unroll
      for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int t = (i == 0 ? tok0 : tok1) + 8 * hh;
          score[i][hh] += knu[gi * SLICE + t] * fmaf(coef * kgm[gi * SLICE + t], term[1][i][hh], term[0][i][hh]);
        }
    }
#pragma unroll
    for (int i = 0; i < MT; ++i) {
      logit[i][0] = a.scale * score[i][0];
      logit[i][1] = a.scale * score[i][1];
    }
  }

  // ---- B) slice maximum per query, exponentials, their sum (fixed order), weight digits (three per weight)
  {
    float mx = -FLT_MAX;
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
        if ((i == 0 ? tok0 : tok1) + 8 * hh < ntok) mx = fmaxf(mx, logit[i][hh]);
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (g8 == 0) red[warp * MAXQ + kq] = mx;
  }
  __syncthreads();
  float smax = red[kq];
#pragma unroll
  for (int w = 1; w < NT / 32; ++w) smax = fmaxf(smax, red[w * MAXQ + kq]);
  float sg[MAXG];   // nu^V < 2^e and p <= 1: w 2^(24 - e) < 2^24
#pragma unroll
  for (int gi = 0; gi < MAXG; ++gi) {
    const int bits = gi < ng ? vmax[gi] : 0;
    sg[gi] = bits > 0 ? pow2f(max(-126, min(127, 24 - (((bits >> 23) & 255) - 126)))) : 1.f;
  }
  {
    float psum = 0.f;
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int t = (i == 0 ? tok0 : tok1) + 8 * hh;
        const bool live = t < ntok && kq < a.qpk;
        const float p = live ? expf(logit[i][hh] - smax) : 0.f;
        psum += p;
#pragma unroll
        for (int gi = 0; gi < MAXG; ++gi)
          if (gi < ng) {
            const uint32_t W = live ? min(__float2uint_rn(p * vnu[gi * SLICE + t] * sg[gi]), 0xffffffu) : 0u;
            unsigned char* col = wt + (gi * WT_ROWS + 3 * kq) * WT_STRIDE + t;
            col[0] = (unsigned char)W;
            col[WT_STRIDE] = (unsigned char)(W >> 8);
            col[2 * WT_STRIDE] = (unsigned char)(W >> 16);
          }
      }
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
    if (g8 == 0) red[(NT / 32) * MAXQ + warp * MAXQ + kq] = psum;
  }
  __syncthreads();   // the weights are complete; region 0 is dead
  if (tid < MAXQ) {
    float* ml = a.part_ml + (size_t)(h * a.nslices + sl) * 2 * MAXQ;
    float s = 0.f, m = red[tid];
    for (int w = 0; w < NT / 32; ++w) {
      s += red[(NT / 32) * MAXQ + w * MAXQ + tid];
      m = fmaxf(m, red[w * MAXQ + tid]);
    }
    ml[tid] = m;
    ml[MAXQ + tid] = s;
  }

  // ---- C) value sums.  Rows of A: weight digit dg of query j at row 3 j + dg (rows 12..15 of the tile carry nothing);
  //         K = the slice's tokens (all eight k-steps: the weights of absent tokens are zero); columns of B: plane bits.
  //         A unit = half a plane word (two 8-column tiles); the units of a group are dealt to the warps; warp gi % 8
  //         also takes the group's column of ones (sum_t w).
  const uint32_t mn = 0x01010101u << g8;
  const uint32_t qrow = 16u * ma.qstride16;                          // bytes per token quad
  const uint32_t vq_s = (uint32_t)__cvta_generic_to_shared(vq) + kq * qrow;
  const uint32_t wt_s = (uint32_t)__cvta_generic_to_shared(wt) + 4 * kq;
  const int row_hi = min(g8 + 8, WT_ROWS - 1);                       // rows 12..15: any row, the results are not stored
  const uint32_t db_s = s_base + (g8 * ma.dstride + 2 * kq) * 4;     // digit row g8, columns 2 kq, 2 kq + 1
  for (int gi = 0; gi < ng; ++gi) {
    const MmaGroup& m = ma.m[gi];
    const int U = 2 * m.v_nw;
    const int ub = U * warp / (NT / 32), ue = U * (warp + 1) / (NT / 32);
    const uint32_t wa_lo = wt_s + (gi * WT_ROWS + g8) * WT_STRIDE, wa_hi = wt_s + (gi * WT_ROWS + row_hi) * WT_STRIDE;
    const bool ones = warp == (gi & (NT / 32 - 1));
    for (int u0 = ub; u0 < ue || (ones && u0 == ub); u0 += 3) {
      uint32_t b0[3], dd[3];
#pragma unroll
      for (int uu = 0; uu < 3; ++uu) {
        const int u = u0 + uu;
        b0[uu] = vq_s + (m.v_w0 + (u >> 1)) * 16 + (u & 1) * 8;
        dd[uu] = db_s + (m.v_pos0 + 16 * u) * 4;
      }
      const bool with_ones = ones && u0 == ub;
      const uint32_t dd_ones = db_s + (ma.vpos + 8 * gi) * 4;
      const int n = min(3, ue - u0);
      if (n == 3) vsum_chunk<3>(wa_lo, wa_hi, b0, dd, 4 * qrow, mn, g8 < 4, 32 * ma.dstride, with_ones, dd_ones);
      else if (n == 2) vsum_chunk<2>(wa_lo, wa_hi, b0, dd, 4 * qrow, mn, g8 < 4, 32 * ma.dstride, with_ones, dd_ones);
      else if (n == 1) vsum_chunk<1>(wa_lo, wa_hi, b0, dd, 4 * qrow, mn, g8 < 4, 32 * ma.dstride, with_ones, dd_ones);
      else vsum_chunk<0>(wa_lo, wa_hi, b0, dd, 4 * qrow, mn, g8 < 4, 32 * ma.dstride, with_ones, dd_ones);
    }
  }
  __syncthreads();

  // ---- item = (coordinate, query): per digit 2 X - sum_t w is a small exact integer (column pos carries the factor
  //      2^(pos % 8)); Horner over the digits in fp32; the coordinate's plane bits added in a fixed order
  const int* dbuf = reinterpret_cast<const int*>(smem_raw);   // [WT_ROWS][dstride]
  const int ncoord = ng * d;
  float* out = a.part_acc + (size_t)(h * a.nslices + sl) * ncoord * MAXQ;
  for (int gi = 0; gi < ng; ++gi) {
    const MmaGroup& m = ma.m[gi];
    const int bits = a.g[gi].v_bits, oc0 = ma.vpos + 8 * gi;
    const float rs = 1.f / sg[gi];
    for (int it = tid; it < d * MAXQ; it += NT) {
      const int c = it >> 2, j = it & 3;
      const int* dj = dbuf + 3 * j * ma.dstride;
      const int o0 = dj[oc0], o1 = dj[ma.dstride + oc0], o2 = dj[2 * ma.dstride + oc0];
      auto plane = [&](int pos, float alpha) -> float {
        const int col = m.v_pos0 + pos, sh = pos & 7;
        const float e0 = (float)(2 * (dj[col] >> sh) - o0), e1 = (float)(2 * (dj[ma.dstride + col] >> sh) - o1);
        const float e2 = (float)(2 * (dj[2 * ma.dstride + col] >> sh) - o2);
        return alpha * fmaf(256.f, fmaf(256.f, e2, e1), e0);
      };
      float s = 0.f;
      if (bits <= 2) {
        for (int o = 0; o < bits; ++o) s += plane(bits * c + o, m.v_alpha[o]);
      } else if (bits == 3) {
        for (int o = 0; o < 3; ++o) s += plane(3 * c + o, m.v_alpha[o]);
        const int sp = 3 * c;
        s += plane(3 * d + 32 * ((sp >> 5) / 3) + (sp & 31), m.v_alpha[3]);
      } else {
        for (int o = 0; o < 4; ++o) s += plane(4 * c + o, m.v_alpha[o]);
        for (int o = 0; o < 4; ++o) s += plane(4 * d + 4 * c + o, m.v_alpha[4 + o]);
      }
      if (TQ_DEVICE_CHECK(h < a.heads && sl < a.nslices && gi * d * MAXQ + it < ncoord * MAXQ, a.status)) out[gi * d * MAXQ + it] = s * rs;
    }
  }
}

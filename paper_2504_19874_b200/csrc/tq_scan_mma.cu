// Packed-code scan (estimator of Section 3.2 evaluated on the codes) with the multiply-accumulate
// on the integer tensor path and the decode reduced to bitwise masks.
//
// Why not table lookups: at d = 1536, b = 4 one pass over 10^6 codes is 0.78 GB (0.12 ms of HBM time)
// but 1.5e9 coordinates; unpack + centroid lookup + FMA on CUDA cores costs >= 6 issue slots per
// coordinate and query, an order of magnitude more than the SMs can issue in that time.
//
// What is done instead.  An antisymmetric codebook (c_{L-1-k} = -c_k, which Lloyd-Max on the even
// density of Lemma 1 always gives) is an odd function of the index bits, so it expands in the odd
// Walsh terms only:   c[idx] = sum_T alpha_T * s_T,   s_T = prod_{i in T} (2 bit_i - 1),  |T| odd.
// For b_m = 1, 2 these are the index bits themselves; b_m = 3 adds the parity of the three bits,
// b_m = 4 the parities of the four 3-subsets.  With s = 2 bit - 1 the estimator becomes
//   sum_j q'_j c[idx_j] = sum_{bits} (2 alpha_T q'_j) * bit  +  const(q),      (same for the QJL signs)
// i.e. a 0/1 matrix (the raw bits of the packed rows plus the few parity words) times a real matrix
// that depends on the query only.  Every 32-bit word w of a packed row yields eight A-operand
// registers of the 8-bit integer MMA by one AND each, (w & (0x01010101 << k)), whose bytes are 0 or
// 2^k; the factor 2^k and the fixed-point scale are folded into the B operand, which holds
// round(2 alpha_T q'_j 2^f / 2^k) as four signed radix-256 digits in four MMA columns.  The int32
// accumulators are exact, so scores do not depend on tiling or summation order.  Since any
// permutation of the K axis is allowed as long as B is permuted alike, bits are consumed in
// whatever order they sit in the registers; no coordinate is ever extracted.
//
// Kernel: persistent CTAs, one TMA producer warp + 12 or 16 consumer warps.  Packed rows travel
// HBM -> shared memory in [rows x 64-byte] boxes (ring of stages, mbarrier full/empty, bounded
// waits), each consumer thread pulls its 16-byte pieces into registers, frees the stage, derives the
// parity words, and issues mma.sync.m16n8k32 (u8 x s8 -> s32) against B fragments resident in
// shared memory.  The epilogue recombines the digit columns exactly (64-bit integer), applies gamma, nu and
// the per-query constants in fp32 and either stores dense scores or appends (score, id) pairs that pass a
// per-query threshold to a candidate list (top-k).
#include <atomic>
#include <algorithm>
#include <cmath>

#include "tq_quantize_tc.h"
#include "tq_scan_mma.h"
#include "tq_tc.cuh"

namespace tq {
namespace mscan {

namespace {

constexpr int LIMBS = 4;                    // signed radix-256 digits per B value
constexpr int MAX_STAGES = 6;
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr size_t kQConstBytes = 256;        // room for the per-query constants of one pass (4 x 48 bytes)

__host__ __device__ constexpr int idx_words(int bm) { return 4 * bm; }
__host__ __device__ constexpr int der_words(int bm) { return bm == 3 ? 4 : (bm == 4 ? 16 : 0); }
__host__ __device__ constexpr int a_words(int bm) { return idx_words(bm) + der_words(bm); }
__host__ __device__ constexpr int ks_a(int bm) { return a_words(bm) / 2 * 8; }
__host__ __device__ constexpr int ks_s(bool prod) { return prod ? 16 : 0; }

// Per-query constants (computed inside bprep_kernel).
struct QConst {
  float sa, ca;    // a = T_a * sa + ca   (MSE term)
  float ss, cs;    // s = T_s * ss + cs   (QJL term)
  int fa, fs;      // fixed-point exponents
  int pad[2];
};

// ------------------------------------------------------------------ K-axis slot -> (coordinate, term)
// One "range" covers 512 coordinates; quad thread t4 owns 128 of them: b_m 16-byte pieces of the idx
// row and one 16-byte piece of the qjl row.  For b_m = 3 the pieces are contiguous (48 bytes, so
// that whole 96-bit groups of 32 coordinates are thread-local); otherwise piece u is taken from the
// u-th 64-byte block of the range (quad-contiguous).
struct Slot {
  int coord;
  int term;   // 0..3: index bit; 4..7: parity terms
};

__host__ __device__ inline Slot a_slot(int bm, int r, int t4, int word, int bitpos) {
  const int ni = 4 * bm;
  if (word < ni) {
    const int byteoff = (bm == 3) ? r * 192 + t4 * 48 + 4 * word
                                  : r * 64 * bm + (word >> 2) * 64 + t4 * 16 + 4 * (word & 3);
    const int gb = byteoff * 8 + bitpos;
    return {gb / bm, gb % bm};
  }
  const int w = word - ni;
  if (bm == 3) {   // parity word of the w-th 96-bit group: bit p holds the coordinate whose field starts there
    const int c0 = r * 512 + t4 * 128 + 32 * w;
    const int m = bitpos % 3;
    const int c = (m == 0) ? bitpos / 3 : (m == 1) ? (32 + bitpos) / 3 : (64 + bitpos) / 3;
    return {c0 + c, 4};
  }
  // bm == 4: parity word w belongs to idx word w; nibble c holds the four 3-subset parities
  const int byteoff = r * 256 + (w >> 2) * 64 + t4 * 16 + 4 * (w & 3);
  return {byteoff * 2 + bitpos / 4, 4 + (bitpos & 3)};
}

__host__ __device__ inline int s_slot(int r, int t4, int word, int bitpos) {
  return (r * 64 + t4 * 16 + 4 * word) * 8 + bitpos;
}

// ------------------------------------------------------------------ B operand
struct BPrepArgs {
  const float* Qcat;   // rotated queries of this pass: row q at Qcat + q*ldq
  int64_t ldq;
  QConst* qc;          // out: per-query constants of this pass (written by block 0)
  int nq_pass;         // valid queries in this pass
  int d, dpad, bm, prod, R, NT;
  double alpha[8];
  double amax, csum;   // max |alpha_T|; alpha_empty - sum_T alpha_T
  uint2* out;          // [NT][R][KS][32]
};

constexpr int kMaxPassQueries = 4;

// Per-query scale and constants.  Every block derives them itself (a few thousand loads from L2),
// in the same order, so that no separate launch is needed; block 0 publishes them for the scan.
__device__ void query_constants(const BPrepArgs& a, QConst* sc /* shared, [kMaxPassQueries] */) {
  __shared__ double red[4][8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int ql = 0; ql < a.nq_pass; ++ql) {
    const float* q = a.Qcat + (int64_t)ql * a.ldq;
    double mx1 = 0.0, sm1 = 0.0, mx2 = 0.0, sm2 = 0.0;
    for (int j = threadIdx.x; j < a.d; j += blockDim.x) {
      const double v = (double)q[j];
      mx1 = fmax(mx1, fabs(v));
      sm1 += v;
      if (a.prod) {
        const double u = (double)q[a.dpad + j];
        mx2 = fmax(mx2, fabs(u));
        sm2 += u;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mx1 = fmax(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
      mx2 = fmax(mx2, __shfl_xor_sync(0xffffffffu, mx2, o));
      sm1 += __shfl_xor_sync(0xffffffffu, sm1, o);
      sm2 += __shfl_xor_sync(0xffffffffu, sm2, o);
    }
    if (lane == 0) {
      red[0][warp] = mx1; red[1][warp] = sm1; red[2][warp] = mx2; red[3][warp] = sm2;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < 8; ++w) {
        mx1 = fmax(mx1, red[0][w]); sm1 += red[1][w];
        mx2 = fmax(mx2, red[2][w]); sm2 += red[3][w];
      }
      // |W| < 2^e with W = 2 alpha q'  ->  |W| 2^(22-e) < 2^22: the fixed-point integers (and their pairwise
      // differences, < 2^23) fit three signed radix-256 digits, the format the tcgen05 engine uses, so that
      // both engines form identical sums; the fourth digit column of this engine stays zero.
      auto expo = [](double wmax) {
        if (!(wmax > 0.0) || !isfinite(wmax)) return 0;
        int e;
        frexp(wmax, &e);
        return 22 - e;
      };
      QConst c;
      c.fa = expo(2.0 * a.amax * mx1);
      c.fs = expo(2.0 * mx2);
      c.sa = (float)ldexp(1.0, -c.fa);
      c.ss = (float)ldexp(1.0, -c.fs);
      c.ca = (float)(a.csum * sm1);
      c.cs = (float)(-sm2);
      c.pad[0] = c.pad[1] = 0;
      sc[ql] = c;
      if (blockIdx.x == 0) a.qc[ql] = c;
    }
    __syncthreads();
  }
}

// 2^e as a double; multiplying by it is the exact scaling ldexp performs, at the cost of one multiply.
__device__ __forceinline__ double pow2_of(int e) {
  if (e < -1000 || e > 1000) return ldexp(1.0, e);
  return __hiloint2double((e + 1023) << 20, 0);
}

__device__ __forceinline__ int digit_of(long long J, int limb) {
  int dg = 0;
  for (int l = 0; l <= limb; ++l) {
    dg = (int)(((J + 128) & 255) - 128);
    J = (J - dg) >> 8;
  }
  return dg;
}

// One thread per output byte (8 per uint2 element): the chain of fp64 and index arithmetic behind a digit is
// long, and this kernel sits in front of every scan call; the 8 bytes meet by a shuffle-OR.
__global__ void __launch_bounds__(256) bprep_kernel(BPrepArgs a) {
  __shared__ QConst sc[kMaxPassQueries];
  query_constants(a, sc);
  const int ksa = ks_a(a.bm), kss = ks_s(a.prod != 0), KS = ksa + kss;
  const int64_t total = (int64_t)a.NT * a.R * KS * 32;
  const int64_t tid8 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t tid = tid8 >> 3;
  if (tid >= total) return;   // total * 8 is a multiple of 256: whole warps leave together
  const int which = (int)(tid8 >> 2) & 1, byte = (int)tid8 & 3;
  const int lane = (int)(tid & 31);
  const int ks = (int)((tid >> 5) % KS);
  const int r = (int)((tid >> 5) / KS % a.R);
  const int nt = (int)((tid >> 5) / KS / a.R);
  const int g = lane >> 2, t4 = lane & 3;
  const int col = nt * 8 + g, ql = col / LIMBS, limb = col % LIMBS;
  uint32_t out[2] = {0u, 0u};
  if (ql < a.nq_pass) {
    const float* q = a.Qcat + (int64_t)ql * a.ldq;
    const QConst c = sc[ql];
    const bool is_s = ks >= ksa;
    const int kk = is_s ? ks - ksa : ks;
    const int p = kk >> 3, k = kk & 7;
    const int fexp = is_s ? c.fs : c.fa;
    const double scale7 = pow2_of(fexp - 7), scalek = pow2_of(fexp - k);
    // Slot (byte, k) and the slot of bit 7 of the same byte: the k = 7 operand is the raw byte
    // (sum_j 2^j bit_j), so the operand of k < 7 carries J_k - J_7.
    auto weight = [&](int bp) -> double {
      double W = 0.0;
      if (!is_s) {
        const Slot s = a_slot(a.bm, r, t4, 2 * p + which, bp);
        if (s.coord < a.d) W = 2.0 * a.alpha[s.term] * (double)q[s.coord];
      } else {
        const int j = s_slot(r, t4, 2 * p + which, bp);
        if (j < a.d) W = 2.0 * (double)q[a.dpad + j];
      }
      return W;
    };
    double Jd = rint(weight(8 * byte + 7) * scale7);
    if (k < 7) Jd = rint(weight(8 * byte + k) * scalek) - Jd;
    if (!(fabs(Jd) <= 8388608.0)) Jd = 0.0;   // non-finite query entries contribute nothing
    const int dg = digit_of((long long)Jd, limb);
    out[which] = (uint32_t)(dg & 255) << (8 * byte);
  }
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) {
    out[0] |= __shfl_xor_sync(0xffffffffu, out[0], o);
    out[1] |= __shfl_xor_sync(0xffffffffu, out[1], o);
  }
  // k-steps 2j and 2j + 1 of a lane sit side by side, so that the scan fetches both with one 16-byte load
  if ((tid8 & 7) == 0) {
    const int64_t pairbase = (tid >> 5) / 2 * 64;   // (nt, r, ks / 2) block of 32 lanes x 2 k-steps
    a.out[pairbase + lane * 2 + (ks & 1)] = make_uint2(out[0], out[1]);
  }
}

// ------------------------------------------------------------------ scan kernel
struct ScanArgs {
  int64_t n;
  int64_t ntiles;
  int R, stages;
  int idx_rb;              // bytes of one idx row (its tail may leave whole 64-byte blocks of the last range empty)
  const uint2* Bfrag;
  int bfrag_u2;            // uint2 elements of Bfrag (multiple of 32)
  const QConst* qc;        // constants of this pass's queries
  int nq_pass;
  const float* gamma;
  const float* norms;      // nullable
  float coef;
  float* scores;           // dense: row q of this pass at scores + q*lds
  int64_t lds;
  const float* tau;        // filter mode (indexed by pass-local query)
  int* count;
  float* cand_s;
  int* cand_i;
  int cap;
  const int* run_if;       // nullable: the launch does nothing when *run_if == 0
  int* status;
};

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ long long shfl_xor_ll(long long v, int m) {
  int lo = (int)(v & 0xffffffffll), hi = (int)(v >> 32);
  lo = __shfl_xor_sync(0xffffffffu, lo, m);
  hi = __shfl_xor_sync(0xffffffffu, hi, m);
  return ((long long)hi << 32) | (unsigned int)lo;
}

// MODE 0: dense scores.  MODE 1: thresholded candidate pairs.
template <int BM, bool PROD, int NW, int MT, int NT, int MODE>
__global__ void __launch_bounds__(32 * (NW + 1), 1)
scan_mma_kernel(const __grid_constant__ CUtensorMap tmIdx, const __grid_constant__ CUtensorMap tmQjl, ScanArgs a) {
  constexpr int NTHREADS = 32 * (NW + 1);          // one TMA producer warp + NW consumer warps
  constexpr int VT = NW * MT * 16;                 // vectors per stage
  constexpr int NBLK = BM + (PROD ? 1 : 0);        // 64-byte column blocks per stage
  constexpr int STAGE_BYTES = NBLK * VT * 64;
  constexpr int NI = idx_words(BM), WA = a_words(BM);
  constexpr int KSA = ks_a(BM), KSS = ks_s(PROD), KS = KSA + KSS;
  constexpr int NQP = NT * 8 / LIMBS;              // queries per pass

  if (a.run_if != nullptr && *a.run_if == 0) return;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* stage_base = smem;
  uint2* Bs = reinterpret_cast<uint2*>(smem + (size_t)a.stages * STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(Bs) + (size_t)a.bfrag_u2 * 8);
  uint64_t* full = bars;
  uint64_t* empty = bars + MAX_STAGES;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * MAX_STAGES);
  QConst* qcs = reinterpret_cast<QConst*>(bars + 2 * MAX_STAGES + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      tc::mbar_init(&full[s], 1);
      tc::mbar_init(&empty[s], NW);
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
    if (BM > 0) tc::tma_prefetch_desc(&tmIdx);
    if (PROD) tc::tma_prefetch_desc(&tmQjl);
  }
  {
    const uint4* src = reinterpret_cast<const uint4*>(a.Bfrag);
    uint4* dst = reinterpret_cast<uint4*>(Bs);
    for (int i = threadIdx.x; i < a.bfrag_u2 / 2; i += NTHREADS) dst[i] = __ldg(src + i);
    if (threadIdx.x < NQP) {
      QConst c = {1.0, 0.0, 1.0, 0.0, 0, 0, {0, 0}};
      if ((int)threadIdx.x < a.nq_pass) c = a.qc[threadIdx.x];
      qcs[threadIdx.x] = c;
    }
  }
  __syncthreads();

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x) {
        const int y = (int)(tile * VT);
        for (int r = 0; r < a.R; ++r) {
          if (!(ok = tc::mbar_wait(&empty[stage], phase ^ 1u, abort_flag, a.status))) break;
          unsigned char* sb = stage_base + (size_t)stage * STAGE_BYTES;
          // 64-byte blocks wholly beyond the row (short rows: d well below a multiple of 512) are not copied at all;
          // the consumers skip their k-steps
          const int nvalid = (BM == 3) ? BM : max(0, min(BM, (a.idx_rb - r * 64 * BM + 63) / 64));
          tc::mbar_arrive_expect_tx(&full[stage], (uint32_t)((nvalid + (PROD ? 1 : 0)) * VT * 64));
#pragma unroll
          for (int u = 0; u < BM; ++u)
            if (u < nvalid) tc::tma_load_2d(sb + u * VT * 64, &tmIdx, &full[stage], r * 64 * BM + u * 64, y);
          if (PROD) tc::tma_load_2d(sb + BM * VT * 64, &tmQjl, &full[stage], r * 64, y);
          if (++stage == a.stages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let copies in flight land
      }
    }
    __syncwarp();
    return;
  }

  // ------------------------------------------------------------------ consumers
  const int cw = warp - 1;
  const int g = lane >> 2, t4 = lane & 3;
  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;
  // Per-row scalars of the epilogue (nu, coef * gamma), requested one tile ahead: with short rows (d = 200: one
  // pipeline step per tile) a request made at the top of its own tile is still in flight when the epilogue needs it.
  float nu_next[MT], gm_next[MT];
  auto request_scalars = [&](int64_t tile) {
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      const int64_t row = tile * VT + cw * (MT * 16) + m * 16 + g + ((t4 & 1) ? 8 : 0);
      const bool in = row < a.n;   // (also false for a tile past the last)
      nu_next[m] = (in && a.norms != nullptr) ? __ldg(a.norms + row) : 1.f;
      gm_next[m] = (PROD && in) ? __ldg(a.gamma + row) : 0.f;   // multiplied by coef where it is used: no wait here
    }
  };
  constexpr bool AHEAD = (NT == 1);   // with two column tiles the longer tile hides the request and the registers cost more
  if (AHEAD) request_scalars(blockIdx.x);
  for (int64_t tile = blockIdx.x; tile < a.ntiles && ok; tile += gridDim.x) {
    int accA[MT][NT][2][4], accS[MT][NT][2][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
          for (int i = 0; i < 4; ++i) accA[m][nt][e][i] = accS[m][nt][e][i] = 0;

    float nu_pre[MT], gm_pre[MT];
    if (!AHEAD) request_scalars(tile);
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      nu_pre[m] = nu_next[m];
      gm_pre[m] = gm_next[m];
    }
    if (AHEAD) request_scalars(tile + gridDim.x);

    for (int r = 0; r < a.R; ++r) {
      if (!(ok = tc::mbar_wait(&full[stage], phase, abort_flag, a.status))) break;
      const unsigned char* sb = stage_base + (size_t)stage * STAGE_BYTES;
      uint32_t w[MT][2][WA > 0 ? WA : 1];
      uint32_t z[MT][2][4];
#pragma unroll
      for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int row = cw * (MT * 16) + m * 16 + h * 8 + g;
#pragma unroll
          for (int u = 0; u < BM; ++u) {
            int blk, off;
            if (BM == 3) {
              const int o = t4 * 48 + u * 16;
              blk = o >> 6;
              off = o & 63;
            } else {
              blk = u;
              off = t4 * 16;
            }
            // (a block that the producer left out holds stale bytes: its k-steps are skipped below)
            const uint4 v = *reinterpret_cast<const uint4*>(sb + blk * VT * 64 + row * 64 + off);
            w[m][h][4 * u] = v.x; w[m][h][4 * u + 1] = v.y; w[m][h][4 * u + 2] = v.z; w[m][h][4 * u + 3] = v.w;
          }
          if (PROD) {
            const uint4 v = *reinterpret_cast<const uint4*>(sb + BM * VT * 64 + row * 64 + t4 * 16);
            z[m][h][0] = v.x; z[m][h][1] = v.y; z[m][h][2] = v.z; z[m][h][3] = v.w;
          }
        }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&empty[stage]);   // the stage now lives in registers
      if (++stage == a.stages) {
        stage = 0;
        phase ^= 1u;
      }

      // parity words
#pragma unroll
      for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (BM == 3) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              const uint32_t w0 = w[m][h][3 * t], w1 = w[m][h][3 * t + 1], w2 = w[m][h][3 * t + 2];
              const uint32_t p0 = w0 ^ __funnelshift_r(w0, w1, 1) ^ __funnelshift_r(w0, w1, 2);
              const uint32_t p1 = w1 ^ __funnelshift_r(w1, w2, 1) ^ __funnelshift_r(w1, w2, 2);
              const uint32_t p2 = w2 ^ (w2 >> 1) ^ (w2 >> 2);
              w[m][h][NI + t] = (p0 & 0x49249249u) | (p1 & 0x92492492u) | (p2 & 0x24924924u);
            }
          } else if (BM == 4) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const uint32_t x = w[m][h][i], s1 = x >> 1, s2 = x >> 2, s3 = x >> 3;
              const uint32_t M = 0x11111111u;
              w[m][h][NI + i] = ((x ^ s1 ^ s2) & M) | (((x ^ s1 ^ s3) & M) << 1) | (((x ^ s2 ^ s3) & M) << 2) |
                                (((s1 ^ s2 ^ s3) & M) << 3);
            }
          }
        }

      uint4 b4[NT];
      const uint4* Bb[NT];   // per lane: the operands of k-steps 2j, 2j + 1 as one 16-byte piece
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) Bb[nt] = reinterpret_cast<const uint4*>(Bs + ((size_t)(nt * a.R + r) * KS) * 32) + lane;

      // 64-byte blocks of this range that hold row bytes at all (short rows: d well below a multiple of 512);
      // the others were not copied (they would be zero fill), and their k-steps, which would add nothing, are skipped
      const int nvalid = (BM == 3) ? BM : max(0, min(BM, (a.idx_rb - r * 64 * BM + 63) / 64));
#pragma unroll
      for (int p = 0; p < WA / 2; ++p) {
        if (BM != 3 && ((2 * p < NI ? 2 * p : 2 * p - NI) >> 2) >= nvalid) continue;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t mk = 0x01010101u << k;
          uint2 b[NT];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            if ((k & 1) == 0) b4[nt] = Bb[nt][((p * 8 + k) >> 1) * 32];
            b[nt] = (k & 1) ? make_uint2(b4[nt].z, b4[nt].w) : make_uint2(b4[nt].x, b4[nt].y);
          }
#pragma unroll
          for (int m = 0; m < MT; ++m) {
            // k = 7 feeds the whole word (all eight bits of every byte): B carries the difference
            const uint32_t a0 = (k == 7) ? w[m][0][2 * p] : (w[m][0][2 * p] & mk);
            const uint32_t a1 = (k == 7) ? w[m][1][2 * p] : (w[m][1][2 * p] & mk);
            const uint32_t a2 = (k == 7) ? w[m][0][2 * p + 1] : (w[m][0][2 * p + 1] & mk);
            const uint32_t a3 = (k == 7) ? w[m][1][2 * p + 1] : (w[m][1][2 * p + 1] & mk);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) mma_u8s8(accA[m][nt][k & 1], a0, a1, a2, a3, b[nt].x, b[nt].y);
          }
        }
      }
      if (PROD) {
#pragma unroll
        for (int p = 0; p < 2; ++p)
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t mk = 0x01010101u << k;
            uint2 b[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              if ((k & 1) == 0) b4[nt] = Bb[nt][((KSA + p * 8 + k) >> 1) * 32];
              b[nt] = (k & 1) ? make_uint2(b4[nt].z, b4[nt].w) : make_uint2(b4[nt].x, b4[nt].y);
            }
#pragma unroll
            for (int m = 0; m < MT; ++m) {
              const uint32_t a0 = (k == 7) ? z[m][0][2 * p] : (z[m][0][2 * p] & mk);
              const uint32_t a1 = (k == 7) ? z[m][1][2 * p] : (z[m][1][2 * p] & mk);
              const uint32_t a2 = (k == 7) ? z[m][0][2 * p + 1] : (z[m][0][2 * p + 1] & mk);
              const uint32_t a3 = (k == 7) ? z[m][1][2 * p + 1] : (z[m][1][2 * p + 1] & mk);
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma_u8s8(accS[m][nt][k & 1], a0, a1, a2, a3, b[nt].x, b[nt].y);
            }
          }
      }
    }
    if (!ok) break;

    // ---------------------------------------------------------------- epilogue
    // Thread (g, t4) holds columns 2 t4, 2 t4 + 1 of rows g and g + 8: two of the four digits of
    // query t4 / 2.  The digit sums are recombined exactly (T = D0 + 256 D1 + 65536 D2 + ... as a 64-bit
    // integer, the same T in both engines although their digit sums differ), then everything is fp32: one
    // rounding of T (2^-24 of sum |W|, three orders below the tolerance) and three FMAs.  The even lane of a
    // pair finishes row g, the odd lane row g + 8: one 64-bit shuffle hands each the other's half.
#pragma unroll
    for (int m = 0; m < MT; ++m) {
      const int64_t row0 = tile * VT + cw * (MT * 16) + m * 16;
      const int64_t row = row0 + g + ((t4 & 1) ? 8 : 0);
      const bool row_ok = row < a.n;
      const float nu = nu_pre[m], gm = PROD ? a.coef * gm_pre[m] : 0.f;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        auto combine = [&](const int (&acc)[2][4]) -> float {
          long long mine[2];
#pragma unroll
          for (int h = 0; h < 2; ++h) {   // digits (0, 1) on the even lane, (2, 3) on the odd lane, as one integer
            const int lo = acc[0][2 * h] + acc[1][2 * h], hi = acc[0][2 * h + 1] + acc[1][2 * h + 1];
            mine[h] = (long long)hi * 256 + lo;
          }
          const long long recv = shfl_xor_ll((t4 & 1) ? mine[0] : mine[1], 1);
          const long long T = (t4 & 1) ? mine[1] * 65536 + recv : recv * 65536 + mine[0];
          return (float)T;   // one rounding of the exact integer: the same value in both engines
        };
        const float Ta = combine(accA[m][nt]);
        const float Ts = PROD ? combine(accS[m][nt]) : 0.f;
        const int ql = nt * 2 + (t4 >> 1);
        const QConst c = qcs[ql];
        const float av = (BM > 0) ? fmaf(Ta, c.sa, c.ca) : 0.f;
        const float sv = PROD ? fmaf(Ts, c.ss, c.cs) : 0.f;
        const float est = __fmul_rn(nu, fmaf(gm, sv, av));
        if (row_ok && ql < a.nq_pass) {
          if (MODE == 0) {
            if (TQ_DEVICE_CHECK(row >= 0 && row < a.n && row < a.lds, a.status)) a.scores[(int64_t)ql * a.lds + row] = est;
          } else if (est >= __ldg(a.tau + ql)) {
            const int slot = atomicAdd(a.count + ql, 1);
            if (slot < a.cap) {
              a.cand_s[(int64_t)ql * a.cap + slot] = est;
              a.cand_i[(int64_t)ql * a.cap + slot] = (int)row;
            }
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------ top-k selection
// One CTA per query: MSD radix select (8-bit digits) on the 64-bit key (ordered score, ~id) for the
// k-th best element, then a bitonic sort of the k survivors.  Keys are distinct because ids are.
struct SelArgs {
  const float* cand_s;
  const int* cand_i;      // nullptr: dense row, id = id0 + position
  const int* count;       // nullptr: m elements
  int cap, m, id0, k, merge;
  float* top_s;
  int* top_i;
  float* kth;             // nullable
  int* overflow;          // nullable: set to 1 when count > cap for this query
  const int* run_if;      // nullable
};

__device__ __forceinline__ unsigned long long make_key(float s, int id) {
  if (s == 0.f) s = 0.f;   // -0 and +0 tie
  uint32_t u = __float_as_uint(s);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return ((unsigned long long)u << 32) | (uint32_t)(~(uint32_t)id);
}

__global__ void __launch_bounds__(1024) select_kernel(SelArgs a) {
  __shared__ int hist[256];
  __shared__ unsigned long long s_prefix;
  __shared__ int s_kk, s_done, s_cnt;
  __shared__ unsigned long long skey[1024];
  if (a.run_if != nullptr && *a.run_if == 0) return;
  const int q = blockIdx.x, tid = threadIdx.x;
  int m_new = a.m;
  if (a.count != nullptr) {
    const int c = a.count[q];
    m_new = min(c, a.cap);
    if (a.overflow != nullptr && c > a.cap && tid == 0) atomicExch(a.overflow, 1);
  }
  const int total = m_new + (a.merge ? a.k : 0);
  const float* src_s = a.cand_s + (int64_t)q * a.cap;
  const int* src_i = a.cand_i ? a.cand_i + (int64_t)q * a.cap : nullptr;
  auto key_at = [&](int i) -> unsigned long long {
    if (i < m_new) {
      const int id = src_i ? src_i[i] : a.id0 + i;
      return id < 0 ? 0ull : make_key(src_s[i], id);
    }
    const int j = i - m_new;
    const int id = a.top_i[(int64_t)q * a.k + j];
    if (id < 0) return 0ull;   // an empty slot of the previous list
    return make_key(a.top_s[(int64_t)q * a.k + j], id);
  };
  // up to 16 keys per thread stay in registers for all rounds (lists up to 16,384 entries)
  const bool cached = total <= 16 * 1024;
  unsigned long long kc[16];
  if (cached) {
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int i = u * 1024 + tid;
      kc[u] = (i < total) ? key_at(i) : 0ull;
    }
  }
  int kk = min(a.k, total);
  const int k_target = kk;
  unsigned long long prefix = 0ull;
  int shift = 56;
  if (kk > 0) {
    for (int round = 0; round < 8; ++round) {
      shift = 56 - 8 * round;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      auto tally = [&](unsigned long long key, bool valid) {
        const bool in = valid && (round == 0 || (key >> (shift + 8)) == prefix);
        // lanes with the same digit add once (scores of one query crowd into a few bins)
        const int dg = in ? (int)((key >> shift) & 255ull) : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, dg);
        if (in && (int)(__ffs(peers) - 1) == (tid & 31)) atomicAdd(&hist[dg], __popc(peers));
      };
      if (cached) {
#pragma unroll
        for (int u = 0; u < 16; ++u) tally(kc[u], u * 1024 + tid < total);
      } else {
        // batches of 8 independent loads per thread, then the (convergent) histogram updates
        for (int base = 0; base < total; base += 8 * blockDim.x) {
          unsigned long long keys[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int i = base + u * blockDim.x + tid;
            keys[u] = (i < total) ? key_at(i) : 0ull;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) tally(keys[u], base + u * (int)blockDim.x + tid < total);
        }
      }
      __syncthreads();
      if (tid < 32) {
        // lane l owns bins 255 - 8l ... 248 - 8l (descending); exclusive prefix of the lane totals by shuffles
        int c[8], tot = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          c[e] = hist[255 - 8 * tid - e];
          tot += c[e];
        }
        int incl = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += v;
        }
        int cum = incl - tot;
        if (cum < kk && incl >= kk) {   // the k-th element lies in this lane's bins
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            if (cum < kk && cum + c[e] >= kk) {
              s_prefix = (prefix << 8) | (unsigned long long)(255 - 8 * tid - e);
              s_kk = kk - cum;
              // stop when the bucket is exactly what is missing, or when everything at or above it fits the
              // final sort, which then settles the order (further rounds would only narrow a small set)
              s_done = (c[e] == kk - cum) || (k_target - (kk - cum) + c[e] <= 1024);
            }
            cum += c[e];
          }
        }
      }
      __syncthreads();
      prefix = s_prefix;
      kk = s_kk;
      const int done = s_done;
      __syncthreads();
      if (done) break;
    }
  }
  // survivors: (key >> shift) >= prefix
  if (tid == 0) s_cnt = 0;
  skey[tid] = 0ull;
  __syncthreads();
  if (min(a.k, total) > 0) {
    auto keep = [&](unsigned long long key) {
      if ((key >> shift) >= prefix && key != 0ull) {
        const int slot = atomicAdd(&s_cnt, 1);
        if (slot < 1024) skey[slot] = key;
      }
    };
    if (cached) {
#pragma unroll
      for (int u = 0; u < 16; ++u) keep(kc[u]);
    } else {
      for (int base = 0; base < total; base += 8 * blockDim.x) {
        unsigned long long keys[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int i = base + u * blockDim.x + tid;
          keys[u] = (i < total) ? key_at(i) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) keep(keys[u]);
      }
    }
  }
  __syncthreads();
  // bitonic sort, descending, of the smallest power of two that holds the survivors (the rest of skey is zero)
  int sort_n = 32;
  while (sort_n < min(s_cnt, 1024)) sort_n <<= 1;
  for (int kb = 2; kb <= sort_n; kb <<= 1) {
    for (int j = kb >> 1; j > 0; j >>= 1) {
      const int p = tid ^ j;
      if (p > tid && p < sort_n) {
        const unsigned long long x = skey[tid], y = skey[p];
        const bool desc = ((tid & kb) == 0);
        if (desc ? (x < y) : (x > y)) {
          skey[tid] = y;
          skey[p] = x;
        }
      }
      __syncthreads();
    }
  }
  if (tid < a.k) {
    const unsigned long long key = skey[tid];
    float s = -INFINITY;
    int id = -1;
    if (key != 0ull) {
      uint32_t u = (uint32_t)(key >> 32);
      u = (u & 0x80000000u) ? (u & 0x7fffffffu) : ~u;
      s = __uint_as_float(u);
      id = (int)(~(uint32_t)(key & 0xffffffffull));
    }
    a.top_s[(int64_t)q * a.k + tid] = s;
    a.top_i[(int64_t)q * a.k + tid] = id;
    if (tid == a.k - 1 && a.kth != nullptr) a.kth[q] = s;
  }
}

// ------------------------------------------------------------------ host side
struct Config {
  int NW, MT, NT, stages;
  size_t smem;
};

size_t bfrag_bytes(const tq_plan* plan, int NT) {
  const int KS = ks_a(plan->mse_bits) + ks_s(plan->mode == TQ_PROD);
  return (size_t)NT * plan->ms.R * KS * 32 * sizeof(uint2);
}

bool pick_config(const tq_plan* plan, int NW, int MT, int NT, Config* out) {
  const int nblk = plan->mse_bits + (plan->mode == TQ_PROD ? 1 : 0);
  const size_t stage = (size_t)nblk * (NW * MT * 16) * 64;
  const size_t fixed = bfrag_bytes(plan, NT) + 1024 /*alignment*/ + 2 * MAX_STAGES * 8 + 16 + 4 * sizeof(QConst);
  if (fixed + 2 * stage > (size_t)SMEM_LIMIT) return false;
  int stages = (int)std::min<size_t>((SMEM_LIMIT - fixed) / stage, MAX_STAGES);
  out->NW = NW;
  out->MT = MT;
  out->NT = NT;
  out->stages = stages;
  out->smem = fixed + (size_t)stages * stage;
  return true;
}

template <int BM, bool PROD, int NW, int MT, int NT, int MODE>
cudaError_t launch_t(const CUtensorMap& mi, const CUtensorMap& mq, const ScanArgs& args, size_t smem, cudaStream_t st) {
  auto kern = scan_mma_kernel<BM, PROD, NW, MT, NT, MODE>;
  // function attributes are per device: the largest size set so far, per device
  static std::atomic<size_t> attr[64];   // zero-initialised; written by any thread that launches
  int attr_dev = 0;
  if (cudaGetDevice(&attr_dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (attr_dev >= 64 || smem > attr[attr_dev].load(std::memory_order_relaxed)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (attr_dev < 64) attr[attr_dev].store(smem, std::memory_order_relaxed);
  }
  const int grid = (int)std::min<int64_t>(args.ntiles, tc::sm_count());
  kern<<<grid, 32 * (NW + 1), smem, st>>>(mi, mq, args);
  count_launches(1);
  return cudaGetLastError();
}

template <int BM, bool PROD>
cudaError_t launch_cfg(const Config& c, bool filter, const CUtensorMap& mi, const CUtensorMap& mq, const ScanArgs& args,
                       cudaStream_t st) {
  if (c.NW == 16 && c.NT == 1)
    return filter ? launch_t<BM, PROD, 16, 1, 1, 1>(mi, mq, args, c.smem, st) : launch_t<BM, PROD, 16, 1, 1, 0>(mi, mq, args, c.smem, st);
  if (c.NW == 12 && c.NT == 2)
    return filter ? launch_t<BM, PROD, 12, 1, 2, 1>(mi, mq, args, c.smem, st) : launch_t<BM, PROD, 12, 1, 2, 0>(mi, mq, args, c.smem, st);
  if (c.NT == 2)
    return filter ? launch_t<BM, PROD, 8, 1, 2, 1>(mi, mq, args, c.smem, st) : launch_t<BM, PROD, 8, 1, 2, 0>(mi, mq, args, c.smem, st);
  return filter ? launch_t<BM, PROD, 8, 1, 1, 1>(mi, mq, args, c.smem, st) : launch_t<BM, PROD, 8, 1, 1, 0>(mi, mq, args, c.smem, st);
}

cudaError_t launch_scan(const tq_plan* plan, const Config& c, bool filter, const CUtensorMap& mi, const CUtensorMap& mq,
                        const ScanArgs& args, cudaStream_t st) {
  const bool prod = plan->mode == TQ_PROD;
  switch (plan->mse_bits) {
    case 0: return launch_cfg<0, true>(c, filter, mi, mq, args, st);
    case 1: return prod ? launch_cfg<1, true>(c, filter, mi, mq, args, st) : launch_cfg<1, false>(c, filter, mi, mq, args, st);
    case 2: return prod ? launch_cfg<2, true>(c, filter, mi, mq, args, st) : launch_cfg<2, false>(c, filter, mi, mq, args, st);
    case 3: return prod ? launch_cfg<3, true>(c, filter, mi, mq, args, st) : launch_cfg<3, false>(c, filter, mi, mq, args, st);
    default: return prod ? launch_cfg<4, true>(c, filter, mi, mq, args, st) : launch_cfg<4, false>(c, filter, mi, mq, args, st);
  }
}

// nq <= 2: one column tile, 16 consumer warps of 16 vectors; nq > 2: two column tiles, 12 (else 8) warps.
// Falls back to the smallest shape when the B operand leaves no room for two stages.
Config config_for(const tq_plan* plan, int nq) {
  Config c{8, 1, 1, 2, 0};
  if (nq > 2 && pick_config(plan, 12, 1, 2, &c)) return c;
  if (nq > 2 && pick_config(plan, 8, 1, 2, &c)) return c;
  if (pick_config(plan, 16, 1, 1, &c)) return c;
  pick_config(plan, 8, 1, 1, &c);
  return c;
}

}  // namespace

void plan_init(tq_plan* plan) {
  plan->ms.ok = 0;
  const int bm = plan->mse_bits, L = 1 << bm;
  if (plan->d < 128 || !plan->tc_ok) return;   // short rows stay on the CUDA-core scan; tensor maps needed
  // Walsh expansion of the codebook over the index bits.
  double coeff[16];
  double cmax = 0.0;
  for (int k = 0; k < L; ++k) cmax = std::max(cmax, std::fabs((double)plan->cb.c[k]));
  for (int T = 0; T < L; ++T) {
    double s = 0.0;
    for (int k = 0; k < L; ++k) {
      int sign = 1;
      for (int i = 0; i < bm; ++i)
        if (((T >> i) & 1) && !((k >> i) & 1)) sign = -sign;
      s += sign * (double)plan->cb.c[k];
    }
    coeff[T] = s / L;
  }
  for (int T = 1; T < L; ++T)
    if (__builtin_popcount(T) % 2 == 0 && std::fabs(coeff[T]) > 1e-7 * cmax) return;   // not antisymmetric
  for (int i = 0; i < 8; ++i) plan->ms.alpha[i] = 0.0;
  for (int i = 0; i < bm; ++i) plan->ms.alpha[i] = coeff[1 << i];
  if (bm == 3) plan->ms.alpha[4] = coeff[7];
  if (bm == 4) {
    plan->ms.alpha[4] = coeff[0b0111];
    plan->ms.alpha[5] = coeff[0b1011];
    plan->ms.alpha[6] = coeff[0b1101];
    plan->ms.alpha[7] = coeff[0b1110];
  }
  double amax = 0.0, asum = 0.0;
  for (int i = 0; i < 8; ++i) {
    amax = std::max(amax, std::fabs(plan->ms.alpha[i]));
    asum += plan->ms.alpha[i];
  }
  plan->ms.amax = amax;
  plan->ms.csum = coeff[0] - asum;
  plan->ms.R = (plan->d + 511) / 512;
  Config c;
  if (!pick_config(plan, 8, 1, 1, &c)) return;   // B operand too large for shared memory at this d
  plan->ms.ok = 1;
}

int queries_per_pass(const tq_plan* plan, int nq) { return config_for(plan, nq).NT * 8 / LIMBS; }


size_t workspace_bytes(const tq_plan* plan) {
  if (!plan->ms.ok) return 0;
  Config c;
  const int nt = pick_config(plan, 8, 1, 2, &c) ? 2 : 1;
  return kQConstBytes + (bfrag_bytes(plan, nt) + 255) / 256 * 256;
}

int prepare(const tq_plan* plan, const float* Qcat, int nqp, void* workspace, cudaStream_t st, const char* who) {
  const Config c = config_for(plan, nqp);
  const bool prod = plan->mode == TQ_PROD;
  const int bm = plan->mse_bits;
  const int ncols = plan->ncat * plan->dpad;
  QConst* qc = static_cast<QConst*>(workspace);
  uint2* bfrag = reinterpret_cast<uint2*>(static_cast<char*>(workspace) + kQConstBytes);
  BPrepArgs ba;
  ba.Qcat = Qcat;
  ba.ldq = ncols;
  ba.qc = qc;
  ba.amax = plan->ms.amax;
  ba.csum = plan->ms.csum;
  ba.nq_pass = nqp;
  ba.d = plan->d;
  ba.dpad = plan->dpad;
  ba.bm = bm;
  ba.prod = prod ? 1 : 0;
  ba.R = plan->ms.R;
  ba.NT = c.NT;
  for (int i = 0; i < 8; ++i) ba.alpha[i] = plan->ms.alpha[i];
  ba.out = bfrag;
  const int64_t total = (int64_t)c.NT * plan->ms.R * (ks_a(bm) + ks_s(prod)) * 32;
  bprep_kernel<<<(unsigned)((total * 8 + 255) / 256), 256, 0, st>>>(ba);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

int run(const tq_plan* plan, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
        const float* norms, float* scores, int64_t lds, const Filter* filter, const int* run_if, const void* workspace,
        cudaStream_t st, const char* who) {
  const Config c = config_for(plan, nqp);
  const bool prod = plan->mode == TQ_PROD;
  const int bm = plan->mse_bits;
  const int VT = c.NW * c.MT * 16;
  CUtensorMap mi, mq;
  if (bm > 0)
    TQ_REQUIRE(tc::make_byte_map(&mi, idx, (uint64_t)n, plan->idx_row_bytes, plan->idx_row_bytes, 64, VT), TQ_ERR_CUDA,
               "%s: cuTensorMapEncodeTiled failed (idx)", who);
  if (prod)
    TQ_REQUIRE(tc::make_byte_map(&mq, qjl, (uint64_t)n, plan->qjl_row_bytes, plan->qjl_row_bytes, 64, VT), TQ_ERR_CUDA,
               "%s: cuTensorMapEncodeTiled failed (qjl)", who);
  if (bm == 0) mi = mq;
  if (!prod) mq = mi;
  ScanArgs sa;
  sa.n = n;
  sa.ntiles = (n + VT - 1) / VT;
  sa.R = plan->ms.R;
  sa.idx_rb = (int)plan->idx_row_bytes;
  sa.stages = c.stages;
  sa.Bfrag = reinterpret_cast<const uint2*>(static_cast<const char*>(workspace) + kQConstBytes);
  sa.bfrag_u2 = c.NT * plan->ms.R * (ks_a(bm) + ks_s(prod)) * 32;
  sa.qc = static_cast<const QConst*>(workspace);
  sa.nq_pass = nqp;
  sa.gamma = gamma;
  sa.norms = norms;
  sa.coef = plan->coef;
  sa.scores = scores;
  sa.lds = lds;
  sa.tau = filter ? filter->tau : nullptr;
  sa.count = filter ? filter->count : nullptr;
  sa.cand_s = filter ? filter->cand_s : nullptr;
  sa.cand_i = filter ? filter->cand_i : nullptr;
  sa.cap = filter ? filter->cap : 0;
  sa.run_if = run_if;
  sa.status = plan->d_status;
  TQ_CHECK_CUDA(launch_scan(plan, c, filter != nullptr, mi, mq, sa, st), who);
  return TQ_OK;
}

cudaError_t select_topk(const float* cand_s, const int* cand_i, const int* count, int cap, int m, int id0, int nq, int k,
                        int merge, float* top_s, int* top_i, float* kth, int* overflow, const int* run_if,
                        cudaStream_t st) {
  SelArgs a;
  a.cand_s = cand_s;
  a.cand_i = cand_i;
  a.count = count;
  a.cap = cap;
  a.m = m;
  a.id0 = id0;
  a.k = k;
  a.merge = merge;
  a.top_s = top_s;
  a.top_i = top_i;
  a.kth = kth;
  a.overflow = overflow;
  a.run_if = run_if;
  select_kernel<<<nq, 1024, 0, st>>>(a);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t select_pairs(const float* cand_s, const int* cand_i, int ld, int m, int nq, int k, float* top_s, int* top_i,
                         cudaStream_t st) {
  return select_topk(cand_s, cand_i, nullptr, ld, m, 0, nq, k, 0, top_s, top_i, nullptr, nullptr, nullptr, st);
}

}  // namespace mscan
}  // namespace tq

// Many-query packed-code scan on tcgen05: the same bit-plane form of the estimator as in
// tq_scan_mma.cu (codebook expanded over the index bits, raw bits and parity words as a 0/1 matrix,
// query weights as fixed-point radix-256 digits, identical integers), but with the multiply-accumulate
// on the 5th-generation tensor cores:
//     D[128 vectors, 96 columns] += A[128, 32] * B[96, 32]^T,   kind::i8, s32 accumulators in TMEM.
// 96 columns hold 32 queries x 3 digits, so one pass over the codes serves 32 queries and the decode
// (one AND per four bits, once per vector) is amortised over all of them.  A tcgen05 MMA of this shape
// costs about the same 55-64 cycles for any N <= 128, which is why this path is for many queries and
// the register-fed mma.sync path for few.
//
// The A operand never touches shared memory: byte-expanded bit planes are 8x the packed codes, and
// writing + reading them there would cost more shared-memory cycles than the MMAs take.  Each
// transform thread owns one vector row = one TMEM lane; it expands the row's four packed words of a
// k-block into 32 registers and stores them with tcgen05.st into the 32 TMEM columns of that k-block,
// from where the MMA takes A directly.
//
// CTA (one per SM, persistent over pairs of 128-vector tiles):
//   warp 0       TMA producer: per k-block (128 K-bytes) one [96 rows x 128 B] box of B (128-byte swizzle); per
//                four k-blocks the packed rows of the pair ([256 rows x 32..64 B], swizzled for row-per-thread reads)
//   warps 1..2   MMA issuers (warp 1 owns TMEM): k-blocks alternate between them, 8 MMAs (K = 32, 4 per tile)
//                + one commit each.  A tcgen05.commit keeps its thread for ~350 cycles while the 8 MMAs take
//                ~420, so a single issuer leaves the tensor pipe idle half of the time (measured: 95 cycles
//                per MMA with one issuing thread, 70 with two).
//   warps 3..10  transform + epilogue (thread = vector row): zero the row's accumulators (tcgen05.st), then per
//                k-block the row's packed bytes from shared memory, 3 index words + their parity word (b_m = 3)
//                -> 32 x (w & (0x01010101 << k)) -> tcgen05.st; after the last k-block the row's accumulators
//                are read back (tcgen05.ld), the digits recombined, estimates emitted.
// Every MMA accumulates onto the zeroed accumulators; the sums are integers, so the order in which the
// k-blocks of the two issuers reach the pipe does not matter.
// TMEM (512 columns): tile t: MSE-part accumulator at 192 t + [0, 96), QJL-part at 192 t + [96, 192);
// A: two k-block slots of 32 columns per tile at 384 + 64 t.  The two tiles share every B box (halves
// the L2 traffic of B).  Rings: 2 A slots (TMEM), 8 B stages and 4 packed-row stages (shared memory) with
// full mbarriers; one tcgen05.commit per k-block releases both the A slot and the B stage; accumulator-full
// barrier (one commit per issuer).  Ring positions and phases are masks and shifts of 32-bit counters: the
// single-lane roles run dependent instruction chains, where 64-bit division costs real time.  All waits
// are bounded.
//
// Calls of more than 32 queries run the wide form of this kernel (tq_scan_tcw.cuh: 64 queries per pass, one tile
// per iteration, four A slots, N = 192); this one serves 7..32 queries and the last, short pass of a longer call.
#include <atomic>
#include <algorithm>
#include <cmath>
#include <cstdlib>

#include "tq_nib_common.cuh"
#include "tq_quantize_tc.h"
#include "tq_scan_tc.h"
#include "tq_tc.cuh"

namespace tq {
namespace tscan {

namespace {

constexpr int TILE = 128;              // vectors per M tile = TMEM lanes
constexpr int LIMBS = 3;               // signed radix-256 digits per weight (|J| < 2^23)
constexpr int NCOL = 96;               // MMA N: 3 digits x 32 queries, digit-major (column = 32 digit + query)
constexpr int KB_BYTES = 128;          // K extent of one k-block (one swizzled row)
constexpr int A_SLOTS = 2;             // k-blocks of A per tile resident in TMEM
constexpr int B_STAGES = 8;            // ring of B tiles in shared memory (TMA from L2); a power of two, so that ring
                                       // positions and phases of 32-bit counters are masks and shifts
constexpr int BTILE_BYTES = NCOL * KB_BYTES;         // 12 KB
constexpr int P_STAGES = 4;            // ring of packed-row groups (4 k-blocks of the pair's 256 rows each)
constexpr int PTILE_BYTES = 2 * TILE * 64;           // 16 KB: 256 rows x at most 64 bytes
constexpr int D_COLS = 2 * NCOL;                     // accumulator columns per tile (MSE part, QJL part)
constexpr int A_COL0 = 2 * D_COLS;                   // first TMEM column of the A slots
constexpr int N_ISSUERS = 2;             // MMA-issuing warps (a tcgen05.commit stalls its thread; a second issuer hides it)
// The barrier rings count on this number: a parity wait also passes when its barrier is two completions behind, so the
// thread that waits for k-block k must itself have waited for the completion before it on the same barrier -- A_SLOTS
// and B_STAGES are multiples of N_ISSUERS.  (Three issuers with rings of 6 / 9 / 16 barriers, as in the 64-query
// kernel, were measured here: 464 against 471 us per pass; this kernel is bound by its transform warps.)
static_assert(A_SLOTS % N_ISSUERS == 0 && B_STAGES % N_ISSUERS == 0, "a waiter has seen the completion before the one it waits for");
constexpr int NTHREADS = 32 * (1 + N_ISSUERS + 8);
constexpr int TMEM_COLS = 512;
constexpr int LBUF = 128;              // candidates per query a CTA collects in shared memory before it appends them
constexpr size_t kConstBytes = 256 * 48;             // per-query constants of one group

struct QConst {
  float sa, ca;    // a = T_a * sa + ca   (MSE term)
  float ss, cs;    // s = T_s * ss + cs   (QJL term)
  int fa, fs;
  int pad[2];
};

struct Geo {
  int bm, d, dpad;
  int widx, wq;    // 32-bit words per idx / qjl row
  int kba, kbs;    // k-blocks of the MSE part and of the QJL part
  // TQ_LAYOUT_NIBBLE: every 64-byte block of the combined row [idx row | qjl row] gives three k-blocks in turn --
  // the h bytes (signed A), the l bytes, the sign bits -- of its 128 coordinates; kba holds their total, kbs = 0
  int nib, nbi, nblk, idx_rb, qjl_rb;
};

__host__ __device__ inline int div_up(int a, int b) { return (a + b - 1) / b; }
// packed idx bytes of one row consumed by a group of four k-blocks
__host__ __device__ constexpr int group_bytes(int bm) { return bm == 3 ? 48 : bm == 4 ? 32 : 64; }

Geo make_geo(const tq_plan* plan) {
  Geo g;
  g.bm = plan->mse_bits;
  g.d = plan->d;
  g.dpad = plan->dpad;
  g.widx = (int)(plan->idx_row_bytes / 4);
  g.wq = (plan->mode == TQ_PROD) ? (int)(plan->qjl_row_bytes / 4) : 0;
  g.kba = g.bm == 0 ? 0 : g.bm == 3 ? div_up(g.widx, 3) : g.bm == 4 ? div_up(g.widx, 2) : div_up(g.widx, 4);
  g.kbs = div_up(g.wq, 4);
  g.nib = plan->layout == TQ_LAYOUT_NIBBLE ? 1 : 0;
  g.nbi = plan->nb.nbi;
  g.nblk = plan->nb.nbi + plan->nb.nbq;
  g.idx_rb = (int)plan->idx_row_bytes;
  g.qjl_rb = (int)plan->qjl_row_bytes;
  if (g.nib) {
    g.kba = 3 * g.nblk;
    g.kbs = 0;
  }
  return g;
}

// K slot (part, k-block, word wl of the block, bit of the word) -> (coordinate, Walsh term).
// MSE part, b_m = 1, 2: four index words per block.  b_m = 3: the three words of one 96-bit group of 32
// coordinates and their parity word.  b_m = 4: two index words and their two words of 3-subset parities.
struct Slot {
  int coord, term;
};
__device__ inline Slot slot_a(const Geo& g, int kb, int wl, int bit) {
  if (g.bm <= 2) {
    const int P = 32 * (4 * kb + wl) + bit;
    return {P / g.bm, P % g.bm};
  }
  if (g.bm == 3) {
    if (wl < 3) {
      const int P = 32 * (3 * kb + wl) + bit;
      return {P / 3, P % 3};
    }
    const int m = bit % 3;
    const int c = (m == 0) ? bit / 3 : (m == 1) ? (32 + bit) / 3 : (64 + bit) / 3;
    return {32 * kb + c, 4};
  }
  if (wl < 2) {
    const int P = 32 * (2 * kb + wl) + bit;
    return {P / 4, P % 4};
  }
  return {8 * (2 * kb + wl - 2) + bit / 4, 4 + (bit & 3)};
}

// ------------------------------------------------------------------ per-query constants
struct StatArgs {
  const float* Qcat;
  int64_t ldq;
  int d, dpad, prod;
  double amax, csum;
  int nib;          // nibble layout: the scales and constants of the table-lookup form
  double delta;
  QConst* out;
};

// Nibble layout: one warp per query, the same reductions in the same order as the register-fed engine's
// (lane-strided maxima in fp32, the sum of q'' in fp64 folded by xor shuffles).
__global__ void __launch_bounds__(32) tstats_nib_kernel(StatArgs a) {
  const int lane = threadIdx.x;
  const float* q = a.Qcat + (int64_t)blockIdx.x * a.ldq;
  float mx1 = 0.f, mx2 = 0.f;
  double sm2 = 0.0;
  for (int j = lane; j < a.d; j += 32) {
    mx1 = fmaxf(mx1, fabsf(q[j]));
    const float u = q[a.dpad + j];
    mx2 = fmaxf(mx2, fabsf(u));
    sm2 += (double)u;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
    mx2 = fmaxf(mx2, __shfl_xor_sync(0xffffffffu, mx2, o));
    sm2 += __shfl_xor_sync(0xffffffffu, sm2, o);
  }
  if (lane == 0) {
    const nib::QScale s = nib::make_scale(mx1, mx2);
    const nib::QConst n = nib::make_const(s, a.delta, sm2);
    QConst c;
    c.sa = n.sa; c.ca = 0.f; c.ss = n.ss; c.cs = n.cs;
    c.fa = s.fh; c.fs = 0;
    // the real scale of the sign-bit weights travels in the two spare words
    c.pad[0] = __double2loint(s.sq); c.pad[1] = __double2hiint(s.sq);
    a.out[blockIdx.x] = c;
  }
}

__global__ void __launch_bounds__(256) tstats_kernel(StatArgs a) {
  __shared__ double red[4][8];
  const float* q = a.Qcat + (int64_t)blockIdx.x * a.ldq;
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
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    red[0][warp] = mx1; red[1][warp] = sm1; red[2][warp] = mx2; red[3][warp] = sm2;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) {
      mx1 = fmax(mx1, red[0][w]); sm1 += red[1][w];
      mx2 = fmax(mx2, red[2][w]); sm2 += red[3][w];
    }
    // |W| < 2^e with W = 2 alpha q'  ->  |W| 2^(22-e) < 2^22: three signed radix-256 digits hold it.  The same
    // exponent as in the register-fed scan, so that both engines form identical integers and estimates.
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
    a.out[blockIdx.x] = c;
  }
}

// ------------------------------------------------------------------ B matrices
// Ba[pass*96 + n][kba*128], Bs[pass*96 + n][kbs*128], n = 32 * digit + (query in pass); K-major int8.
// Byte kappa of a k-block = (2 wl + k / 4) * 16 + (k % 4) * 4 + i  <->  bit 8 i + k of word wl: the order in
// which the transform threads lay out their registers.
struct BPrepArgs {
  const float* Qcat;
  int64_t ldq;
  const QConst* qc;
  int nqg;
  Geo g;
  double alpha[8];
  uint8_t* Ba;
  uint8_t* Bs;
};

__device__ __forceinline__ int digit_of(long long J, int limb) {
  int dg = 0;
  for (int l = 0; l <= limb; ++l) {
    dg = (int)(((J + 128) & 255) - 128);
    J = (J - dg) >> 8;
  }
  return dg;
}

__global__ void __launch_bounds__(256) tbprep_kernel(BPrepArgs a, int part, int rows) {
  const int nkb = part ? a.g.kbs : a.g.kba;
  const int64_t total = (int64_t)rows * nkb * 4;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (tid >= total) return;
  const int wl = (int)(tid & 3);
  const int kb = (int)((tid >> 2) % nkb);
  const int row = (int)((tid >> 2) / nkb);      // pass * 96 + n
  const int ql = (row / NCOL) * kQueriesPerPass + (row % NCOL) % kQueriesPerPass, limb = (row % NCOL) / kQueriesPerPass;
  uint32_t out[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
  if (ql < a.nqg) {
    const float* q = a.Qcat + (int64_t)ql * a.ldq;
    const QConst c = a.qc[ql];
    for (int k = 0; k < 8; ++k) {
      for (int i = 0; i < 4; ++i) {
        const int bit = 8 * i + k;
        double W = 0.0;
        int f;
        if (!part) {
          const Slot s = slot_a(a.g, kb, wl, bit);
          if (s.coord < a.g.d) W = 2.0 * a.alpha[s.term] * (double)q[s.coord];
          f = c.fa;
        } else {
          const int j = 32 * (4 * kb + wl) + bit;
          if (j < a.g.d) W = 2.0 * (double)q[a.g.dpad + j];
          f = c.fs;
        }
        double Jd = rint(ldexp(W, f - k));
        if (!(fabs(Jd) <= 8388608.0)) Jd = 0.0;   // non-finite query entries contribute nothing
        out[k] |= (uint32_t)(digit_of((long long)Jd, limb) & 255) << (8 * i);
      }
    }
  }
  uint8_t* dst = (part ? a.Bs : a.Ba) + (size_t)row * nkb * KB_BYTES + (size_t)kb * KB_BYTES + wl * 32;
  *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
  *reinterpret_cast<uint4*>(dst + 16) = make_uint4(out[4], out[5], out[6], out[7]);
}

// Nibble layout: one B matrix Bn[pass*96 + n][3 nblk * 128]; k-block 3 b + type of block b.  K-byte kappa of an h or l
// k-block <-> coordinate kappa of the block; of a sign k-block: register kappa / 4 = 2 word + parity, byte i = kappa % 4
// <-> coordinate 8 word + 2 i + parity (low nibbles, parity 0, have the value 8 and carry 16 J; high nibbles 128 and J).
__global__ void __launch_bounds__(256) tbprep_nib_kernel(BPrepArgs a, int rows) {
  const int nkb = a.g.kba;
  const int64_t total = (int64_t)rows * nkb * 4;
  const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (tid >= total) return;
  const int wl = (int)(tid & 3);
  const int kb = (int)((tid >> 2) % nkb);
  const int row = (int)((tid >> 2) / nkb);      // pass * 96 + n
  const int ql = (row / NCOL) * kQueriesPerPass + (row % NCOL) % kQueriesPerPass, limb = (row % NCOL) / kQueriesPerPass;
  const int b = kb / 3, type = kb % 3;
  uint32_t out[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
  if (ql < a.nqg) {
    const float* q = a.Qcat + (int64_t)ql * a.ldq;
    const QConst c = a.qc[ql];
    nib::QScale sc;
    sc.fh = c.fa;
    sc.sq = __hiloint2double(c.pad[1], c.pad[0]);
    for (int r = 0; r < 8; ++r)
      for (int i = 0; i < 4; ++i) {
        const int kappa = 32 * wl + 4 * r + i;
        int cib, mul = 1;
        if (type < 2) {
          cib = kappa;
        } else {
          const int reg = kappa >> 2;
          cib = 8 * (reg >> 1) + 2 * i + (reg & 1);
          mul = (reg & 1) ? 1 : 16;
        }
        const int coord = nib::coord_of_block(a.g.nbi, a.g.idx_rb, a.g.qjl_rb, a.g.d, b, cib);
        if (coord < 0) continue;
        const long long J = mul * nib::weight(sc, type, q[(type < 2 ? 0 : a.g.dpad) + coord]);
        out[r] |= (uint32_t)(nib::digit_of(J, limb) & 255) << (8 * i);
      }
  }
  uint8_t* dst = a.Ba + (size_t)row * nkb * KB_BYTES + (size_t)kb * KB_BYTES + wl * 32;
  *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
  *reinterpret_cast<uint4*>(dst + 16) = make_uint4(out[4], out[5], out[6], out[7]);
}

// ------------------------------------------------------------------ scan kernel
struct ScanArgs {
  int64_t n, npairs;
  uint32_t hi_a, hi_b, lo_a, lo_b;   // nibble layout: the 16-bit centroid table as bytes (h of entries 0..3, 4..7; l alike)
  Geo g;
  int pass, nqp;
  const QConst* qc;        // constants of this pass's queries
  const uint8_t* idx;
  size_t idx_rb;
  const uint8_t* qjl;
  size_t qjl_rb;
  const float* gamma;
  const float* norms;
  float coef;
  float* scores;
  int64_t lds;
  const float* tau;
  int* count;
  float* cand_s;
  int* cand_i;
  int cap;
  const int* run_if;
  int* status;
};

// D[tmem] (+)= A[tmem] * B[smem]^T: A is taken from TMEM (row = lane, 4 K-bytes per 32-bit column).
__device__ __forceinline__ void umma_i8_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same over a CTA pair (M = 256: the leader's thread issues for both CTAs, each CTA holds its own rows of A and D in
// TMEM and half of B's rows in shared memory).
__device__ __forceinline__ void umma_i8_ts_pair(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// kind::i8: D = s32, A = unsigned 8-bit, B = signed 8-bit, both K-major.
__host__ __device__ constexpr uint32_t idesc_i8(int M, int N, bool a_signed = false) {
  return (2u << 4) | ((a_signed ? 1u : 0u) << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

template <int BM, int MODE, bool NIB = false>
__global__ void __launch_bounds__(NTHREADS, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap tmBa, const __grid_constant__ CUtensorMap tmBs,
               const __grid_constant__ CUtensorMap tmPa, const __grid_constant__ CUtensorMap tmPs, ScanArgs a) {
  if (a.run_if != nullptr && *a.run_if == 0) return;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* bring = smem;
  unsigned char* pring = smem + B_STAGES * BTILE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(pring + P_STAGES * PTILE_BYTES);
  uint64_t* afull = bars;                           // [A_SLOTS]   transform warps -> MMA
  uint64_t* bfull = afull + A_SLOTS;                // [B_STAGES]  TMA -> MMA
  // One tcgen05.commit per k-block: the issuing thread pays ~350 cycles per commit (measured), so the release
  // of the A slot (2 k-blocks later) and of the B stage (8 k-blocks later) share one ring of barriers.
  uint64_t* kdone = bfull + B_STAGES;               // [B_STAGES]  MMAs of k-block f complete
  uint64_t* pfull = kdone + B_STAGES;               // [P_STAGES]  TMA (packed rows) -> transform warps
  uint64_t* pempty = pfull + P_STAGES;              // [P_STAGES]  transform warps -> TMA producer
  uint64_t* dfull = pempty + P_STAGES;              // accumulators complete -> epilogue
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dfull + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  QConst* qcs = reinterpret_cast<QConst*>(dfull + 4);
  float* taus = reinterpret_cast<float*>(qcs + kQueriesPerPass);   // [32] admission thresholds (filter mode)
  // Filter mode: admitted pairs are collected per CTA and appended to the global lists in one piece per query at
  // the end: one atomic per (CTA, query) instead of one per pair on 32 contended counters.
  int* lcnt = reinterpret_cast<int*>(taus + kQueriesPerPass);       // [32]
  uint2* lbuf = reinterpret_cast<uint2*>(lcnt + kQueriesPerPass);   // [32][LBUF] (score bits, row)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb_total = a.g.kba + a.g.kbs;

  if (threadIdx.x == 0) {
    for (int s = 0; s < A_SLOTS; ++s) tc::mbar_init(&afull[s], 8);
    for (int s = 0; s < B_STAGES; ++s) {
      tc::mbar_init(&bfull[s], 1);
      tc::mbar_init(&kdone[s], 1);
    }
    for (int s = 0; s < P_STAGES; ++s) {
      tc::mbar_init(&pfull[s], 1);
      tc::mbar_init(&pempty[s], 8);
    }
    tc::mbar_init(dfull, N_ISSUERS);
    *abort_flag = 0;
    tc::fence_barrier_init();
    if (a.g.kba > 0) tc::tma_prefetch_desc(&tmBa);
    if (a.g.kbs > 0) tc::tma_prefetch_desc(&tmBs);
    if (a.g.kba > 0) tc::tma_prefetch_desc(&tmPa);
    if (a.g.kbs > 0) tc::tma_prefetch_desc(&tmPs);
  }
  if (threadIdx.x < kQueriesPerPass) {
    QConst c = {1.f, 0.f, 1.f, 0.f, 0, 0, {0, 0}};
    if ((int)threadIdx.x < a.nqp) c = a.qc[threadIdx.x];
    qcs[threadIdx.x] = c;
    taus[threadIdx.x] = (MODE == 1 && (int)threadIdx.x < a.nqp) ? a.tau[threadIdx.x] : 0.f;
    lcnt[threadIdx.x] = 0;
  }
  if (warp == 1) tc::tmem_alloc(tmem_slot, TMEM_COLS);
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer of B
    if (lane == 0) {
      int stage = 0, pstage = 0;
      uint32_t phase = 0, pphase = 0;
      bool ok = true;
      long long kc = 0;   // k-blocks issued so far by this CTA
      for (int64_t pair = blockIdx.x; pair < a.npairs && ok; pair += gridDim.x) {
        for (int f = 0; f < nkb_total; ++f, ++kc) {
          const bool part_s = f >= a.g.kba;
          const int kb = part_s ? f - a.g.kba : f;
          if (NIB ? (kb % 3 == 0) : ((kb & 3) == 0)) {   // the packed rows of the pair for the next group of k-blocks
            if (!(ok = tc::mbar_wait(&pempty[pstage], pphase ^ 1u, abort_flag, a.status))) break;
            const int gb = (part_s || NIB) ? 64 : group_bytes(BM);
            tc::mbar_arrive_expect_tx(&pfull[pstage], (uint32_t)(2 * TILE * gb));
            if (NIB) {   // block kb / 3 of the combined row: from the idx rows, then from the qjl rows
              const int b = kb / 3;
              tc::tma_load_2d(pring + pstage * PTILE_BYTES, b < a.g.nbi ? &tmPa : &tmPs, &pfull[pstage],
                              64 * (b < a.g.nbi ? b : b - a.g.nbi), (int)(pair * (2 * TILE)));
            } else {
              tc::tma_load_2d(pring + pstage * PTILE_BYTES, part_s ? &tmPs : &tmPa, &pfull[pstage], (kb >> 2) * gb,
                              (int)(pair * (2 * TILE)));
            }
            if (++pstage == P_STAGES) {
              pstage = 0;
              pphase ^= 1u;
            }
          }
          // B stage kc % B_STAGES was last read by the MMAs of k-block kc - B_STAGES
          if (kc >= B_STAGES && !(ok = tc::mbar_wait(&kdone[stage], phase ^ 1u, abort_flag, a.status))) break;
          tc::mbar_arrive_expect_tx(&bfull[stage], BTILE_BYTES);
          tc::tma_load_2d(bring + stage * BTILE_BYTES, part_s ? &tmBs : &tmBa, &bfull[stage], kb * KB_BYTES, a.pass * NCOL);
          if (++stage == B_STAGES) {
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
  } else if (warp <= N_ISSUERS) {
    // ---------------------------------------------------------------- MMA issuers
    // The k-blocks are dealt in turn to the issuing warps: 8 MMAs (4 per tile) + one commit each.  The
    // accumulators are zeroed by the transform warps, every MMA accumulates, and integer sums do not depend
    // on the order in which the k-blocks of different threads reach the tensor pipe.
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_i8(TILE, NCOL);
      const int me = warp - 1;
      bool ok = true;
      uint32_t kc = 0;    // k-blocks of this CTA so far
      int turn = 0;       // whose k-block comes next
      const uint64_t bdesc0 = tc::smem_desc_sw128(tc::smem_u32(bring));
      for (int64_t pair = blockIdx.x; pair < a.npairs && ok; pair += gridDim.x) {
        for (int f = 0; f < nkb_total; ++f, ++kc) {
          const bool mine = turn == me;
          if (++turn == N_ISSUERS) turn = 0;
          if (!mine) continue;
          const uint32_t bstage = kc & (B_STAGES - 1), stage = kc & (A_SLOTS - 1);
          if (!(ok = tc::mbar_wait(&bfull[bstage], (kc / B_STAGES) & 1u, abort_flag, a.status))) break;
          if (!(ok = tc::mbar_wait(&afull[stage], (kc / A_SLOTS) & 1u, abort_flag, a.status))) break;
          tc::tc_fence_after();
          // nibble layout: k-blocks of h bytes (signed A), l bytes and sign bits in turn; the sign bits have the
          // second accumulator
          const int kind = NIB ? f % 3 : 0;
          const bool part_s = NIB ? kind == 2 : f >= a.g.kba;
          const uint32_t idesc_f = (NIB && kind == 0) ? idesc_i8(TILE, NCOL, true) : idesc;
          const uint64_t bdesc = bdesc0 + (uint64_t)(bstage * (BTILE_BYTES >> 4));
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const uint32_t a_tmem = tmem_base + (uint32_t)(A_COL0 + t * (A_SLOTS * 32) + stage * 32);
            const uint32_t d_tmem = tmem_base + (uint32_t)(t * D_COLS + (part_s ? NCOL : 0));
#pragma unroll
            for (int step = 0; step < 4; ++step)   // 32 K-bytes per MMA: 8 TMEM columns of A, +32 bytes inside B's swizzled row
              umma_i8_ts(d_tmem, a_tmem + 8 * step, bdesc + 2 * step, idesc_f, 1u);
          }
          tc::umma_commit(&kdone[bstage]);   // A slot and B stage reusable once these MMAs have read them
        }
        if (ok) tc::umma_commit(dfull);   // all MMAs this thread issued for the pair
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- transform + epilogue (thread = vector row)
    const int e = warp - 1 - N_ISSUERS;
    const int t = e >> 2;                   // which tile of the pair
    const int quad = warp & 3;              // TMEM lane group this warp may access
    const int r = quad * 32 + lane;         // row inside the tile
    int stage = 0, pstage_keep = 0;
    uint32_t pphase_keep = 0;
    uint32_t kt = 0;    // k-blocks expanded so far by this warp
    bool ok = true;
    int64_t it = 0;
    // the row's scalars are requested one pair ahead, so that their latency hides behind a pair's k-blocks
    auto load_nu = [&](int64_t pr) -> float {
      const int64_t rw = pr * (2 * TILE) + t * TILE + r;
      return (pr < a.npairs && rw < a.n && a.norms != nullptr) ? __ldg(a.norms + rw) : 1.f;
    };
    auto load_gm = [&](int64_t pr) -> float {
      const int64_t rw = pr * (2 * TILE) + t * TILE + r;
      return (pr < a.npairs && rw < a.n && (a.g.kbs > 0 || NIB)) ? __ldg(a.gamma + rw) : 0.f;   // times coef where it is used, so that nothing waits for the load here
    };
    float nu_next = load_nu(blockIdx.x), gm_next = load_gm(blockIdx.x);
    for (int64_t pair = blockIdx.x; pair < a.npairs && ok; pair += gridDim.x, ++it) {
      const int64_t row = pair * (2 * TILE) + t * TILE + r;
      const bool row_ok = row < a.n;
      const float nu = nu_next, gm = gm_next;
      nu_next = load_nu(pair + gridDim.x);
      gm_next = load_gm(pair + gridDim.x);

      // this row's accumulators start from zero (the previous pair's epilogue, by this same thread, has read
      // them; the stores complete before the row's first A tile is announced)
#pragma unroll
      for (int c = 0; c < D_COLS; c += 16) tc::tmem_fill16(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(t * D_COLS + c), 0u);

      // stores one k-block's 32 A registers of this row into the current A slot and announces it
      auto store_a = [&](const uint32_t (&v)[32]) -> bool {
        // A slot kt % 2 was last read by the MMAs of k-block kt - 2: completion number (kt - 2) / B_STAGES of its barrier
        if (kt >= A_SLOTS) {
          const uint32_t kp = kt - A_SLOTS;
          if (!tc::mbar_wait(&kdone[kp & (B_STAGES - 1)], (kp / B_STAGES) & 1u, abort_flag, a.status)) return false;
        }
        tc::tc_fence_after();
        tc::tmem_st32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(A_COL0 + t * (A_SLOTS * 32) + stage * 32), v);
        tc::tmem_st_wait();
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&afull[stage]);
        if (++stage == A_SLOTS) stage = 0;
        ++kt;
        return true;
      };
      // expands one k-block's words into the row's 128 bytes of the A tile of the current stage
      auto emit = [&](uint32_t (&w)[4], int f) -> bool {
        if (f >= nkb_total) return true;
        if (f < a.g.kba) {
          if (BM == 3) {
            const uint32_t p0 = w[0] ^ __funnelshift_r(w[0], w[1], 1) ^ __funnelshift_r(w[0], w[1], 2);
            const uint32_t p1 = w[1] ^ __funnelshift_r(w[1], w[2], 1) ^ __funnelshift_r(w[1], w[2], 2);
            const uint32_t p2 = w[2] ^ (w[2] >> 1) ^ (w[2] >> 2);
            w[3] = (p0 & 0x49249249u) | (p1 & 0x92492492u) | (p2 & 0x24924924u);
          } else if (BM == 4) {
            const uint32_t M = 0x11111111u;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              const uint32_t x = w[i], s1 = x >> 1, s2 = x >> 2, s3 = x >> 3;
              w[2 + i] = ((x ^ s1 ^ s2) & M) | (((x ^ s1 ^ s3) & M) << 1) | (((x ^ s2 ^ s3) & M) << 2) | (((s1 ^ s2 ^ s3) & M) << 3);
            }
          }
        }
        // the row's 128 A bytes of this k-block: register 4 c + e = (word c / 2, bit 4 (c % 2) + e of every byte)
        uint32_t v[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t x = w[c >> 1];
          const int k0 = (c & 1) * 4;
#pragma unroll
          for (int e2 = 0; e2 < 4; ++e2) v[4 * c + e2] = x & (0x01010101u << (k0 + e2));
        }
        return store_a(v);
      };
      // groups of four k-blocks: the pair's packed rows arrive by TMA ([256 rows x group bytes], swizzled so that
      // row-per-thread 16-byte reads are conflict-free); the thread copies its row's bytes to registers, frees the
      // stage and expands the four k-blocks
      const int prow = t * TILE + r;   // row inside the pair
      int pstage = pstage_keep;
      uint32_t pphase = pphase_keep;
      if (NIB) {
        // nibble layout: a group is one 64-byte block of the combined row = 16 code words = 128 coordinates, expanded
        // into three k-blocks: h bytes and l bytes by byte permutes with the masked word as selector, sign bits by masks
        for (int f0 = 0; f0 < nkb_total && ok; f0 += 3) {
          if (!(ok = tc::mbar_wait(&pfull[pstage], pphase, abort_flag, a.status))) break;
          const unsigned char* ps = pring + pstage * PTILE_BYTES;
          uint32_t x[16];
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // 64 bytes per row, 64-byte swizzle: chunk c at c ^ ((row >> 1) & 3)
            const uint4 v4 = *reinterpret_cast<const uint4*>(ps + prow * 64 + ((j ^ ((prow >> 1) & 3)) << 4));
            x[4 * j] = v4.x; x[4 * j + 1] = v4.y; x[4 * j + 2] = v4.z; x[4 * j + 3] = v4.w;
          }
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&pempty[pstage]);
          if (++pstage == P_STAGES) {
            pstage = 0;
            pphase ^= 1u;
          }
          uint32_t v[32];
#pragma unroll
          for (int wd = 0; wd < 16; ++wd) {
            const uint32_t sl = x[wd] & 0x77777777u;
            v[2 * wd] = prmt(a.hi_a, a.hi_b, sl);
            v[2 * wd + 1] = prmt(a.hi_a, a.hi_b, sl >> 16);
          }
          ok = ok && store_a(v);
#pragma unroll
          for (int wd = 0; wd < 16; ++wd) {
            const uint32_t sl = x[wd] & 0x77777777u;
            v[2 * wd] = prmt(a.lo_a, a.lo_b, sl);
            v[2 * wd + 1] = prmt(a.lo_a, a.lo_b, sl >> 16);
          }
          ok = ok && store_a(v);
#pragma unroll
          for (int wd = 0; wd < 16; ++wd) {
            v[2 * wd] = x[wd] & 0x08080808u;
            v[2 * wd + 1] = x[wd] & 0x80808080u;
          }
          ok = ok && store_a(v);
        }
      }
      for (int f0 = 0; !NIB && f0 < nkb_total && ok; f0 += 4) {
        // a part boundary inside a group cannot happen: each part starts a new group
        const bool part_s = f0 >= a.g.kba;
        if (!(ok = tc::mbar_wait(&pfull[pstage], pphase, abort_flag, a.status))) break;
        const unsigned char* ps = pring + pstage * PTILE_BYTES;
        uint32_t w[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j][0] = w[j][1] = w[j][2] = w[j][3] = 0u;
        if (part_s || BM <= 2) {           // 64 bytes per row, 64-byte swizzle: chunk c at c ^ ((row >> 1) & 3)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint4 v = *reinterpret_cast<const uint4*>(ps + prow * 64 + ((j ^ ((prow >> 1) & 3)) << 4));
            w[j][0] = v.x; w[j][1] = v.y; w[j][2] = v.z; w[j][3] = v.w;
          }
        } else if (BM == 3) {              // 48 bytes per row, plain: three words per k-block
          uint32_t x[12];
#pragma unroll
          for (int j = 0; j < 3; ++j) {
            const uint4 v = *reinterpret_cast<const uint4*>(ps + prow * 48 + j * 16);
            x[4 * j] = v.x; x[4 * j + 1] = v.y; x[4 * j + 2] = v.z; x[4 * j + 3] = v.w;
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            w[j][0] = x[3 * j]; w[j][1] = x[3 * j + 1]; w[j][2] = x[3 * j + 2];
          }
        } else {                           // b_m = 4: 32 bytes per row, 32-byte swizzle: chunk c at c ^ ((row >> 2) & 1)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const uint4 v = *reinterpret_cast<const uint4*>(ps + prow * 32 + ((j ^ ((prow >> 2) & 1)) << 4));
            w[2 * j][0] = v.x; w[2 * j][1] = v.y; w[2 * j + 1][0] = v.z; w[2 * j + 1][1] = v.w;
          }
        }
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&pempty[pstage]);
        if (++pstage == P_STAGES) {
          pstage = 0;
          pphase ^= 1u;
        }
        const int fend = part_s ? nkb_total : a.g.kba;   // k-blocks of this part end here
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if (f0 + j < fend) ok = ok && emit(w[j], f0 + j);
        if (!part_s && f0 + 4 >= a.g.kba) f0 = a.g.kba - 4;   // the next group starts the QJL part
      }
      pstage_keep = pstage;
      pphase_keep = pphase;
      if (!ok) break;

      // ---- epilogue: this thread's row of the four accumulators
      if (!(ok = tc::mbar_wait(dfull, (uint32_t)(it & 1), abort_flag, a.status))) break;
      tc::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(t * D_COLS);
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {   // 16 queries per half: digit l of query 16 h + qq sits in column 32 l + 16 h + qq
        if (h * 16 >= a.nqp) break;   // a short last pass: columns of absent queries are not read
        uint32_t va[LIMBS][16], vs[LIMBS][16];
#pragma unroll
        for (int l = 0; l < LIMBS; ++l) {
          if (a.g.kba > 0) tc::tmem_ld16(taddr + l * 32 + h * 16, va[l]);
          if (a.g.kbs > 0 || NIB) tc::tmem_ld16(taddr + NCOL + l * 32 + h * 16, vs[l]);
        }
        tc::tmem_ld_wait();
#pragma unroll
        for (int qq = 0; qq < 16; ++qq) {
          const int ql = h * 16 + qq;
          if (ql >= a.nqp) break;
          // digits recombined exactly (64-bit integer: the same T as in the register-fed engine), then fp32
          const QConst c = qcs[ql];
          float av = 0.f, sv = 0.f;
          if (a.g.kba > 0) {
            const long long T = ((long long)(int)va[2][qq] * 256 + (int)va[1][qq]) * 256 + (int)va[0][qq];
            av = fmaf((float)T, c.sa, c.ca);
          }
          if (a.g.kbs > 0 || NIB) {
            const long long T = ((long long)(int)vs[2][qq] * 256 + (int)vs[1][qq]) * 256 + (int)vs[0][qq];
            sv = fmaf((float)T, c.ss, c.cs);
          }
          const float est = __fmul_rn(nu, fmaf(__fmul_rn(a.coef, gm), sv, av));
          if (row_ok && ql < a.nqp) {
            if (MODE == 0) {
              if (TQ_DEVICE_CHECK(row >= 0 && row < a.n && row < a.lds, a.status)) a.scores[(int64_t)ql * a.lds + row] = est;
            } else if (est >= taus[ql]) {
              const int ls = atomicAdd(&lcnt[ql], 1);
              if (ls < LBUF) {
                lbuf[ql * LBUF + ls] = make_uint2(__float_as_uint(est), (uint32_t)row);
              } else {   // the CTA's buffer is full: straight to the global list
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
      tc::tc_fence_before();
    }
  }

  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (MODE == 1 && warp > N_ISSUERS) {   // the eight transform warps append four queries' collected pairs each
    for (int ql = (warp - 1 - N_ISSUERS) * 4; ql < (warp - N_ISSUERS) * 4; ++ql) {
      const int m = min(lcnt[ql], LBUF);
      if (m == 0 || ql >= a.nqp) continue;
      int base = 0;
      if (lane == 0) base = atomicAdd(a.count + ql, m);
      base = __shfl_sync(0xffffffffu, base, 0);
      for (int i = lane; i < m; i += 32) {
        const int slot = base + i;
        if (slot < a.cap) {
          const uint2 e = lbuf[ql * LBUF + i];
          a.cand_s[(int64_t)ql * a.cap + slot] = __uint_as_float(e.x);
          a.cand_i[(int64_t)ql * a.cap + slot] = (int)e.y;
        }
      }
    }
  }
}

// at least 120 KB so that a second CTA can never share the SM (the kernel allocates all of TMEM)
#include "tq_scan_tcw.cuh"

constexpr size_t kSmemUsed = B_STAGES * BTILE_BYTES + P_STAGES * PTILE_BYTES + 1024 + 512 + kQueriesPerPass * (sizeof(QConst) + sizeof(float) + sizeof(int) + LBUF * sizeof(uint2));
constexpr size_t kSmemBytes = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;

template <int BM, int MODE, bool NIB = false>
cudaError_t launch_t(const CUtensorMap& ma, const CUtensorMap& ms, const CUtensorMap& pa, const CUtensorMap& ps,
                     const ScanArgs& args, cudaStream_t st) {
  auto kern = scan_tc_kernel<BM, MODE, NIB>;
  // function attributes are per device: remember the devices this launcher has prepared
  static std::atomic<unsigned long long> attr_devices{0};   // written by any thread that launches
  int attr_dev = 0;
  if (cudaGetDevice(&attr_dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (attr_dev >= 64 || !((attr_devices.load(std::memory_order_relaxed) >> attr_dev) & 1ull)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    if (attr_dev < 64) attr_devices.fetch_or(1ull << attr_dev, std::memory_order_relaxed);
  }
  const int grid = (int)std::min<int64_t>(args.npairs, tc::sm_count());
  kern<<<grid, NTHREADS, kSmemBytes, st>>>(ma, ms, pa, ps, args);
  count_launches(1);
  return cudaGetLastError();
}

template <int BM, int MODE, bool NIB, int CTAS>
cudaError_t launch_wide_c(const CUtensorMap& ma, const CUtensorMap& ms, const CUtensorMap& pa, const CUtensorMap& ps,
                          const ScanArgs& args, cudaStream_t st) {
  auto kern = scan_tcw_kernel<BM, MODE, NIB, CTAS>;
  static std::atomic<unsigned long long> attr_devices{0};
  int attr_dev = 0;
  if (cudaGetDevice(&attr_dev) != cudaSuccess) return cudaErrorInvalidDevice;
  if (attr_dev >= 64 || !((attr_devices.load(std::memory_order_relaxed) >> attr_dev) & 1ull)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWideSmemBytes);
    if (e != cudaSuccess) return e;
    if (attr_dev < 64) attr_devices.fetch_or(1ull << attr_dev, std::memory_order_relaxed);
  }
  count_launches(1);
  const int64_t ntiles = (args.n + TILE - 1) / TILE;
  if (CTAS == 1) {
    kern<<<(int)std::min<int64_t>(ntiles, tc::sm_count()), W_NTHREADS, kWideSmemBytes, st>>>(ma, ms, pa, ps, args);
    return cudaGetLastError();
  }
  const int units = (int)std::min<int64_t>((ntiles + CTAS - 1) / CTAS, tc::sm_count() / CTAS);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(units * CTAS));
  cfg.blockDim = dim3(W_NTHREADS);
  cfg.dynamicSmemBytes = kWideSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, ma, ms, pa, ps, args);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// pairs = true: ma / ms are the B maps with boxes of half the rows
template <int BM, int MODE, bool NIB = false>
cudaError_t launch_wide_t(bool pairs, const CUtensorMap& ma, const CUtensorMap& ms, const CUtensorMap& pa, const CUtensorMap& ps,
                          const ScanArgs& args, cudaStream_t st) {
  return pairs ? launch_wide_c<BM, MODE, NIB, 2>(ma, ms, pa, ps, args, st) : launch_wide_c<BM, MODE, NIB, 1>(ma, ms, pa, ps, args, st);
}

template <int MODE>
cudaError_t launch_wide(int bm, bool pairs, const CUtensorMap& ma, const CUtensorMap& ms, const CUtensorMap& pa, const CUtensorMap& ps,
                        const ScanArgs& args, cudaStream_t st) {
  if (args.g.nib) return launch_wide_t<3, MODE, true>(pairs, ma, ms, pa, ps, args, st);
  switch (bm) {
    case 0: return launch_wide_t<0, MODE>(pairs, ma, ms, pa, ps, args, st);
    case 1: return launch_wide_t<1, MODE>(pairs, ma, ms, pa, ps, args, st);
    case 2: return launch_wide_t<2, MODE>(pairs, ma, ms, pa, ps, args, st);
    case 3: return launch_wide_t<3, MODE>(pairs, ma, ms, pa, ps, args, st);
    default: return launch_wide_t<4, MODE>(pairs, ma, ms, pa, ps, args, st);
  }
}

template <int MODE>
cudaError_t launch_bm(int bm, const CUtensorMap& ma, const CUtensorMap& ms, const CUtensorMap& pa, const CUtensorMap& ps,
                      const ScanArgs& args, cudaStream_t st) {
  if (args.g.nib) return launch_t<3, MODE, true>(ma, ms, pa, ps, args, st);
  switch (bm) {
    case 0: return launch_t<0, MODE>(ma, ms, pa, ps, args, st);
    case 1: return launch_t<1, MODE>(ma, ms, pa, ps, args, st);
    case 2: return launch_t<2, MODE>(ma, ms, pa, ps, args, st);
    case 3: return launch_t<3, MODE>(ma, ms, pa, ps, args, st);
    default: return launch_t<4, MODE>(ma, ms, pa, ps, args, st);
  }
}

size_t b_bytes(const Geo& g, int part) {
  return (size_t)kPassesPerGroup * NCOL * (part ? g.kbs : g.kba) * KB_BYTES;
}

}  // namespace

bool available(const tq_plan* plan) { return plan->ms.ok != 0; }

// The wide form can be switched off (TQ_SCAN_WIDE=0) to compare the two kernels on one machine.
int queries_per_pass(int nq) {
  static const bool wide = [] {
    const char* e = std::getenv("TQ_SCAN_WIDE");
    return e == nullptr || e[0] != '0';
  }();
  return wide && nq > kQueriesPerPass ? W_QPP : kQueriesPerPass;
}

size_t workspace_bytes(const tq_plan* plan) {
  if (!available(plan)) return 0;
  const Geo g = make_geo(plan);
  return kConstBytes + b_bytes(g, 0) + b_bytes(g, 1);
}

int prepare_group(const tq_plan* plan, const float* Qcat, int nqg, void* workspace, cudaStream_t st, const char* who) {
  const Geo g = make_geo(plan);
  const int ncols = plan->ncat * plan->dpad;
  QConst* qc = static_cast<QConst*>(workspace);
  uint8_t* Ba = static_cast<uint8_t*>(workspace) + kConstBytes;
  uint8_t* Bs = Ba + b_bytes(g, 0);
  StatArgs sa;
  sa.Qcat = Qcat;
  sa.ldq = ncols;
  sa.d = plan->d;
  sa.dpad = plan->dpad;
  sa.prod = plan->mode == TQ_PROD ? 1 : 0;
  sa.amax = plan->ms.amax;
  sa.csum = plan->ms.csum;
  sa.nib = g.nib;
  sa.delta = plan->nb.delta;
  sa.out = qc;
  if (g.nib) tstats_nib_kernel<<<nqg, 32, 0, st>>>(sa);
  else tstats_kernel<<<nqg, 256, 0, st>>>(sa);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  BPrepArgs ba;
  ba.Qcat = Qcat;
  ba.ldq = ncols;
  ba.qc = qc;
  ba.nqg = nqg;
  ba.g = g;
  for (int i = 0; i < 8; ++i) ba.alpha[i] = plan->ms.alpha[i];
  ba.Ba = Ba;
  ba.Bs = Bs;
  const int passes = (nqg + kQueriesPerPass - 1) / kQueriesPerPass;
  const int rows = passes * NCOL;
  if (g.nib) {
    const int64_t total = (int64_t)rows * g.kba * 4;
    tbprep_nib_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(ba, rows);
    count_launches(1);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
    return TQ_OK;
  }
  for (int part = 0; part < 2; ++part) {
    const int nkb = part ? g.kbs : g.kba;
    if (nkb == 0) continue;
    const int64_t total = (int64_t)rows * nkb * 4;
    tbprep_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(ba, part, rows);
    count_launches(1);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
  }
  return TQ_OK;
}

int run_pass(const tq_plan* plan, int pass, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
             const float* norms, float* scores, int64_t lds, const mscan::Filter* filter, const int* run_if,
             const void* workspace, cudaStream_t st, const char* who) {
  const Geo g = make_geo(plan);
  const QConst* qc = static_cast<const QConst*>(workspace);
  const uint8_t* Ba = static_cast<const uint8_t*>(workspace) + kConstBytes;
  const uint8_t* Bs = Ba + b_bytes(g, 0);
  // more than 32 queries: the wide kernel takes the B rows of this pass and the next as one box of 192 rows and one
  // 128-vector tile at a time
  const bool wide = nqp > kQueriesPerPass;
  TQ_REQUIRE(nqp <= (wide ? W_QPP : kQueriesPerPass) && (!wide || (pass % 2 == 0 && pass + 2 <= kPassesPerGroup)), TQ_ERR_INVALID_ARG,
             "%s: pass %d of %d queries", who, pass, nqp);
  // The wide kernel runs on CTA pairs wherever there is more than one tile (M = 256, each CTA loads half of a B box's
  // rows into one of twelve half-size stages: measured 316 against 339 us per 32 queries at d = 1536, n = 10^6).
  // TQ_SCAN_PAIRS=0 keeps single CTAs, to compare the two on one machine.
  static const bool pairs_on = [] {
    const char* e = std::getenv("TQ_SCAN_PAIRS");
    return e == nullptr || e[0] != '0';
  }();
  const bool pairs = wide && pairs_on && n > TILE;
  const uint32_t brows = wide ? (pairs ? W_NCOL / 2 : W_NCOL) : NCOL, prows = wide ? TILE : 2 * TILE;
  CUtensorMap ma, ms;
  const uint64_t rows = (uint64_t)kPassesPerGroup * NCOL;
  if (g.kba > 0)
    TQ_REQUIRE(tc::make_byte_map(&ma, Ba, rows, (uint64_t)g.kba * KB_BYTES, (uint64_t)g.kba * KB_BYTES, KB_BYTES, brows, 128),
               TQ_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (B, MSE part)", who);
  if (g.kbs > 0)
    TQ_REQUIRE(tc::make_byte_map(&ms, Bs, rows, (uint64_t)g.kbs * KB_BYTES, (uint64_t)g.kbs * KB_BYTES, KB_BYTES, brows, 128),
               TQ_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (B, QJL part)", who);
  if (g.kba == 0) ma = ms;
  if (g.kbs == 0) ms = ma;
  // packed rows: boxes of [256 rows x group bytes]; 64- and 32-byte boxes are swizzled (row-per-thread reads)
  CUtensorMap pa, ps;
  const int gb = g.nib ? 64 : group_bytes(g.bm);
  if (g.nib) {
    TQ_REQUIRE(tc::make_byte_map(&pa, idx, (uint64_t)n, plan->idx_row_bytes, plan->idx_row_bytes, 64, prows, 64) &&
                   tc::make_byte_map(&ps, qjl, (uint64_t)n, plan->qjl_row_bytes, plan->qjl_row_bytes, 64, prows, 64),
               TQ_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (code rows)", who);
  } else if (g.kba > 0)
    TQ_REQUIRE(tc::make_byte_map(&pa, idx, (uint64_t)n, plan->idx_row_bytes, plan->idx_row_bytes, gb, prows,
                                 gb == 64 ? 64 : gb == 32 ? 32 : 0),
               TQ_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (idx rows)", who);
  if (!g.nib && g.kbs > 0)
    TQ_REQUIRE(tc::make_byte_map(&ps, qjl, (uint64_t)n, plan->qjl_row_bytes, plan->qjl_row_bytes, 64, prows, 64), TQ_ERR_CUDA,
               "%s: cuTensorMapEncodeTiled failed (qjl rows)", who);
  if (!g.nib && g.kba == 0) pa = ps;
  if (!g.nib && g.kbs == 0) ps = pa;
  ScanArgs a;
  a.n = n;
  a.npairs = (n + 2 * TILE - 1) / (2 * TILE);
  a.hi_a = plan->nb.hi_a; a.hi_b = plan->nb.hi_b; a.lo_a = plan->nb.lo_a; a.lo_b = plan->nb.lo_b;
  a.g = g;
  a.pass = pass;
  a.nqp = nqp;
  a.qc = qc + (size_t)pass * kQueriesPerPass;
  a.idx = idx;
  a.idx_rb = plan->idx_row_bytes;
  a.qjl = qjl;
  a.qjl_rb = plan->qjl_row_bytes;
  a.gamma = gamma;
  a.norms = norms;
  a.coef = plan->coef;
  a.scores = scores;
  a.lds = lds;
  a.tau = filter ? filter->tau : nullptr;
  a.count = filter ? filter->count : nullptr;
  a.cand_s = filter ? filter->cand_s : nullptr;
  a.cand_i = filter ? filter->cand_i : nullptr;
  a.cap = filter ? filter->cap : 0;
  a.run_if = run_if;
  a.status = plan->d_status;
  if (wide) TQ_CHECK_CUDA(filter ? launch_wide<1>(g.bm, pairs, ma, ms, pa, ps, a, st) : launch_wide<0>(g.bm, pairs, ma, ms, pa, ps, a, st), who);
  else TQ_CHECK_CUDA(filter ? launch_bm<1>(g.bm, ma, ms, pa, ps, a, st) : launch_bm<0>(g.bm, ma, ms, pa, ps, a, st), who);
  return TQ_OK;
}

}  // namespace tscan
}  // namespace tq

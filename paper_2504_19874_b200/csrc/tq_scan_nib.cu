// Packed-code scan for TQ_LAYOUT_NIBBLE (estimator of Section 3.2 evaluated on the codes of a TQ_PROD plan
// with a 3-bit MSE stage): the centroid of a coordinate is looked up, not expanded.
//
// Layout.  The three index bits and the QJL sign bit of coordinate j share nibble j of one combined row
// (byte j >> 1, bits 4 (j & 1) .. 4 (j & 1) + 3: index in the low three bits, sign bit on top).  The combined
// row is stored across the two arrays the ABI already has: its first tq_idx_row_bytes bytes in the idx row,
// the rest in the qjl row.  Same bytes per vector as the bit-stream layout, an exact permutation of its bits.
//
// Arithmetic.  The codebook is rounded once to 16-bit integers, c_i ~ delta * t_i with t_i = 256 h_i + l_i
// (h signed, l unsigned byte; delta chosen so that all t_i are nearly integers), so that
//     sum_j q'_j c[idx_j]  =  delta * ( 256 sum_j q'_j h[idx_j] + sum_j q'_j l[idx_j] ).
// A byte permute with the masked code word as selector (PRMT: four 3-bit selectors pick four bytes out of an
// eight-byte table) turns four coordinates into four A-operand bytes of the 8-bit integer MMA: one
// instruction per four K-elements and two K-elements per coordinate, against one AND per four K-elements and
// four K-elements per coordinate (three index bits + their parity) in the bit-plane form; the sign bits cost
// one AND per four as before.  That is 9 instead of 15 mma.sync.m16n8k32 per vector at d = 1536, and fewer
// instructions beside them, which is what bounds this scan (it is issue-bound, not HBM-bound).
// The query side holds fixed-point weights as signed radix-256 digits: Wh = round(q' 2^fh) (three digits) for
// the h bytes, Wl = round(q' 2^(fh-8)) (two digits) for the l bytes, J = round(q'' s_q) (two digits; s_q is a
// real scale, so that J uses the whole two-digit range) for the sign bits, whose two bit positions (values 8
// and 128) go to accumulators of their own.  All sums are exact integers, recombined in 64 bits; results do
// not depend on tiling, order or on the queries sharing a pass.
//
// Two shapes of the query-side operand: up to two queries with the digits of a query in neighbouring MMA
// columns (3 MMAs per code word), or up to eight queries with one column per query and one MMA per digit
// (7 MMAs per code word).
#include <algorithm>
#include <cmath>

#include "tq_nib_common.cuh"
#include "tq_quantize_tc.h"
#include "tq_scan_nib.h"
#include "tq_tc.cuh"

namespace tq {
namespace nscan {

namespace {

constexpr int NW = 16;                      // consumer warps
constexpr int VT = NW * 16;                 // vectors per tile
constexpr int BLOCK_BYTES = VT * 64;        // one 64-byte column block of the combined row, all rows of a tile
constexpr int MAX_STAGES = 6;
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr int KPB_COL = 12, KPB_TILE = 28;  // operand elements (uint2) per lane and 64-byte block (two word pairs)
constexpr size_t kQConstBytes = 256;

using NQConst = nib::QConst;
using QScale = nib::QScale;

// Coordinate whose nibble is nibble `nib` (0..7) of code word `wd` (0..3) that quad thread t4 holds of block b
// (thread t4 owns bytes 16 t4 .. 16 t4 + 15 of a block), or -1 when that nibble lies in the zero fill.
__host__ __device__ inline int coord_of(int nbi, int idx_rb, int qjl_rb, int d, int b, int t4, int wd, int nibble) {
  return nib::coord_of_block(nbi, idx_rb, qjl_rb, d, b, 32 * t4 + 8 * wd + nibble);
}

// ------------------------------------------------------------------ query-side operand
struct PrepArgs {
  const float* Qcat;   // rotated queries of this pass: row q at Qcat + q*ldq, [q' | q''] with q'' at dpad
  int64_t ldq;
  NQConst* qc;
  int nq_pass, d, dpad;
  int nbi, idx_rb, qjl_rb, nblocks, tiled;
  double delta;
  uint2* out;          // [nblocks][KPB][32], k-steps 2j and 2j + 1 of a lane side by side
};

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may start while its
// predecessor in the stream still runs; it must pass this wait before touching anything the predecessor
// writes or reads.  launch_dependents lets the successor's CTAs be scheduled as this grid's CTAs drain.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Warp `ql` of every block derives the scales of query ql itself (a few thousand loads from L2, the same
// values in the same order everywhere); block 0 publishes the constants the scan needs.
__device__ void query_scales(const PrepArgs& a, QScale* sc /* shared, [8] */) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < a.nq_pass) {
    const float* q = a.Qcat + (int64_t)warp * a.ldq;
    float mx1 = 0.f, mx2 = 0.f;
    double sm2 = 0.0;
    for (int j = lane; j < a.d; j += 32) {
      mx1 = fmaxf(mx1, fabsf(q[j]));
      const float u = q[a.dpad + j];
      mx2 = fmaxf(mx2, fabsf(u));
      if (blockIdx.x == 0) sm2 += (double)u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
      mx2 = fmaxf(mx2, __shfl_xor_sync(0xffffffffu, mx2, o));
      sm2 += __shfl_xor_sync(0xffffffffu, sm2, o);
    }
    if (lane == 0) {
      const QScale s = nib::make_scale(mx1, mx2);
      sc[warp] = s;
      if (blockIdx.x == 0) a.qc[warp] = nib::make_const(s, a.delta, sm2);
    }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(256) nprep_kernel(PrepArgs a) {
  __shared__ QScale sc[8];
  grid_dependency_wait();   // the rotated queries come from the kernel before; the operand may still be in use
  grid_launch_dependents();
  query_scales(a, sc);
  const int KPB = a.tiled ? KPB_TILE : KPB_COL;
  const int total = a.nblocks * KPB * 32;
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= total) return;
  const int lane = e & 31, ks = (e >> 5) % KPB, b = (e >> 5) / KPB;
  const int g = lane >> 2, t4 = lane & 3;
  int p, type, wsel, digit, ql;   // type 0: h bytes, 1: l bytes, 2: sign bits of value 8, 3: of value 128
  if (a.tiled) {
    p = ks / 14;
    const int slot = ks % 14;
    ql = g;
    if (slot < 10) {
      wsel = slot / 5;
      const int r = slot % 5;
      type = r < 3 ? 0 : 1;
      digit = r < 3 ? r : r - 3;
    } else {
      wsel = 0;
      type = slot < 12 ? 2 : 3;
      digit = slot & 1;
    }
  } else {
    p = ks / 6;
    const int slot = ks % 6;
    ql = g >> 2;
    digit = g & 3;
    if (slot < 4) {
      wsel = slot >> 1;
      type = slot & 1;
    } else {
      wsel = 0;
      type = slot - 2;
    }
    if (digit > (type == 0 ? 2 : 1)) ql = a.nq_pass;   // column unused by this operand
  }
  uint32_t regs[2] = {0u, 0u};
  if (ql < a.nq_pass) {
    const float* q = a.Qcat + (int64_t)ql * a.ldq;
    const QScale qs = sc[ql];
#pragma unroll
    for (int half = 0; half < 2; ++half)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int wd, nib;
        if (type < 2) {
          wd = 2 * p + wsel;
          nib = 4 * half + i;
        } else {
          wd = 2 * p + half;
          nib = 2 * i + (type == 3 ? 1 : 0);
        }
        const int coord = coord_of(a.nbi, a.idx_rb, a.qjl_rb, a.d, b, t4, wd, nib);
        if (coord < 0) continue;
        const long long J = nib::weight(qs, type < 2 ? type : 2, q[(type < 2 ? 0 : a.dpad) + coord]);
        regs[half] |= (uint32_t)(nib::digit_of(J, digit) & 255) << (8 * i);
      }
  }
  a.out[((size_t)b * KPB + (ks & ~1)) * 32 + lane * 2 + (ks & 1)] = make_uint2(regs[0], regs[1]);
}

// ------------------------------------------------------------------ scan kernel
struct ScanArgs {
  int64_t n, ntiles;
  int nsteps, stages;
  int nbi, nblocks;        // 64-byte blocks of the idx row; of the combined sequence
  uint32_t hi_a, hi_b, lo_a, lo_b;   // centroid bytes: entries 0..3 and 4..7 of the h and l tables
  const uint2* Bfrag;
  int bfrag_u2;
  const NQConst* qc;
  int nq_pass;
  const float* gamma;
  const float* norms;      // nullable
  float coef;
  float* scores;
  int64_t lds;
  const float* tau;        // filter mode
  int* count;
  float* cand_s;
  int* cand_i;
  int cap;
  const int* run_if;
  int* status;
};

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_s8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
__device__ __forceinline__ long long shfl_xor_ll(long long v, int m) {
  int lo = (int)(v & 0xffffffffll), hi = (int)(v >> 32);
  lo = __shfl_xor_sync(0xffffffffu, lo, m);
  hi = __shfl_xor_sync(0xffffffffu, hi, m);
  return ((long long)hi << 32) | (unsigned int)lo;
}
// A load that stays where it is written (the compiler would otherwise sink it to its first use, the epilogue).
__device__ __forceinline__ float ldg_now(const float* p) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(32 * NW) : "memory"); }

// TILED 0: up to 2 queries, digits in columns.  TILED 1: up to 8 queries, one MMA per digit.
// MODE 0: dense scores.  MODE 1: thresholded candidate pairs.  SB: 64-byte blocks per pipeline stage.
template <int TILED, int MODE, int SB>
__global__ void __launch_bounds__(32 * (NW + 1), 1)
scan_nib_kernel(const __grid_constant__ CUtensorMap tmIdx, const __grid_constant__ CUtensorMap tmQjl, ScanArgs a) {
  constexpr int KPB = TILED ? KPB_TILE : KPB_COL;
  constexpr int NQP = TILED ? 8 : 2;
  constexpr int NT_T = TILED ? 3 : 2;   // accumulators of the centroid term: digit tiles, or (h, l) kept apart
  constexpr int NT_Q = TILED ? 2 : 1;   // per sign-bit position
  constexpr int STAGE_BYTES = SB * BLOCK_BYTES;

  // the switch may be written by the kernel before this one
  if (a.run_if != nullptr) {
    grid_dependency_wait();
    if (*a.run_if == 0) return;
  }

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* stage_base = smem;
  uint2* Bs = reinterpret_cast<uint2*>(smem + (size_t)a.stages * STAGE_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(Bs) + (size_t)a.bfrag_u2 * 8);
  uint64_t* full = bars;
  uint64_t* empty = bars + MAX_STAGES;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * MAX_STAGES);
  NQConst* qcs = reinterpret_cast<NQConst*>(bars + 2 * MAX_STAGES + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      tc::mbar_init(&full[s], 1);
      tc::mbar_init(&empty[s], NW);
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmIdx);
    tc::tma_prefetch_desc(&tmQjl);
  }
  __syncthreads();

  // This CTA's contiguous range of rows: the 16-row units are dealt evenly, so that every CTA ends with the same
  // fraction of a tile instead of some running a whole tile more than the others (10^6 rows on 148 CTAs: 26.4
  // tiles each instead of 26 or 27: measured 1.3 % faster with two queries, 2.3 % with eight).  Rows of a last, partial tile beyond the range belong to the next CTA.
  const int64_t units = (a.n + 15) / 16;
  const int64_t row_begin = 16 * (units * blockIdx.x / gridDim.x);
  const int64_t row_end = min(a.n, 16 * (units * (blockIdx.x + 1) / gridDim.x));

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    // The codes are inputs of the call: their copies start at once, also while the kernel that builds the
    // query-side operand is still running.
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t rt = row_begin; rt < row_end && ok; rt += VT) {
        const int y = (int)rt;
        for (int s = 0; s < a.nsteps; ++s) {
          if (!(ok = tc::mbar_wait(&empty[stage], phase ^ 1u, abort_flag, a.status))) break;
          unsigned char* sb = stage_base + (size_t)stage * STAGE_BYTES;
          const int b0 = SB * s, nb = min(SB, a.nblocks - b0);
          tc::mbar_arrive_expect_tx(&full[stage], nb * BLOCK_BYTES);
          for (int u = 0; u < nb; ++u) {
            const int b = b0 + u;
            if (b < a.nbi) tc::tma_load_2d(sb + u * BLOCK_BYTES, &tmIdx, &full[stage], 64 * b, y);
            else tc::tma_load_2d(sb + u * BLOCK_BYTES, &tmQjl, &full[stage], 64 * (b - a.nbi), y);
          }
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
  grid_dependency_wait();   // the query-side operand and constants are the previous kernel's output
  {
    const uint4* src = reinterpret_cast<const uint4*>(a.Bfrag);
    uint4* dst = reinterpret_cast<uint4*>(Bs);
    const int ct = threadIdx.x - 32;
    for (int i = ct; i < a.bfrag_u2 / 2; i += 32 * NW) dst[i] = __ldg(src + i);
    if (ct < NQP) {
      NQConst c = {0.f, 0.f, 0.f, 0};
      if (ct < a.nq_pass) c = a.qc[ct];
      qcs[ct] = c;
    }
  }
  consumer_barrier();

  const int cw = warp - 1;
  const int g = lane >> 2, t4 = lane & 3;
  const uint32_t hi_a = a.hi_a, hi_b = a.hi_b, lo_a = a.lo_a, lo_b = a.lo_b;
  const uint32_t lane_off = (uint32_t)((cw * 16 + g) * 64 + t4 * 16);   // this thread's 16 bytes of row g of a block
  int stage = 0;
  uint32_t phase = 0;
  bool ok = true;
  for (int64_t rt = row_begin; rt < row_end && ok; rt += VT) {
    const bool active = rt + cw * 16 < row_end;   // a warp without rows in a partial tile only keeps the pipeline's pace
    int accT[NT_T][4], accQ3[NT_Q][4], accQ7[NT_Q][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int t = 0; t < NT_T; ++t) accT[t][i] = 0;
#pragma unroll
      for (int t = 0; t < NT_Q; ++t) accQ3[t][i] = accQ7[t][i] = 0;
    }
    // per-row scalars of the epilogue, requested now so that their latency hides behind the tile
    float nu_pre[2], gm_pre[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int64_t row = rt + cw * 16 + g + 8 * h;
      nu_pre[h] = (row < row_end && a.norms != nullptr) ? ldg_now(a.norms + row) : 1.f;
      gm_pre[h] = (row < row_end) ? ldg_now(a.gamma + row) : 0.f;
    }

    for (int s = 0; s < a.nsteps; ++s) {
      if (!(ok = tc::mbar_wait(&full[stage], phase, abort_flag, a.status))) break;
      const unsigned char* sb = stage_base + (size_t)stage * STAGE_BYTES + lane_off;
      uint32_t w[2][4 * SB];
      if (active) {
#pragma unroll
        for (int u = 0; u < SB; ++u)
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint4 v = *reinterpret_cast<const uint4*>(sb + u * BLOCK_BYTES + h * 512);
            w[h][4 * u] = v.x; w[h][4 * u + 1] = v.y; w[h][4 * u + 2] = v.z; w[h][4 * u + 3] = v.w;
          }
      }
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&empty[stage]);   // the stage now lives in registers
      if (++stage == a.stages) {
        stage = 0;
        phase ^= 1u;
      }
      if (!active) continue;
      // blocks of the last step that do not exist hold stale bytes; their operand is zero
      const uint4* Bb = reinterpret_cast<const uint4*>(Bs + (size_t)s * (SB * KPB) * 32) + lane;
#pragma unroll
      for (int p = 0; p < 2 * SB; ++p) {
        const uint32_t x0 = w[0][2 * p], x1 = w[1][2 * p], y0 = w[0][2 * p + 1], y1 = w[1][2 * p + 1];
        const uint32_t sx0 = x0 & 0x77777777u, sx1 = x1 & 0x77777777u, sy0 = y0 & 0x77777777u, sy1 = y1 & 0x77777777u;
        const uint32_t tx0 = sx0 >> 16, tx1 = sx1 >> 16, ty0 = sy0 >> 16, ty1 = sy1 >> 16;
        // A operands: h and l bytes of the eight coordinates of a word (rows g, g + 8)
        const uint32_t hx0 = prmt(hi_a, hi_b, sx0), hx1 = prmt(hi_a, hi_b, sx1), hx2 = prmt(hi_a, hi_b, tx0), hx3 = prmt(hi_a, hi_b, tx1);
        const uint32_t lx0 = prmt(lo_a, lo_b, sx0), lx1 = prmt(lo_a, lo_b, sx1), lx2 = prmt(lo_a, lo_b, tx0), lx3 = prmt(lo_a, lo_b, tx1);
        const uint32_t hy0 = prmt(hi_a, hi_b, sy0), hy1 = prmt(hi_a, hi_b, sy1), hy2 = prmt(hi_a, hi_b, ty0), hy3 = prmt(hi_a, hi_b, ty1);
        const uint32_t ly0 = prmt(lo_a, lo_b, sy0), ly1 = prmt(lo_a, lo_b, sy1), ly2 = prmt(lo_a, lo_b, ty0), ly3 = prmt(lo_a, lo_b, ty1);
        // sign bits: value 8 (low nibbles) and value 128 (high nibbles) of both words
        const uint32_t q30 = x0 & 0x08080808u, q31 = x1 & 0x08080808u, q32 = y0 & 0x08080808u, q33 = y1 & 0x08080808u;
        const uint32_t q70 = x0 & 0x80808080u, q71 = x1 & 0x80808080u, q72 = y0 & 0x80808080u, q73 = y1 & 0x80808080u;
        if (TILED) {
          const uint4 v0 = Bb[(7 * p + 0) * 32], v1 = Bb[(7 * p + 1) * 32], v2 = Bb[(7 * p + 2) * 32], v3 = Bb[(7 * p + 3) * 32];
          mma_s8s8(accT[0], hx0, hx1, hx2, hx3, v0.x, v0.y);
          mma_s8s8(accT[1], hx0, hx1, hx2, hx3, v0.z, v0.w);
          mma_s8s8(accT[NT_T - 1], hx0, hx1, hx2, hx3, v1.x, v1.y);
          mma_u8s8(accT[0], lx0, lx1, lx2, lx3, v1.z, v1.w);
          mma_u8s8(accT[1], lx0, lx1, lx2, lx3, v2.x, v2.y);
          const uint4 v4 = Bb[(7 * p + 4) * 32], v5 = Bb[(7 * p + 5) * 32], v6 = Bb[(7 * p + 6) * 32];
          mma_s8s8(accT[0], hy0, hy1, hy2, hy3, v2.z, v2.w);
          mma_s8s8(accT[1], hy0, hy1, hy2, hy3, v3.x, v3.y);
          mma_s8s8(accT[NT_T - 1], hy0, hy1, hy2, hy3, v3.z, v3.w);
          mma_u8s8(accT[0], ly0, ly1, ly2, ly3, v4.x, v4.y);
          mma_u8s8(accT[1], ly0, ly1, ly2, ly3, v4.z, v4.w);
          mma_u8s8(accQ3[0], q30, q31, q32, q33, v5.x, v5.y);
          mma_u8s8(accQ3[NT_Q - 1], q30, q31, q32, q33, v5.z, v5.w);
          mma_u8s8(accQ7[0], q70, q71, q72, q73, v6.x, v6.y);
          mma_u8s8(accQ7[NT_Q - 1], q70, q71, q72, q73, v6.z, v6.w);
        } else {
          const uint4 v0 = Bb[(3 * p + 0) * 32], v1 = Bb[(3 * p + 1) * 32], v2 = Bb[(3 * p + 2) * 32];
          mma_s8s8(accT[0], hx0, hx1, hx2, hx3, v0.x, v0.y);
          mma_u8s8(accT[1], lx0, lx1, lx2, lx3, v0.z, v0.w);
          mma_u8s8(accQ3[0], q30, q31, q32, q33, v2.x, v2.y);
          mma_s8s8(accT[0], hy0, hy1, hy2, hy3, v1.x, v1.y);
          mma_u8s8(accT[1], ly0, ly1, ly2, ly3, v1.z, v1.w);
          mma_u8s8(accQ7[0], q70, q71, q72, q73, v2.z, v2.w);
        }
      }
    }
    if (!ok) break;

    // ---------------------------------------------------------------- epilogue
    if (!active) continue;
    const int64_t row0 = rt + cw * 16;
    auto finish = [&](long long T, long long TQ, int ql, int64_t row, float nu, float gamma) {
      const NQConst c = qcs[ql];
      const float av = __fmul_rn((float)T, c.sa);
      const float sv = fmaf((float)TQ, c.ss, c.cs);
      const float est = __fmul_rn(nu, fmaf(__fmul_rn(a.coef, gamma), sv, av));
      if (row < row_end && ql < a.nq_pass) {
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
    };
    if (TILED) {
      // thread (g, t4): rows g, g + 8, queries 2 t4, 2 t4 + 1; the digit tiles of a query sit in this thread
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int e = 2 * h + c;
          const long long T = (long long)accT[0][e] + 256ll * accT[1][e] + 65536ll * accT[NT_T - 1][e];
          const long long TQ = 16ll * ((long long)accQ3[0][e] + 256ll * accQ3[NT_Q - 1][e]) +
                               ((long long)accQ7[0][e] + 256ll * accQ7[NT_Q - 1][e]);
          finish(T, TQ, 2 * t4 + c, row0 + g + 8 * h, nu_pre[h], gm_pre[h]);
        }
    } else {
      // thread (g, t4) holds columns 2 t4, 2 t4 + 1 of rows g, g + 8: digits (0, 1) of query t4 / 2 on the even
      // lane of a pair, digit 2 on the odd lane.  The even lane finishes row g, the odd lane row g + 8.
      const bool odd = (t4 & 1) != 0;
      long long low[2], tq[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const long long c0 = (long long)accT[0][2 * h] + accT[1][2 * h], c1 = (long long)accT[0][2 * h + 1] + accT[1][2 * h + 1];
        low[h] = odd ? c0 : c0 + 256ll * c1;   // odd lane: digit 2 alone
        tq[h] = 16ll * ((long long)accQ3[0][2 * h] + 256ll * accQ3[0][2 * h + 1]) +
                ((long long)accQ7[0][2 * h] + 256ll * accQ7[0][2 * h + 1]);
      }
      const long long recvT = shfl_xor_ll(odd ? low[0] : low[1], 1);
      const long long recvQ = shfl_xor_ll(tq[1], 1);
      const long long T = odd ? recvT + 65536ll * low[1] : low[0] + 65536ll * recvT;
      const long long TQ = odd ? recvQ : tq[0];
      finish(T, TQ, t4 >> 1, row0 + g + (odd ? 8 : 0), nu_pre[odd ? 1 : 0], gm_pre[odd ? 1 : 0]);
    }
  }
}

// ------------------------------------------------------------------ layout conversion
// One warp per row, one lane per group of 32 coordinates (three idx words + one qjl word <-> four words of the
// combined nibble row).  In place: a warp holds its whole row in registers before it writes any of it.
struct ConvArgs {
  int64_t n;
  uint8_t* idx;
  uint8_t* qjl;
  int d, idx_rb, qjl_rb, to_nibble;
};

constexpr int CONV_MAX_GROUPS_PER_LANE = TQ_MAX_D / 32 / 32;   // 8

__global__ void __launch_bounds__(256) convert_kernel(ConvArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= a.n) return;
  uint32_t* ri = reinterpret_cast<uint32_t*>(a.idx + (size_t)row * a.idx_rb);
  uint32_t* rq = reinterpret_cast<uint32_t*>(a.qjl + (size_t)row * a.qjl_rb);
  const int wi = a.idx_rb / 4, wq = a.qjl_rb / 4;
  const int ngroups = (a.d + 31) / 32;
  // word w of the combined row [idx row | qjl row]
  auto comb = [&](int w) -> uint32_t* { return w < wi ? ri + w : rq + (w - wi); };
  uint32_t in[CONV_MAX_GROUPS_PER_LANE][4];
#pragma unroll
  for (int t = 0; t < CONV_MAX_GROUPS_PER_LANE; ++t) {
    const int g = lane + 32 * t;
#pragma unroll
    for (int i = 0; i < 4; ++i) in[t][i] = 0u;
    if (g >= ngroups) continue;
    if (a.to_nibble) {
#pragma unroll
      for (int i = 0; i < 3; ++i)
        if (3 * g + i < wi) in[t][i] = ri[3 * g + i];
      if (g < wq) in[t][3] = rq[g];
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (4 * g + i < wi + wq) in[t][i] = *comb(4 * g + i);
    }
  }
  __syncwarp();
#pragma unroll
  for (int t = 0; t < CONV_MAX_GROUPS_PER_LANE; ++t) {
    const int g = lane + 32 * t;
    if (g >= ngroups) continue;
    const int valid = min(32, a.d - 32 * g);   // coordinates of this group that exist
    uint32_t out[4] = {0u, 0u, 0u, 0u};
    if (a.to_nibble) {
      const unsigned long long lo = (unsigned long long)in[t][0] | ((unsigned long long)in[t][1] << 32);
      const uint32_t hi = in[t][2], z = in[t][3];
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        const int bp = 3 * c;
        uint32_t f;
        if (bp + 3 <= 64) f = (uint32_t)(lo >> bp) & 7u;
        else if (bp >= 64) f = (hi >> (bp - 64)) & 7u;
        else f = ((uint32_t)(lo >> bp) | (hi << (64 - bp))) & 7u;
        const uint32_t nib = c < valid ? (f | (((z >> c) & 1u) << 3)) : 0u;
        out[c >> 3] |= nib << (4 * (c & 7));
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (4 * g + i < wi + wq) *comb(4 * g + i) = out[i];
    } else {
      unsigned long long lo = 0ull;
      uint32_t hi = 0u, z = 0u;
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        const uint32_t nib = c < valid ? (in[t][c >> 3] >> (4 * (c & 7))) & 15u : 0u;
        const int bp = 3 * c;
        const unsigned long long f = nib & 7u;
        if (bp < 64) lo |= f << bp;
        if (bp + 3 > 64) hi |= bp >= 64 ? (uint32_t)f << (bp - 64) : (uint32_t)(f >> (64 - bp));
        z |= (nib >> 3) << c;
      }
      out[0] = (uint32_t)lo; out[1] = (uint32_t)(lo >> 32); out[2] = hi;
#pragma unroll
      for (int i = 0; i < 3; ++i)
        if (3 * g + i < wi) ri[3 * g + i] = out[i];
      if (g < wq) rq[g] = z;
    }
  }
  // words that no group owns (row padding) are zero in either layout
  if (a.to_nibble) {
    for (int w = 4 * ngroups + lane; w < wi + wq; w += 32) *comb(w) = 0u;
  } else {
    for (int w = 3 * ngroups + lane; w < wi; w += 32) ri[w] = 0u;
    for (int w = ngroups + lane; w < wq; w += 32) rq[w] = 0u;
  }
}

// ------------------------------------------------------------------ host side
struct Config {
  int sb;        // 64-byte blocks per stage
  int stages;
  size_t smem;
};

int nblocks_of(const tq_plan* plan) { return plan->nb.nbi + plan->nb.nbq; }

size_t bfrag_bytes(const tq_plan* plan, bool tiled) {
  // whole stages of 2, 3 or 4 blocks, so that every stage size finds its operand
  return (size_t)((nblocks_of(plan) + 11) / 12 * 12) * (tiled ? KPB_TILE : KPB_COL) * 32 * sizeof(uint2);
}

// Blocks per stage: as measured at d = 1536 on 10^6 rows, the two-query shape runs best on three (or more) stages
// of three blocks (166 us against 172 us on two stages of four: its consumers outrun a shallow pipeline), the
// eight-query shape, whose operand leaves room for two large or four small stages, on two stages of four (244 us
// against 251 us: fewer, longer steps).
bool pick_config(const tq_plan* plan, bool tiled, Config* out) {
  const size_t fixed = bfrag_bytes(plan, tiled) + 1024 /*alignment*/ + 2 * MAX_STAGES * 8 + 16 + 8 * sizeof(NQConst);
  const int order[2][3] = {{3, 2, 4}, {4, 3, 2}};
  for (int sb : order[tiled ? 1 : 0]) {
    const size_t stage = (size_t)sb * BLOCK_BYTES;
    if (fixed + 2 * stage > (size_t)SMEM_LIMIT) continue;
    out->sb = sb;
    out->stages = (int)std::min<size_t>((SMEM_LIMIT - fixed) / stage, MAX_STAGES);
    out->smem = fixed + (size_t)out->stages * stage;
    return true;
  }
  return false;
}

// Launch with the programmatic-stream-serialisation attribute: the kernel may be scheduled while its
// predecessor in the stream drains; it orders itself with griddepcontrol.wait.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
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
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

template <int TILED, int MODE, int SB>
cudaError_t launch_t(const CUtensorMap& mi, const CUtensorMap& mq, const ScanArgs& args, size_t smem, bool dependent,
                     cudaStream_t st) {
  auto kern = scan_nib_kernel<TILED, MODE, SB>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const int grid = (int)std::min<int64_t>(args.ntiles, tc::sm_count());
  if (dependent) e = launch_dependent(kern, dim3(grid), dim3(32 * (NW + 1)), smem, st, mi, mq, args);
  else kern<<<grid, 32 * (NW + 1), smem, st>>>(mi, mq, args);
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <int TILED, int MODE>
cudaError_t launch_sb(int sb, const CUtensorMap& mi, const CUtensorMap& mq, const ScanArgs& args, size_t smem, bool dependent,
                      cudaStream_t st) {
  return sb == 4   ? launch_t<TILED, MODE, 4>(mi, mq, args, smem, dependent, st)
         : sb == 3 ? launch_t<TILED, MODE, 3>(mi, mq, args, smem, dependent, st)
                   : launch_t<TILED, MODE, 2>(mi, mq, args, smem, dependent, st);
}

}  // namespace

void plan_init(tq_plan* plan) {
  plan->nb.ok = 0;
  if (plan->mode != TQ_PROD || plan->mse_bits != 3 || !plan->ms.ok) return;
  const float* c = plan->cb.c;
  for (int i = 0; i < 4; ++i)
    if (c[i] != -c[7 - i]) return;   // the table below relies on exact antisymmetry
  const double cmax = std::fabs((double)c[0]);
  if (!(cmax > 0.0)) return;
  // delta = cmax / m for an integer top entry m <= 32767: the m that brings the other three centroids closest
  // to integers (their fractional errors then are a few hundredths instead of up to one half)
  double best = 2.0;
  int best_m = 32767;
  for (int m = 32767; m >= 16384; --m) {
    double worst = 0.0;
    for (int i = 1; i < 4; ++i) {
      const double t = std::fabs((double)c[i]) * m / cmax;
      worst = std::max(worst, std::fabs(t - std::nearbyint(t)));
    }
    if (worst < best) {
      best = worst;
      best_m = m;
    }
  }
  plan->nb.delta = cmax / best_m;
  uint32_t hi[2] = {0u, 0u}, lo[2] = {0u, 0u};
  for (int i = 0; i < 8; ++i) {
    const int t = (int)std::nearbyint((double)c[i] / plan->nb.delta);   // |t| <= 32767, t_i = -t_{7-i}
    const int h = t >> 8, l = t & 255;                                  // t = 256 h + l, h signed, l unsigned
    hi[i >> 2] |= (uint32_t)(h & 255) << (8 * (i & 3));
    lo[i >> 2] |= (uint32_t)l << (8 * (i & 3));
  }
  plan->nb.hi_a = hi[0]; plan->nb.hi_b = hi[1]; plan->nb.lo_a = lo[0]; plan->nb.lo_b = lo[1];
  plan->nb.nbi = (int)((plan->idx_row_bytes + 63) / 64);
  plan->nb.nbq = (int)((plan->qjl_row_bytes + 63) / 64);
  Config cfg;
  if (!pick_config(plan, false, &cfg)) return;   // query-side operand too large for shared memory at this d
  plan->nb.ok = 1;
}

int queries_per_pass(const tq_plan* plan, int nq) {
  Config c;
  return (nq > 2 && pick_config(plan, true, &c)) ? 8 : 2;
}

size_t workspace_bytes(const tq_plan* plan) {
  Config c;
  return kQConstBytes + (bfrag_bytes(plan, pick_config(plan, true, &c)) + 255) / 256 * 256;
}

int prepare(const tq_plan* plan, const float* Qcat, int nqp, void* workspace, cudaStream_t st, const char* who) {
  const bool tiled = queries_per_pass(plan, nqp) == 8;
  PrepArgs pa;
  pa.Qcat = Qcat;
  pa.ldq = (int64_t)plan->ncat * plan->dpad;
  pa.qc = static_cast<NQConst*>(workspace);
  pa.nq_pass = nqp;
  pa.d = plan->d;
  pa.dpad = plan->dpad;
  pa.nbi = plan->nb.nbi;
  pa.idx_rb = (int)plan->idx_row_bytes;
  pa.qjl_rb = (int)plan->qjl_row_bytes;
  pa.nblocks = (nblocks_of(plan) + 11) / 12 * 12;   // blocks beyond the rows get a zero operand
  pa.tiled = tiled ? 1 : 0;
  pa.delta = plan->nb.delta;
  pa.out = reinterpret_cast<uint2*>(static_cast<char*>(workspace) + kQConstBytes);
  const int total = pa.nblocks * (tiled ? KPB_TILE : KPB_COL) * 32;
  cudaError_t e = launch_dependent(nprep_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, st, pa);
  count_launches(1);
  TQ_CHECK_CUDA(e != cudaSuccess ? e : cudaGetLastError(), who);
  return TQ_OK;
}

int run(const tq_plan* plan, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
        const float* norms, float* scores, int64_t lds, const mscan::Filter* filter, const int* run_if,
        const void* workspace, bool codes_final, cudaStream_t st, const char* who) {
  const bool tiled = queries_per_pass(plan, nqp) == 8;
  Config c;
  TQ_REQUIRE(pick_config(plan, tiled, &c), TQ_ERR_UNSUPPORTED, "%s: no shared-memory configuration for d=%d", who, plan->d);
  CUtensorMap mi, mq;
  TQ_REQUIRE(tc::make_byte_map(&mi, idx, (uint64_t)n, plan->idx_row_bytes, plan->idx_row_bytes, 64, VT), TQ_ERR_CUDA,
             "%s: cuTensorMapEncodeTiled failed (idx)", who);
  TQ_REQUIRE(tc::make_byte_map(&mq, qjl, (uint64_t)n, plan->qjl_row_bytes, plan->qjl_row_bytes, 64, VT), TQ_ERR_CUDA,
             "%s: cuTensorMapEncodeTiled failed (qjl)", who);
  ScanArgs sa;
  sa.n = n;
  sa.ntiles = (n + VT - 1) / VT;
  sa.nblocks = nblocks_of(plan);
  sa.nsteps = (sa.nblocks + c.sb - 1) / c.sb;
  sa.stages = c.stages;
  sa.nbi = plan->nb.nbi;
  sa.hi_a = plan->nb.hi_a; sa.hi_b = plan->nb.hi_b; sa.lo_a = plan->nb.lo_a; sa.lo_b = plan->nb.lo_b;
  sa.Bfrag = reinterpret_cast<const uint2*>(static_cast<const char*>(workspace) + kQConstBytes);
  sa.bfrag_u2 = (int)(bfrag_bytes(plan, tiled) / sizeof(uint2));
  sa.qc = static_cast<const NQConst*>(workspace);
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
  cudaError_t e;
  // the early start reads the codes before the kernel ahead in the stream has finished: only when that kernel
  // is one of this call's own (the caller says so), never a writer of the codes
  const bool dep = codes_final;
  if (tiled) e = filter ? launch_sb<1, 1>(c.sb, mi, mq, sa, c.smem, dep, st) : launch_sb<1, 0>(c.sb, mi, mq, sa, c.smem, dep, st);
  else e = filter ? launch_sb<0, 1>(c.sb, mi, mq, sa, c.smem, dep, st) : launch_sb<0, 0>(c.sb, mi, mq, sa, c.smem, dep, st);
  TQ_CHECK_CUDA(e, who);
  return TQ_OK;
}

int convert(const tq_plan* plan, int64_t n, uint8_t* idx, uint8_t* qjl, int to_layout, cudaStream_t st, const char* who) {
  if (n == 0) return TQ_OK;
  ConvArgs a;
  a.n = n;
  a.idx = idx;
  a.qjl = qjl;
  a.d = plan->d;
  a.idx_rb = (int)plan->idx_row_bytes;
  a.qjl_rb = (int)plan->qjl_row_bytes;
  a.to_nibble = to_layout == TQ_LAYOUT_NIBBLE ? 1 : 0;
  convert_kernel<<<(unsigned)((n + 7) / 8), 256, 0, st>>>(a);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

}  // namespace nscan
}  // namespace tq

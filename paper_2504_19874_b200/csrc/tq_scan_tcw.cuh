// The wide form of the tcgen05 scan: 64 queries per pass over the codes on one 128-vector tile,
//     D[128 vectors, 192 columns] += A[128, 32] * B[192, 32]^T,   kind::i8, s32 accumulators in TMEM.
// Included by tq_scan_tc.cu inside tq::tscan's unnamed namespace (same operands, constants and integers as
// scan_tc_kernel: the 192 columns are the B rows of two consecutive 32-query passes, column = 96 (q / 32) +
// 32 digit + q % 32).
//
// Why a second form.  With clock64 counters in a scratch build of scan_tc_kernel a transform warp is busy ~530
// cycles per k-block (expansion ~350, tcgen05.st ~120, barriers ~60) plus ~160 for the epilogue, and waits
// ~300 for its A slot: with two slots per tile the round trip store -> MMA -> commit -> barrier (~1700 cycles)
// and the warp's own dependent chain both sit near 900 cycles per k-block, so neither more slots (TMEM is full
// with two tiles) nor more issuers helped.  Here
//   - one expansion of a row serves 64 queries instead of 32: half as many tcgen05.st, PRMT/LOP and barrier
//     rounds per (vector, query);
//   - one tile per iteration leaves room for four A slots beside the two 192-column accumulators
//     (384 + 4 x 32 = 512 TMEM columns);
//   - the eight transform warps form two sets that take the row groups (64-byte blocks of the nibble layout,
//     groups of four k-blocks of the bit streams) in turn, so that two warps work on every lane quadrant's chain;
//     a set's threads read back and emit 32 of the 64 queries each;
//   - a k-block is 4 MMAs of N = 192 instead of 8 of N = 96 (an MMA of N = 96 costs as much as one of N = 128).
// The accumulators are single-buffered: the issuers wait (dfree) until both sets have read their columns of the
// previous tile into registers and zeroed them.
//
// CTA (one per SM, persistent over tiles), 384 threads:
//   warp 0       TMA producer: per k-block one [192 rows x 128 B] box of B (6 stages); per row group the tile's packed
//                rows ([128 rows x 32..64 B], 4 stages), requested as far ahead as their ring allows
//   warps 1..3   MMA issuers, k-blocks in turn.  A thread issues an MMA every ~82 cycles and does not get to its next
//                k-block before the MMAs it committed have completed (~1000 cycles per k-block and thread): two
//                threads fed 4 MMAs of ~97 cycles every ~500 cycles, three keep the pipe busy between epilogues.
//   warps 4..11  transform + epilogue: set = (warp - 4) / 4, lane quadrant = warp % 4, thread = vector row; a set takes
//                every second row group of the CTA's running count
// CTAS = 2 (the default where there is more than one tile): two CTAs of a cluster run in lockstep on their own tiles
// and share every B box -- each loads half of its rows (no multicast) into one of twelve half-size stages, the
// leader's issuers run the MMAs with M = 256 (cta_group::2), the commits reach both CTAs' barriers.  Halving the B
// traffic from L2 alone gave nothing; the deeper ring in the same bytes and the third issuer together 7 %.
// All waits are bounded.
#pragma once

constexpr int W_QPP = 2 * kQueriesPerPass;      // 64 queries per pass
constexpr int W_NCOL = 2 * NCOL;                // 192 MMA columns
constexpr int W_SLOTS = 4;                      // k-blocks of A resident in TMEM
constexpr int W_BSTAGES = 6;                    // ring of B boxes (a CTA of a pair holds half of each: 12 stages in the same bytes)
constexpr int W_BTILE = W_NCOL * KB_BYTES;      // 24 KB
constexpr int W_PSTAGES = 4;                    // ring of packed-row groups
constexpr int W_PTILE = TILE * 64;              // 8 KB: 128 rows x at most 64 bytes
constexpr int W_ACOL0 = 2 * W_NCOL;             // first TMEM column of the A slots
constexpr int W_ISSUERS = 3;                    // MMA-issuing warps: a thread that has committed a k-block's MMAs does not get to its
                                                // next k-block before they have completed (~1000 cycles per k-block and thread),
                                                // so two threads feed 4 MMAs of ~97 cycles every ~500 cycles, three every ~333
constexpr int W_NTHREADS = 32 * (1 + W_ISSUERS + 8);
constexpr int W_LBUF = 64;                      // candidates per query a CTA collects before it appends them
static_assert(W_ACOL0 + W_SLOTS * 32 <= TMEM_COLS, "TMEM columns");
static_assert((W_SLOTS & (W_SLOTS - 1)) == 0 && (W_PSTAGES & (W_PSTAGES - 1)) == 0, "ring sizes used as masks");

constexpr size_t kWideSmemBytes = 1024 + W_BSTAGES * W_BTILE + W_PSTAGES * W_PTILE + 512 +
                                  W_QPP * (sizeof(QConst) + sizeof(float) + sizeof(int) + W_LBUF * sizeof(uint2));

// Row group g of a tile: its first k-block, its k-blocks, which part they belong to, and where its packed bytes
// start in the idx / qjl rows.
struct RowGroup {
  int f0, cnt;
  bool part_s;    // bit streams: the QJL part (its own rows and B matrix)
  bool from_qjl;  // the packed bytes come from the qjl rows
  int x;          // byte offset in those rows
  int bytes;      // bytes per row
};
template <int BM, bool NIB>
__device__ __forceinline__ RowGroup row_group(const Geo& g, int gi) {
  RowGroup rg;
  if (NIB) {   // block gi of the combined row [idx row | qjl row]: three k-blocks
    rg.f0 = 3 * gi;
    rg.cnt = 3;
    rg.part_s = false;
    rg.from_qjl = gi >= g.nbi;
    rg.x = 64 * (rg.from_qjl ? gi - g.nbi : gi);
    rg.bytes = 64;
    return rg;
  }
  const int ga = (g.kba + 3) >> 2;
  if (gi < ga) {
    rg.f0 = 4 * gi;
    rg.cnt = min(4, g.kba - 4 * gi);
    rg.part_s = rg.from_qjl = false;
    rg.bytes = group_bytes(BM);
    rg.x = gi * rg.bytes;
  } else {
    const int gq = gi - ga;
    rg.f0 = g.kba + 4 * gq;
    rg.cnt = min(4, g.kbs - 4 * gq);
    rg.part_s = rg.from_qjl = true;
    rg.bytes = 64;
    rg.x = gq * 64;
  }
  return rg;
}

template <int BM, int MODE, bool NIB, int CTAS>
__global__ void __launch_bounds__(W_NTHREADS, 1)
scan_tcw_kernel(const __grid_constant__ CUtensorMap tmBa, const __grid_constant__ CUtensorMap tmBs,
                const __grid_constant__ CUtensorMap tmPa, const __grid_constant__ CUtensorMap tmPs, ScanArgs a) {
  if (a.run_if != nullptr && *a.run_if == 0) return;
  // B ring of this CTA: a CTA of a pair holds half of every box, so the same shared memory gives twice the stages --
  // the boxes arrive ~2500 cycles after they are requested (all SMs read the same lines of L2 at about the same time),
  // and the number of boxes in flight, not the bytes, sets the rate at which they arrive
  constexpr int BST = W_BSTAGES * CTAS, BTILE = W_BTILE / CTAS;
  // The completion barriers of the k-blocks form a ring of their own, kdone[k % KD].  Several threads issue, so the
  // k-blocks complete out of order, and a waiter must never find that its barrier has completed twice since the
  // k-block it waits for (the parity would look unchanged): the producer waits for k - BST before it loads k, the
  // transform warps for k - W_SLOTS before they store k, and the next k-block on either's barrier, k - BST + KD resp.
  // k - W_SLOTS + KD, cannot complete before k itself is loaded resp. k + W_SLOTS stored when KD >= BST and
  // KD >= 2 W_SLOTS.  (With kdone[k % 6] and three issuers k + 2 could complete before k was stored.)
  constexpr int KD = CTAS == 2 ? 16 : 8;
  // A parity wait also passes when its barrier is two completions behind, so whoever waits for a completion must
  // itself have seen the one before it.  The "A stored" barriers therefore form a ring of lcm(issuers, slots) = 12:
  // the thread that issues k-block k waited on afull[k % 12] for k - 12 (with afull[k % 4] the completion before k's
  // is k - 4's, another thread's, and k - 4 may not be stored yet when the other set is ahead).  The B rings (6 and
  // 12 stages) are multiples of the issuer count for the same reason.
  constexpr int AF = 12;
  static_assert(AF % W_ISSUERS == 0 && AF % W_SLOTS == 0 && BST % W_ISSUERS == 0, "a waiter has seen the completion before the one it waits for");
  static_assert(KD >= BST && KD >= 2 * W_SLOTS && (KD & (KD - 1)) == 0, "ring of completion barriers");
  const int rank = CTAS == 2 ? (int)tc::cluster_ctarank() : 0;
  // a unit = one CTA or one pair of CTAs; in round i unit u's CTA `rank` takes tile (u + i nunits) CTAS + rank
  const int64_t unit = blockIdx.x / CTAS, nunits = gridDim.x / CTAS;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* bring = smem;
  unsigned char* pring = smem + W_BSTAGES * W_BTILE;
  uint64_t* bars = reinterpret_cast<uint64_t*>(pring + W_PSTAGES * W_PTILE);
  uint64_t* afull = bars;                           // [AF]   k-block k stored by the owning set's four warps (afull[k % AF]) -> MMA
  uint64_t* bfull = afull + AF;                // [BST]  TMA -> MMA
  uint64_t* kdone = bfull + BST;                    // [KD]   MMAs of k-block k complete (kdone[k % KD]): its B stage and A slot are free
  uint64_t* pfull = kdone + KD;              // [W_PSTAGES]  TMA (packed rows) -> the owning set
  uint64_t* pempty = pfull + W_PSTAGES;             // [W_PSTAGES]  the owning set -> TMA producer
  uint64_t* dfull = pempty + W_PSTAGES;             // accumulators complete -> epilogue
  uint64_t* dfree = dfull + 1;                      // accumulators read and zeroed -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dfree + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  QConst* qcs = reinterpret_cast<QConst*>(reinterpret_cast<unsigned char*>(bars) + 512);
  float* taus = reinterpret_cast<float*>(qcs + W_QPP);             // [64] admission thresholds (filter mode)
  int* lcnt = reinterpret_cast<int*>(taus + W_QPP);                // [64]
  uint2* lbuf = reinterpret_cast<uint2*>(lcnt + W_QPP);            // [64][W_LBUF] (score bits, row)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb_total = a.g.kba + a.g.kbs;
  const int ngroups = NIB ? a.g.nblk : ((a.g.kba + 3) >> 2) + ((a.g.kbs + 3) >> 2);
  const int64_t ntiles = (a.n + TILE - 1) / TILE, nrounds = (ntiles + CTAS - 1) / CTAS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < AF; ++s) tc::mbar_init(&afull[s], 4 * CTAS);   // the leader's: the owning set of both CTAs
    for (int s = 0; s < BST; ++s) tc::mbar_init(&bfull[s], 1);
    for (int s = 0; s < KD; ++s) tc::mbar_init(&kdone[s], 1);
    for (int s = 0; s < W_PSTAGES; ++s) {
      tc::mbar_init(&pfull[s], 1);
      tc::mbar_init(&pempty[s], 4);
    }
    tc::mbar_init(dfull, W_ISSUERS);
    tc::mbar_init(dfree, 8 * CTAS);
    *abort_flag = 0;
    tc::fence_barrier_init();
    if (a.g.kba > 0) tc::tma_prefetch_desc(&tmBa);
    if (a.g.kbs > 0) tc::tma_prefetch_desc(&tmBs);
    if (a.g.kba > 0) tc::tma_prefetch_desc(&tmPa);
    if (a.g.kbs > 0) tc::tma_prefetch_desc(&tmPs);
  }
  if (threadIdx.x < W_QPP) {
    QConst c = {1.f, 0.f, 1.f, 0.f, 0, 0, {0, 0}};
    if ((int)threadIdx.x < a.nqp) c = a.qc[threadIdx.x];
    qcs[threadIdx.x] = c;
    taus[threadIdx.x] = (MODE == 1 && (int)threadIdx.x < a.nqp) ? a.tau[threadIdx.x] : 0.f;
    lcnt[threadIdx.x] = 0;
  }
  if (warp == 1) {
    if (CTAS == 2) tc::tmem_alloc_pair(tmem_slot, TMEM_COLS);
    else tc::tmem_alloc(tmem_slot, TMEM_COLS);
  }
  tc::tc_fence_before();
  if (CTAS == 2) tc::cluster_sync();   // the partner's barriers exist before anything arrives on them
  else __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int bst = 0;
      uint32_t kc = 0, gc = 0;   // k-blocks and row groups reached so far by this CTA
      bool ok = true;
      // The packed rows run ahead of the B boxes as far as their own ring allows: a row group's bytes are wanted by its
      // set as soon as the set has stored its previous group, several k-blocks before the MMAs free a B stage for it.
      int64_t prnd = unit;
      int pgi = 0;
      uint32_t pgc = 0;                   // row groups whose packed rows have been requested
      auto load_rows = [&]() {
        const RowGroup rg = row_group<BM, NIB>(a.g, pgi);
        const uint32_t pst = pgc & (W_PSTAGES - 1);
        tc::mbar_arrive_expect_tx(&pfull[pst], (uint32_t)(TILE * rg.bytes));
        tc::tma_load_2d(pring + pst * W_PTILE, rg.from_qjl ? &tmPs : &tmPa, &pfull[pst], rg.x, (int)((prnd * CTAS + rank) * TILE));
        ++pgc;
        if (++pgi == ngroups) {
          pgi = 0;
          prnd += nunits;
        }
      };
      for (int64_t rnd = unit; rnd < nrounds && ok; rnd += nunits) {   // a tile past the last one (odd count) reads zeros
        for (int gi = 0; gi < ngroups && ok; ++gi, ++gc) {
          const RowGroup rg = row_group<BM, NIB>(a.g, gi);
          while (pgc <= gc) {   // this group's rows at the latest now
            if (!(ok = tc::mbar_wait(&pempty[pgc & (W_PSTAGES - 1)], ((pgc / W_PSTAGES) & 1u) ^ 1u, abort_flag, a.status))) break;
            load_rows();
          }
          if (!ok) break;
          for (int j = 0; j < rg.cnt; ++j, ++kc) {
            // one more row group ahead when its stage is free (a test, not a wait)
            if (prnd < nrounds && tc::mbar_test_wait(&pempty[pgc & (W_PSTAGES - 1)], ((pgc / W_PSTAGES) & 1u) ^ 1u)) load_rows();
            const int f = rg.f0 + j;
            const int kb = rg.part_s ? f - a.g.kba : f;
            // B stage kc % BST was last read by the MMAs of k-block kc - BST
            if (kc >= BST && !(ok = tc::mbar_wait(&kdone[(kc - BST) & (KD - 1)], ((kc - BST) / KD) & 1u, abort_flag, a.status))) break;
            if (CTAS == 2) {   // each CTA loads half of the box's rows; the bytes of both are counted on the leader's barrier
              if (rank == 0) tc::mbar_arrive_expect_tx(&bfull[bst], W_BTILE);
              tc::tma_load_2d_pair(bring + bst * BTILE, rg.part_s ? &tmBs : &tmBa, &bfull[bst], kb * KB_BYTES,
                                   a.pass * NCOL + rank * (W_NCOL / 2));
            } else {
              tc::mbar_arrive_expect_tx(&bfull[bst], W_BTILE);
              tc::tma_load_2d(bring + bst * BTILE, rg.part_s ? &tmBs : &tmBa, &bfull[bst], kb * KB_BYTES, a.pass * NCOL);
            }
            if (++bst == BST) bst = 0;
          }
        }
      }
      if (!ok) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let copies in flight land
      }
    }
    __syncwarp();
  } else if (warp <= W_ISSUERS) {
    // ---------------------------------------------------------------- MMA issuers
    if (lane == 0 && rank == 0) {   // the leader's threads issue for both CTAs of a pair (M = 256)
      constexpr uint32_t idesc = idesc_i8(TILE * CTAS, W_NCOL);
      const int me = warp - 1;
      bool ok = true;
      uint32_t kc = 0, it = 0;
      int turn = 0;
      const uint64_t bdesc0 = tc::smem_desc_sw128(tc::smem_u32(bring));
      for (int64_t rnd = unit; rnd < nrounds && ok; rnd += nunits, ++it) {
        // both sets (of both CTAs) have read the previous tile's accumulators and zeroed them
        if (!(ok = tc::mbar_wait(dfree, it & 1u, abort_flag, a.status))) break;
        for (int f = 0; f < nkb_total; ++f, ++kc) {
          const bool mine = turn == me;
          if (++turn == W_ISSUERS) turn = 0;
          if (!mine) continue;
          const uint32_t bst = kc % BST, slot = kc & (W_SLOTS - 1);
          if (!(ok = tc::mbar_wait(&bfull[bst], (kc / BST) & 1u, abort_flag, a.status))) break;
          if (!(ok = tc::mbar_wait(&afull[kc % AF], (kc / AF) & 1u, abort_flag, a.status))) break;
          tc::tc_fence_after();
          const int kind = NIB ? f % 3 : 0;   // nibble layout: h bytes (signed A), l bytes, sign bits (second accumulator)
          const bool part_s = NIB ? kind == 2 : f >= a.g.kba;
          const uint32_t idesc_f = (NIB && kind == 0) ? idesc_i8(TILE * CTAS, W_NCOL, true) : idesc;
          const uint64_t bdesc = bdesc0 + (uint64_t)(bst * (BTILE >> 4));
          const uint32_t a_tmem = tmem_base + (uint32_t)(W_ACOL0 + slot * 32);
          const uint32_t d_tmem = tmem_base + (uint32_t)(part_s ? W_NCOL : 0);
#pragma unroll
          for (int step = 0; step < 4; ++step) {   // 32 K-bytes per MMA: 8 TMEM columns of A, +32 bytes inside B's swizzled row
            if (CTAS == 2) umma_i8_ts_pair(d_tmem, a_tmem + 8 * step, bdesc + 2 * step, idesc_f, 1u);
            else umma_i8_ts(d_tmem, a_tmem + 8 * step, bdesc + 2 * step, idesc_f, 1u);
          }
          // A slot and B stage (of both CTAs) reusable once these MMAs have read them
          if (CTAS == 2) tc::umma_commit_pair(&kdone[kc & (KD - 1)]);
          else tc::umma_commit(&kdone[kc & (KD - 1)]);
        }
        if (ok) {   // all MMAs this thread issued for the tile
          if (CTAS == 2) tc::umma_commit_pair(dfull);
          else tc::umma_commit(dfull);
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- transform + epilogue (thread = vector row)
    const int e = warp - 1 - W_ISSUERS;
    const int set = e >> 2;                 // takes the row groups gi % 2 == set and the queries [32 set, 32 set + 32)
    const int quad = warp & 3;              // TMEM lane group this warp may access
    const int r = quad * 32 + lane;         // row inside the tile
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    bool ok = true;
    uint32_t it = 0;
    auto load_nu = [&](int64_t tl) -> float {
      const int64_t rw = tl * TILE + r;
      return (rw < a.n && a.norms != nullptr) ? __ldg(a.norms + rw) : 1.f;
    };
    auto load_gm = [&](int64_t tl) -> float {
      const int64_t rw = tl * TILE + r;
      return (rw < a.n && (a.g.kbs > 0 || NIB)) ? __ldg(a.gamma + rw) : 0.f;   // times coef where it is used, so that nothing waits for the load here
    };
    // zeroes this thread's columns of both accumulators and tells the issuers (before the first tile, and in every
    // epilogue as soon as the columns have been read into registers)
    auto release_accumulators = [&]() {
#pragma unroll
      for (int c = 0; c < NCOL; c += 16) {
        tc::tmem_fill16(lane_addr + (uint32_t)(NCOL * set + c), 0u);
        tc::tmem_fill16(lane_addr + (uint32_t)(W_NCOL + NCOL * set + c), 0u);
      }
      tc::tmem_st_wait();
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (CTAS == 2) tc::mbar_arrive_leader(dfree);
        else tc::mbar_arrive(dfree);
      }
    };
    release_accumulators();
    float nu_next = load_nu(unit * CTAS + rank), gm_next = load_gm(unit * CTAS + rank);
    for (int64_t rnd = unit; rnd < nrounds && ok; rnd += nunits, ++it) {
      const int64_t tile = rnd * CTAS + rank;
      const int64_t row = tile * TILE + r;
      const bool row_ok = row < a.n;
      const float nu = nu_next, gm = gm_next;
      nu_next = load_nu(tile + nunits * CTAS);
      gm_next = load_gm(tile + nunits * CTAS);

      const uint32_t kt0 = it * (uint32_t)nkb_total;   // this tile's first k-block in the CTA's count
      // stores k-block kt's 32 A registers of this row into slot kt % W_SLOTS and announces it
      auto store_a = [&](const uint32_t (&v)[32], uint32_t kt) -> bool {
        const uint32_t slot = kt & (W_SLOTS - 1);
        if (kt >= W_SLOTS) {   // the slot was last read by the MMAs of k-block kt - W_SLOTS
          const uint32_t kp = kt - W_SLOTS;
          if (!tc::mbar_wait(&kdone[kp & (KD - 1)], (kp / KD) & 1u, abort_flag, a.status)) return false;
        }
        tc::tc_fence_after();
        tc::tmem_st32(lane_addr + (uint32_t)(W_ACOL0 + slot * 32), v);
        tc::tmem_st_wait();
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (CTAS == 2) tc::mbar_arrive_leader(&afull[kt % AF]);
          else tc::mbar_arrive(&afull[kt % AF]);
        }
        return true;
      };
      // expands one k-block's words of the bit streams into the row's 128 bytes of A
      auto emit = [&](uint32_t (&w)[4], int f) -> bool {
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
        // register 4 c + e2 = (word c / 2, bit 4 (c % 2) + e2 of every byte)
        uint32_t v[32];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint32_t x = w[c >> 1];
          const int k0 = (c & 1) * 4;
#pragma unroll
          for (int e2 = 0; e2 < 4; ++e2) v[4 * c + e2] = x & (0x01010101u << (k0 + e2));
        }
        return store_a(v, kt0 + (uint32_t)f);
      };

      // the sets take the row groups in turn by the CTA's running count of groups (not by the group's number inside the
      // tile, which changes sides from tile to tile when a tile has an odd number of groups): a set then meets a
      // packed-row stage every second time it is used, always after it has itself waited for the use before
      for (int gi = (set + (int)((it * (uint32_t)ngroups) & 1u)) & 1; gi < ngroups && ok; gi += 2) {
        const RowGroup rg = row_group<BM, NIB>(a.g, gi);
        const uint32_t gc = it * (uint32_t)ngroups + (uint32_t)gi;
        const uint32_t pst = gc & (W_PSTAGES - 1), pph = (gc / W_PSTAGES) & 1u;
        if (!(ok = tc::mbar_wait(&pfull[pst], pph, abort_flag, a.status))) break;
        const unsigned char* ps = pring + pst * W_PTILE;
        if (NIB) {
          // one 64-byte block of the combined row = 16 code words = 128 coordinates: h bytes and l bytes by byte
          // permutes with the masked word as selector, sign bits by masks
          uint32_t x[16];
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // 64 bytes per row, 64-byte swizzle: chunk c at c ^ ((row >> 1) & 3)
            const uint4 v4 = *reinterpret_cast<const uint4*>(ps + r * 64 + ((j ^ ((r >> 1) & 3)) << 4));
            x[4 * j] = v4.x; x[4 * j + 1] = v4.y; x[4 * j + 2] = v4.z; x[4 * j + 3] = v4.w;
          }
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&pempty[pst]);
          const uint32_t kt = kt0 + (uint32_t)rg.f0;
          uint32_t v[32];
#pragma unroll
          for (int wd = 0; wd < 16; ++wd) {
            const uint32_t sl = x[wd] & 0x77777777u;
            v[2 * wd] = prmt(a.hi_a, a.hi_b, sl);
            v[2 * wd + 1] = prmt(a.hi_a, a.hi_b, sl >> 16);
          }
          ok = ok && store_a(v, kt);
#pragma unroll
          for (int wd = 0; wd < 16; ++wd) {
            const uint32_t sl = x[wd] & 0x77777777u;
            v[2 * wd] = prmt(a.lo_a, a.lo_b, sl);
            v[2 * wd + 1] = prmt(a.lo_a, a.lo_b, sl >> 16);
          }
          ok = ok && store_a(v, kt + 1);
#pragma unroll
          for (int wd = 0; wd < 16; ++wd) {
            v[2 * wd] = x[wd] & 0x08080808u;
            v[2 * wd + 1] = x[wd] & 0x80808080u;
          }
          ok = ok && store_a(v, kt + 2);
        } else {
          uint32_t w[4][4];
#pragma unroll
          for (int j = 0; j < 4; ++j) w[j][0] = w[j][1] = w[j][2] = w[j][3] = 0u;
          if (rg.part_s || BM <= 2) {        // 64 bytes per row, 64-byte swizzle: chunk c at c ^ ((row >> 1) & 3)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint4 v = *reinterpret_cast<const uint4*>(ps + r * 64 + ((j ^ ((r >> 1) & 3)) << 4));
              w[j][0] = v.x; w[j][1] = v.y; w[j][2] = v.z; w[j][3] = v.w;
            }
          } else if (BM == 3) {              // 48 bytes per row, plain: three words per k-block
            uint32_t x[12];
#pragma unroll
            for (int j = 0; j < 3; ++j) {
              const uint4 v = *reinterpret_cast<const uint4*>(ps + r * 48 + j * 16);
              x[4 * j] = v.x; x[4 * j + 1] = v.y; x[4 * j + 2] = v.z; x[4 * j + 3] = v.w;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              w[j][0] = x[3 * j]; w[j][1] = x[3 * j + 1]; w[j][2] = x[3 * j + 2];
            }
          } else {                           // b_m = 4: 32 bytes per row, 32-byte swizzle: chunk c at c ^ ((row >> 2) & 1)
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const uint4 v = *reinterpret_cast<const uint4*>(ps + r * 32 + ((j ^ ((r >> 2) & 1)) << 4));
              w[2 * j][0] = v.x; w[2 * j][1] = v.y; w[2 * j + 1][0] = v.z; w[2 * j + 1][1] = v.w;
            }
          }
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&pempty[pst]);
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (j < rg.cnt) ok = ok && emit(w[j], rg.f0 + j);
        }
      }
      if (!ok) break;

      // ---- epilogue: this thread's row, the set's 32 queries
      if (!(ok = tc::mbar_wait(dfull, it & 1u, abort_flag, a.status))) break;
      tc::tc_fence_after();
      const uint32_t taddr = lane_addr + (uint32_t)(NCOL * set);
      // halves of 16 queries; a short last pass: columns of absent queries are not read
      const int nh = min(2, max(0, (a.nqp - 32 * set + 15) >> 4));
      if (nh == 0) release_accumulators();
#pragma unroll 1
      for (int h = 0; h < nh; ++h) {   // digit l of query 32 set + 16 h + qq sits in column 96 set + 32 l + 16 h + qq
        uint32_t va[LIMBS][16], vs[LIMBS][16];
#pragma unroll
        for (int l = 0; l < LIMBS; ++l) {
          if (a.g.kba > 0) tc::tmem_ld16(taddr + l * 32 + h * 16, va[l]);
          if (a.g.kbs > 0 || NIB) tc::tmem_ld16(taddr + W_NCOL + l * 32 + h * 16, vs[l]);
        }
        tc::tmem_ld_wait();
        // the last columns are in registers: the next tile's MMAs may start while their estimates are formed
        if (h == nh - 1) release_accumulators();
#pragma unroll
        for (int qq = 0; qq < 16; ++qq) {
          const int ql = 32 * set + h * 16 + qq;
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
          if (row_ok) {
            if (MODE == 0) {
              if (TQ_DEVICE_CHECK(row >= 0 && row < a.n && row < a.lds, a.status)) a.scores[(int64_t)ql * a.lds + row] = est;
            } else if (est >= taus[ql]) {
              const int ls = atomicAdd(&lcnt[ql], 1);
              if (ls < W_LBUF) {
                lbuf[ql * W_LBUF + ls] = make_uint2(__float_as_uint(est), (uint32_t)row);
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
  if (CTAS == 2) tc::cluster_sync();   // neither CTA leaves while the partner may still arrive on its barriers
  else __syncthreads();
  if (warp == 1) {
    tc::tc_fence_after();
    if (CTAS == 2) tc::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    else tc::tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (MODE == 1 && warp > W_ISSUERS) {   // the eight transform warps append eight queries' collected pairs each
    for (int ql = (warp - 1 - W_ISSUERS) * 8; ql < (warp - W_ISSUERS) * 8; ++ql) {
      const int m = min(lcnt[ql], W_LBUF);
      if (m == 0 || ql >= a.nqp) continue;
      int base = 0;
      if (lane == 0) base = atomicAdd(a.count + ql, m);
      base = __shfl_sync(0xffffffffu, base, 0);
      for (int i = lane; i < m; i += 32) {
        const int slot = base + i;
        if (slot < a.cap) {
          const uint2 e = lbuf[ql * W_LBUF + i];
          a.cand_s[(int64_t)ql * a.cap + slot] = __uint_as_float(e.x);
          a.cand_i[(int64_t)ql * a.cap + slot] = (int)e.y;
        }
      }
    }
  }
}

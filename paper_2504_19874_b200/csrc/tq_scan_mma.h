// Interface of the tensor-path packed-code scan (tq_scan_mma.cu) towards the API layer.
#pragma once

#include "tq_internal.h"

namespace tq {
namespace mscan {

// Decides whether the plan's codebook / dimension admit the bit-plane scan and fills plan->ms.
void plan_init(tq_plan* plan);

// Queries served by one pass over the codes when nq queries remain (2 or 4).
int queries_per_pass(const tq_plan* plan, int nq);

// Bytes of workspace one pass needs: per-query constants + the B operand (query-side matrix).
size_t workspace_bytes(const tq_plan* plan);

struct Filter {          // top-k candidate collection for the queries of one pass
  const float* tau;      // [nqp] admission threshold per query (score >= tau is kept)
  int* count;            // [nqp] candidates appended so far (may exceed cap: the excess was dropped)
  float* cand_s;         // [nqp, cap]
  int* cand_i;           // [nqp, cap]  ids = row numbers
  int cap;
};

// Builds the per-query constants and the B operand of one pass (nqp <= queries_per_pass) from the
// rotated queries Qcat[nqp, ncat*dpad] into `workspace`.
int prepare(const tq_plan* plan, const float* Qcat, int nqp, void* workspace, cudaStream_t st, const char* who);

// One pass over vectors [0, n) with the operand prepared in `workspace`: dense estimates into
// scores[nqp, lds], or, with a filter, only the (score, row) pairs it admits.  When run_if is not null
// the kernel returns at once if *run_if == 0 (device-side switch, read at launch).
int run(const tq_plan* plan, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
        const float* norms, float* scores, int64_t lds, const Filter* filter, const int* run_if, const void* workspace,
        cudaStream_t st, const char* who);

// The k best (score desc, id asc) per query out of `count[q]` (clamped to cap) candidate pairs, or, when
// cand_i is nullptr, out of the dense row cand_s[q*cap .. +m) with ids id0 + position.  Optionally merges
// the previous best list (top_s/top_i, when merge != 0) and writes the k-th score to kth[q].
// *overflow is set to 1 if some count exceeded cap; run_if as above.
cudaError_t select_topk(const float* cand_s, const int* cand_i, const int* count, int cap, int m, int id0, int nq, int k,
                        int merge, float* top_s, int* top_i, float* kth, int* overflow, const int* run_if,
                        cudaStream_t st);

// The k best of m candidate pairs per query (row stride ld); pairs with id < 0 are skipped.
cudaError_t select_pairs(const float* cand_s, const int* cand_i, int ld, int m, int nq, int k, float* top_s, int* top_i,
                         cudaStream_t st);

}  // namespace mscan
}  // namespace tq

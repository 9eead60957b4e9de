// Interface of the nibble-layout packed-code scan (tq_scan_nib.cu) towards the API layer.
#pragma once

#include "tq_internal.h"
#include "tq_scan_mma.h"

namespace tq {
namespace nscan {

// Fills plan->nb: whether this plan may use TQ_LAYOUT_NIBBLE (TQ_PROD with a 3-bit MSE stage, antisymmetric
// codebook, d >= 128, shared-memory room for the query-side operand) and the 16-bit centroid table.
void plan_init(tq_plan* plan);

// Queries served by one pass over the codes when nq queries remain (2 or 8).
int queries_per_pass(const tq_plan* plan, int nq);

// Bytes of workspace one pass needs: per-query constants + the query-side operand.
size_t workspace_bytes(const tq_plan* plan);

// Builds the per-query constants and the query-side operand of one pass (nqp <= queries_per_pass) from the
// rotated queries Qcat[nqp, 2*dpad] into `workspace`.
int prepare(const tq_plan* plan, const float* Qcat, int nqp, void* workspace, cudaStream_t st, const char* who);

// One pass over vectors [0, n); arguments as mscan::run.  codes_final: the kernel ahead of this one in the
// stream is one of the same API call (query preparation, selection), so the codes were complete before that
// call began and the scan may start copying them while that kernel still runs (programmatic dependent launch).
int run(const tq_plan* plan, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
        const float* norms, float* scores, int64_t lds, const mscan::Filter* filter, const int* run_if,
        const void* workspace, bool codes_final, cudaStream_t st, const char* who);

// Rewrites n rows of (idx, qjl) in place from one layout into the other (an exact permutation of the bits).
int convert(const tq_plan* plan, int64_t n, uint8_t* idx, uint8_t* qjl, int to_layout, cudaStream_t st, const char* who);

}  // namespace nscan
}  // namespace tq

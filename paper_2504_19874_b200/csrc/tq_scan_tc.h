// Interface of the many-query packed-code scan on tcgen05 (tq_scan_tc.cu) towards the API layer.
#pragma once

#include "tq_internal.h"
#include "tq_scan_mma.h"

namespace tq {
namespace tscan {

constexpr int kQueriesPerPass = 32;    // 96 MMA columns = 32 queries x 3 radix-256 digits
constexpr int kPassesPerGroup = 8;     // B operands are built for up to 8 passes (256 queries) at a time

// Queries one pass over the codes serves when a call has nq of them: 32, or 64 (the wide kernel) beyond 32 queries.
int queries_per_pass(int nq);

// Whether the plan can use this path (same conditions as the bit-plane scan, plus shared-memory room).
bool available(const tq_plan* plan);

// Bytes of workspace for one group of passes: per-query constants + both B matrices.
size_t workspace_bytes(const tq_plan* plan);

// Builds constants and B matrices for queries [0, nqg) of a group (nqg <= 256), rotated queries in Qcat.
int prepare_group(const tq_plan* plan, const float* Qcat, int nqg, void* workspace, cudaStream_t st, const char* who);

// One pass of up to 32 queries (pass index `pass` inside the prepared group), or of 33 to 64 queries (the queries of
// passes `pass` and `pass + 1`, `pass` even), over vectors [0, n): dense estimates into scores[nqp, lds] or the pairs
// admitted by the filter.  run_if as in mscan::run.
int run_pass(const tq_plan* plan, int pass, int nqp, int64_t n, const uint8_t* idx, const uint8_t* qjl, const float* gamma,
             const float* norms, float* scores, int64_t lds, const mscan::Filter* filter, const int* run_if,
             const void* workspace, cudaStream_t st, const char* who);

}  // namespace tscan
}  // namespace tq

/*
 * tq.h -- C ABI of the TurboQuant hot path for NVIDIA B200 (sm_100a).
 *
 * TurboQuant (arxiv 2504.19874) quantises a vector x in R^d in two ways:
 *   TurboQuant_mse  (Algorithm 1): y = Pi x with a random rotation Pi, then the index of the
 *                   nearest centroid of a precomputed scalar codebook for every coordinate.
 *   TurboQuant_prod (Algorithm 2): the same at b-1 bits, plus the sign bits of S r for the
 *                   residual r = x - DeQuant_mse(idx) (the QJL map of Definition 1) and ||r||.
 * This library computes those maps, their inverses, and the inner-product estimator of
 * Section 3.2 evaluated directly on the packed codes (dense scores or top-k).
 *
 * Notation used below: n vectors, d dimensions, b total bits per coordinate, b_m = bits of
 * the MSE stage (b for TQ_MSE, b-1 for TQ_PROD), nu = ||x||, u = x/nu, gamma = ||r||.
 * Following Section 1.3 the stored norm nu is kept in floating point, the unit vector u is
 * what gets quantised, and every reconstruction / estimate is rescaled by nu.
 *
 * Conventions for every entry point
 *   - returns 0 (TQ_OK) or a TQ_ERR_* code; tq_last_error() gives a thread-local message.
 *     No exception crosses the boundary.  Invalid arguments are rejected on the host before
 *     anything is launched.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA global memory of the
 *     current device, owned by the caller, 16-byte aligned, never retained after the call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).  Device work
 *     is only enqueued; the calls do not synchronise and allocate nothing (callers pass
 *     scratch sized by tq_workspace_bytes).  tq_plan_create/destroy are the exceptions.
 *   - n = 0 (or nq = 0) is a no-op that returns TQ_OK.
 *
 * Packed layouts (the paper says only "b-bit integers"; this layout is the library's)
 *   idx row : little-endian bit stream, coordinate j in bits [j*b_m, (j+1)*b_m); bit p of the
 *             row is bit (p & 7) of byte (p >> 3); value k names the k-th centroid in
 *             ascending order (0-based).  Row stride tq_idx_row_bytes(d, b_m); pad bits are 0.
 *   qjl row : bit j = 1 iff (S r)_j >= 0 (sign(0) = +1).  Row stride tq_qjl_row_bytes(d).
 *   gamma, norms : float32 arrays of length n.
 * This is TQ_LAYOUT_CANONICAL, the layout of every plan unless tq_plan_set_layout chose the other one:
 *   TQ_LAYOUT_NIBBLE (TQ_PROD plans with b = 4 only): the three index bits and the sign bit of coordinate j
 *             share nibble j of one combined row of ceil(d/2) bytes -- byte j >> 1, bits 4 (j & 1) .. 4 (j & 1) + 3,
 *             index in the low three bits, sign bit on top.  The combined row is stored across the same two
 *             arrays with the same strides: its first tq_idx_row_bytes(d, 3) bytes in the idx row, the
 *             remaining bytes in the qjl row; unused nibbles are 0.  Same bytes per vector, an exact
 *             permutation of the canonical bits (tq_convert_layout goes either way); the scan reads four
 *             coordinates' centroids with one byte-permute instruction in this layout, which makes
 *             tq_score / tq_topk about 1.5 times faster than on the bit streams.
 */
#ifndef TQ_H_
#define TQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  TQ_OK = 0,
  TQ_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, inconsistent arguments           */
  TQ_ERR_UNSUPPORTED = 2,   /* d, bits, k or dtype outside the supported range               */
  TQ_ERR_ALIGNMENT = 3,     /* a device pointer or leading dimension is not aligned          */
  TQ_ERR_CUDA = 4,          /* a CUDA runtime call failed (message has the CUDA error)       */
  TQ_ERR_NOT_CONVERGED = 5, /* Lloyd-Max iteration did not converge                          */
  TQ_ERR_TIMEOUT = 6,       /* a bounded device-side wait ran out                            */
  TQ_ERR_WORKSPACE = 7,     /* scratch / workspace smaller than tq_workspace_bytes says      */
  TQ_ERR_BOUNDS = 8         /* a TQ_DEBUG build of the library found an index outside its array */
};
enum { TQ_MSE = 0, TQ_PROD = 1 };              /* plan mode                                   */
enum { TQ_F32 = 0, TQ_BF16 = 1 };              /* element type of X / Q                       */
enum { TQ_ORTHOGONAL = 0, TQ_GAUSSIAN = 1 };   /* tq_rotation kind                            */
enum { TQ_LAYOUT_CANONICAL = 0, TQ_LAYOUT_NIBBLE = 1 };   /* arrangement of the code rows, see above */
enum { TQ_OP_QUANTIZE = 0, TQ_OP_SCORE = 1, TQ_OP_TOPK = 2, TQ_OP_WSUM = 3, TQ_OP_DEQUANTIZE = 4 };

#define TQ_MAX_D 8192
#define TQ_MAX_K 1024

typedef struct tq_plan tq_plan;

/* Message of the last error raised on the calling thread ("" if none). Never NULL. */
const char* tq_last_error(void);

/* Number of kernels this library has enqueued so far in this process (all threads, all
 * devices).  Diagnostic only: lets a harness verify that the CUDA path did the work. */
uint64_t tq_launch_count(void);

/*
 * Lloyd-Max codebook of Eq. (4): the 2^bits centroids c_1 <= ... <= c_{2^bits} in [-1,1] that
 * minimise the scalar k-means cost for the coordinate density of Lemma 1,
 * f_X(x) = Gamma(d/2) / (sqrt(pi) Gamma((d-1)/2)) (1 - x^2)^((d-3)/2)  (exact for this d, not its
 * Gaussian limit).  Host only, fp64 inside, results rounded to float32.
 *   d          2..TQ_MAX_D;   bits 0..4 (bits = 0 gives the single centroid 0)
 *   centroids  host, 2^bits floats, ascending, exactly antisymmetric (c_i = -c_{2^bits-1-i})
 *   boundaries host, 2^bits - 1 floats or NULL: fl32(0.5f * (c_i + c_{i+1})), the decision
 *              thresholds of the nearest-centroid rule of Algorithm 1 (step idx_j)
 */
int tq_codebook(int d, int bits, float* centroids, float* boundaries);

/*
 * Seeded d x d matrix, host, row-major float32.
 *   TQ_GAUSSIAN   i.i.d. N(0,1) entries: the matrix S of Definition 1 / Algorithm 2.  Entry
 *                 e = r*d + c is sqrt(-2 ln u1) cos(2 pi u2) with u1 = ((h(2e) >> 11) + 0.5) 2^-53,
 *                 u2 = (h(2e+1) >> 11) 2^-53, h(t) = mix(mix(seed + G) + t*G), mix = SplitMix64
 *                 finaliser, G = 0x9E3779B97F4A7C15 (64-bit wrap-around arithmetic).
 *   TQ_ORTHOGONAL the rotation Pi of Section 3.1: Q of the QR decomposition of that Gaussian
 *                 matrix, columns signed so that R has a positive diagonal.  fp64 Householder.
 */
int tq_rotation(int d, uint64_t seed, int kind, float* out);

/* Row strides in bytes.  ceil(d*bits/8) rounded up to a multiple of 16; rows shorter than
 * 16 bytes are rounded up to a power of two (at least 4) instead.  bits = 0 gives 0. */
size_t tq_idx_row_bytes(int d, int bits);
size_t tq_qjl_row_bytes(int d);

/*
 * Builds the per-(d, b, mode) state ("global parameters" of Algorithms 1 and 2) on the current
 * device: copies Pi, S and the codebook, forms S' = S Pi^T (fp64 on the device, rounded to
 * fp32), the decision boundaries and the operand splits the kernels use.
 *   d         2..TQ_MAX_D
 *   bits      total bits b per coordinate: TQ_MSE 1..4; TQ_PROD 1..5 (b_m = b-1, so b = 1 has a
 *             0-bit MSE stage: idx arrays are then unused and may be NULL)
 *   Pi        host, d*d floats, row-major: y = Pi x
 *   S         host, d*d floats, row-major (TQ_PROD); ignored / may be NULL for TQ_MSE
 *   centroids host, 2^b_m floats, ascending
 *   out       receives the plan; free with tq_plan_destroy.  The plan owns device memory only.
 * Allocates device memory and synchronises the device.
 */
int tq_plan_create(int d, int bits, int mode, const float* Pi, const float* S,
                   const float* centroids, tq_plan** out);
int tq_plan_destroy(tq_plan* plan);

/*
 * Chooses the arrangement of the idx / qjl rows that this plan's calls write (tq_quantize_prod) and read
 * (tq_score, tq_topk, tq_dequantize, tq_wsum, tq_score_static).  The paper fixes no layout ("b-bit integers",
 * Algorithm 1), so this is the library's choice; the codes themselves are the same.
 *   layout  TQ_LAYOUT_CANONICAL (default, every plan) or TQ_LAYOUT_NIBBLE (TQ_PROD, b = 4, d >= 128 and
 *           small enough for the scan's shared-memory operand: d <= 4096 is always accepted)
 * Returns TQ_ERR_UNSUPPORTED for a plan that cannot use the requested layout.  Host-side switch, no device
 * work; arrays written under one layout must be converted before they are read under the other.
 * tq_attend_decode / tq_kv_append take canonical plans only.
 */
int tq_plan_set_layout(tq_plan* plan, int layout);
int tq_plan_layout(const tq_plan* plan);   /* TQ_LAYOUT_*; -1 for a NULL plan */

/*
 * Rewrites n rows of codes in place from layout `from` into layout `to` (TQ_LAYOUT_*): an exact permutation
 * of the bits of each (idx row, qjl row) pair; gamma and norms are not touched.  from == to is a no-op.
 *   idx, qjl  device, the arrays of tq_quantize_prod (same strides in both layouts)
 * Errors: TQ_ERR_UNSUPPORTED when the plan cannot use TQ_LAYOUT_NIBBLE; the usual argument checks.
 */
int tq_convert_layout(const tq_plan* plan, int64_t n, uint8_t* idx, uint8_t* qjl, int from, int to, void* stream);

/* Synchronises the device and reports whether any kernel launched for this plan since the
 * last call gave up one of its bounded device-side waits (TQ_ERR_TIMEOUT; the outputs of that
 * call are then invalid).  Every producer/consumer wait inside the tensor-core kernels has a
 * time limit so that a stalled pipeline ends as this status instead of a hung GPU.
 * A library built with -DTQ_DEBUG (`python -m paper_2504_19874_b200.build --debug`, libtq_debug.so) also checks the
 * row, column and slot indices of its kernels' global stores and of the caller's channel lists on the device: an
 * index outside its array is not stored through; TQ_ERR_BOUNDS is recorded and reported here. */
int tq_plan_status(tq_plan* plan);

/* Self test of that mechanism, for test suites: enqueues a one-warp kernel that waits, through the same bounded
 * wait the tensor-core kernels use, on a barrier nobody arrives at, with a limit of `limit_cycles` SM cycles
 * (1 .. 1e8) instead of the seconds-long production limit.  The kernel returns on its own; the next
 * tq_plan_status(plan) must report TQ_ERR_TIMEOUT.  Nothing faults, traps or hangs. */
int tq_selftest_wait_timeout(tq_plan* plan, long long limit_cycles, void* stream);

/* Bytes of device scratch the given operation asks for (0 if none).  For TQ_OP_QUANTIZE and
 * TQ_OP_TOPK this is the preferred size; a smaller buffer is accepted down to the value returned
 * for n = 128 (QUANTIZE) resp. n = 4096 (TOPK) and means more, smaller launches (for TOPK also the
 * slower block-by-block selection instead of the thresholded single pass).
 * op = TQ_OP_*;  nq, k ignored where they do not apply.  Scratch must be 256-byte aligned. */
size_t tq_workspace_bytes(const tq_plan* plan, int op, int64_t n, int nq, int k);

/*
 * Quant_mse of Algorithm 1 for n vectors (plan mode TQ_MSE).
 *   X        device, n rows of d elements (x_dtype), row stride ldx elements (ldx >= d)
 *   idx      device out, n rows of tq_idx_row_bytes(d, b) bytes
 *   norms    device out, n floats: nu = ||x||.  NULL: rows are taken as already unit-norm and
 *            quantised as they are.  A zero row gives nu = 0 and the codes of y = 0.
 * Nearest centroid = number of boundaries strictly below y_j (a coordinate exactly on a
 * boundary takes the lower index).
 */
int tq_quantize_mse(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx,
                    uint8_t* idx, float* norms, void* scratch, size_t scratch_bytes, void* stream);
/*   scratch  device, sized by tq_workspace_bytes(plan, TQ_OP_QUANTIZE, n, 0, 0): holds the bf16
 *            operand splits of a block of rows (d >= 128); may be NULL when that size is 0. */

/*
 * Quant_prod of Algorithm 2 for n vectors (plan mode TQ_PROD): idx at b-1 bits, qjl = sign(S r)
 * and gamma = ||r|| for r = u - DeQuant_mse(idx).  Uses r = Pi^T (Pi u - c[idx]), so that
 * ||r|| = ||Pi u - c[idx]|| and S r = S' (Pi u - c[idx]) -- two d x d products instead of three.
 *   idx, norms as above;  qjl device out, n rows of tq_qjl_row_bytes(d);  gamma device out, n floats
 *   scratch  device, scratch_bytes >= tq_workspace_bytes(plan, TQ_OP_QUANTIZE, n, 0, 0)
 * A zero row gives gamma = 0 and all qjl bits 1.
 */
int tq_quantize_prod(const tq_plan* plan, const void* X, int x_dtype, int64_t n, int64_t ldx,
                     uint8_t* idx, uint8_t* qjl, float* gamma, float* norms,
                     void* scratch, size_t scratch_bytes, void* stream);

/*
 * DeQuant_mse / DeQuant_prod: Xhat = nu * (Pi^T c[idx] + sqrt(pi/2)/d * gamma * S^T qjl).
 *   qjl, gamma  used for TQ_PROD plans only;  norms NULL means nu = 1
 *   Xhat        device out, n rows of d floats, row stride ldxh
 */
int tq_dequantize(const tq_plan* plan, int64_t n, const uint8_t* idx, const uint8_t* qjl,
                  const float* gamma, const float* norms, float* Xhat, int64_t ldxh, void* stream);

/*
 * Inner-product estimator of Section 3.2 for every (query, vector) pair, evaluated on the codes:
 *   est = nu * ( sum_j (Pi q)_j c[idx_j]  +  sqrt(pi/2)/d * gamma * sum_i (S q)_i z_i ),  z_i = +-1
 * which equals <q, DeQuant(code)> because Pi is orthogonal.
 *   Q       device, nq rows of d elements (q_dtype), row stride ldq
 *   scores  device out, nq rows of n floats, row stride lds
 *   workspace  >= tq_workspace_bytes(plan, TQ_OP_SCORE, n, nq, 0)
 */
int tq_score(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
             const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms,
             float* scores, int64_t lds, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Queries prepared once and scanned many times (a search over several segments or shards of a database, a
 * cache that grows between decoding steps): tq_query_prepare does the query-side work of tq_score -- the
 * rotations q' = Pi q, q'' = S q and the scan's fixed-point operand -- into a caller buffer, tq_score_prepared
 * runs only the scan over the codes.  tq_score(Q) == tq_query_prepare(Q) followed by tq_score_prepared, bit for bit.
 *   prepared   device, 256-byte aligned, >= tq_query_bytes(plan, nq); valid for this plan, its current layout
 *              and exactly this nq until overwritten
 */
size_t tq_query_bytes(const tq_plan* plan, int nq);
int tq_query_prepare(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq,
                     void* prepared, size_t prepared_bytes, void* stream);
int tq_score_prepared(const tq_plan* plan, const void* prepared, int nq, int64_t n,
                      const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms,
                      float* scores, int64_t lds, void* stream);

/*
 * tq_score without caller-provided workspace and without any allocation (the paper has no
 * counterpart: this is a packaging variant of tq_score with the same arithmetic and the same scan kernels;
 * its estimates equal tq_score's bit for bit).
 *
 * Who needs it: callers that are not allowed to obtain device memory at the time they score --
 * an inference server that gave the whole GPU to its own memory pool at start-up, a plug-in whose
 * host forbids driver allocations after initialisation, a latency-critical loop that cannot afford
 * the device-wide synchronisation cudaMalloc / cudaFree imply.  Such a caller has nowhere to take
 * the workspace from (rotated queries and the scan's query-side operand), so the library keeps it: a fixed
 * array of TQ_STATIC_SCRATCH_BYTES that lives in the library's device image.  Every GPU that loads the
 * library holds that array until the process exits, whether or not this function is ever called.
 *
 *   arguments   as tq_score, minus workspace / workspace_bytes
 *   limit       rotated queries (nq * ncat * dpad * 4 bytes, ncat = 1 for TQ_MSE, 2 for TQ_PROD, dpad = d rounded
 *               up to a multiple of 8) plus one scan operand must fit in TQ_STATIC_SCRATCH_BYTES;
 *               tq_score_static_max_queries(plan) gives the largest accepted nq (75 at d = 1536 TQ_PROD b = 4).
 *               Larger requests return TQ_ERR_WORKSPACE and launch nothing.  Where the many-query engine's
 *               operand does not fit, the few-query engine runs instead (more passes, same estimates).
 *   first call  the first call on each device looks up the array's device address (with that
 *               device current) and remembers it; make that first call outside any stream capture.
 *   sharing     all calls on a device use the same array and it keeps whatever the previous call
 *               left there.  Nothing in it needs to start at zero: each call overwrites the part
 *               it reads before reading it.  Two calls whose kernels may overlap on the GPU
 *               (different streams, no dependency between them) race on the array; serialise them.
 * Calls no cudaMalloc / cudaFree and no allocating library routine.
 */
#define TQ_STATIC_SCRATCH_BYTES (1u << 20)
int tq_score_static(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
                    const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms,
                    float* scores, int64_t lds, void* stream);
int tq_score_static_max_queries(const tq_plan* plan);

/*
 * The k vectors with the largest estimate per query (nearest-neighbour search by estimated
 * inner product, Section 4.4), sorted by descending score, equal scores by ascending id.
 * The nq x n score matrix is never formed.
 *   k 1..min(n, TQ_MAX_K);  top_scores device out [nq, k] floats;  top_ids device out [nq, k] int32
 */
int tq_topk(const tq_plan* plan, const void* Q, int q_dtype, int nq, int64_t ldq, int64_t n,
            const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms, int k,
            float* top_scores, int32_t* top_ids, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The k best of m candidate (score, id) pairs per query, sorted like tq_topk's output (descending
 * score, equal scores by ascending id).  This is the merge step of a sharded search: every shard
 * returns its local top-k (the search of Section 4.4 is independent per database vector), the lists
 * are concatenated per query and reduced to the global top-k here.  Pairs with a negative id are
 * empty slots and are ignored; ids must be distinct within a query.
 *   cand_scores, cand_ids  device, nq rows of m entries, row stride ld
 *   k 1..TQ_MAX_K;  top_scores / top_ids device out [nq, k] (may not alias the candidates);
 *   if fewer than k candidates exist the tail is filled with (-inf, -1)
 */
int tq_select_topk(const float* cand_scores, const int32_t* cand_ids, int nq, int64_t m, int64_t ld, int k,
                   float* top_scores, int32_t* top_ids, void* stream);

/*
 * Weighted sum of dequantised vectors (the value side of attention over a compressed cache,
 * Section 4.3):   out[w, :] = sum_t W[w, t] * Xhat_t,   Xhat_t as in tq_dequantize.
 * Formed in the code domain -- sum_t W nu c[idx_t] and coef * sum_t W nu gamma z_t per coordinate,
 * then one product with Pi (and S) per output row -- so no token is dequantised.
 *   W    device, nw rows of n floats (e.g. softmax weights), row stride ldw
 *   out  device out, nw rows of d floats, row stride ldo;  n = 0 gives zeros
 *   workspace  >= tq_workspace_bytes(plan, TQ_OP_WSUM, n, nw, 0)
 * Partial sums are combined in a fixed order: results are deterministic.
 */
int tq_wsum(const tq_plan* plan, const float* W, int nw, int64_t ldw, int64_t n,
            const uint8_t* idx, const uint8_t* qjl, const float* gamma, const float* norms,
            float* out, int64_t ldo, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Attention weights from estimated scores: W[w, t] = softmax over t of scale * (s1[w, t] + s2[w, t]).
 * Two score arrays are accepted because a head whose channels are split into two separately
 * quantised groups (the outlier / regular split of Section 4.3) has its score as the sum of the two
 * groups' estimates; s2 may be NULL.
 *   s1, s2  device, nw rows of n floats, row stride lds;   W device out, row stride ldw (may alias s1)
 */
int tq_softmax(const float* s1, const float* s2, int nw, int64_t n, int64_t lds, float scale,
               float* W, int64_t ldw, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Decode attention over a compressed KV cache, all KV heads of a layer in one call (the use of the
 * two quantisers in Section 4.3: keys with TurboQuant_prod so that q.k is estimated without bias,
 * values with TurboQuant_mse; channels of a head may be split into groups of different bit widths,
 * the outlier treatment of that section).  For query head r = h * q_per_kv + j of KV head h:
 *     logit_t = scale * sum_groups  estimate of < q_r[channels of the group], k_t[those channels] >
 *               (estimator of Section 3.2 on the group's codes; Algorithm 1 when the key plan is _mse),
 *     out_r   = sum_t softmax(logit)_t * v~_t,   v~_t = DeQuant_mse of the value codes (Algorithm 1),
 * evaluated on the packed codes: nothing is dequantised per token, Pi_V^T is applied once per output
 * row.  Equal to tq_score per (head, group) + tq_softmax + tq_wsum within fp32 rounding.
 *
 * One tq_kv_group per channel group.  All plans share one dimension d (a multiple of 32, <= 128) and
 * one device; the key plan may be TQ_PROD or TQ_MSE, the value plan is TQ_MSE.  Code arrays hold the
 * rows of all heads, head-major: row h * head_stride + t, head_stride >= tokens being the capacity of
 * the cache.  All pointers are device pointers owned by the caller; nothing is retained after the call.
 * tq_attend_decode only reads the code arrays, tq_kv_append writes one row per head.
 */
#define TQ_MAX_KV_GROUPS 4
typedef struct tq_kv_group {
  const tq_plan* plan_k;
  const tq_plan* plan_v;
  uint8_t* k_idx;       /* [heads*head_stride, tq_idx_row_bytes(d, b_m of plan_k)], 4-byte aligned; NULL if b_m = 0 */
  uint8_t* k_qjl;       /* [heads*head_stride, tq_qjl_row_bytes(d)] (TQ_PROD), 4-byte aligned, else NULL */
  float* k_gamma;       /* [heads*head_stride] residual norms (TQ_PROD), else NULL */
  float* k_norms;       /* [heads*head_stride] key norms, or NULL for unit norms */
  uint8_t* v_idx;       /* [heads*head_stride, tq_idx_row_bytes(d, b of plan_v)], 4-byte aligned */
  float* v_norms;       /* [heads*head_stride] value norms, or NULL */
  const int32_t* k_channels;  /* [heads, d] column of Q that is coordinate c of this group for KV head h */
  const int32_t* v_channels;  /* [heads, d] column of out that receives coordinate c of this group */
} tq_kv_group;

/* Bytes of workspace tq_attend_decode needs (query-side operands + per-slice partial results). */
size_t tq_attend_decode_workspace_bytes(int ngroups, int heads, int64_t tokens, int d);

/*   groups     host array of ngroups (1..TQ_MAX_KV_GROUPS) descriptors
 *   tokens     tokens attended to (rows 0 .. tokens-1 of every head); head_stride >= tokens
 *   Q          device, [heads*q_per_kv rows, row stride ldq elements] of q_dtype (TQ_F32 / TQ_BF16); 1 <= q_per_kv <= 4
 *   out        device fp32, [heads*q_per_kv rows, row stride ldo]; only the columns named by v_channels are written
 *   workspace  device, 256-byte aligned, >= tq_attend_decode_workspace_bytes(...)
 * tokens == 0 writes zeros to those columns.  Results do not depend on timing (fixed reduction orders).
 * Three launches: query preparation, one CTA per (head, slice of 256 tokens), merge of the slices.  Codebooks that are
 * antisymmetric (c[i] = -c[last - i], as every codebook of tq_codebook is) run on the integer tensor path (scores of
 * the Section 3.2 estimator and the value sums as bit-plane MMAs with exact int32 accumulation); any other codebook
 * runs on table-lookup CUDA-core kernels with the same results up to fp32 rounding.  The launches are programmatic
 * dependents: the first may be scheduled while the kernel ahead of it in the stream drains and waits for it before
 * it reads Q, so ordering against earlier work in the stream is what it would be for plain launches.
 * Errors: TQ_ERR_INVALID_ARG / _UNSUPPORTED / _ALIGNMENT / _WORKSPACE / _CUDA as for the other calls.
 */
int tq_attend_decode(const tq_kv_group* groups, int ngroups, int heads, int64_t tokens, int64_t head_stride, int q_per_kv,
                     const void* Q, int q_dtype, int64_t ldq, float scale, float* out, int64_t ldo,
                     void* workspace, size_t workspace_bytes, void* stream);

/* Appends one token to a compressed KV cache (the streaming use of Section 4.3: keys and values are
 * quantised as they are generated): for every KV head h and channel group, Quant_prod / Quant_mse
 * (Algorithms 2 / 1) of the group's channels of K[h] and V[h], written to row h * head_stride + position
 * of the group's code arrays (idx, qjl, gamma, norms; norms arrays may be NULL when unit norms are
 * implied).  Same comparisons as tq_quantize_*: codes agree with them up to fp32 summation order.
 *   K, V   device, [heads rows, row strides ldk / ldv elements] of kv_dtype (TQ_F32 / TQ_BF16), full head rows
 * Errors: TQ_ERR_INVALID_ARG (NULL pointers, position outside [0, head_stride)), TQ_ERR_UNSUPPORTED,
 * TQ_ERR_ALIGNMENT, TQ_ERR_CUDA.
 */
int tq_kv_append(const tq_kv_group* groups, int ngroups, int heads, int64_t head_stride, int64_t position,
                 const void* K, const void* V, int kv_dtype, int64_t ldk, int64_t ldv, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Entropy coding of the indices (Section 3.1, the paragraph on entropy encoding the codebook pointers): index
 * value l occurs with probability p_l, the mass of the l-th cell under the density of Lemma 1, so a lossless
 * prefix code stores the indices in about the entropy of {p_l} instead of b bits per coordinate (3.8 bits at
 * b = 4).  The paper leaves the code open; here it is a Huffman code given by its lengths, with code words assigned
 * canonically (symbols sorted by (length, symbol) take consecutive values, shifted left when the length grows).
 * Every vector is coded on its own.  Row stream: bit p is bit (p & 7) of byte (p >> 3); code words follow one
 * another without gaps, each from its most significant bit; a row occupies a whole number of 32-bit words.
 * Storage / transfer format only: the scans read the fixed-width rows (tq_entropy_unpack restores them exactly).
 * Plans with TQ_LAYOUT_CANONICAL and b_m >= 1.
 */
/* Huffman code lengths (1..15 in general; the coder accepts up to 12) for the 2^bits index values of the given
 * codebook in dimension d.  Host only.  centroids: host, 2^bits ascending; lengths: host out, 2^bits bytes. */
int tq_entropy_lengths(int d, int bits, const float* centroids, uint8_t* lengths);
/* Bytes of device workspace tq_entropy_measure needs for n rows. */
size_t tq_entropy_workspace_bytes(int64_t n);
/* Byte offset of every row's stream: row_offsets[i] for i < n, and row_offsets[n] = total bytes of the packed
 * array (read it back to size the output of tq_entropy_pack).
 *   lengths  host, 2^b_m code lengths (from tq_entropy_lengths or the caller's own; must satisfy Kraft's inequality)
 *   idx      device, n canonical rows;  row_offsets device out, n + 1 values;  workspace device, 256-byte aligned */
int tq_entropy_measure(const tq_plan* plan, const uint8_t* lengths, int64_t n, const uint8_t* idx,
                       uint64_t* row_offsets, void* workspace, size_t workspace_bytes, void* stream);
/* Writes the rows' streams at their offsets.  out: device, 4-byte aligned, out_bytes >= row_offsets[n]; if it is
 * smaller the rows that do not fit are skipped and the next tq_plan_status(plan) reports an error. */
int tq_entropy_pack(const tq_plan* plan, const uint8_t* lengths, int64_t n, const uint8_t* idx,
                    const uint64_t* row_offsets, uint8_t* out, size_t out_bytes, void* stream);
/* The inverse: n canonical idx rows (pad bits zero) from the packed streams. */
int tq_entropy_unpack(const tq_plan* plan, const uint8_t* lengths, int64_t n, const uint8_t* packed,
                      const uint64_t* row_offsets, uint8_t* idx, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TQ_H_ */

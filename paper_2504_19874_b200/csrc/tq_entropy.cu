// Entropy coding of the indices (Section 3.1, "entropy encoding codebook pointers"): index value l occurs with
// probability p_l (mass of the l-th cell of the codebook under the density of Lemma 1), so a lossless prefix code
// brings the average width from b bits towards the entropy of {p_l} (3.8 bits at b = 4, about 5 % saved).
//
// The code is given by its lengths (tq_entropy_lengths builds the Huffman lengths from the cell masses); code
// words are assigned canonically from the lengths: symbols sorted by (length, symbol) receive consecutive
// values, shifted left whenever the length grows.  Every vector is coded on its own, so rows are decoded in
// parallel.  Row stream: bit p is bit (p & 7) of byte (p >> 3); code words follow one another without gaps,
// each written from its most significant bit; a row occupies a whole number of 32-bit words.
//
//   measure   one warp per row: lane l sums the code lengths of its chunk of coordinates; row bytes -> sizes
//   offsets   exclusive prefix sum of the row sizes (one CTA walks the rows in pieces of 1024 with a carry)
//   pack      one warp per row: warp scan of the lanes' bit counts gives every lane its bit offset; a lane
//             shifts its code words into a 64-bit buffer and flushes whole words (the first and last word of
//             a lane's chunk, shared with its neighbours, by atomic OR into the zeroed output)
//   unpack    one thread per row: table look-up on the next maxlen bits gives (symbol, length)
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "tq_internal.h"

namespace tq {
namespace entropy {

namespace {

constexpr int kMaxLen = 12;   // longest code word accepted (look-up table of 2^12 entries in shared memory)

struct Code {
  uint8_t len[16];
  uint16_t word[16];   // canonical code word, most significant bit first
  int bits;            // b_m
  int maxlen;
};

struct Args {
  int64_t n;
  int d;
  const uint8_t* idx;
  size_t idx_rb;
  Code code;
};

__device__ __forceinline__ int symbol_at(const uint8_t* row, int j, int bits) {
  const int bp = j * bits, b0 = bp >> 3, sh = bp & 7;
  unsigned v = row[b0];
  if (sh + bits > 8) v |= (unsigned)row[b0 + 1] << 8;
  return (v >> sh) & ((1u << bits) - 1u);
}

// Row sizes in bytes (multiple of 4).
__global__ void __launch_bounds__(256) measure_kernel(Args a, uint32_t* __restrict__ sizes) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= a.n) return;
  const uint8_t* r = a.idx + (size_t)row * a.idx_rb;
  const int chunk = (a.d + 31) / 32;
  int bits = 0;
  for (int j = lane * chunk; j < min(a.d, (lane + 1) * chunk); ++j) bits += a.code.len[symbol_at(r, j, a.code.bits)];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, o);
  if (lane == 0) sizes[row] = (uint32_t)((bits + 31) / 32 * 4);
}

// offsets[i] = sum of sizes[0 .. i-1], offsets[n] = total.  One CTA of 1024 threads.
__global__ void __launch_bounds__(1024) offsets_kernel(const uint32_t* __restrict__ sizes, int64_t n, uint64_t* __restrict__ offsets) {
  __shared__ unsigned long long warp_tot[32];
  __shared__ unsigned long long carry;
  if (threadIdx.x == 0) carry = 0ull;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int64_t base = 0; base < n; base += 1024) {
    const int64_t i = base + threadIdx.x;
    const unsigned long long v = i < n ? sizes[i] : 0ull;
    unsigned long long incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      unsigned long long w = warp_tot[lane], wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += t;
      }
      warp_tot[lane] = wi - w;   // exclusive
    }
    __syncthreads();
    const unsigned long long excl = carry + warp_tot[warp] + incl - v;
    if (i < n) offsets[i] = excl;
    __syncthreads();
    if (threadIdx.x == 1023) carry = excl + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) offsets[n] = carry;
}

__global__ void __launch_bounds__(256) pack_kernel(Args a, const uint64_t* __restrict__ offsets, uint8_t* __restrict__ out,
                                                   size_t out_bytes, int* status) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= a.n) return;
  if (offsets[row + 1] > out_bytes) {   // the caller's buffer is smaller than the measured total
    if (lane == 0) atomicExch(status, TQ_ERR_WORKSPACE);
    return;
  }
  const uint8_t* r = a.idx + (size_t)row * a.idx_rb;
  uint32_t* dst = reinterpret_cast<uint32_t*>(out + offsets[row]);
  const int chunk = (a.d + 31) / 32;
  const int j0 = lane * chunk, j1 = min(a.d, (lane + 1) * chunk);
  int bits = 0;
  for (int j = j0; j < j1; ++j) bits += a.code.len[symbol_at(r, j, a.code.bits)];
  int incl = bits;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  const int start = incl - bits, end = incl;   // this lane's bits occupy [start, end) of the row stream
  if (bits == 0) return;
  int word = start >> 5, fill = start & 31;    // current output word and the bits of it already in `buf`
  unsigned long long buf = 0ull;
  const int first_word = word, last_word = (end - 1) >> 5;
  auto flush = [&](uint32_t v) {
    // words shared with a neighbouring lane: the first of the chunk (unless it starts on a word boundary) and the last
    // (unless it ends on one); the output was zeroed, so OR composes them
    if ((word == first_word && (start & 31)) || (word == last_word && (end & 31))) atomicOr(dst + word, v);
    else dst[word] = v;
    ++word;
  };
  for (int j = j0; j < j1; ++j) {
    const int s = symbol_at(r, j, a.code.bits);
    const int l = a.code.len[s];
    // the code word from its most significant bit = stream order: reverse its l bits into LSB-first order
    const unsigned rev = __brev((unsigned)a.code.word[s]) >> (32 - l);
    buf |= (unsigned long long)rev << fill;
    fill += l;
    if (fill >= 32) {
      flush((uint32_t)buf);
      buf >>= 32;
      fill -= 32;
    }
  }
  if (fill > 0) flush((uint32_t)buf);
}

__global__ void __launch_bounds__(128) unpack_kernel(Args a, const uint64_t* __restrict__ offsets, const uint8_t* __restrict__ packed,
                                                     uint8_t* __restrict__ idx_out) {
  __shared__ uint16_t lut[1 << kMaxLen];   // next maxlen stream bits (LSB first) -> symbol | length << 8
  const int L = a.code.maxlen;
  for (int u = threadIdx.x; u < (1 << L); u += blockDim.x) {
    uint16_t e = 0;
    for (int s = 0; s < (1 << a.code.bits); ++s) {
      const int l = a.code.len[s];
      if (l == 0) continue;
      const unsigned rev = __brev((unsigned)a.code.word[s]) >> (32 - l);
      if ((u & ((1u << l) - 1u)) == rev) e = (uint16_t)(s | (l << 8));
    }
    lut[u] = e;
  }
  __syncthreads();
  const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= a.n) return;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(packed + offsets[row]);
  const int nwords = (int)((offsets[row + 1] - offsets[row]) / 4);
  uint32_t* dst = reinterpret_cast<uint32_t*>(idx_out + (size_t)row * a.idx_rb);
  const int row_words = (int)(a.idx_rb / 4);
  unsigned long long in = 0ull, outbuf = 0ull;
  int have = 0, rd = 0, ofill = 0, ow = 0;
  const unsigned mask = (1u << L) - 1u;
  for (int j = 0; j < a.d; ++j) {
    if (have < L) {   // a zero word past the end of the row stream only pads the look-up of the last code words
      in |= (unsigned long long)(rd < nwords ? src[rd] : 0u) << have;
      ++rd;
      have += 32;
    }
    const uint16_t e = lut[(unsigned)in & mask];
    const int l = e >> 8;
    in >>= l;
    have -= l;
    outbuf |= (unsigned long long)(e & 255u) << ofill;
    ofill += a.code.bits;
    if (ofill >= 32) {
      dst[ow++] = (uint32_t)outbuf;
      outbuf >>= 32;
      ofill -= 32;
    }
  }
  if (ofill > 0) dst[ow++] = (uint32_t)outbuf;
  for (; ow < row_words; ++ow) dst[ow] = 0u;   // pad words of the row
}

int make_code(const tq_plan* plan, const uint8_t* lengths, Code* c, const char* who) {
  const int L = 1 << plan->mse_bits;
  std::memset(c, 0, sizeof(*c));
  c->bits = plan->mse_bits;
  double kraft = 0.0;
  std::vector<std::pair<int, int>> order;
  for (int s = 0; s < L; ++s) {
    TQ_REQUIRE(lengths[s] >= 1 && lengths[s] <= kMaxLen, TQ_ERR_UNSUPPORTED, "%s: code length %d of symbol %d outside 1..%d", who,
               (int)lengths[s], s, kMaxLen);
    c->len[s] = lengths[s];
    c->maxlen = std::max(c->maxlen, (int)lengths[s]);
    kraft += std::ldexp(1.0, -(int)lengths[s]);
    order.push_back({(int)lengths[s], s});
  }
  TQ_REQUIRE(kraft <= 1.0, TQ_ERR_INVALID_ARG, "%s: the lengths violate Kraft's inequality (no prefix code has them)", who);
  std::sort(order.begin(), order.end());
  unsigned code = 0;
  int prev = 0;
  for (const auto& e : order) {
    code <<= e.first - prev;
    c->word[e.second] = (uint16_t)code;
    ++code;
    prev = e.first;
  }
  return TQ_OK;
}

int check(const tq_plan* plan, const char* who, const uint8_t* lengths, int64_t n) {
  TQ_REQUIRE(plan != nullptr, TQ_ERR_INVALID_ARG, "%s: plan is NULL", who);
  int dev = -1;
  TQ_CHECK_CUDA(cudaGetDevice(&dev), who);
  TQ_REQUIRE(dev == plan->device, TQ_ERR_INVALID_ARG, "%s: plan was created on device %d, current device is %d", who, plan->device, dev);
  TQ_REQUIRE(plan->mse_bits >= 1, TQ_ERR_UNSUPPORTED, "%s: the plan has no index array (0-bit MSE stage)", who);
  TQ_REQUIRE(plan->layout == TQ_LAYOUT_CANONICAL, TQ_ERR_UNSUPPORTED, "%s: the plan must use the canonical code layout", who);
  TQ_REQUIRE(lengths != nullptr && n >= 0, TQ_ERR_INVALID_ARG, "%s: lengths is NULL or n is negative", who);
  return TQ_OK;
}

}  // namespace
}  // namespace entropy

// Mass of every cell of the codebook under the density of Lemma 1 (defined in tq_host.cu).
int cell_masses(int d, int levels, const float* centroids, double* p_out);

}  // namespace tq

using namespace tq;

extern "C" int tq_entropy_lengths(int d, int bits, const float* centroids, uint8_t* lengths) {
  const char* who = "tq_entropy_lengths";
  TQ_REQUIRE(d >= 2 && d <= TQ_MAX_D && bits >= 1 && bits <= 4, TQ_ERR_UNSUPPORTED, "%s: d=%d bits=%d unsupported", who, d, bits);
  TQ_REQUIRE(centroids != nullptr && lengths != nullptr, TQ_ERR_INVALID_ARG, "%s: NULL argument", who);
  const int L = 1 << bits;
  double p[16];
  int rc = cell_masses(d, L, centroids, p);
  if (rc) return rc;
  // Huffman: merge the two least probable nodes; among equals the one created earlier goes first
  struct Node { double p; int order; unsigned mask; };
  std::vector<Node> nodes;
  int depth[16] = {0};
  for (int s = 0; s < L; ++s) nodes.push_back({p[s], s, 1u << s});
  int created = L;
  while (nodes.size() > 1) {
    std::sort(nodes.begin(), nodes.end(), [](const Node& a, const Node& b) { return a.p != b.p ? a.p < b.p : a.order < b.order; });
    const Node a = nodes[0], b = nodes[1];
    for (int s = 0; s < L; ++s)
      if ((a.mask | b.mask) >> s & 1u) ++depth[s];
    nodes.erase(nodes.begin(), nodes.begin() + 2);
    nodes.push_back({a.p + b.p, created++, a.mask | b.mask});
  }
  for (int s = 0; s < L; ++s) lengths[s] = (uint8_t)depth[s];
  return TQ_OK;
}

extern "C" size_t tq_entropy_workspace_bytes(int64_t n) { return n > 0 ? (size_t)((n * 4 + 255) / 256 * 256) : 0; }

extern "C" int tq_entropy_measure(const tq_plan* plan, const uint8_t* lengths, int64_t n, const uint8_t* idx, uint64_t* row_offsets,
                                  void* workspace, size_t workspace_bytes, void* stream) {
  const char* who = "tq_entropy_measure";
  TQ_RANGE(who);
  int rc = entropy::check(plan, who, lengths, n);
  if (rc) return rc;
  TQ_REQUIRE(row_offsets != nullptr && (n == 0 || idx != nullptr), TQ_ERR_INVALID_ARG, "%s: NULL argument", who);
  TQ_REQUIRE(workspace_bytes >= tq_entropy_workspace_bytes(n) && (n == 0 || workspace != nullptr), TQ_ERR_WORKSPACE,
             "%s: workspace of %zu bytes, %zu needed", who, workspace_bytes, tq_entropy_workspace_bytes(n));
  entropy::Args a;
  if ((rc = entropy::make_code(plan, lengths, &a.code, who))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  a.n = n; a.d = plan->d; a.idx = idx; a.idx_rb = plan->idx_row_bytes;
  uint32_t* sizes = static_cast<uint32_t*>(workspace);
  if (n > 0) {
    entropy::measure_kernel<<<(unsigned)((n + 7) / 8), 256, 0, st>>>(a, sizes);
    TQ_CHECK_CUDA(cudaGetLastError(), who);
  }
  entropy::offsets_kernel<<<1, 1024, 0, st>>>(sizes, n, row_offsets);
  count_launches(n > 0 ? 2 : 1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

extern "C" int tq_entropy_pack(const tq_plan* plan, const uint8_t* lengths, int64_t n, const uint8_t* idx, const uint64_t* row_offsets,
                               uint8_t* out, size_t out_bytes, void* stream) {
  const char* who = "tq_entropy_pack";
  TQ_RANGE(who);
  int rc = entropy::check(plan, who, lengths, n);
  if (rc) return rc;
  if (n == 0) return TQ_OK;
  TQ_REQUIRE(idx != nullptr && row_offsets != nullptr && out != nullptr, TQ_ERR_INVALID_ARG, "%s: NULL argument", who);
  TQ_REQUIRE((reinterpret_cast<uintptr_t>(out) & 3) == 0, TQ_ERR_ALIGNMENT, "%s: out is not 4-byte aligned", who);
  entropy::Args a;
  if ((rc = entropy::make_code(plan, lengths, &a.code, who))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  a.n = n; a.d = plan->d; a.idx = idx; a.idx_rb = plan->idx_row_bytes;
  TQ_CHECK_CUDA(cudaMemsetAsync(out, 0, out_bytes, st), who);
  entropy::pack_kernel<<<(unsigned)((n + 7) / 8), 256, 0, st>>>(a, row_offsets, out, out_bytes, plan->d_status);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

extern "C" int tq_entropy_unpack(const tq_plan* plan, const uint8_t* lengths, int64_t n, const uint8_t* packed,
                                 const uint64_t* row_offsets, uint8_t* idx, void* stream) {
  const char* who = "tq_entropy_unpack";
  TQ_RANGE(who);
  int rc = entropy::check(plan, who, lengths, n);
  if (rc) return rc;
  if (n == 0) return TQ_OK;
  TQ_REQUIRE(idx != nullptr && row_offsets != nullptr && packed != nullptr, TQ_ERR_INVALID_ARG, "%s: NULL argument", who);
  TQ_REQUIRE((reinterpret_cast<uintptr_t>(packed) & 3) == 0 && (reinterpret_cast<uintptr_t>(idx) & 15) == 0, TQ_ERR_ALIGNMENT,
             "%s: packed / idx is misaligned", who);
  entropy::Args a;
  if ((rc = entropy::make_code(plan, lengths, &a.code, who))) return rc;
  a.n = n; a.d = plan->d; a.idx = nullptr; a.idx_rb = plan->idx_row_bytes;
  entropy::unpack_kernel<<<(unsigned)((n + 127) / 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(a, row_offsets, packed, idx);
  count_launches(1);
  TQ_CHECK_CUDA(cudaGetLastError(), who);
  return TQ_OK;
}

// What the two scan engines of TQ_LAYOUT_NIBBLE (register-fed in tq_scan_nib.cu, tcgen05 in tq_scan_tc.cu) must
// agree on so that they form identical integers, hence identical estimates: the fixed-point scales of a query and
// its three kinds of weights.
//   T  = sum_j Wh_j h[idx_j] + sum_j Wl_j l[idx_j],   Wh = round(q' 2^fh), Wl = round(q' 2^(fh-8)),  c_i ~ delta (256 h_i + l_i)
//   TQ = sum_i J_i (16 * 8 z_i  or  128 z_i),          J = round(q'' sq)   (low-nibble coordinates carry the 16)
//   estimate = nu ( delta 2^(8-fh) T  +  coef gamma ( TQ / (64 sq) - sum_i q''_i ) )
#pragma once

#include <cstdint>

namespace tq {
namespace nib {

struct QScale {
  int fh;      // Wh = round(q' 2^fh)
  double sq;   // J = round(q'' sq)
};

struct QConst {
  float sa;   // centroid term = T  * sa
  float ss;   // sign term     = TQ * ss + cs
  float cs;
  int pad;
};

// From max |q'|, max |q''| (exact in fp32) and sum q''.
__device__ __forceinline__ QScale make_scale(float mx1, float mx2) {
  QScale s;
  // |v| < 2^e  ->  |v| 2^(22 - e) < 2^22: Wh in three signed radix-256 digits, Wl = Wh / 256 in two
  s.fh = 0;
  if (mx1 > 0.f && isfinite(mx1)) {
    int e;
    frexpf(mx1, &e);
    s.fh = 22 - e;
  }
  // J in two signed digits (|J| <= 127 * 257): the scale need not be a power of two, so all of that range is used
  s.sq = (mx2 > 0.f && isfinite(mx2)) ? 32639.0 / (double)mx2 : 1.0;
  return s;
}

__device__ __forceinline__ QConst make_const(const QScale& s, double delta, double sum_q2) {
  QConst c;
  c.sa = (float)(delta * ldexp(1.0, 8 - s.fh));
  c.ss = (float)(1.0 / (64.0 * s.sq));
  c.cs = (float)(-sum_q2);
  c.pad = 0;
  return c;
}

__device__ __forceinline__ double pow2_of(int e) {
  if (e < -1000 || e > 1000) return ldexp(1.0, e);
  return __hiloint2double((e + 1023) << 20, 0);
}

// type 0: Wh, 1: Wl, 2: J.  Non-finite query entries contribute nothing.
__device__ __forceinline__ long long weight(const QScale& s, int type, float q) {
  const double scale = type == 0 ? pow2_of(s.fh) : type == 1 ? pow2_of(s.fh - 8) : s.sq;
  const double bound = type == 0 ? 4194304.0 : type == 1 ? 16384.0 : 32639.0;
  double J = rint((double)q * scale);
  if (!(fabs(J) <= bound)) J = 0.0;
  return (long long)J;
}

__device__ __forceinline__ int digit_of(long long J, int limb) {
  int dg = 0;
  for (int l = 0; l <= limb; ++l) {
    dg = (int)(((J + 128) & 255) - 128);
    J = (J - dg) >> 8;
  }
  return dg;
}

// Coordinate stored in nibble `cib` (0..127) of 64-byte block b of the sequence [idx row | qjl row], or -1 when that
// nibble lies in the zero fill.
__host__ __device__ inline int coord_of_block(int nbi, int idx_rb, int qjl_rb, int d, int b, int cib) {
  int coord;
  if (b < nbi) {
    const int byte = 64 * b + (cib >> 1);
    if (byte >= idx_rb) return -1;
    coord = 2 * byte + (cib & 1);
  } else {
    const int byte = 64 * (b - nbi) + (cib >> 1);
    if (byte >= qjl_rb) return -1;
    coord = 2 * idx_rb + 2 * byte + (cib & 1);
  }
  return coord < d ? coord : -1;
}

}  // namespace nib
}  // namespace tq

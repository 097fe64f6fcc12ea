// The two stochastic quantizers of the encoder (device code shared by the packet and the unframed writers).
#pragma once

#include "cvlc_common.cuh"

namespace cvlc {

#ifdef __CUDACC__

// PQ: stochastic rounding of num = x - lo onto the 2^y uniform centroids of [lo, hi]; den = hi - lo > 0, Lc = 2^y - 1,
// scale = Lc / den, u = the coordinate's random word / 2^32.  t = (num / den) * Lc decides floor(t) and [u < frac(t)].
// num * scale is within a few ulp of it; unless its fraction sits that close to 0, 1 or u, both decisions are the same
// and the division is not needed.
__device__ __forceinline__ uint32_t pq_quantize(double num, double den, double Lc, double scale, double u) {
  const double tf = __dmul_rn(num, scale);
  const double jf = floor(tf);
  const double ff = __dsub_rn(tf, jf);
  const double eps = __dmul_rn(tf, 0x1p-48) + 0x1p-1000;
  if (ff > eps && ff < 1.0 - eps && fabs(ff - u) > eps && jf < Lc) return __double2uint_rz(jf) + ((u < ff) ? 1u : 0u);
  const double t = __dmul_rn(__ddiv_rn(num, den), Lc);
  double j0 = floor(t);
  if (j0 > Lc) j0 = Lc;
  const double frac = __dsub_rn(t, j0);
  return __double2uint_rz(j0) + ((u < frac) ? 1u : 0u);
}

// QSGD: level of a = |x| against the packet's norm dn > 0 on a grid of sq = sqd steps; scale = sqd / dn
__device__ __forceinline__ uint32_t qsgd_quantize_level(double a, double dn, double sqd, uint32_t sq, double scale, double u) {
  const double tf = __dmul_rn(a, scale);
  const double jf = floor(tf);
  const double ff = __dsub_rn(tf, jf);
  const double eps = __dmul_rn(tf, 0x1p-48) + 0x1p-1000;
  if (ff > eps && ff < 1.0 - eps && fabs(ff - u) > eps && jf < sqd) return __double2uint_rz(jf) + ((u < ff) ? 1u : 0u);
  const double t = __dmul_rn(__ddiv_rn(a, dn), sqd);
  double j0 = floor(t);
  if (j0 > sqd) j0 = sqd;
  const double frac = __dsub_rn(t, j0);
  uint32_t level = __double2uint_rz(j0) + ((u < frac) ? 1u : 0u);
  if (level > sq) level = sq;
  return level;
}

// the l2-norm of P values whose exact squares sit in sqv, added in the given order in double, rounded to fp32
// (FLT_MAX beyond the fp32 range); one thread walks the chain: the order is part of the stream's definition
__device__ __forceinline__ float qsgd_norm_of_squares(const double* sqv, uint32_t P) {
  double sum = 0.0;
  uint32_t j = 0;
  for (; j + 8 <= P; j += 8) {
    double v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = sqv[j + u];
#pragma unroll
    for (int u = 0; u < 8; ++u) sum = __dadd_rn(sum, v[u]);
  }
  for (; j < P; ++j) sum = __dadd_rn(sum, sqv[j]);
  const double rt = __dsqrt_rn(sum);
  return (rt > 3.4028234663852886e38) ? 3.4028234663852886e38f : __double2float_rn(rt);
}

#endif  // __CUDACC__

}  // namespace cvlc

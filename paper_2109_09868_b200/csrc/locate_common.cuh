// Device helpers shared by the two locator kernels (Algorithm 2): warp arg-min with the paper-independent
// tie rule "lower index first", and Householder reflectors over statically bounded row ranges.
#pragma once
#include "common.cuh"

namespace approxifer {
namespace locate_detail {

constexpr unsigned kFull = 0xffffffffu;

// Lexicographic "smaller (key, index)" butterfly: returns the index of the
// minimum over the warp; ties go to the lower index.
__device__ __forceinline__ int warp_argmin(double key, int idx) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const double k2 = __shfl_xor_sync(kFull, key, o);
    const int i2 = __shfl_xor_sync(kFull, idx, o);
    if (k2 < key || (k2 == key && i2 < idx)) {
      key = k2;
      idx = i2;
    }
  }
  return idx;
}

// Normalised reflector of `col` restricted to rows >= ROW0:
// v = (x - akk e_ROW0) / sqrt(c), c = |x|(|x| + |x_ROW0|), so that H = I - v v^T
// maps x to akk e_ROW0.  v_out[r] is written for r >= (ROW0 rounded down to even);
// returns akk (0 and v = 0 when the sub-column is exactly zero).
template <int NMAX, int ROW0>
__device__ __forceinline__ double make_reflector(const double (&col)[NMAX], double* v_out) {
  double s2a = 0.0, s2b = 0.0;
#pragma unroll
  for (int r = ROW0; r < NMAX; r += 2) {
    s2a = fma(col[r], col[r], s2a);
    if (r + 1 < NMAX) s2b = fma(col[r + 1], col[r + 1], s2b);
  }
  const double s2 = s2a + s2b;
  const double x0 = col[ROW0];
  const bool nz = s2 > 0.0;
  const double normx = nz ? s2 * rsqrt(s2) : 0.0;
  const double akk = (x0 >= 0.0) ? -normx : normx;
  const double c = fma(fabs(x0), normx, s2);
  const double scale = nz ? rsqrt(c) : 0.0;
  if (ROW0 & 1) v_out[ROW0 - 1] = 0.0;
  v_out[ROW0] = (x0 - akk) * scale;
#pragma unroll
  for (int r = ROW0 + 1; r < NMAX; ++r) v_out[r] = col[r] * scale;
  return akk;
}

// col <- (I - v v^T) col for a reflector whose entries before ROW0 are zero.
template <int NMAX, int ROW0>
__device__ __forceinline__ void apply_reflector(double (&col)[NMAX], const double* v) {
  constexpr int R0 = ROW0 & ~1;
  double2 vv[(NMAX - R0) / 2];
  double sa = 0.0, sb = 0.0;
#pragma unroll
  for (int r = R0; r < NMAX; r += 2) {
    vv[(r - R0) / 2] = *reinterpret_cast<const double2*>(v + r);
    sa = fma(vv[(r - R0) / 2].x, col[r], sa);
    sb = fma(vv[(r - R0) / 2].y, col[r + 1], sb);
  }
  const double s = -(sa + sb);
#pragma unroll
  for (int r = R0; r < NMAX; r += 2) {
    col[r] = fma(s, vv[(r - R0) / 2].x, col[r]);
    col[r + 1] = fma(s, vv[(r - R0) / 2].y, col[r + 1]);
  }
}

}  // namespace locate_detail
}  // namespace approxifer

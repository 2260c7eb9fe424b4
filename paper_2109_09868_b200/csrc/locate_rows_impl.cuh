// ApproxIFER Byzantine-worker locator (Algorithm 2), thread-per-class variant for K+E <= 15; also (K+E <= 13) Algorithm 1's
// homogeneous system and Algorithm 3's rational function as alternative last steps (see the kernel's MODE).
//
// Same mathematics as locate_kernel (locate.cu): the P-part of the per-class least-squares problem is
// eliminated with an orthonormal basis N of the complement of {polynomials of degree < M} on the available
// nodes (M = K+E), which depends on the mask only, and the Q-part solves the (n-M) x (M-1) problem
//     B q = -b0,   B[r][l] = sum_i N[i][r] y_i b_i^l (l = 1..M-1),   b0[r] = sum_i N[i][r] y_i.
// Different parallelisation: after one warp per group has produced N (from the basis of the full node set by a
// few small reflectors when few workers are missing, else by Householder reflectors of the group's own
// Vandermonde block applied to unit vectors), every (group, class) pair gets ONE THREAD.
// The thread generates the rows of [B | -b0] one at a time from N (shared memory, shared by the group's
// threads) and its own 22-odd predictions (shared memory, one column per thread) and folds each row into a
// square-root-free triangular factor (Gentleman's form of the Givens row update).  The factor (at most
// 45 + 9 doubles) lives in registers with static indices; the rows are never stored.  No lane waits for
// another lane: there is no serial single-lane section, and all 32 lanes of a warp work on different
// problems.  The thread then evaluates a_r = Q(b_r) for every available worker, picks the E smallest |a_r|
// (ties to the lower worker) and votes with shared-memory atomics; a warp per group elects the E most voted
// workers.  Everything runs in fp64.
#pragma once
#include <type_traits>

#include "common.cuh"
#include "locate_common.cuh"

namespace approxifer {

namespace {

using namespace locate_detail;

static_assert(sizeof(LocateArgs) + sizeof(LocateTables) + sizeof(LocateBasis) + sizeof(DecodeTables) + 16 <= 32764,
              "locator kernel parameters exceed the launch limit (blocks above 4 KB need CUDA 12.1 or later)");

constexpr int kRowsThreads = 128;
constexpr int kRowsWarps = kRowsThreads / 32;
constexpr int kMaxGroupsPerCta = 16;

template <int NMAX, int M>
struct GroupSmem {
  static constexpr int MP = (M + 1) / 2 * 2;  // powers padded to pairs: rows stay 16-byte aligned
  double nt[NMAX - M][NMAX];                  // nt[r][i] = N[i][r]
  double pw[NMAX][MP];                        // pw[i][k] = b_i^k
  double xs[NMAX];                            // b_i
  long long yoff[NMAX];                       // element offset of the i-th available worker's row
  int votes[NMAX];
  uint32_t mask;
  int n;  // workers available; -1: fewer than 2(K+E), nothing to locate
  uint32_t status;
  int pad;
};

// Bytes of the per-CTA scratch: the threads' predictions, or (during set-up) the warps' reflectors and the
// transposed full-set basis, whichever is larger.
template <int NMAX, int M>
__host__ __device__ constexpr size_t scratch_bytes() {
  const size_t y_bytes = (size_t)NMAX * kRowsThreads * sizeof(float);
  const size_t setup_bytes = ((size_t)kRowsWarps * M + (NMAX - M)) * NMAX * sizeof(double);
  return y_bytes > setup_bytes ? y_bytes : setup_bytes;
}

// The k-th of M ranks spread evenly over 0 .. n-1 (first and last included).
template <int M>
__host__ __device__ __forceinline__ int spread_rank(int k, int n) {
  return (k * (n - 1)) / (M - 1);
}

template <int NMAX, int M, int K0 = 0>
__device__ __forceinline__ void rows_pblock_factor(double (&col)[NMAX], int lane, double (*refl)[NMAX]) {
  if constexpr (K0 < M) {
    if (lane == K0) make_reflector<NMAX, K0>(col, refl[K0]);
    __syncwarp();
    if (lane > K0 && lane < M) apply_reflector<NMAX, K0>(col, refl[K0]);
    rows_pblock_factor<NMAX, M, K0 + 1>(col, lane, refl);
  }
}
// col <- H_0 H_1 .. H_{M-1} col (reflectors applied last to first)
template <int NMAX, int M, int K0 = M - 1>
__device__ __forceinline__ void rows_apply_q(double (&col)[NMAX], double (*refl)[NMAX]) {
  if constexpr (K0 >= 0) {
    apply_reflector<NMAX, K0>(col, refl[K0]);
    rows_apply_q<NMAX, M, K0 - 1>(col, refl);
  }
}

// Index of the r-th (0-based) set bit of m; r < popc(m).  Five halving steps on population counts.
__device__ __forceinline__ int nth_set_bit(uint32_t m, int r) {
  int pos = 0;
#pragma unroll
  for (int w = 16; w > 0; w >>= 1) {
    const uint32_t low = m & ((1u << w) - 1u);
    const int c = __popc(low);
    const bool up = r >= c;
    r = up ? r - c : r;
    m = up ? (m >> w) : low;
    pos += up ? w : 0;
  }
  return pos;
}

// 1/h for a positive, normal h: hardware seed (about 20 bits) and two Newton steps, no special cases.
__device__ __forceinline__ double rcp_pos(double h) {
  double y;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(y) : "d"(h));
  double e = fma(-h, y, 1.0);
  y = fma(y, e, y);
  e = fma(-h, y, 1.0);
  y = fma(y, e, y);
  return y;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;  // the same value, bit for bit, in every lane
}

// The complement basis of a group with only a few workers missing, derived from the basis Nf of the full node
// set.  A vector that is orthogonal to the polynomials on the available nodes is, padded with zeros at the
// missing nodes, orthogonal to them on all nodes; so the group's complement is { Nf c : (Nf c)_i = 0 for every
// missing i }, and with Q = H_0 .. H_{s-1} the Householder factor of the (W-M) x s matrix of the missing
// workers' rows of Nf, the columns s .. W-M-1 of Nf Q restricted to the available workers are an orthonormal
// basis of it.  Cost: s small reflectors of length W-M (lane = column of Nf) and their application to one row of
// Nf per lane (lane = available worker), instead of M reflectors of length n and n-M long back-transformations.
//   nft[d * NMAX + i] = Nf[i][d] (zero beyond W or W-M), vq: scratch of SMAX * (NMAX-M) doubles.
template <int NMAX, int M>
__device__ __forceinline__ void rows_basis_from_full(GroupSmem<NMAX, M>& sm, const double* nft, double* vq, uint32_t mask,
                                                     int W, int n, int my_worker, int lane) {
  constexpr int DN = NMAX - M;
  constexpr int SMAX = M / 2 + 1;
  const int s = W - n;
  const uint32_t absent = ~mask & worker_bits(W);
  if (s > 0) {
    double arow[SMAX];  // lane = d: arow[t] = Nf[t-th missing worker][d]
#pragma unroll
    for (int t = 0; t < SMAX; ++t) {
      const int it = (t < s) ? nth_set_bit(absent, t) : 0;
      arow[t] = (t < s && lane < DN) ? nft[lane * NMAX + it] : 0.0;
    }
#pragma unroll
    for (int t = 0; t < SMAX; ++t) {
      if (t < s) {  // uniform over the warp
        const double x = (lane >= t) ? arow[t] : 0.0;
        const double s2 = warp_sum(x * x);
        const double x0 = __shfl_sync(kFull, arow[t], t);
        const bool nz = s2 > 0.0;
        const double normx = nz ? s2 * rsqrt(s2) : 0.0;
        const double akk = (x0 >= 0.0) ? -normx : normx;
        const double c = fma(fabs(x0), normx, s2);
        const double scale = nz ? rsqrt(c) : 0.0;
        const double v = (lane == t) ? (x0 - akk) * scale : x * scale;
        if (lane < DN) vq[t * DN + lane] = v;
#pragma unroll
        for (int t2 = t + 1; t2 < SMAX; ++t2) {
          if (t2 < s) {
            const double dot = warp_sum(v * arow[t2]);
            arow[t2] = fma(-dot, v, arow[t2]);
          }
        }
      }
    }
    __syncwarp();
  }
  // lane = rank of an available worker: its row of Nf, times H_0 .. H_{s-1}
  if (lane < NMAX) {
    double x[DN];
#pragma unroll
    for (int d = 0; d < DN; ++d) x[d] = (lane < n) ? nft[d * NMAX + my_worker] : 0.0;
#pragma unroll
    for (int t = 0; t < SMAX; ++t) {
      if (t < s) {
        const double* v = vq + t * DN;
        double da = 0.0, db = 0.0;
#pragma unroll
        for (int d = 0; d < DN; d += 2) {
          da = fma(x[d], v[d], da);
          if (d + 1 < DN) db = fma(x[d + 1], v[d + 1], db);
        }
        const double dot = -(da + db);
#pragma unroll
        for (int d = 0; d < DN; ++d) x[d] = fma(dot, v[d], x[d]);
      }
    }
#pragma unroll
    for (int d = 0; d < DN; ++d)
      if (d >= s) sm.nt[d - s][lane] = x[d];
  }
}

// One warp: nodes, powers and the complement basis N of one group.
template <int NMAX, int M>
__device__ __forceinline__ void rows_setup_group(GroupSmem<NMAX, M>& sm, double (*refl)[NMAX], const double* nft,
                                                 const LocateArgs& a, const LocateTables& tab, int64_t g, int lane) {
  using SM = GroupSmem<NMAX, M>;
  const uint32_t mask = a.mask[g] & worker_bits(a.W);
  const int n = __popc(mask);
  if (lane == 0) {
    sm.mask = mask;
    sm.n = (n < 2 * M) ? -1 : n;  // Algorithm 1's condition N-S+1 >= 2(K+E)
    sm.status = (n < 2 * M) ? kStLocateUnderdetermined : 0u;
  }
  if (lane < NMAX) sm.votes[lane] = 0;
  if (n < 2 * M) return;
  const int my_worker = (lane < n) ? nth_set_bit(mask, lane) : -1;
  if (lane < NMAX) {
    const double b = (lane < n) ? tab.beta[my_worker] : 0.0;
    sm.xs[lane] = b;
    sm.yoff[lane] = (lane < n) ? (a.rows.on ? (long long)a.rows.off[my_worker] : (long long)my_worker * a.y_rs) : 0;
    double p = 1.0;
#pragma unroll
    for (int k = 0; k < SM::MP; ++k) {
      sm.pw[lane][k] = (lane < n && k < M) ? p : 0.0;
      p *= b;
    }
  }
  __syncwarp();
  if (a.W - n <= M / 2 + 1) {
    rows_basis_from_full<NMAX, M>(sm, nft, &refl[0][0], mask, a.W, n, my_worker, lane);
    return;
  }
  // many workers missing: Householder reflectors of the group's own Vandermonde block, applied to unit vectors
  double col[NMAX];
#pragma unroll
  for (int r = 0; r < NMAX; ++r) col[r] = (lane < M) ? sm.pw[r][lane] : 0.0;
  rows_pblock_factor<NMAX, M>(col, lane, refl);
  __syncwarp();
  // lane r < NMAX-M: column M+r of Q = H_0 .. H_{M-1}
#pragma unroll
  for (int r = 0; r < NMAX; ++r) col[r] = (r == M + lane) ? 1.0 : 0.0;
  if (lane < NMAX - M) {
    rows_apply_q<NMAX, M>(col, refl);
#pragma unroll
    for (int r = 0; r < NMAX; ++r) sm.nt[lane][r] = col[r];
  }
}


// MODE 0: Algorithm 2 (Q_0 = 1).  MODE 1: Algorithm 1's homogeneous system (Q_0 free) solved in the least-squares
// sense with |Q| = 1; basis, rows, selection and vote are shared.  MODE 2: Algorithm 3 -- the same per-class
// solve as mode 0, then no selection and no vote: P is recovered and r = P/Q is evaluated at the K nodes alpha_j
// (a decoder that absorbs up to E wrong predictions instead of locating them).
// MODE 3: mode 0 followed, in the same launch, by the decoding of every group from the workers that are present and
// were not located (Section 3, "ApproxIFER Decoding", steps 1 and 2 in one pass): the same terms in the same order
// as the decoder kernels, so the result is bit-identical to the two launches.
constexpr int kModeLocate = 0, kModeHomogeneous = 1, kModeRational = 2, kModeLocateDecode = 3;

template <int NMAX, int M, int MODE>
__global__ void __launch_bounds__(kRowsThreads, M > 10 ? 2 : 3) locate_rows_kernel(const __grid_constant__ LocateArgs a,
                                                                      const __grid_constant__ LocateTables tab,
                                                                      const __grid_constant__ LocateBasis basis,
                                                                      const __grid_constant__ DecodeTables dtab,
                                                                      const int gpb) {
  using SM = GroupSmem<NMAX, M>;
  constexpr int MP = SM::MP;
  constexpr int NQ = M - 1;  // unknowns Q_1 .. Q_{M-1}
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SM* groups = reinterpret_cast<SM*>(smem_raw);
  // the thread's own predictions, ysm[i][tid]: shared memory rather than registers, which the factor needs
  // (the same bytes serve, during set-up, as each warp's scratch for the reflectors of the Vandermonde block)
  unsigned char* scratch = smem_raw + (size_t)gpb * sizeof(SM);
  float* ysm = reinterpret_cast<float*>(scratch) + threadIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr bool HOMOG = MODE == kModeHomogeneous;
  const int E = a.E;
  const int64_t g_first = (int64_t)blockIdx.x * gpb;
  const int ng = (int)min((int64_t)gpb, a.G - g_first);

  // (Algorithm 3 only) per group, behind the scratch: the K x M table that carries P from M nodes to the alpha_j
  double* lgs = reinterpret_cast<double*>(scratch + scratch_bytes<NMAX, M>());

  // ---- set-up, one warp per group ------------------------------------------------------------------
  {
    // the full-set basis, transposed and zero-padded, behind the warps' reflector scratch
    double* nft = reinterpret_cast<double*>(scratch) + kRowsWarps * M * NMAX;
    // (the host lays the table out exactly as it is used here: consecutive threads copy consecutive entries)
    for (int idx = tid; idx < (NMAX - M) * NMAX; idx += kRowsThreads) nft[idx] = basis.nft[idx];
    __syncthreads();
    double(*refl)[NMAX] = reinterpret_cast<double(*)[NMAX]>(scratch) + warp * M;
    for (int s = warp; s < ng; s += kRowsWarps) {
      rows_setup_group<NMAX, M>(groups[s], refl, nft, a, tab, g_first + s, lane);
      __syncwarp();  // the scratch is reused by this warp's next group
      if constexpr (MODE == kModeRational) {
        // P has degree < M, so its values on M of the available nodes (spread over the whole range) fix it:
        // lg[j][k] = Lagrange basis of those nodes at alpha_j, lane = j
        const SM& sm = groups[s];
        if (sm.n >= 0 && lane < a.K) {
          double* lg = lgs + (size_t)s * M * M + lane * M;
          const double z = tab.alpha[lane];
#pragma unroll 1
          for (int k = 0; k < M; ++k) {
            const double xk = sm.xs[spread_rank<M>(k, sm.n)];
            double num = 1.0, den = 1.0;
            for (int l = 0; l < M; ++l) {
              if (l == k) continue;
              const double xl = sm.xs[spread_rank<M>(l, sm.n)];
              num *= z - xl;
              den *= xk - xl;
            }
            lg[k] = num / den;
          }
        }
      }
    }
  }
  __syncthreads();

  // ---- one thread per (group, class) -----------------------------------------------------------------
  const int64_t n_tasks = (int64_t)ng * a.C;
  for (int64_t t = tid; t < n_tasks; t += kRowsThreads) {
    const int s = (int)(t / a.C);
    const int64_t c = t - (int64_t)s * a.C;
    SM& sm = groups[s];
    const int n = sm.n;
    if (n < 0) {
      if constexpr (MODE == kModeRational)  // nothing can be solved: the group's output is zero-filled
        for (int j = 0; j < a.K; ++j) a.Yh[(g_first + s) * a.o_gs + j * a.o_rs + c] = 0.f;
      continue;
    }
    const float* Yc = a.Yt + (g_first + s) * a.y_gs + c;

#pragma unroll
    for (int i = 0; i < NMAX; ++i) ysm[i * kRowsThreads] = (i < n) ? __ldg(Yc + sm.yoff[i]) : 0.f;

    // Square-root-free triangular factor: R = sqrt(D) U with U unit upper triangular (only j > k is ever
    // touched) and the transformed right-hand side sqrt(D) d.  Folding a row costs two multiply-adds per
    // entry and one reciprocal per column, no square roots, and the unknowns come out of U q = d directly.
    // (homogeneous form: column 0 is one more unknown instead of the right-hand side, NC = M columns)
    constexpr int NC = HOMOG ? M : NQ;   // columns of the factor
    constexpr int C0 = HOMOG ? 0 : 1;    // row[] index of the factor's first column
    double U[NC][NC], dg[NC], d[NQ];
#pragma unroll
    for (int k = 0; k < NC; ++k) {
      dg[k] = 0.0;
#pragma unroll
      for (int j = 0; j < NC; ++j) U[k][j] = 0.0;
    }
#pragma unroll
    for (int k = 0; k < NQ; ++k) d[k] = 0.0;

    const int rows = n - M;
#pragma unroll 1
    for (int r = 0; r < rows; ++r) {
      // row[l] = sum_i N[i][r] y_i b_i^l, l = 0..M-1  (row[0] = b0[r])
      double row[MP];
#pragma unroll
      for (int l = 0; l < MP; ++l) row[l] = 0.0;
      const double* nr = sm.nt[r];
#pragma unroll 2
      for (int i = 0; i < n; i += 2) {  // an odd n reads one padded (zero) entry
        const double2 nn = *reinterpret_cast<const double2*>(nr + i);
        const double u0 = nn.x * (double)ysm[i * kRowsThreads], u1 = nn.y * (double)ysm[(i + 1) * kRowsThreads];
        if constexpr (M >= 14) {
          // The largest factors leave no registers to spare and spill; there the powers b_i^l are rebuilt on the
          // way (the same products in the same order as the table holds, so the same values) instead of being
          // loaded: one multiplication per power against five 128-bit shared-memory loads per worker, each of
          // which costs one pass per group that the warp's threads belong to.  Measured on 65,536 groups of 10
          // classes: K+E = 14: 1.87 -> 1.50 ms, 15: 2.99 -> 2.59 ms; for K+E <= 13 the table is as fast or faster.
          const double2 bb = *reinterpret_cast<const double2*>(&sm.xs[i]);
          double p0 = bb.x, p1 = bb.y;
          row[0] = fma(u0, 1.0, row[0]);
          row[0] = fma(u1, 1.0, row[0]);
#pragma unroll
          for (int l = 1; l < M; ++l) {
            row[l] = fma(u0, p0, row[l]);
            row[l] = fma(u1, p1, row[l]);
            if (l + 1 < M) {
              p0 *= bb.x;
              p1 *= bb.y;
            }
          }
        } else {
#pragma unroll
          for (int l = 0; l < MP; l += 2) {
            const double2 p0 = *reinterpret_cast<const double2*>(&sm.pw[i][l]);
            const double2 p1 = *reinterpret_cast<const double2*>(&sm.pw[i + 1][l]);
            row[l] = fma(u0, p0.x, row[l]);
            row[l + 1] = fma(u0, p0.y, row[l + 1]);
            row[l] = fma(u1, p1.x, row[l]);
            row[l + 1] = fma(u1, p1.y, row[l + 1]);
          }
        }
      }
      // fold the equation  sum_k row[k+1] q_k = -row[0]  (weight w, 1 at the start) into (D, U, d): the
      // square-root-free form of a Givens rotation per column (Gentleman's row update)
      double rhs = -row[0];
      double w = 1.0;
#pragma unroll
      for (int k = 0; k < NC; ++k) {
        const double xk = row[k + C0];
        const double wx = w * xk;
        const double dn = fma(wx, xk, dg[k]);
        if (dn > 1e-290) {  // (an exactly zero column leaves the factor as it is)
          const double inv = rcp_pos(dn);
          const double sb = wx * inv;
          w *= dg[k] * inv;
          dg[k] = dn;
#pragma unroll
          for (int j = k + 1; j < NC; ++j) {
            row[j + C0] = fma(-xk, U[k][j], row[j + C0]);
            U[k][j] = fma(sb, row[j + C0], U[k][j]);
          }
          if constexpr (!HOMOG) {
            rhs = fma(-xk, d[k], rhs);
            d[k] = fma(sb, rhs, d[k]);
          }
        }
      }
    }

    // q[k] = Q_{k+1} (Algorithm 2) or Q_k (homogeneous form)
    double q[NC];
    if constexpr (!HOMOG) {
      // back substitution (unit diagonal); a column that never received a non-zero entry keeps its unknown at 0
#pragma unroll
      for (int k = NQ - 1; k >= 0; --k) {
        double v = d[k];
#pragma unroll
        for (int j = k + 1; j < NQ; ++j) v = fma(-U[k][j], q[j], v);
        q[k] = v;
      }
    } else {
      // The unit vector q that minimises |R q|, R^T R = U^T D U: inverse iteration (two unit-triangular solves
      // and a diagonal scaling per step), stopped when the direction no longer moves, then two more steps.
      double dmax = 0.0;
#pragma unroll
      for (int k = 0; k < NC; ++k) dmax = fmax(dmax, dg[k]);
      const double floor_d = fmax(dmax * 1e-30, 1e-300);
#pragma unroll
      for (int k = 0; k < NC; ++k) dg[k] = 1.0 / fmax(dg[k], floor_d);  // from here on: 1/D (floored)
#pragma unroll
      for (int k = 0; k < NC; ++k) q[k] = 0.3 + 0.07 * k;
      int extra = 2;
#pragma unroll 1
      for (int it = 0; it < 300 && extra >= 0; ++it) {
        double t[NC];
#pragma unroll
        for (int k = 0; k < NC; ++k) {  // U^T t = q
          double v = q[k];
#pragma unroll
          for (int j = 0; j < k; ++j) v = fma(-U[j][k], t[j], v);
          t[k] = v;
        }
#pragma unroll
        for (int k = 0; k < NC; ++k) t[k] *= dg[k];
#pragma unroll
        for (int k = NC - 1; k >= 0; --k) {  // U z = t, in place
          double v = t[k];
#pragma unroll
          for (int j = k + 1; j < NC; ++j) v = fma(-U[k][j], t[j], v);
          t[k] = v;
        }
        double n2 = 0.0, dot = 0.0;
#pragma unroll
        for (int k = 0; k < NC; ++k) {
          n2 = fma(t[k], t[k], n2);
          dot = fma(t[k], q[k], dot);
        }
        const double inv = rsqrt(n2);
        // q is a unit vector after the first step; |dot| * inv = |cos| of the angle between the two iterates
        const bool settled = it > 0 && (1.0 - fabs(dot) * inv) <= 4e-16;
        if (settled || extra < 2) --extra;
#pragma unroll
        for (int k = 0; k < NC; ++k) q[k] = t[k] * inv;
      }
    }

    if constexpr (MODE == kModeRational) {
      // Algorithm 3, Step 2.  For this Q the best P is the least-squares polynomial through (b_i, y_i Q(b_i)):
      // on the nodes, P = t - N (N^T t) with t_i = y_i a_i.  Its values on M spread nodes carry it to alpha_j.
      double z[NMAX - M];
#pragma unroll
      for (int r = 0; r < NMAX - M; ++r) z[r] = 0.0;
#pragma unroll 2
      for (int i = 0; i < NMAX; ++i) {
        const double b = sm.xs[i];
        double h = q[NC - 1];
#pragma unroll
        for (int k = NC - 2; k >= 0; --k) h = fma(h, b, q[k]);
        const double ti = (i < n) ? fma(h, b, 1.0) * (double)ysm[i * kRowsThreads] : 0.0;
#pragma unroll
        for (int r = 0; r < NMAX - M; ++r)
          if (r < rows) z[r] = fma(sm.nt[r][i], ti, z[r]);  // N has n-M columns; the rest of nt is not meaningful
      }
      double pk[M];
#pragma unroll
      for (int k = 0; k < M; ++k) {
        const int i = spread_rank<M>(k, n);
        const double b = sm.xs[i];
        double h = q[NC - 1];
#pragma unroll
        for (int kk = NC - 2; kk >= 0; --kk) h = fma(h, b, q[kk]);
        double v = fma(h, b, 1.0) * (double)ysm[i * kRowsThreads];
#pragma unroll
        for (int r = 0; r < NMAX - M; ++r)
          if (r < rows) v = fma(-sm.nt[r][i], z[r], v);
        pk[k] = v;
      }
      const double* lg = lgs + (size_t)s * M * M;
      float* out = a.Yh + (g_first + s) * a.o_gs + (t - (int64_t)s * a.C);
      bool nonfin = false;
      for (int j = 0; j < a.K; ++j) {
        double pv = 0.0;
#pragma unroll
        for (int k = 0; k < M; ++k) pv = fma(lg[j * M + k], pk[k], pv);
        const double zj = tab.alpha[j];
        double h = q[NC - 1];
#pragma unroll
        for (int kk = NC - 2; kk >= 0; --kk) h = fma(h, zj, q[kk]);
        const float o = (float)(pv / fma(h, zj, 1.0));
        nonfin |= !isfinite(o);
        out[j * a.o_rs] = o;
      }
      if (nonfin) atomicOr(&sm.status, kStNonfinite);
      continue;
    }

    // a_i = Q(b_i) = 1 + sum_k q_k b_i^(k+1); the E smallest |a_i| (ties to the lower worker) get a vote
    double mag[NMAX];
    bool nonfinite = false;
#pragma unroll
    for (int i = 0; i < NMAX; ++i) {
      const double b = sm.xs[i];
      double h = q[NC - 1];
#pragma unroll
      for (int k = NC - 2; k >= 0; --k) h = fma(h, b, q[k]);
      const double av = HOMOG ? h : fma(h, b, 1.0);
      const bool fin = isfinite(av);
      mag[i] = fin ? fabs(av) : INFINITY;
      nonfinite |= (i < n) && !fin;
    }
    if (nonfinite) atomicOr(&sm.status, kStNonfinite);
    uint32_t taken = 0;
    for (int e = 0; e < E; ++e) {
      int best = -1;
      double bestv = 0.0;
#pragma unroll
      for (int i = 0; i < NMAX; ++i) {
        const bool cand = (i < n) && !((taken >> i) & 1u) && (best < 0 || mag[i] < bestv);
        if (cand) {
          best = i;
          bestv = mag[i];
        }
      }
      taken |= 1u << best;
      atomicAdd(&sm.votes[best], 1);
    }
  }
  __syncthreads();

  if constexpr (MODE == kModeRational) {
    if (a.status != nullptr && tid < ng) a.status[g_first + tid] = groups[tid].status;
    return;
  }
  // ---- the E most voted workers of each group, ties to the lower index; lane = rank ----------------
  for (int s = warp; s < ng; s += kRowsWarps) {
    SM& sm = groups[s];
    const int64_t g = g_first + s;
    const uint32_t mask = sm.mask;
    if (sm.n < 0) {
      for (int e = lane; e < E; e += 32) a.adv[g * E + e] = -1;
      if (lane == 0) {
        a.trusted[g] = mask;
        sm.pad = (int)mask;  // (kept for the decoding tail)
        if (a.status) a.status[g] = sm.status;
      }
      continue;
    }
    const int n = sm.n;
    const int my_worker = (lane < n) ? nth_set_bit(mask, lane) : 0;
    int v = (lane < n) ? sm.votes[lane] : -1;
    int idx = (lane < n) ? lane : 64 + lane;
    uint32_t picked = 0;
    for (int e = 0; e < E; ++e) {
      const int win = warp_argmin((double)(-v), idx);
      picked |= 1u << win;
      if (win == lane) {
        v = -1;
        idx = 64 + lane;
      }
    }
    const bool elected = (picked >> lane) & 1u;
    const uint32_t wbits = __reduce_or_sync(kFull, elected ? (1u << my_worker) : 0u);
    if (elected) a.adv[g * E + __popc(picked & ((1u << lane) - 1u))] = my_worker;
    if (lane == 0) {
      a.trusted[g] = mask & ~wbits;
      sm.pad = (int)(mask & ~wbits);
      if (a.status) a.status[g] = sm.status;
    }
  }

  if constexpr (MODE == kModeLocateDecode) {
    // ---- decoding from the trusted workers, one thread per (group, class) again ----------------------
    // Yhat[g][j][c] = sum_i s_i rg_ij y_ic / sum_i s_i rg_ij over the trusted workers i in ascending order,
    // rg_ij = 1/(alpha_j - beta_i): the decoder kernels' terms, order and roundings.  The predictions come
    // back from global memory (L2: this CTA has just read them); the table sits where the threads' prediction
    // columns were.
    constexpr int KMAX = M - 1;  // K = M - E, E >= 1
    __syncthreads();  // the trusted masks are in shared memory, the prediction columns are dead
    float* rgs = reinterpret_cast<float*>(scratch);
    const int K = a.K, W = a.W;
    for (int idx = tid; idx < W * K; idx += kRowsThreads) rgs[idx] = dtab.rg[idx];
    __syncthreads();
    const bool literal = (a.flags & kFlagSignWorkerIndex) != 0;
    for (int64_t t = tid; t < n_tasks; t += kRowsThreads) {
      const int s = (int)(t / a.C);
      const int64_t c = t - (int64_t)s * a.C;
      const int64_t g = g_first + s;
      const uint32_t trusted = (uint32_t)groups[s].pad;
      const float* Yc = a.Yt + g * a.y_gs + c;
      float acc[KMAX], den[KMAX];
#pragma unroll
      for (int j = 0; j < KMAX; ++j) acc[j] = den[j] = 0.f;
      int r = 0;
      for (uint32_t m = trusted; m; m &= m - 1, ++r) {
        const int i = __ffs((int)m) - 1;
        const float y = __ldg(Yc + (int64_t)i * a.y_rs);
        const uint32_t odd = ((literal ? (uint32_t)i : (uint32_t)r) & 1u) << 31;
#pragma unroll
        for (int j = 0; j < KMAX; ++j) {
          if (j < K) {
            const float w = __uint_as_float(__float_as_uint(rgs[i * K + j]) ^ odd);
            acc[j] = fmaf(w, y, acc[j]);
            den[j] = __fadd_rn(den[j], w);
          }
        }
      }
      const int n = r;
#pragma unroll
      for (int j = 0; j < KMAX; ++j) {
        if (j < K) {
          const int cq = dtab.any_coin ? (int)dtab.coin[j] : -1;  // alpha_j == beta_cq: the interpolant takes that value
          float v = acc[j] * __frcp_rn(den[j]);
          if (cq >= 0 && ((trusted >> cq) & 1u)) v = __ldg(Yc + (int64_t)cq * a.y_rs);
          if (n == 0) v = 0.f;
          a.Yh[g * a.o_gs + (int64_t)j * a.o_rs + c] = v;
        }
      }
      if (c == 0) {
        if (a.n_used) a.n_used[g] = n;
        if (a.decode_status) a.decode_status[g] = (n == 0 ? kStNoWorkers : 0u) | (n < K ? kStFewWorkers : 0u);
      }
    }
  }
}

template <int NMAX, int M>
cudaError_t launch_rows_nm(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  // as many groups per CTA as give every thread a class, within the shared-memory budget of two CTAs per SM
  int64_t gpb = a.C >= kRowsThreads ? 1 : kRowsThreads / a.C;
  if (gpb > kMaxGroupsPerCta) gpb = kMaxGroupsPerCta;
  // per group: its block, and for Algorithm 3 the M x M table that carries P to the alpha nodes
  const size_t per_group = sizeof(GroupSmem<NMAX, M>) + ((a.Yh != nullptr && !a.fuse_decode) ? (size_t)M * M * sizeof(double) : 0);
  // per-thread predictions, aliased with the set-up scratch (the warps' reflectors and the transposed full-set basis)
  const size_t y_bytes = scratch_bytes<NMAX, M>();
  // shared memory for three CTAs per SM (K+E <= 10: 168 registers per thread) or two (the larger factors
  // of K+E = 11..15 take 255 registers, and from 14 on a little local memory)
  const size_t budget = (M > 10 ? 110 : 74) * 1024;
  while (gpb > 1 && gpb * per_group + y_bytes > budget) --gpb;
  if (gpb > a.G) gpb = a.G;
  const size_t smem = (size_t)gpb * per_group + y_bytes;
  const int64_t blocks = (a.G + gpb - 1) / gpb;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  auto run = [&](auto mode) -> cudaError_t {
    constexpr int MODE = decltype(mode)::value;
    if (smem > 48 * 1024) {
      const DeviceInfo* di = nullptr;
      cudaError_t e = current_device_info(&di);
      if (e != cudaSuccess) return e;
      struct Tag {};
      if ((e = ensure_dynamic_smem<Tag>(locate_rows_kernel<NMAX, M, MODE>, di->ordinal, (int)smem)) != cudaSuccess) return e;
    }
    locate_rows_kernel<NMAX, M, MODE><<<(unsigned)blocks, kRowsThreads, smem, stream>>>(a, tab, locate_basis(a.W, M),
                                                                                        decode_tables(a.K, a.W), (int)gpb);
    count_launch();
    return cudaGetLastError();
  };
  if constexpr (M <= kLocateFuseMaxM) {
    if (a.fuse_decode) return run(std::integral_constant<int, kModeLocateDecode>{});
  }
  if (a.fuse_decode) return cudaErrorInvalidConfiguration;
  if constexpr (M <= kLocateAltMaxM) {
    if (a.Yh != nullptr) return run(std::integral_constant<int, kModeRational>{});
    if (a.flags & kFlagLocateHomogeneous) return run(std::integral_constant<int, kModeHomogeneous>{});
  }
  return run(std::integral_constant<int, kModeLocate>{});
}

template <int NMAX, int M = 2>
cudaError_t dispatch_rows_m(int m, const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  if constexpr (M > NMAX / 2 || M > kLocateRowsMaxM) {
    return cudaErrorInvalidValue;
  } else {
    if (m == M) return launch_rows_nm<NMAX, M>(a, tab, stream);
    return dispatch_rows_m<NMAX, M + 1>(m, a, tab, stream);
  }
}

}  // namespace

// One translation unit per row bound (the kernels are compiled per (rows, K+E, mode): four files build in
// parallel); APPROXIFER_ROWS_NMAX is set by the including .cu file.
#define APPROXIFER_ROWS_ENTRY2(n) launch_locate_rows_##n
#define APPROXIFER_ROWS_ENTRY(n) APPROXIFER_ROWS_ENTRY2(n)
cudaError_t APPROXIFER_ROWS_ENTRY(APPROXIFER_ROWS_NMAX)(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  return dispatch_rows_m<APPROXIFER_ROWS_NMAX>(a.K + a.E, a, tab, stream);
}

}  // namespace approxifer

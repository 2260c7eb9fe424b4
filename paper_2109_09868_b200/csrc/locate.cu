// ApproxIFER Byzantine-worker locator (Algorithm 2; inner step = Algorithm 1).
//
// Per group and class c the paper asks for the least-squares solution of
//     sum_k P_k b_r^k - y_r sum_{k>=1} Q_k b_r^k = y_r,   r = 0..n-1
// (b_r = beta of the r-th available worker, m = K+E, unknowns P_0..P_{m-1},
// Q_1..Q_{m-1}), then a_r = Q(b_r), the E smallest |a_r|, and a vote over the
// classes.  Only Q is ever used, so P is eliminated first: with V = [b_r^k]
// (n x m) and V = H_0..H_{m-1} [R;0] its Householder factorisation, the Q-part
// of the minimiser solves the (n-m) x (m-1) problem obtained by applying
// H_{m-1}..H_0 to the columns -y_r b_r^k and to the right-hand side y and
// keeping rows m..n-1.  The reflectors of V depend on the mask only and are
// shared by all classes of the group.  Everything runs in fp64.
//
// Warp-parallel layout: one warp per group; a lane owns one COLUMN of the
// current matrix (n <= 32 entries in registers), so applying a reflector is
// lane-local (a dot product and an axpy against a vector broadcast from shared
// memory) and needs no cross-lane reduction.  floor(32/m) classes (at most 8)
// are factorised side by side in one warp.  The selection steps (E smallest
// |a_r|, E most voted) are warp arg-min / arg-max butterflies with lane = worker.
//
// The kernel is compiled per (NMAX, M): NMAX = rows rounded up to 8, M = K+E.
// With M fixed at compile time every loop over rows and columns has static
// bounds: reflector k of the P-block touches rows k.., reflector k of the
// reduced problem rows M+k.., and no element is masked by a run-time predicate.
#include "common.cuh"
#include "locate_common.cuh"

namespace approxifer {

namespace {

using namespace locate_detail;

constexpr int kLocateWarps = 4;
constexpr int kLocateThreads = kLocateWarps * 32;
constexpr int kMaxSlots = 8;

template <int NMAX, int M>
struct WarpSmem {
  static constexpr int kSlots = (32 / M) < kMaxSlots ? (32 / M) : kMaxSlots;
  double refl[M][NMAX];            // normalised reflectors of the P-block (H = I - v v^T)
  double pw[NMAX][M];              // pw[r][k] = b_r^k
  double vbuf[2][kSlots][NMAX];    // reflector being broadcast, per class slot, double-buffered
  double rs[32][M];                // rs[lane][k'] = row k' of that lane's column of the reduced R | rhs
  double qs[32];                   // Q_1.. of each slot
  double xs[NMAX];                 // b_r
  long long yoff[NMAX];            // element offset of worker F[r]'s row
};

// Compile-time loops over reflector indices.
template <int NMAX, int M, int K0 = 0>
__device__ __forceinline__ void pblock_factor(double (&col)[NMAX], int lane, WarpSmem<NMAX, M>& sm) {
  if constexpr (K0 < M) {
    if (lane == K0) make_reflector<NMAX, K0>(col, sm.refl[K0]);
    __syncwarp();
    if (lane > K0 && lane < M) apply_reflector<NMAX, K0>(col, sm.refl[K0]);
    pblock_factor<NMAX, M, K0 + 1>(col, lane, sm);
  }
}
template <int NMAX, int M, int K0 = 0>
__device__ __forceinline__ void pblock_apply(double (&col)[NMAX], const WarpSmem<NMAX, M>& sm) {
  if constexpr (K0 < M) {
    apply_reflector<NMAX, K0>(col, sm.refl[K0]);
    pblock_apply<NMAX, M, K0 + 1>(col, sm);
  }
}
template <int NMAX, int M, int K0 = 0>
__device__ __forceinline__ void reduced_factor(double (&col)[NMAX], bool active, int l, int slot, double& diag,
                                               WarpSmem<NMAX, M>& sm) {
  if constexpr (K0 < M - 1) {
    double* vb = sm.vbuf[K0 & 1][slot];
    if (active && l == K0) diag = make_reflector<NMAX, M + K0>(col, vb);
    __syncwarp();
    if (active && l > K0) apply_reflector<NMAX, M + K0>(col, vb);
    reduced_factor<NMAX, M, K0 + 1>(col, active, l, slot, diag, sm);
  }
}

template <int NMAX, int M>
__global__ void __launch_bounds__(kLocateThreads) locate_kernel(const __grid_constant__ LocateArgs a,
                                                                const __grid_constant__ LocateTables tab) {
  using SM = WarpSmem<NMAX, M>;
  constexpr int kSlots = SM::kSlots;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  SM& sm = reinterpret_cast<SM*>(smem_raw)[warp];

  const int64_t g = (int64_t)blockIdx.x * kLocateWarps + warp;
  if (g >= a.G) return;  // whole warp leaves together

  const int E = a.E;
  const uint32_t mask = a.mask[g] & worker_bits(a.W);
  const int n = __popc(mask);
  if (n < 2 * M) {  // Algorithm 1's condition N-S+1 >= 2(K+E) does not hold
    for (int e = lane; e < E; e += 32) a.adv[g * E + e] = -1;
    if (lane == 0) {
      a.trusted[g] = mask;
      if (a.status) a.status[g] = kStLocateUnderdetermined;
    }
    return;
  }

  // ---- lane = available worker r: its index, node, powers --------------------
  const int my_worker = (lane < n) ? (int)__fns(mask, 0, lane + 1) : -1;
  if (lane < NMAX) {
    const double b = (lane < n) ? tab.beta[my_worker] : 0.0;
    sm.xs[lane] = b;
    sm.yoff[lane] = (lane < n) ? (a.rows.on ? (long long)a.rows.off[my_worker] : (long long)my_worker * a.y_rs) : 0;
    double p = 1.0;
#pragma unroll
    for (int k = 0; k < M; ++k) {
      sm.pw[lane][k] = (lane < n) ? p : 0.0;
      p *= b;
    }
  }
  __syncwarp();

  // ---- P-block: Householder reflectors of V = [b_r^k], lane = column k --------
  double col[NMAX];
#pragma unroll
  for (int r = 0; r < NMAX; ++r) col[r] = (lane < M) ? sm.pw[r][lane] : 0.0;
  pblock_factor<NMAX, M>(col, lane, sm);
  __syncwarp();

  // ---- classes, kSlots at a time; lane = (slot, column l) ----------------------
  const int slot_raw = lane / M, l = lane - slot_raw * M;
  const bool lane_in_slot = slot_raw < kSlots;
  const int slot = lane_in_slot ? slot_raw : 0;
  const float* Yg = a.Yt + g * a.y_gs;

  int votes = 0;  // lane = worker r again: how often it was among the E smallest
  uint32_t st = 0;

  for (int64_t c0 = 0; c0 < a.C; c0 += kSlots) {
    const int64_t c = c0 + slot_raw;
    const bool active = lane_in_slot && c < a.C;

    // column l < M-1: -y_r b_r^(l+1);  column M-1: the right-hand side y_r  (rows >= n are zero)
    {
      const int lp = (l < M - 1) ? l + 1 : 0;
      const double sgn = (l < M - 1) ? -1.0 : 1.0;  // pw[r][0] = 1 on present rows
#pragma unroll
      for (int r = 0; r < NMAX; ++r) {
        double v = 0.0;
        if (active && r < n) v = sgn * (double)__ldg(Yg + sm.yoff[r] + c) * sm.pw[r][lp];
        col[r] = v;
      }
    }
    // eliminate P: apply H_0 .. H_{M-1}
    pblock_apply<NMAX, M>(col, sm);

    // reduced problem on rows M..n-1: Householder QR, one column per step
    double diag = 0.0;
    reduced_factor<NMAX, M>(col, active, l, slot, diag, sm);

    // R (upper triangle, rows M..2M-2 of the columns) and rhs -> shared memory
    if (active) {
#pragma unroll
      for (int r = M; r < 2 * M - 1; ++r) sm.rs[lane][r - M] = col[r];
    }
    __syncwarp();

    // back substitution, lane = (slot, row l) for l < M-1
    if constexpr (M > 1) {
      double rhs = 0.0, rrow[M - 1];
      const int base = slot * M;
      const bool row_lane = active && l < M - 1;
#pragma unroll
      for (int k = 0; k < M - 1; ++k) rrow[k] = row_lane ? sm.rs[base + k][l] : 0.0;
      if (row_lane) rhs = sm.rs[base + M - 1][l];
      const double invd = (diag != 0.0) ? 1.0 / diag : 0.0;  // a zero column leaves its unknown at 0
#pragma unroll
      for (int k = M - 2; k >= 0; --k) {
        const int src = lane_in_slot ? base + k : lane;
        const double qk = __shfl_sync(kFull, rhs * invd, src);
        if (l < k) rhs = fma(-rrow[k], qk, rhs);
      }
      if (row_lane) sm.qs[lane] = rhs * invd;
    }
    __syncwarp();

    // a_r = Q(b_r) = 1 + sum_{k>=1} Q_k b_r^k, lane = worker r; then the E smallest |a_r|
    for (int s = 0; s < kSlots && c0 + s < a.C; ++s) {
      double mag = INFINITY;
      if (lane < n) {
        const double b = sm.xs[lane];
        double q = 1.0, p = b;
#pragma unroll
        for (int k = 0; k < M - 1; ++k) {
          q = fma(sm.qs[s * M + k], p, q);
          p *= b;
        }
        mag = fabs(q);
        if (!isfinite(q)) {
          mag = INFINITY;
          st |= kStNonfinite;
        }
      }
      int idx = (lane < n) ? lane : 64 + lane;
      for (int e = 0; e < E; ++e) {
        const int win = warp_argmin(mag, idx);
        if (win == lane) {
          votes += 1;
          mag = INFINITY;
          idx = 64 + lane;
        }
      }
    }
    __syncwarp();
  }

  // ---- the E most voted workers, ties to the lower index ----------------------
  uint32_t picked = 0;  // bit r = r-th available worker elected
  {
    int v = (lane < n) ? votes : -1;
    int idx = (lane < n) ? lane : 64 + lane;
    for (int e = 0; e < E; ++e) {
      const int win = warp_argmin((double)(-v), idx);
      picked |= 1u << win;
      if (win == lane) {
        v = -1;
        idx = 64 + lane;
      }
    }
  }
  const uint32_t any_st = __reduce_or_sync(kFull, st);
  const bool elected = (picked >> lane) & 1u;
  // worker-index bitmask of the elected ranks
  const uint32_t wbits = __reduce_or_sync(kFull, elected ? (1u << my_worker) : 0u);
  if (elected) {
    const int pos = __popc(picked & ((1u << lane) - 1u));  // ascending in r = ascending in worker index
    a.adv[g * E + pos] = my_worker;
  }
  if (lane == 0) {
    a.trusted[g] = mask & ~wbits;
    if (a.status) a.status[g] = any_st;
  }
}

template <int NMAX, int M>
cudaError_t launch_nm(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  const size_t smem = sizeof(WarpSmem<NMAX, M>) * kLocateWarps;
  if (smem > 48 * 1024) {  // opt in to more than the default dynamic shared memory (once per device)
    const DeviceInfo* di = nullptr;
    cudaError_t e = current_device_info(&di);
    if (e != cudaSuccess) return e;
    struct Tag {};
    if ((e = ensure_dynamic_smem<Tag>(locate_kernel<NMAX, M>, di->ordinal, (int)smem)) != cudaSuccess) return e;
  }
  const int64_t blocks = (a.G + kLocateWarps - 1) / kLocateWarps;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  locate_kernel<NMAX, M><<<(unsigned)blocks, kLocateThreads, smem, stream>>>(a, tab);
  count_launch();
  return cudaGetLastError();
}

// m = K + E runs over 2 .. NMAX/2 (the entry point has checked 2m <= W <= NMAX).
template <int NMAX, int M = 2>
cudaError_t dispatch_m(int m, const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  if constexpr (M > NMAX / 2) {
    return cudaErrorInvalidValue;
  } else {
    if (m == M) return launch_nm<NMAX, M>(a, tab, stream);
    return dispatch_m<NMAX, M + 1>(m, a, tab, stream);
  }
}

}  // namespace

// Locate and decode in one pass: Algorithm 2's form of the per-class step, a thread per (group, class) with all
// classes of a group in one CTA, and a factor small enough to leave the decoding tail its registers.
bool locate_fuse_eligible(const LocateArgs& a) {
  return !(a.flags & kFlagLocateHomogeneous) && a.K + a.E <= kLocateFuseMaxM && a.C <= kLocateFuseMaxC;
}

cudaError_t launch_locate(const LocateArgs& a, cudaStream_t stream) {
  if (a.G == 0) return cudaSuccess;
  const LocateTables& tab = locate_tables(a.K, a.W);
  const int m = a.K + a.E;
  // (the homogeneous form and Algorithm 3 exist in the thread-per-class kernel only; the entry points have checked K+E)
  const bool alt = (a.flags & kFlagLocateHomogeneous) || a.Yh != nullptr;  // (the fused pass is one of them: api.cu has checked its range)
  if (alt ? m <= kLocateAltMaxM : (m <= kLocateRowsMaxM && !a.force_warp_kernel))
    return launch_locate_rows(a, tab, stream);
  if (a.W <= 8) return dispatch_m<8>(m, a, tab, stream);
  if (a.W <= 16) return dispatch_m<16>(m, a, tab, stream);
  if (a.W <= 24) return dispatch_m<24>(m, a, tab, stream);
  return dispatch_m<32>(m, a, tab, stream);
}

}  // namespace approxifer

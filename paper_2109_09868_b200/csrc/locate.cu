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
#include "common.cuh"

namespace approxifer {

namespace {

constexpr int kLocateWarps = 4;
constexpr int kLocateThreads = kLocateWarps * 32;
constexpr int kMaxSlots = 8;
constexpr unsigned kFull = 0xffffffffu;

template <int NMAX>
struct WarpSmem {
  static constexpr int MMAX = NMAX / 2;
  double refl[MMAX][NMAX];          // normalised reflectors of the P-block (H = I - v v^T)
  double pw[NMAX][MMAX];            // pw[r][k] = b_r^k
  double vbuf[2][kMaxSlots][NMAX];  // reflector being broadcast, per class slot, double-buffered
  double rs[32][MMAX];              // rs[lane][k'] = row k' of that lane's column of the reduced R | rhs
  double qs[32];                    // Q_1.. of each slot
  double xs[NMAX];                  // b_r
  long long yoff[NMAX];             // element offset of worker F[r]'s row
};

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

// Builds the normalised reflector of `col` restricted to rows >= row0:
// v = x - akk e_row0 scaled so that H = I - v v^T maps x to akk e_row0.
// Returns akk (0 and v = 0 when the sub-column is exactly zero).
template <int NMAX>
__device__ __forceinline__ double make_reflector(const double (&col)[NMAX], int row0, double* v_out) {
  double s2 = 0.0, x0 = 0.0;
#pragma unroll
  for (int r = 0; r < NMAX; ++r) {
    const double x = (r >= row0) ? col[r] : 0.0;
    s2 = fma(x, x, s2);
    x0 = (r == row0) ? col[r] : x0;
  }
  const double normx = sqrt(s2);
  const double akk = (x0 >= 0.0) ? -normx : normx;
  // v^T v = s2 - x0^2 + (x0 - akk)^2 = 2 (s2 - x0 akk) = 2 normx (normx + |x0|)
  const double vv = 2.0 * (s2 - x0 * akk);
  const double scale = (vv > 0.0) ? sqrt(2.0 / vv) : 0.0;
#pragma unroll
  for (int r = 0; r < NMAX; ++r) {
    double v = (r > row0) ? col[r] : 0.0;
    v = (r == row0) ? (x0 - akk) : v;
    v_out[r] = v * scale;
  }
  return (vv > 0.0) ? akk : 0.0;
}

template <int NMAX>
__device__ __forceinline__ void apply_reflector(double (&col)[NMAX], const double* v) {
  double s = 0.0;
#pragma unroll
  for (int r = 0; r < NMAX; r += 2) {
    const double2 vv = *reinterpret_cast<const double2*>(v + r);
    s = fma(vv.x, col[r], s);
    s = fma(vv.y, col[r + 1], s);
  }
#pragma unroll
  for (int r = 0; r < NMAX; r += 2) {
    const double2 vv = *reinterpret_cast<const double2*>(v + r);
    col[r] = fma(-s, vv.x, col[r]);
    col[r + 1] = fma(-s, vv.y, col[r + 1]);
  }
}

template <int NMAX>
__global__ void __launch_bounds__(kLocateThreads) locate_kernel(const __grid_constant__ LocateArgs a,
                                                                const __grid_constant__ LocateTables tab) {
  constexpr int MMAX = NMAX / 2;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  WarpSmem<NMAX>& sm = reinterpret_cast<WarpSmem<NMAX>*>(smem_raw)[warp];

  const int64_t g = (int64_t)blockIdx.x * kLocateWarps + warp;
  if (g >= a.G) return;  // whole warp leaves together

  const int E = a.E, m = a.K + E;
  const uint32_t mask = a.mask[g] & worker_bits(a.W);
  const int n = __popc(mask);
  if (n < 2 * m) {  // Algorithm 1's condition N-S+1 >= 2(K+E) does not hold
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
    sm.yoff[lane] = (lane < n) ? (long long)my_worker * a.y_rs : 0;
    double p = 1.0;
    for (int k = 0; k < m; ++k) {
      sm.pw[lane][k] = (lane < n) ? p : 0.0;
      p *= b;
    }
  }
  __syncwarp();

  // ---- P-block: Householder reflectors of V = [b_r^k], lane = column k --------
  double col[NMAX];
  {
#pragma unroll
    for (int r = 0; r < NMAX; ++r) col[r] = (lane < m) ? sm.pw[r][lane] : 0.0;
    for (int k = 0; k < m; ++k) {
      if (lane == k) make_reflector<NMAX>(col, k, sm.refl[k]);
      __syncwarp();
      if (lane > k && lane < m) apply_reflector<NMAX>(col, sm.refl[k]);
    }
  }
  __syncwarp();

  // ---- classes, `slots` at a time; lane = (slot, column l) ---------------------
  int slots = 32 / m;
  if (slots > kMaxSlots) slots = kMaxSlots;
  const int slot = lane / m, l = lane - slot * m;
  const bool lane_in_slot = slot < slots;
  const float* Yg = a.Yt + g * a.y_gs;

  int votes = 0;       // lane = worker r again: how often it was among the E smallest
  uint32_t st = 0;

  for (int64_t c0 = 0; c0 < a.C; c0 += slots) {
    const int64_t c = c0 + slot;
    const bool active = lane_in_slot && c < a.C;

    // column l < m-1: -y_r b_r^(l+1);  column m-1: the right-hand side y_r
#pragma unroll
    for (int r = 0; r < NMAX; ++r) {
      double v = 0.0;
      if (active && r < n) {
        const double y = (double)__ldg(Yg + sm.yoff[r] + c);
        v = (l < m - 1) ? -y * sm.pw[r][l + 1] : y;
      }
      col[r] = v;
    }
    // eliminate P: apply H_0 .. H_{m-1}
    for (int k = 0; k < m; ++k) apply_reflector<NMAX>(col, sm.refl[k]);

    // reduced problem on rows m..n-1: Householder QR, one column per step
    double diag = 0.0;
    for (int k = 0; k < m - 1; ++k) {
      double* vb = sm.vbuf[k & 1][lane_in_slot ? slot : 0];
      if (active && l == k) diag = make_reflector<NMAX>(col, m + k, vb);
      __syncwarp();
      if (active && l > k) apply_reflector<NMAX>(col, vb);
    }
    // R (upper triangle, rows m..2m-2 of the columns) and rhs -> shared memory
    if (active) {
#pragma unroll
      for (int r = 0; r < NMAX; ++r)
        if (r >= m && r < 2 * m - 1) sm.rs[lane][r - m] = col[r];
    }
    __syncwarp();

    // back substitution, lane = (slot, row l) for l < m-1
    {
      double rhs = 0.0, rrow[MMAX];
      const int base = slot * m;
#pragma unroll
      for (int k = 0; k < MMAX; ++k) rrow[k] = (active && k < m - 1 && l < m - 1) ? sm.rs[base + k][l] : 0.0;
      if (active && l < m - 1) rhs = sm.rs[base + m - 1][l];
      const double invd = (diag != 0.0) ? 1.0 / diag : 0.0;  // a zero column leaves its unknown at 0
#pragma unroll
      for (int k = MMAX - 2; k >= 0; --k) {
        if (k < m - 1) {
          const int src = lane_in_slot ? base + k : lane;
          const double qk = __shfl_sync(kFull, rhs * invd, src);
          if (l < k) rhs = fma(-rrow[k], qk, rhs);
        }
      }
      if (active && l < m - 1) sm.qs[lane] = rhs * invd;
    }
    __syncwarp();

    // a_r = Q(b_r) = 1 + sum_{k>=1} Q_k b_r^k, lane = worker r; then the E smallest |a_r|
    for (int s = 0; s < slots && c0 + s < a.C; ++s) {
      double mag = INFINITY;
      if (lane < n) {
        const double b = sm.xs[lane];
        double q = 1.0, p = b;
        for (int k = 0; k < m - 1; ++k) {
          q = fma(sm.qs[s * m + k], p, q);
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

template <int NMAX>
cudaError_t launch_n(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  const size_t smem = sizeof(WarpSmem<NMAX>) * kLocateWarps;
  if (smem > 48 * 1024) {  // opt in to more than the default dynamic shared memory (per device, idempotent)
    cudaError_t e = cudaFuncSetAttribute(locate_kernel<NMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const int64_t blocks = (a.G + kLocateWarps - 1) / kLocateWarps;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  locate_kernel<NMAX><<<(unsigned)blocks, kLocateThreads, smem, stream>>>(a, tab);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_locate(const LocateArgs& a, cudaStream_t stream) {
  if (a.G == 0) return cudaSuccess;
  LocateTables tab;
  build_locate_tables(a.W, &tab);
  if (a.W <= 8) return launch_n<8>(a, tab, stream);
  if (a.W <= 16) return launch_n<16>(a, tab, stream);
  if (a.W <= 24) return launch_n<24>(a, tab, stream);
  return launch_n<32>(a, tab, stream);
}

}  // namespace approxifer

// ApproxIFER decoder, short-payload variant (Section 3, "Decoding", step 2) for predictions of a few
// classes (C <= 32: the paper's own workloads have C = 10) in dense [G][W][C] / [G][K][C] buffers.
//
// Same arithmetic as decode_kernel, term by term and rounding by rounding, but one thread per
// (group, QUERY) instead of one per (group, class): the thread walks the present workers once, forms the
// signed weight s_i/(alpha_j - beta_i) and the denominator of its query once, and applies the weight to all
// C classes of the worker's row.  The per-class kernel repeats the weight and denominator work for every
// class, which dominates when C is small.  The predictions of a CTA's groups are one contiguous piece of
// memory: they are copied into shared memory with 128-bit loads (rows of absent workers come along and are
// never used), the results leave the same way.
#include "common.cuh"

namespace approxifer {

namespace {

constexpr int kSmallThreads = 256;
constexpr int kSmallMaxC = 32;
constexpr int kSmallSmemBudget = 44 * 1024;  // payload + results of one CTA

// CP: the number of classes rounded up to an even number; a thread reads CP floats of a row (for an odd C the
// last one belongs to the next row or to the slack behind the buffer: finite or not, it only reaches an
// accumulator that is never stored).  V2: C is even (= CP), rows start on 8-byte boundaries and are read and
// written as 64-bit words.
template <int CP, bool V2>
__global__ void __launch_bounds__(kSmallThreads) decode_small_kernel(const __grid_constant__ DecodeArgs a,
                                                                    const __grid_constant__ DecodeTables tab, const int gpb) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x;
  const int W = a.W, K = a.K;
  const int C = V2 ? CP : (int)a.C;  // an even class count is instantiated exactly, an odd one is CP - 1 (or 1)
  const int64_t g_first = (int64_t)blockIdx.x * gpb;
  const int ng = (int)min((int64_t)gpb, a.G - g_first);
  const int in_floats = ng * W * C, out_floats = ng * K * C;
  // shared memory: ys[gpb*W*C (+ slack)] | os[gpb*K*C] | rg[W*K] | mask[gpb]
  float* ys = reinterpret_cast<float*>(smem_raw);
  float* os = ys + ((gpb * W * C + kSmallMaxC + 3) & ~3);
  float* rgs = os + ((gpb * K * C + 3) & ~3);
  uint32_t* masks = reinterpret_cast<uint32_t*>(rgs + W * K);

  // ---- stage: predictions (dense, so one contiguous range), table, masks ------------------------------
  {
    const float4* src = reinterpret_cast<const float4*>(a.Yt + g_first * a.y_gs);
    float4* dst = reinterpret_cast<float4*>(ys);
    const int n4 = in_floats >> 2;  // gpb is a multiple of 4 and the base is 16-byte aligned: whole float4s ...
    for (int idx = tid; idx < n4; idx += kSmallThreads) dst[idx] = ld_stream(src + idx);
    for (int idx = (n4 << 2) + tid; idx < in_floats; idx += kSmallThreads)  // ... except in the last CTA
      ys[idx] = ld_stream(a.Yt + g_first * a.y_gs + idx);
    for (int idx = tid; idx < W * K; idx += kSmallThreads) rgs[idx] = tab.rg[idx];
    if (tid < ng) masks[tid] = a.mask[g_first + tid] & worker_bits(W);
  }
  __syncthreads();

  // ---- one thread per (group, query) -----------------------------------------------------------------
  const int s = tid / K, j = tid - s * K;
  if (s < ng) {
    const uint32_t mask = masks[s];
    const uint32_t literal = (a.flags & kFlagSignWorkerIndex) ? 1u : 0u;
    const int coin = tab.any_coin ? (int)tab.coin[j] : -1;  // the worker whose node equals alpha_j, if any
    const float* yg = ys + s * W * C;
    const float* rgj = rgs + j;
    float acc[CP];
#pragma unroll
    for (int c = 0; c < CP; ++c) acc[c] = 0.f;
    float den = 0.f;
    int r = 0;
    for (uint32_t m = mask; m; m &= m - 1, ++r) {
      const int i = __ffs(m) - 1;
      // the signed weight; (s rg) y rounds like rg (s y), the sign being exact
      const uint32_t odd = (literal ? (uint32_t)i : (uint32_t)r) & 1u;
      const float srg = __uint_as_float(__float_as_uint(rgj[i * K]) ^ (odd << 31));
      const float* y = yg + i * C;
      if constexpr (V2) {
#pragma unroll
        for (int c = 0; c < CP; c += 2) {
          const float2 v = *reinterpret_cast<const float2*>(y + c);
          acc[c] = fmaf(srg, v.x, acc[c]);
          if (c + 1 < CP) acc[c + 1] = fmaf(srg, v.y, acc[c + 1]);
        }
      } else {
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[c] = fmaf(srg, y[c], acc[c]);
      }
      den = __fadd_rn(den, srg);
    }
    const int n = r;
    const bool pinned = coin >= 0 && ((mask >> coin) & 1u);  // alpha_j == beta_coin: the interpolant takes that value
    const float inv = __frcp_rn(den);
    float* o = os + (s * K + j) * C;
    if (n == 0) {
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] = 0.f;
    } else if (pinned) {
      const float* yp = yg + coin * C;
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] = (c < C) ? yp[c] : 0.f;
    } else {
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] *= inv;
    }
    if constexpr (V2) {
#pragma unroll
      for (int c = 0; c < CP; c += 2) *reinterpret_cast<float2*>(o + c) = make_float2(acc[c], acc[c + 1]);
    } else {
#pragma unroll
      for (int c = 0; c < CP; ++c)
        if (c < C) o[c] = acc[c];
    }
    if (j == 0) {
      if (a.n_used) a.n_used[g_first + s] = n;
      if (a.status) a.status[g_first + s] = (n == 0 ? kStNoWorkers : 0u) | (n < K ? kStFewWorkers : 0u);
    }
  }
  __syncthreads();

  // ---- results out: again one contiguous range --------------------------------------------------------
  {
    float4* dst = reinterpret_cast<float4*>(a.Yh + g_first * a.o_gs);
    const float4* src = reinterpret_cast<const float4*>(os);
    const int n4 = out_floats >> 2;
    for (int idx = tid; idx < n4; idx += kSmallThreads) st_stream(dst + idx, src[idx]);
    for (int idx = (n4 << 2) + tid; idx < out_floats; idx += kSmallThreads) st_stream(a.Yh + g_first * a.o_gs + idx, os[idx]);
  }
}

bool g_small_disabled = false;

int groups_per_cta(const DecodeArgs& a) {
  const int C = (int)a.C;
  int gpb = kSmallThreads / a.K;
  const int per_group = (a.W + a.K) * C * 4 + 4;
  const int fixed = (kSmallMaxC + 8) * 4 + a.W * a.K * 4;
  while (gpb > 4 && gpb * per_group + fixed > kSmallSmemBudget) --gpb;
  return gpb & ~3;  // a multiple of 4 groups: every CTA's ranges start on 16-byte boundaries
}

template <int CP, bool V2>
cudaError_t launch_small(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  const int gpb = groups_per_cta(a);
  const int C = (int)a.C;
  const size_t smem = (size_t)(((gpb * a.W * C + kSmallMaxC + 3) & ~3) + ((gpb * a.K * C + 3) & ~3) + a.W * a.K + gpb) * 4;
  const int64_t blocks = (a.G + gpb - 1) / gpb;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  decode_small_kernel<CP, V2><<<(unsigned)blocks, kSmallThreads, smem, stream>>>(a, tab, gpb);
  count_launch();
  return cudaGetLastError();
}

template <int CP = 2>
cudaError_t dispatch_cp(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  if constexpr (CP > kSmallMaxC) {
    return cudaErrorInvalidValue;
  } else {
    if (a.C == CP) return launch_small<CP, true>(a, tab, stream);       // even C: compiled for exactly C classes
    if (a.C == CP - 1) return launch_small<CP, false>(a, tab, stream);  // odd C: one padding class
    return dispatch_cp<CP + 2>(a, tab, stream);
  }
}

}  // namespace

void decode_small_config(int disable) { g_small_disabled = disable != 0; }

// Dense buffers (rows and groups back to back), 16-byte aligned, at most 32 classes, and room for at least
// four groups per CTA.
bool decode_small_eligible(const DecodeArgs& a) {
  if (g_small_disabled || a.C > kSmallMaxC) return false;
  if (a.y_rs != a.C || a.y_gs != (int64_t)a.W * a.C || a.o_rs != a.C || a.o_gs != (int64_t)a.K * a.C) return false;
  if (!aligned16(a.Yt) || !aligned16(a.Yh)) return false;
  return groups_per_cta(a) >= 4;
}

cudaError_t launch_decode_small(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  return dispatch_cp<>(a, tab, stream);
}

}  // namespace approxifer

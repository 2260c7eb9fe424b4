// ApproxIFER decoder kernels (Section 3, "Decoding", step 2):
//   Yhat[g][j][:] = r_g(alpha_j),
//   r_g(z) = sum_{i in F} [s_i/(z-beta_i)] Yt[g][i][:] / sum_{i in F} s_i/(z-beta_i)
// evaluated in its barycentric form: the numerator sum and the denominator sum
// are accumulated side by side over the workers present in the group's mask and
// divided once at the end, so the only per-group "weight generation" is K
// reciprocals.  1/(alpha_j - beta_i) comes from a launch-constant table staged
// in shared memory; the rank of a worker inside F (which fixes its sign) falls
// out of walking the mask's set bits in ascending order.
#include "common.cuh"

namespace approxifer {

namespace {

constexpr int kDecodeThreads = 256;

template <typename V>
struct Vec;
template <>
struct Vec<float4> {
  static constexpr int kLanes = 4;
  static __device__ __forceinline__ float4 zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
  static __device__ __forceinline__ float4 scale(float s, float4 x) { return make_float4(s * x.x, s * x.y, s * x.z, s * x.w); }
  static __device__ __forceinline__ float4 fma(float w, float4 x, float4 a) {
    return make_float4(fmaf(w, x.x, a.x), fmaf(w, x.y, a.y), fmaf(w, x.z, a.z), fmaf(w, x.w, a.w));
  }
};
template <>
struct Vec<float> {
  static constexpr int kLanes = 1;
  static __device__ __forceinline__ float zero() { return 0.f; }
  static __device__ __forceinline__ float scale(float s, float x) { return s * x; }
  static __device__ __forceinline__ float fma(float w, float x, float a) { return fmaf(w, x, a); }
};

// Generic decoder: one thread per (group, V-wide column).  Works for every
// shape, alignment and mask; threads of one warp may belong to different
// groups when C is small.
template <int K, typename P>
__global__ void __launch_bounds__(kDecodeThreads) decode_kernel(const __grid_constant__ DecodeArgs a,
                                                                const __grid_constant__ DecodeTables tab) {
  using V = typename P::Vec;
  using S = typename P::Store;
  using Ops = Vec<V>;
  constexpr int KP = (K + 3) / 4 * 4;              // table rows padded to whole float4s
  __shared__ __align__(16) float s_rg[kMaxW * KP];  // [i][j] = 1/(alpha_j - beta_i), 0 beyond K
  for (int idx = threadIdx.x; idx < a.W * KP; idx += kDecodeThreads) {
    const int i = idx / KP, j = idx - i * KP;
    s_rg[idx] = (j < K) ? tab.rg[i * K + j] : 0.f;
  }
  __syncthreads();

  const uint32_t Cv = (uint32_t)(a.C / Ops::kLanes);
  const int64_t first = (int64_t)blockIdx.x * kDecodeThreads;
  const int64_t g0 = first / Cv;
  const uint32_t t = (uint32_t)(first - g0 * Cv) + threadIdx.x;
  const uint32_t dg = t / Cv;
  const uint32_t v = t - dg * Cv;
  const int64_t g = g0 + dg;
  if (g >= a.G) return;

  const uint32_t mask = a.mask[g] & worker_bits(a.W);
  const int n = __popc(mask);
  const S* in = reinterpret_cast<const S*>(reinterpret_cast<const unsigned char*>(a.Yt) + g * a.y_gs * P::kElemBytes) + v;
  const int64_t in_rs = a.y_rs / Ops::kLanes;
  const bool literal = (a.flags & kFlagSignWorkerIndex) != 0;
  const bool any_coin = tab.any_coin != 0;

  V acc[K];
  float den[K];
#pragma unroll
  for (int j = 0; j < K; ++j) {
    acc[j] = Ops::zero();
    den[j] = 0.f;
  }
  uint32_t pinned = 0;  // queries whose node coincides with a present worker's

  auto use_row = [&](int i, int r, V y) {
    const float sgn = ((literal ? i : r) & 1) ? -1.f : 1.f;
    const V ys = Ops::scale(sgn, y);
    float rg[KP];
#pragma unroll
    for (int q = 0; q < KP / 4; ++q) {
      const float4 w4 = *reinterpret_cast<const float4*>(s_rg + i * KP + 4 * q);
      rg[4 * q] = w4.x, rg[4 * q + 1] = w4.y, rg[4 * q + 2] = w4.z, rg[4 * q + 3] = w4.w;
    }
    if (!any_coin) {
#pragma unroll
      for (int j = 0; j < K; ++j) {
        acc[j] = Ops::fma(rg[j], ys, acc[j]);
        den[j] = fmaf(sgn, rg[j], den[j]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < K; ++j) {
        if (tab.coin[j] == i) {  // alpha_j == beta_i: the interpolant takes this worker's value
          acc[j] = y;
          pinned |= 1u << j;
        } else if (!((pinned >> j) & 1u)) {
          acc[j] = Ops::fma(rg[j], ys, acc[j]);
          den[j] = fmaf(sgn, rg[j], den[j]);
        }
      }
    }
  };

  // Walk the present workers in ascending order.
  if (Ops::kLanes == 1) {
    // 4-byte columns (narrow or unaligned payloads): sweep the W workers eight at a time; the loads of the
    // present ones are issued together, then consumed in ascending order (r counts the present workers).
    int r = 0;
    for (int i0 = 0; i0 < a.W; i0 += 8) {
      const uint32_t bits = (mask >> i0) & 0xffu;
      if (bits == 0) continue;
      V y[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if ((bits >> u) & 1u) y[u] = P::load(in + (a.rows.on ? a.rows.off[i0 + u] / Ops::kLanes : (i0 + u) * in_rs));
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if ((bits >> u) & 1u) {
          use_row(i0 + u, r, y[u]);
          ++r;
        }
    }
  } else {
    // 16-byte columns: four rows in flight at a time.
    uint32_t m = mask;
    int r = 0;
    while (m) {
      int i[4];
      V y[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        i[u] = m ? (__ffs(m) - 1) : -1;
        m &= m - 1;  // 0 stays 0
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i[u] >= 0) y[u] = P::load(in + (a.rows.on ? a.rows.off[i[u]] / Ops::kLanes : i[u] * in_rs));
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i[u] >= 0) use_row(i[u], r + u, y[u]);
      r += 4;
    }
  }

  S* out = reinterpret_cast<S*>(reinterpret_cast<unsigned char*>(a.Yh) + g * a.o_gs * P::kElemBytes) + v;
  const int64_t out_rs = a.o_rs / Ops::kLanes;
#pragma unroll
  for (int j = 0; j < K; ++j) {
    V o;
    if (n == 0)
      o = Ops::zero();
    else if ((pinned >> j) & 1u)
      o = acc[j];
    else
      o = Ops::scale(__frcp_rn(den[j]), acc[j]);  // correctly rounded, like 1.0f / den
    P::store(out + j * out_rs, o);
  }
  if (v == 0) {
    if (a.n_used) a.n_used[g] = n;
    if (a.status) a.status[g] = (n == 0 ? kStNoWorkers : 0u) | (n < a.K ? kStFewWorkers : 0u);
  }
}

template <int K, typename V>
cudaError_t launch_one(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  const int64_t Cv = a.C / V::kLanes;
  const int64_t items = a.G * Cv;
  const int64_t blocks = (items + kDecodeThreads - 1) / kDecodeThreads;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  decode_kernel<K, V><<<(unsigned)blocks, kDecodeThreads, 0, stream>>>(a, tab);
  count_launch();
  return cudaGetLastError();
}

template <typename V, int K = 1>
cudaError_t dispatch_k(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  if constexpr (K > kMaxK) {
    return cudaErrorInvalidValue;
  } else {
    if (a.K == K) return launch_one<K, V>(a, tab, stream);
    return dispatch_k<V, K + 1>(a, tab, stream);
  }
}

// Test hook: normalised decoder weights of one mask, computed with the same
// table, order and arithmetic as decode_kernel.
__global__ void debug_decode_weights_kernel(int K, int W, uint32_t flags, uint32_t mask_in, const __grid_constant__ DecodeTables tab,
                                            float* w, int32_t* idx, int32_t* n_out) {
  const int j = threadIdx.x;
  const uint32_t mask = mask_in & worker_bits(W);
  const int n = __popc(mask);
  if (j == 0) {
    *n_out = n;
    int r = 0;
    for (uint32_t m = mask; m; m &= m - 1) idx[r++] = __ffs(m) - 1;
    for (; r < W; ++r) idx[r] = -1;
  }
  if (j >= K) return;
  const bool literal = (flags & kFlagSignWorkerIndex) != 0;
  float den = 0.f;
  int hit = -1, r = 0;
  for (uint32_t m = mask; m; m &= m - 1, ++r) {
    const int i = __ffs(m) - 1;
    const float sgn = ((literal ? i : r) & 1) ? -1.f : 1.f;
    if (tab.coin[j] == i) hit = r;
    den = fmaf(sgn, tab.rg[i * K + j], den);
  }
  const float inv = 1.0f / den;
  r = 0;
  for (uint32_t m = mask; m; m &= m - 1, ++r) {
    const int i = __ffs(m) - 1;
    const float sgn = ((literal ? i : r) & 1) ? -1.f : 1.f;
    w[j * W + r] = hit >= 0 ? (r == hit ? 1.f : 0.f) : inv * (sgn * tab.rg[i * K + j]);
  }
  for (; r < W; ++r) w[j * W + r] = 0.f;
}

__global__ void debug_encode_weights_kernel(int K, int W, const __grid_constant__ EncodeTables tab, float* w) {
  for (int idx = threadIdx.x; idx < K * W; idx += blockDim.x) w[idx] = tab.w[idx];
}

}  // namespace

cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream) {
  if (a.G == 0) return cudaSuccess;
  const DecodeTables& tab = decode_tables(a.K, a.W);
  bool by4 = a.C % 4 == 0 && a.y_gs % 4 == 0 && (a.rows.on || a.y_rs % 4 == 0) && a.o_gs % 4 == 0 && a.o_rs % 4 == 0;
  if (a.rows.on) {  // gathered rows: the packed-groups kernel where it takes the shape, else the per-column kernel
                    // follows the offset table
    if (!a.bf16 && decode_pack_eligible(a)) return launch_decode_pack(a, tab, stream);
    for (int i = 0; i < a.W; ++i) by4 = by4 && a.rows.off[i] % 4 == 0;
    if (by4 && aligned16(a.Yt) && aligned16(a.Yh)) return dispatch_k<PayloadF32x4>(a, tab, stream);
    return dispatch_k<PayloadF32>(a, tab, stream);
  }
  if (a.bf16) {  // bfloat16 payloads: the bulk-copy staged kernel for long rows, else the per-column kernel, four
                 // elements (8 bytes) per thread where it can
    if (decode_staged_eligible(a)) return launch_decode_staged(a, tab, stream);
    if (by4 && aligned8(a.Yt) && aligned8(a.Yh)) return dispatch_k<PayloadBf16x4>(a, tab, stream);
    return dispatch_k<PayloadBf16>(a, tab, stream);
  }
  if (decode_pack_eligible(a)) return launch_decode_pack(a, tab, stream);
  if (decode_small_eligible(a)) return launch_decode_small(a, tab, stream);
  if (decode_staged_eligible(a)) return launch_decode_staged(a, tab, stream);
  if (by4 && aligned16(a.Yt) && aligned16(a.Yh)) return dispatch_k<PayloadF32x4>(a, tab, stream);
  return dispatch_k<PayloadF32>(a, tab, stream);
}

cudaError_t launch_debug_weights(int K, int W, uint32_t flags, uint32_t mask, int which, float* w, int32_t* idx,
                                 int32_t* n, cudaStream_t stream) {
  if (which == 0) {
    EncodeTables tab;
    build_encode_tables(K, W, &tab);
    debug_encode_weights_kernel<<<1, 256, 0, stream>>>(K, W, tab, w);
  } else {
    DecodeTables tab;
    build_decode_tables(K, W, &tab);
    debug_decode_weights_kernel<<<1, 32, 0, stream>>>(K, W, flags, mask, tab, w, idx, n);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace approxifer

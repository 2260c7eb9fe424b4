// ApproxIFER decoder, short- and medium-payload variant (Section 3, "Decoding", step 2) for predictions of
// up to a few hundred classes (the paper's own workloads have C = 10; 100 classes is the next common size) in
// dense [G][W][C] / [G][K][C] buffers (the predictions may also be stored worker-major, [W][G][C]).
//
// Same arithmetic as decode_kernel, term by term and rounding by rounding, but one thread per
// (group, QUERY, chunk of CP <= 32 classes) instead of one per (group, 16-byte column): the thread walks the
// present workers once, forms the signed weight s_i/(alpha_j - beta_i) and the denominator of its query once,
// and applies the weight to its CP classes of the worker's row.  The per-column kernel repeats the weight and
// denominator work for every column and keeps all K accumulators per thread, which costs instructions when C
// is small and occupancy when K is large.  The predictions of a CTA's groups are one contiguous piece of
// memory: they are copied into shared memory with 128-bit loads (rows of absent workers come along and are
// never used), the results leave the same way.
#include "common.cuh"

namespace approxifer {

namespace {

constexpr int kSmallThreads = 256;
constexpr int kSmallMaxChunk = 32;            // classes per thread
constexpr int kSmallMaxC = 511;               // from 512 on: the bulk-copy staged kernel
constexpr int kSmallSmemBudget = 100 * 1024;  // payload + results of one CTA (two CTAs per SM)

// CP: classes per thread.  V = 1: C = CP - 1 (or 1) is odd, one chunk per row, scalar shared-memory accesses, the
// CP-th float a thread reads belongs to the next row or to the slack behind the buffer and only reaches an
// accumulator that is never stored.  V = 2 / 4: C is a multiple of CP, rows and chunks start on 8- / 16-byte
// boundaries and are read and written as 64- / 128-bit words.
template <int CP, int V>
__global__ void __launch_bounds__(kSmallThreads) decode_small_kernel(const __grid_constant__ DecodeArgs a,
                                                                    const __grid_constant__ DecodeTables tab, const int gpb,
                                                                    const int nch) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x;
  const int W = a.W, K = a.K, C = (int)a.C;
  const int64_t g_first = (int64_t)blockIdx.x * gpb;
  const int ng = (int)min((int64_t)gpb, a.G - g_first);
  const int in_floats = ng * W * C, out_floats = ng * K * C;
  // shared memory: ys[gpb*W*C (+ slack)] | os[gpb*K*C] | rg[W*K] | mask[gpb]
  float* ys = reinterpret_cast<float*>(smem_raw);
  float* os = ys + ((gpb * W * C + kSmallMaxChunk + 3) & ~3);
  float* rgs = os + ((gpb * K * C + 3) & ~3);
  uint32_t* masks = reinterpret_cast<uint32_t*>(rgs + W * K);

  // ---- stage: predictions, table, masks --------------------------------------------------------------
  {
    if (a.y_rs == a.C) {
      // group-major ([G][W][C] dense): the CTA's groups are one contiguous range
      const float4* src = reinterpret_cast<const float4*>(a.Yt + g_first * a.y_gs);
      float4* dst = reinterpret_cast<float4*>(ys);
      const int n4 = in_floats >> 2;  // every CTA's range starts on a 16-byte boundary: whole float4s ...
      for (int idx = tid; idx < n4; idx += kSmallThreads) dst[idx] = ld_stream(src + idx);
      for (int idx = (n4 << 2) + tid; idx < in_floats; idx += kSmallThreads)  // ... except at the end of the last CTA
        ys[idx] = ld_stream(a.Yt + g_first * a.y_gs + idx);
    } else {
      // worker-major ([W][G][C]: y_gs == C, one batch per worker): W contiguous ranges of ng * C floats, read
      // with 128-bit loads where they are whole 16-byte columns and scattered into the group-major layout
      const int per_worker = ng * C;
      const int n4 = per_worker >> 2;
      for (int idx = tid; idx < W * n4; idx += kSmallThreads) {
        const int i = idx / n4, q = idx - i * n4;
        const float4 v = ld_stream(reinterpret_cast<const float4*>(a.Yt + (int64_t)i * a.y_rs + g_first * (int64_t)C) + q);
        const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          const int f = 4 * q + t, sgrp = f / C, c = f - sgrp * C;
          ys[(sgrp * W + i) * C + c] = e[t];
        }
      }
      const int rem = per_worker - (n4 << 2);  // ragged end of the last CTA
      for (int idx = tid; idx < W * rem; idx += kSmallThreads) {
        const int i = idx / rem, f = (n4 << 2) + idx - i * rem, sgrp = f / C, c = f - sgrp * C;
        ys[(sgrp * W + i) * C + c] = ld_stream(a.Yt + (int64_t)i * a.y_rs + g_first * (int64_t)C + f);
      }
    }
    for (int idx = tid; idx < W * K; idx += kSmallThreads) rgs[idx] = tab.rg[idx];
    if (tid < ng) masks[tid] = a.mask[g_first + tid] & worker_bits(W);
  }
  __syncthreads();

  // ---- one thread per (group, query, chunk) -----------------------------------------------------------
  const int sj = tid / nch, ch = tid - sj * nch;  // consecutive threads: consecutive chunks of one (group, query)
  const int s = sj / K, j = sj - s * K;
  if (s < ng) {
    const uint32_t mask = masks[s];
    const uint32_t literal = (a.flags & kFlagSignWorkerIndex) ? 1u : 0u;
    const int coin = tab.any_coin ? (int)tab.coin[j] : -1;  // the worker whose node equals alpha_j, if any
    // a thread's classes are interleaved with those of the other chunks of its row, one shared-memory word
    // (V floats) at a time: word q of thread ch is word q*nch + ch of the row, so that the threads of a row
    // read consecutive words and no two of them meet in a bank
    const float* yg = ys + s * W * C + ch * V;
    const int step = nch * V;  // floats between two words of this thread
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
      if constexpr (V == 4) {
#pragma unroll
        for (int c = 0; c < CP; c += 4) {
          const float4 v = *reinterpret_cast<const float4*>(y + (c / 4) * step);
          acc[c] = fmaf(srg, v.x, acc[c]);
          acc[c + 1] = fmaf(srg, v.y, acc[c + 1]);
          acc[c + 2] = fmaf(srg, v.z, acc[c + 2]);
          acc[c + 3] = fmaf(srg, v.w, acc[c + 3]);
        }
      } else if constexpr (V == 2) {
#pragma unroll
        for (int c = 0; c < CP; c += 2) {
          const float2 v = *reinterpret_cast<const float2*>(y + (c / 2) * step);
          acc[c] = fmaf(srg, v.x, acc[c]);
          acc[c + 1] = fmaf(srg, v.y, acc[c + 1]);
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
    float* o = os + (s * K + j) * C + ch * V;
    if (n == 0) {
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] = 0.f;
    } else if (pinned) {
      const float* yp = yg + coin * C;
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] = (V > 1 || c < C) ? yp[(c / V) * step + c % V] : 0.f;
    } else {
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] *= inv;
    }
    if constexpr (V == 4) {
#pragma unroll
      for (int c = 0; c < CP; c += 4)
        *reinterpret_cast<float4*>(o + (c / 4) * step) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
    } else if constexpr (V == 2) {
#pragma unroll
      for (int c = 0; c < CP; c += 2) *reinterpret_cast<float2*>(o + (c / 2) * step) = make_float2(acc[c], acc[c + 1]);
    } else {
#pragma unroll
      for (int c = 0; c < CP; ++c)
        if (c < C) o[c] = acc[c];
    }
    if (j == 0 && ch == 0) {
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

// How a row of C classes is cut into per-thread chunks: CP classes each, V floats per shared-memory access.
struct ChunkPlan {
  int cp = 0, v = 0, nch = 0;
};

ChunkPlan plan_chunks(int64_t C) {
  ChunkPlan p;
  if (C < 1 || C > kSmallMaxC) return p;
  if (C % 2 == 1) {  // odd: a single chunk with one padding class
    if (C + 1 > kSmallMaxChunk) return p;
    p.cp = (int)C + 1, p.v = 1, p.nch = 1;
    return p;
  }
  // even: the largest chunk width <= 32 that divides C (at least 8 unless C itself is smaller), 128-bit if it can
  for (int cp = kSmallMaxChunk; cp >= 2; cp -= 2) {
    if (C % cp) continue;
    if (cp < 8 && C > cp) return p;  // e.g. C = 508 = 4 x 127: too many tiny chunks, leave it to the per-column kernel
    p.cp = cp, p.nch = (int)(C / cp), p.v = (cp % 4 == 0 && C % 4 == 0) ? 4 : 2;
    return p;
  }
  return p;
}

int groups_per_cta(const DecodeArgs& a, const ChunkPlan& p) {
  const int C = (int)a.C;
  int gpb = kSmallThreads / (a.K * p.nch);
  const int64_t per_group = (int64_t)(a.W + a.K) * C * 4 + 4;
  const int64_t fixed = (kSmallMaxChunk + 8) * 4 + a.W * a.K * 4;
  while (gpb > 0 && gpb * per_group + fixed > kSmallSmemBudget) --gpb;
  // every CTA's ranges must start on 16-byte boundaries: any number of groups if a group is whole float4s,
  // else a multiple of 4 groups
  if (((int64_t)a.W * C) % 4 != 0 || ((int64_t)a.K * C) % 4 != 0 || (a.y_rs != a.C && C % 4 != 0)) gpb &= ~3;
  return gpb;
}

template <int CP, int V>
cudaError_t launch_small(const DecodeArgs& a, const DecodeTables& tab, const ChunkPlan& p, cudaStream_t stream) {
  const int gpb = groups_per_cta(a, p);
  const int C = (int)a.C;
  const size_t smem = (size_t)(((gpb * a.W * C + kSmallMaxChunk + 3) & ~3) + ((gpb * a.K * C + 3) & ~3) + a.W * a.K + gpb) * 4;
  const int64_t blocks = (a.G + gpb - 1) / gpb;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  if (smem > 48 * 1024) {
    const DeviceInfo* di = nullptr;
    cudaError_t e = current_device_info(&di);
    if (e != cudaSuccess) return e;
    struct Tag {};
    if ((e = ensure_dynamic_smem<Tag>(decode_small_kernel<CP, V>, di->ordinal, (int)smem)) != cudaSuccess) return e;
  }
  decode_small_kernel<CP, V><<<(unsigned)blocks, kSmallThreads, smem, stream>>>(a, tab, gpb, p.nch);
  count_launch();
  return cudaGetLastError();
}

template <int CP = 2>
cudaError_t dispatch_cp(const DecodeArgs& a, const DecodeTables& tab, const ChunkPlan& p, cudaStream_t stream) {
  if constexpr (CP > kSmallMaxChunk) {
    return cudaErrorInvalidValue;
  } else {
    if (p.cp == CP) {
      if (p.v == 1) return launch_small<CP, 1>(a, tab, p, stream);
      if constexpr (CP % 4 == 0) {
        if (p.v == 4) return launch_small<CP, 4>(a, tab, p, stream);
      }
      return launch_small<CP, 2>(a, tab, p, stream);
    }
    return dispatch_cp<CP + 2>(a, tab, p, stream);
  }
}

}  // namespace

// Dense buffers (rows and groups back to back), 16-byte aligned, a class count that cuts into chunks (see
// plan_chunks), and room for at least one group per CTA.
bool decode_small_eligible(const DecodeArgs& a) {
  if (a.tune.kernel != 0 && a.tune.kernel != 2) return false;
  // predictions group-major and dense, or worker-major ([W][G][C]: groups C apart, workers' batches whole
  // 16-byte columns apart); results dense
  const bool group_major = a.y_rs == a.C && a.y_gs == (int64_t)a.W * a.C;
  const bool worker_major = a.y_gs == a.C && a.y_rs >= a.G * a.C && a.y_rs % 4 == 0;
  if (!(group_major || worker_major) || a.o_rs != a.C || a.o_gs != (int64_t)a.K * a.C) return false;
  if (!aligned16(a.Yt) || !aligned16(a.Yh)) return false;
  const ChunkPlan p = plan_chunks(a.C);
  if (p.cp == 0 || a.K * p.nch > kSmallThreads) return false;
  // Where it pays (measured on 3 GB problems against the per-column kernel, K = 4 .. 24, C = 10 .. 400): short
  // rows, where the per-column kernel redoes the weights for every column (1.2-2.1x at C <= 36), and many
  // queries, where that kernel's K accumulators per thread cost occupancy (1.2-1.7x at K >= 14, C < 64; from 64
  // on the bulk-copy staged kernel takes over).
  // Elsewhere below 64 the per-column kernel is as fast or faster (both reach 3-3.5 TB/s there).
  if (!(a.C <= 36 || (a.K >= 14 && a.C < 64))) return false;
  // ... except (measured on 1.5 GB problems, K = 4 .. 16; left to the per-column kernel unless this one is asked
  // for): rows of 2 or 4 classes, where one 16-byte column per thread is already the whole row or half of it
  // (per-column 1.1-1.8x), and rows of exactly 32 classes with K <= 12, where every row starts in the same
  // shared-memory banks (per-column 1.2-1.7x).
  if (a.tune.kernel == 0 && group_major && (a.C <= 4 || (a.C == 32 && a.K <= 12))) return false;
  return groups_per_cta(a, p) >= 1;
}

cudaError_t launch_decode_small(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  return dispatch_cp<>(a, tab, plan_chunks(a.C), stream);
}

}  // namespace approxifer

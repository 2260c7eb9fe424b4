// ApproxIFER decoder, wide-payload variant (Section 3, "Decoding", step 2).
//
// Same arithmetic as decode_kernel (barycentric numerator / denominator over
// the workers present in the mask, terms added in ascending worker order),
// different data movement: persistent CTAs pull the rows of PRESENT workers
// only into a shared-memory ring with bulk asynchronous copies
// (cp.async.bulk global -> shared, completion counted on an mbarrier), so the
// HBM reads of the next work items are in flight while the current item is
// reduced from shared memory.  Nothing waits on a register-staged load and the
// register file holds only the accumulators.
//
// A work item is (group, tile of COLS 16-byte columns).  SPLIT*COLS compute threads work on it:
// thread = (thread group h, column); group h forms the queries j = h*KT .. h*KT+KT-1 (KT = ceil(K/SPLIT)).
// With SPLIT = 1 (the default where it fits: K <= 16, COLS = 256, one CTA per SM; K = 9 .. 12 on 16,384 groups or more take SPLIT = 2) every payload word is read
// from shared memory once and a thread keeps all K accumulators per payload element; with SPLIT = 2 or 4 the
// thread groups share each column's payload, every thread keeps only KT accumulators, and there are more warps
// per byte of ring (two CTAs per SM).  The FMAs are packed (fma.rn.f32x2: the weights of two adjacent
// queries times one payload element, each half an ordinary round-to-nearest fp32 FMA).  One more warp is
// the producer: for each item it waits for a free ring slot, writes the item's
// signed weights (by rank) and K reciprocal denominators into the slot, and
// starts the copies of the present rows; slots are handed over and back
// through "full" / "empty" mbarriers, so producer and compute warps never meet
// at a CTA-wide barrier.  Every wait is bounded.  Items are dealt round-robin
// to the CTAs.  Every copy targets the issuing CTA's own shared memory.
#include <type_traits>

#include "common.cuh"

namespace approxifer {

__device__ unsigned int g_decode_wait_timeouts = 0;  // bounded waits that gave up (never, in a correct run)

namespace {

constexpr int kMaxStages = 4;
constexpr uint32_t kWaitLimit = 1u << 22;  // try_wait attempts before a wait gives up
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking probe of a phase (the test hook's short waits poll with this one, so that their length is a
// number of probes and not a multiple of try_wait's system-dependent blocking time).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the phase did not complete within `limit` attempts.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit, bool probe) {
  for (uint32_t it = 0; it < limit; ++it)
    if (probe ? mbar_test_wait(bar, parity) : mbar_try_wait(bar, parity)) return true;
  return false;
}
// 1-D bulk copy global -> this CTA's shared memory; src, dst and bytes are multiples of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;  // two independent round-to-nearest fp32 FMAs on the packed halves
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t dup(uint32_t v) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %1};" : "=l"(d) : "r"(v));
  return d;
}
__device__ __forceinline__ float lo_f(uint64_t v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float hi_f(uint64_t v) { return __uint_as_float((uint32_t)(v >> 32)); }

struct StagedPlan {
  int32_t tiles;       // column tiles per group
  int32_t stages;      // ring depth
  int64_t n_items;     // G * tiles
};

constexpr int kWeightsOff = 16 + 128;  // header, reciprocal denominators
__host__ __device__ constexpr int ktp4(int KT) { return (KT + 3) / 4 * 4;  }  // weights of one half, padded to float4s
// Per-slot item block: n (16 B) | 1/denominators (32 floats) | weights of the present workers, by rank:
//   float w[r][h][jj] = s_r / (alpha_j - beta_{F[r]}), j = h*KT + jj (0 beyond K or KT).
__host__ __device__ constexpr int meta_bytes(int W, int KT, int SPLIT) { return (kWeightsOff + W * SPLIT * ktp4(KT) * 4 + 127) / 128 * 128; }
constexpr int kTableOff = 128;  // float rg[W][K] after the mbarriers and the abort flag
__host__ __device__ constexpr int slots_off(int W, int K) { return (kTableOff + W * (K | 1) * 4 + 127) / 128 * 128; }
// (cb: bytes of a column of four elements -- 16 for fp32 payloads, 8 for bfloat16)
__host__ __device__ constexpr int slot_bytes(int W, int KT, int SPLIT, int COLS, int cb = 16) { return meta_bytes(W, KT, SPLIT) + W * COLS * cb; }
// Resident CTAs per SM the kernel is compiled and launched for.  The 96-thread configuration (rows of 17 .. 32
// columns: C = 68 .. 128) runs 8 per SM with up to 6 queries per thread (measured 1.19-1.30x over 6: its items are
// small and what hides their latency is more warps); with 7 or 8 queries per thread the registers that 8, or 7,
// CTAs leave cost more than the extra warps gain (0.9x), and 12 CTAs of 64 threads or 5 of 160 changed nothing or
// lost 2 %.
__host__ __device__ constexpr int min_ctas(int KT, int threads) {
  return KT > 8 ? 1 : (threads <= 64 ? 10 : (threads <= 96 ? (KT <= 6 ? 8 : 6) : (threads <= 160 ? 4 : (threads <= 288 ? 2 : 1))));
}

// Shared memory: full[4] empty[4] mbarriers, abort flag | rg[W][K] | S slots, each = item block + W rows of COLS*16 B.
// The producer compacts on the way in: the r-th PRESENT worker's row lands in row r of the slot and its signed
// weights in row r of the item block, so the compute threads index both by rank with constant strides.
// BF16: the payload elements are bfloat16 (a column of four is 8 bytes); they are widened exactly on their way
// out of shared memory and the results rounded to nearest-even on their way out, everything between is the same.
template <int KT, int COLS, int SPLIT, bool BF16 = false>
__global__ void __launch_bounds__(SPLIT* COLS + 32, min_ctas(KT, SPLIT* COLS + 32))
    decode_staged_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ DecodeTables tab,
                         const __grid_constant__ StagedPlan plan) {
  constexpr uint32_t CB = BF16 ? 8u : 16u;   // bytes of a column of four elements
  constexpr int ES = BF16 ? 2 : 4;           // bytes of an element
  constexpr int KTP4 = ktp4(KT);
  constexpr int NP = KTP4 / 2;                   // query pairs per thread
  constexpr int kThreads = SPLIT * COLS;         // compute threads
  constexpr int kConsumerWarps = kThreads / 32;
  constexpr uint32_t kRowBytes = COLS * CB;      // one worker's row inside a ring slot
  constexpr int kWRowF = SPLIT * KTP4;           // floats of one rank's weights
  extern __shared__ __align__(128) unsigned char smem_raw[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw);
  uint64_t* empty = full + kMaxStages;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_raw + 64);
  float* s_rg = reinterpret_cast<float*>(smem_raw + kTableOff);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int W = a.W, K = a.K, S = plan.stages;
  const uint32_t wb = worker_bits(W);
  const uint32_t Cv = (uint32_t)(a.C / 4);
  unsigned char* slots = smem_raw + slots_off(W, K);
  const uint32_t slot_sz = (uint32_t)slot_bytes(W, KT, SPLIT, COLS, (int)CB);
  const uint32_t meta_sz = (uint32_t)meta_bytes(W, KT, SPLIT);
  const bool producer = warp == kConsumerWarps;  // the last warp moves data and prepares items; the others compute
  const bool literal = (a.flags & kFlagSignWorkerIndex) != 0;

  const int KS = K | 1;  // odd row stride: a column of the table falls into distinct banks
  for (int idx = tid; idx < W * K; idx += kThreads + 32) s_rg[(idx / K) * KS + idx % K] = tab.rg[idx];
  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(smem_u32(full + s), 2);  // the copies' expect_tx arrival + the item block's arrival
      mbar_init(smem_u32(empty + s), kConsumerWarps);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();

  const int64_t first = blockIdx.x, stride = gridDim.x;
  const int64_t my_items = first < plan.n_items ? (plan.n_items - first + stride - 1) / stride : 0;

  // Bounded wait that also gives up when another warp of the CTA has given up.
  const bool probe = a.tune.wait_limit != 0;  // (test hook: a short limit, counted in non-blocking probes)
  const uint32_t wait_limit = probe ? a.tune.wait_limit : kWaitLimit;
  auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < wait_limit; ++it) {
      if (probe ? mbar_test_wait(addr, parity) : mbar_try_wait(addr, parity)) return true;
      if ((it & 255u) == 255u && *abort_flag) return false;
    }
    return false;
  };
  auto give_up = [&]() {
    if (lane == 0) {
      *abort_flag = 1;
      atomicAdd(&g_decode_wait_timeouts, 1u);
    }
  };

  if (producer) {
    // This warp's work per item is a serial chain, so it is kept short: no 64-bit division (the item's group
    // and tile advance incrementally), ranks from prefix population counts (lane = worker), conflict-free
    // shared-memory traffic, and the masks of the next 32 items fetched together, one per lane, so that the
    // latency of a global load is paid once per 32 items.
    const int64_t dq = stride / plan.tiles;
    const int32_t dr = (int32_t)(stride - dq * plan.tiles);
    int64_t g = first / plan.tiles;
    int32_t tile = (int32_t)(first - g * plan.tiles);
    int64_t g_batch = g;  // group / tile of the first item of the next mask batch
    int32_t tile_batch = tile;
    uint32_t mask_batch = 0;
    int64_t k = 0;
    int stage = 0;
    uint32_t phase = 1;  // parity of the slot's previous "empty" phase; first used on the second lap of the ring
    for (; k < my_items; ++k) {
      if ((k & 31) == 0) {
        // lane l fetches the mask of item k + l: its group is g_batch advanced l times
        int64_t gl = g_batch + dq * lane;
        const int64_t tl = (int64_t)tile_batch + (int64_t)dr * lane;
        gl += tl / plan.tiles;
        mask_batch = (k + lane < my_items) ? a.mask[gl] : 0u;
        // advance the batch origin by 32 items
        const int64_t t32 = (int64_t)tile_batch + (int64_t)dr * 32;
        g_batch += dq * 32 + t32 / plan.tiles;
        tile_batch = (int32_t)(t32 % plan.tiles);
      }
      if (k >= S && !wait(empty + stage, phase)) break;  // compute warps are done with the slot
      const uint32_t col0 = (uint32_t)tile * COLS;
      const uint32_t row_bytes = min((uint32_t)COLS, Cv - col0) * CB;
      unsigned char* mb = slots + (size_t)stage * slot_sz;
      int32_t* hdr = reinterpret_cast<int32_t*>(mb);  // [0] = n, [1] = first column, [2..3] = group
      float* inv_den = reinterpret_cast<float*>(mb + 16);
      float* w = reinterpret_cast<float*>(mb + kWeightsOff);
      const uint32_t m = __shfl_sync(kFull, mask_batch, (int)(k & 31)) & wb;
      const int n = __popc(m);
      const bool present = (m >> lane) & 1u;               // lane = worker i
      const int rank = __popc(m & ((1u << lane) - 1u));   // its position among the present workers
      // 1. payload first, so that it is in flight while the item block is being written
      const uint32_t bar = smem_u32(full + stage);
      if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)n * row_bytes);
      __syncwarp();
      if (present) {
        const unsigned char* src = reinterpret_cast<const unsigned char*>(a.Yt) + (g * a.y_gs + (int64_t)lane * a.y_rs + (int64_t)col0 * 4) * ES;
        bulk_g2s(smem_u32(mb) + meta_sz + (uint32_t)rank * kRowBytes, src, row_bytes, bar);
      }
      // 2. signed weights by rank, lane = worker: w[rank][c] = +-rg[i][j(c)].  The column is rotated by the
      //    lane so that the 32 stores of one step spread over the banks.
      if (present) {
        const bool neg = ((literal ? lane : rank) & 1) != 0;
        const float* src = s_rg + lane * KS;
        float* wr = w + rank * kWRowF;
#pragma unroll
        for (int c0 = 0; c0 < kWRowF; ++c0) {
          const int c = (c0 + lane) % kWRowF;
          const int h = c / KTP4, jj = c - h * KTP4;
          const int j = h * KT + jj;
          const float v = (jj < KT && j < K) ? src[j] : 0.f;
          wr[c] = neg ? -v : v;
        }
      }
      if (lane == 0) {
        hdr[0] = n;
        hdr[1] = (int32_t)col0;
        *reinterpret_cast<int64_t*>(hdr + 2) = g;
        if (col0 == 0) {
          if (a.n_used) a.n_used[g] = n;
          if (a.status) a.status[g] = (n == 0 ? kStNoWorkers : 0u) | (n < K ? kStFewWorkers : 0u);
        }
      }
      __syncwarp();
      // 3. reciprocal denominators, lane = query j: the signed weights of query j summed in ascending worker
      //    order, four loads at a time (rows beyond n contribute an exact 0)
      {
        float d = 0.f;
        const int hq = lane / KT, jq = lane - hq * KT;
        const float* wj = w + ((lane < K) ? hq * KTP4 + jq : 0);
        for (int r0 = 0; r0 < n; r0 += 4) {
          float t[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) t[u] = (r0 + u < n) ? wj[(r0 + u) * kWRowF] : 0.f;
#pragma unroll
          for (int u = 0; u < 4; ++u) d += t[u];
        }
        inv_den[lane] = 1.0f / d;
      }
      __syncwarp();  // the whole item block is written before lane 0 publishes it
      // (test hook: the item of one chosen group is staged but never announced, so the waits for it run out)
      if (lane == 0 && g != a.tune.withhold_group) mbar_arrive(bar);
      // next item of this CTA
      if (++stage == S) {
        stage = 0;
        phase ^= 1u;
      }
      g += dq;
      tile += dr;
      if (tile >= plan.tiles) {
        tile -= plan.tiles;
        ++g;
      }
    }
    if (k < my_items) {
      // A wait gave up (here or in a compute warp).  Let the copies already started land (bounded), then leave.
      give_up();
      for (int64_t q = (k > S ? k - S : 0); q < k; ++q)
        (void)mbar_wait(smem_u32(full + (q % S)), (uint32_t)((q / S) & 1), wait_limit, probe);
    }
    return;
  }

  const int half = tid / COLS;
  const uint32_t col = (uint32_t)(tid - half * COLS);

  int stage = 0;
  uint32_t phase = 0;
  for (int64_t k = 0; k < my_items; ++k) {
    if (!wait(full + stage, phase)) {
      give_up();
      // this CTA's items from here on are not (fully) written: say so in their groups' status words
      if (tid == 0 && a.status != nullptr)
        for (int64_t q = k; q < my_items; ++q) a.status[(first + q * stride) / plan.tiles] = kStTimeout;
      return;
    }
    // the producer left the item's coordinates in the slot's header
    const unsigned char* mb = slots + (size_t)stage * slot_sz;
    const int4 hdr = *reinterpret_cast<const int4*>(mb);
    const int n = hdr.x;
    const uint32_t col0 = (uint32_t)hdr.y;
    const int64_t g = (int64_t)(((uint64_t)(uint32_t)hdr.w << 32) | (uint32_t)hdr.z);
    const uint32_t ncols = min((uint32_t)COLS, Cv - col0);
    const float* inv_den = reinterpret_cast<const float*>(mb + 16);
    // idle threads (beyond the last column) shadow column 0 and store nothing
    const bool active = col < ncols;
    using Col = typename std::conditional<BF16, uint2, uint4>::type;  // a column of four payload elements as stored
    auto widen = [](Col c) -> uint4 {  // ... and as the four fp32 bit patterns the arithmetic uses
      if constexpr (BF16) return make_uint4(c.x << 16, c.x & 0xffff0000u, c.y << 16, c.y & 0xffff0000u);
      else return c;
    };
    const Col* yp = reinterpret_cast<const Col*>(mb + meta_sz) + (active ? col : 0u);                    // + r * COLS
    const ulonglong2* wp = reinterpret_cast<const ulonglong2*>(mb + kWeightsOff) + half * (KTP4 / 4);  // + r * kWRowF / 4

    // acc[p][e] = (numerator of query 2p, numerator of query 2p+1) for payload element e of this column
    uint64_t acc[NP][4];
#pragma unroll
    for (int p = 0; p < NP; ++p)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[p][e] = 0ull;

    if (n > 0) {
      // software pipeline over the ranks: the next row's payload and weights are loaded before this row's FMAs
      Col yn = yp[0];
      ulonglong2 wn[KTP4 / 4];
#pragma unroll
      for (int q = 0; q < KTP4 / 4; ++q) wn[q] = wp[q];
#pragma unroll 2
      for (int r = 0; r < n; ++r) {
        const uint4 y = widen(yn);
        uint64_t wpair[NP];
#pragma unroll
        for (int q = 0; q < KTP4 / 4; ++q) {
          wpair[2 * q] = wn[q].x;
          wpair[2 * q + 1] = wn[q].y;
        }
        const int rn = min(r + 1, n - 1);
        yn = yp[rn * COLS];
#pragma unroll
        for (int q = 0; q < KTP4 / 4; ++q) wn[q] = wp[rn * (kWRowF / 4) + q];
        const uint64_t yd[4] = {dup(y.x), dup(y.y), dup(y.z), dup(y.w)};
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          if (2 * p < KT) {  // pairs made only of padding are never touched
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[p][e] = ffma2(wpair[p], yd[e], acc[p][e]);
          }
        }
      }
    }

    float inv[KT];
#pragma unroll
    for (int jj = 0; jj < KT; ++jj) inv[jj] = (half * KT + jj < K) ? inv_den[half * KT + jj] : 0.f;
    // this warp no longer needs the slot
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(empty + stage));
    if (++stage == S) {
      stage = 0;
      phase ^= 1u;
    }

    Col* out = reinterpret_cast<Col*>(reinterpret_cast<unsigned char*>(a.Yh) + g * a.o_gs * ES) + col0 + col;
    const int64_t out_rs = a.o_rs / 4;
#pragma unroll
    for (int jj = 0; jj < KT; ++jj) {
      const int j = half * KT + jj;
      if (j < K && active) {
        const int p = jj / 2;
        float4 o;
        if (jj & 1)
          o = make_float4(inv[jj] * hi_f(acc[p][0]), inv[jj] * hi_f(acc[p][1]), inv[jj] * hi_f(acc[p][2]), inv[jj] * hi_f(acc[p][3]));
        else
          o = make_float4(inv[jj] * lo_f(acc[p][0]), inv[jj] * lo_f(acc[p][1]), inv[jj] * lo_f(acc[p][2]), inv[jj] * lo_f(acc[p][3]));
        if (n == 0) o = make_float4(0.f, 0.f, 0.f, 0.f);
        if constexpr (BF16) __stcs(out + j * out_rs, make_uint2(pack_bf16x2(o.x, o.y), pack_bf16x2(o.z, o.w)));
        else st_stream(reinterpret_cast<float4*>(out + j * out_rs), o);
      }
    }
  }
}

template <int KT, int COLS, int SPLIT, bool BF16 = false>
cudaError_t launch_kt(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  const int64_t Cv = a.C / 4;
  StagedPlan plan;
  plan.tiles = (int32_t)((Cv + COLS - 1) / COLS);
  plan.n_items = a.G * plan.tiles;
  const int64_t slot = slot_bytes(a.W, KT, SPLIT, COLS, BF16 ? 8 : 16);

  const DeviceInfo* di = nullptr;
  cudaError_t e = current_device_info(&di);
  if (e != cudaSuccess) return e;
  const int sms = di->sms, smem_sm = di->smem_per_sm;
  const int fixed = slots_off(a.W, a.K);
  // as many CTAs per SM as fit with a two-slot ring (up to min_ctas), then the ring as deep as the rest allows
  int ctas = min_ctas(KT, SPLIT * COLS + 32);
  if (a.tune.ctas_per_sm > 0 && a.tune.ctas_per_sm < ctas) ctas = a.tune.ctas_per_sm;
  while (ctas > 1 && (int64_t)ctas * (fixed + 2 * slot + 1024) > smem_sm) --ctas;
  int stages = (int)(((int64_t)smem_sm / ctas - 1024 - fixed) / slot);  // 1 KB per CTA is reserved
  if (stages < 2) return cudaErrorInvalidConfiguration;
  if (stages > kMaxStages) stages = kMaxStages;
  if (a.tune.stages >= 2 && a.tune.stages < stages) stages = a.tune.stages;
  plan.stages = stages;
  const size_t smem = (size_t)fixed + (size_t)stages * slot;
  int64_t grid = (int64_t)sms * ctas;
  if (grid > plan.n_items) grid = plan.n_items;

  struct Tag {};
  if ((e = ensure_dynamic_smem<Tag>(decode_staged_kernel<KT, COLS, SPLIT, BF16>, di->ordinal, (int)smem)) != cudaSuccess) return e;
  decode_staged_kernel<KT, COLS, SPLIT, BF16><<<(unsigned)grid, SPLIT * COLS + 32, smem, stream>>>(a, tab, plan);
  count_launch();
  return cudaGetLastError();
}

constexpr int kWholeMaxK = 16;  // most queries one thread forms (SPLIT = 1)
constexpr int kStagedMinC = 64;
constexpr int kStagedMinCManyQueries = 52;  // K >= 8: rows of 52 .. 60 floats too (2 GB problems: 1.12-1.36x the
                                            // per-column kernel at K = 8, 12; with K = 4 it is 0.5x, below 52 it loses)

// Columns per work item.  Long contiguous pieces are what HBM likes: with 256 columns an item of workload 4
// (rows of 250 float4) is whole rows -- one 4000-byte copy per present worker instead of two copies of about 2 KB
// issued by different CTAs at different times -- and the kernel runs 6 % faster (one CTA of 16 compute warps per
// SM instead of two of 8).  256 is taken when a two-slot ring of such items fits in shared memory and wastes no
// more threads on the ragged last tile than 128 would.
template <int KT, int SPLIT>
bool fits_256(const DecodeArgs& a) {
  // 544 threads (two thread groups) leave 112 registers each: enough for 8 queries per thread; a single thread
  // group of 256 carries up to 16
  if (SPLIT == 4 || (SPLIT == 2 && KT > 8) || (SPLIT == 1 && KT > kWholeMaxK)) return false;
  const DeviceInfo* di = nullptr;
  if (current_device_info(&di) != cudaSuccess) return false;
  const int smem_sm = di->smem_per_sm;
  return (int64_t)slots_off(a.W, a.K) + 2 * (int64_t)slot_bytes(a.W, KT, SPLIT, 256, a.bf16 ? 8 : 16) + 1024 <= smem_sm;
}

template <int KT, int SPLIT>
int auto_cols(const DecodeArgs& a) {
  const int64_t Cv = a.C / 4;
  if (Cv <= 16 && SPLIT == 2) return 16;  // the shortest rows: one compute warp and one producer warp per CTA
  if (Cv <= 32 && SPLIT == 2) return 32;  // short rows: small items, six CTAs per SM
  if (Cv <= 64) return 64;
  if (!fits_256<KT, SPLIT>(a)) return 128;
  const int64_t waste256 = (Cv + 255) / 256 * 256 - Cv, waste128 = (Cv + 127) / 128 * 128 - Cv;
  return waste256 <= waste128 ? 256 : 128;
}

template <int SPLIT, int KT = 1>
cudaError_t dispatch_kt(int kt, const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  if constexpr (KT > kMaxK / SPLIT) {
    return cudaErrorInvalidValue;
  } else {
    if (kt == KT) {
      int cols = a.tune.cols ? a.tune.cols : auto_cols<KT, SPLIT>(a);
      if (cols == 256 && !fits_256<KT, SPLIT>(a)) cols = 128;  // (a forced setting that cannot be honoured)
      if constexpr (SPLIT == 2) {
        if (cols == 16) return launch_kt<KT, 16, SPLIT>(a, tab, stream);
        if (cols == 32) return launch_kt<KT, 32, SPLIT>(a, tab, stream);
      }
      if (cols == 64 || cols == 32 || cols == 16) return launch_kt<KT, 64, SPLIT>(a, tab, stream);
      if constexpr (SPLIT == 2 && KT <= 8) {
        if (cols == 256) return launch_kt<KT, 256, SPLIT>(a, tab, stream);
      }
      return launch_kt<KT, 128, SPLIT>(a, tab, stream);
    }
    return dispatch_kt<SPLIT, KT + 1>(kt, a, tab, stream);
  }
}

}  // namespace

// Rows of at least 64 floats (52 with K >= 8) on the 128-bit path (measured against the other two decoders on 3 GB problems,
// K = 8 .. 16: 3.6-4.9 TB/s at C = 64, 3.8-4.5 TB/s at C = 96-100, 5.0-5.7 TB/s at C = 128, 4.9-5.9 TB/s from
// C = 200 on, where they reach 2.1-3.8 TB/s; at C = 40-48 they are as fast or faster).  Narrower payloads, and
// the (K, W) pairs in which some alpha_j equals some beta_i (the row-copy case), stay on the other kernels.
bool decode_staged_eligible(const DecodeArgs& a) {
  if (a.tune.kernel != 0 && a.tune.kernel != 3) return false;
  bool vec = aligned16(a.Yt) && aligned16(a.Yh) && a.C % 4 == 0 && a.y_gs % 4 == 0 && a.y_rs % 4 == 0 &&
             a.o_gs % 4 == 0 && a.o_rs % 4 == 0;
  // bfloat16: a column of four elements is 8 bytes, and every bulk copy must start and end on 16-byte boundaries
  if (a.bf16) vec = vec && a.C % 8 == 0 && a.y_gs % 8 == 0 && a.y_rs % 8 == 0 && a.K <= kWholeMaxK;
  const int64_t min_c = (a.K >= 8 && !a.bf16) ? kStagedMinCManyQueries : kStagedMinC * (a.bf16 ? 2 : 1);
  if (!(vec && a.C >= min_c)) return false;
  for (int j = 0; j < a.K; ++j)
    for (int i = 0; i < a.W; ++i)
      if (nodes_coincide(a.K, a.W, j, i)) return false;
  return true;
}

// One thread group forming all K queries of a column, 256-column items: the fewest shared-memory reads and
// register moves per multiply-add (each payload word is fetched and duplicated once, not once per thread group).
// Under the power cap that a long run of this kernel hits, it sustains 6.2 ms on workload 4 where two groups of
// 8 queries sustain 6.4 ms (both 5.7 ms while the clocks last).
template <int KT = 1>
cudaError_t dispatch_whole(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream, bool* taken) {
  if constexpr (KT > kWholeMaxK) {
    *taken = false;
    return cudaSuccess;
  } else {
    if (a.K == KT) {
      const int64_t Cv = a.C / 4;
      const int64_t waste256 = (Cv + 255) / 256 * 256 - Cv, waste128 = (Cv + 127) / 128 * 128 - Cv;
      // (K = 9 .. 12: two thread groups of up to 6 queries on the same 256-column items measured 1.07-1.09x
      // this plan on 3 GB problems, K = 10, 12, C = 1000, 2000; equal at K = 8, 1.01x at K = 16, where the single
      // group sustains better under the power cap)
      // ... and only from 16,384 groups on: on 4,096 groups (28 items per CTA, run right after the encoder under
      // the power cap) the single group measured 2-5 % faster.
      const bool two_groups_better = a.K >= 9 && a.K <= 12 && a.G >= 16384;
      const bool want = a.tune.split == 1 || (a.tune.split == 0 && (a.tune.cols == 0 || a.tune.cols == 256) &&
                                              waste256 <= waste128 && !two_groups_better);
      *taken = (want || a.bf16) && fits_256<KT, 1>(a);
      if (*taken && a.bf16) return launch_kt<KT, 256, 1, true>(a, tab, stream);
      return *taken ? launch_kt<KT, 256, 1>(a, tab, stream) : cudaSuccess;
    }
    return dispatch_whole<KT + 1>(a, tab, stream, taken);
  }
}

cudaError_t launch_decode_staged(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  bool taken = false;
  const cudaError_t e = dispatch_whole<>(a, tab, stream, &taken);
  if (taken) return e;
  if (a.bf16) return cudaErrorInvalidConfiguration;  // (decode_staged_eligible admits bfloat16 only where the whole-row plan fits)
  if (a.tune.split == 4) return dispatch_kt<4>((a.K + 3) / 4, a, tab, stream);
  return dispatch_kt<2>((a.K + 1) / 2, a, tab, stream);
}

cudaError_t reset_decode_wait_timeouts() {
  const unsigned int zero = 0;
  return cudaMemcpyToSymbol(g_decode_wait_timeouts, &zero, sizeof(unsigned int));
}

cudaError_t read_decode_wait_timeouts(unsigned int* out) {
  return cudaMemcpyFromSymbol(out, g_decode_wait_timeouts, sizeof(unsigned int));
}

}  // namespace approxifer

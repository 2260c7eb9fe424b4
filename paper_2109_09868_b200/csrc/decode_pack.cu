// ApproxIFER decoder for short payloads in dense buffers (Section 3, "Decoding", step 2): predictions of an even
// number of classes up to 62 -- the paper's own workloads have C = 10 -- stored back to back ([G][W][C] in,
// [G][K][C] out), or one batch per worker ([W][G][C], or W buffers of [G][C] given by a table of offsets: the
// form in which the workers' answers arrive).
//
// Same arithmetic as decode_kernel, term by term and rounding by rounding (barycentric numerator and
// denominator over the present workers in ascending order, one reciprocal per query), different data movement
// and work split:
//
//  * Every WARP is a pipeline of its own.  A warp's work item is a block of GW consecutive groups (a few KB,
//    one contiguous range: rows this short are shorter than a DRAM burst, so the absent workers' rows come
//    along and are simply never used).  Lane 0 brings items into the warp's private shared-memory ring with
//    bulk asynchronous copies, one item ahead of the one being reduced (the ring has two slots: deeper rings
//    measured slower, and cost registers), completion counted on one mbarrier per slot; a slot is refilled by the warp that has just finished reading it, so there are no "empty"
//    barriers, no producer warp and no CTA-wide barrier in the main loop.  With a dozen such warps per SM
//    there are always tens of KB of loads in flight and always some warp with arithmetic to do.  With one batch
//    per worker an item is W pieces (a worker's rows of the item's groups), copied by W lanes, one piece each,
//    onto the same mbarrier; inside the slot the rows then lie worker by worker.
//  * Lane = (group of the item, tile of two queries, word lane).  A thread forms two queries for NW words
//    (pairs of adjacent classes): every payload word it loads from shared memory feeds two packed
//    multiply-adds (fma.rn.f32x2: both halves ordinary round-to-nearest fp32 FMAs), and the signed weights
//    and denominators of its queries are formed once per worker.  All lanes step through the workers
//    0 .. W-1 together and skip (by predicate) those absent from their group's mask, so a warp reads one
//    table row and one row position at a time; a worker's rank (its sign) is a running population count.
//  * Results are collected in the ring slot they were computed from (its predictions are no longer needed, and
//    K rows never take more room than W) and streamed out by the whole warp with 128-bit stores, again one
//    contiguous range.  (A bulk copy out of shared memory frees its source only after
//    several microseconds; waiting for that dominated every variant that used one.)
//  * The masks of an item come with it: a second bulk copy on the same mbarrier brings the 16-byte columns of
//    the mask array that hold them (an ordinary load per item cost a tenth of the run time).
//  * Shared memory, not DRAM, bounds this kernel (its load/store pipe is 60-80 % busy), and an item's groups are
//    as far apart in shared memory as in DRAM, so groups can start in the same banks.  Where they do, some
//    groups take the words of their rows in an order rotated by one (register slot u holds word u + 1), which
//    puts the lanes that execute the same load or store into different banks; the host picks the groups with a
//    model of the bank rules (see choose_rotation).
//
// Every wait is bounded.  Every bulk copy targets, or reads, the issuing CTA's own shared memory.
#include <mutex>
#include <vector>

#include "common.cuh"

namespace approxifer {

__device__ unsigned int g_pack_wait_timeouts = 0;  // bounded waits that gave up (never, in a correct run)

namespace {

constexpr int kPackMaxWarps = 24;  // 768 threads: 80 registers each
__host__ __device__ constexpr int pack_max_warps(int) { return kPackMaxWarps; }
constexpr int kPackStages = 2;  // ring slots per warp
constexpr int kPackMaxNW = 5;  // words (float2) per thread and row
constexpr int kPackMaxC = 62;
constexpr int kPackMaskBytes = 160;  // up to 32 masks, widened to whole 16-byte columns of the mask array
constexpr uint32_t kPackWaitLimit = 1u << 22;
constexpr unsigned kFullMask = 0xffffffffu;

__device__ __forceinline__ uint32_t p_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void p_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void p_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void p_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool p_try_wait(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool p_test_wait(uint32_t bar, uint32_t parity) {  // non-blocking probe
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
// global -> this CTA's shared memory; src, dst and bytes are multiples of 16
__device__ __forceinline__ void p_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint64_t p_ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t p_dup(float v) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %1};" : "=l"(d) : "r"(__float_as_uint(v)));
  return d;
}

struct PackPlan {
  int32_t gw;         // groups per warp item
  int32_t nch;        // lanes sharing the words of one (group, query tile)
  int32_t jt;         // query tiles per group = ceil(K / 2)
  int32_t warps;      // warps per CTA
  int32_t in_bytes;   // one ring slot: gw * W * C floats padded to 128 B, then the item's masks (kPackMaskBytes)
  int32_t mask_off;   // where a slot's masks start
  int32_t table_bytes;
  // sizes the kernel would otherwise keep in registers (as kernel parameters they are read where they are used)
  uint32_t row_bytes;      // C floats
  uint32_t group_bytes;    // W rows
  uint32_t y_group_step;   // bytes between two groups' rows of one worker inside a ring slot
  uint32_t y_row_step;     // ... between two workers' rows of one group
  uint32_t result_bytes;   // K rows
  uint32_t wrow_bytes;     // one worker's row of the weight table: KP entries of 8 bytes
  uint32_t sign_bytes;     // between the two signs of the weight table (padded: the two copies of a row sit in
                           // different halves of the banks, since the lanes of a warp read both at once)
  uint32_t coin_off;       // where coin[32] starts
  uint32_t rot_groups;     // bit s: the lanes of the item's group s keep their row's words rotated by one
  uint32_t wait_limit;     // probes of a wait before it gives up
  int32_t probe;           // (test hook) non-blocking probes
  int64_t n_items;
};

__device__ __forceinline__ float p_lo(uint64_t v) { return __uint_as_float((uint32_t)v); }
__device__ __forceinline__ float p_hi(uint64_t v) { return __uint_as_float((uint32_t)(v >> 32)); }

// Shared memory: wtab[2][W][KP] (8 bytes each) | coin[32] | per warp: full[2] mbarriers (64 B) | 2 ring slots.
// wtab[sg][i][j] = (w, w) with w = (-1)^sg / (alpha_j - beta_i): the signed weight, already duplicated for the
// packed multiply-add (the sign flip is exact, so (s rg) y rounds like rg (s y)).
// SIMPLE: one lane owns all the words of its rows (nch == 1, NW == C/2), so every offset is a compile-time constant.
template <int NW, bool SIMPLE, bool ROT, bool WM, bool DEEP>
__global__ void __launch_bounds__(pack_max_warps(NW) * 32, 1)
    decode_pack_kernel(const __grid_constant__ DecodeArgs a, const __grid_constant__ DecodeTables tab,
                       const __grid_constant__ PackPlan plan) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int W = a.W, K = a.K, C = (int)a.C, GW = plan.gw;
  constexpr int S = kPackStages;
  const int KP = (K + 1) & ~1;
  uint64_t* wtab = reinterpret_cast<uint64_t*>(smem_raw);    // [2][W][KP], 0 beyond K
  int* coins = reinterpret_cast<int*>(smem_raw + plan.coin_off);  // [32]
  const uint32_t per_warp = 64u + (uint32_t)S * (uint32_t)plan.in_bytes;
  unsigned char* mine = smem_raw + plan.table_bytes + (size_t)warp * per_warp;
  uint64_t* full = reinterpret_cast<uint64_t*>(mine);
  unsigned char* slots = mine + 64;
  const uint32_t wb = worker_bits(W);

  for (int idx = tid; idx < 2 * W * KP; idx += blockDim.x) {
    const int sg = idx / (W * KP), rem = idx - sg * (W * KP);
    const int i = rem / KP, j = rem - i * KP;
    const float w = (j < K) ? tab.rg[i * K + j] : 0.f;
    wtab[(sg ? plan.sign_bytes / 8u : 0u) + (uint32_t)rem] = p_dup(sg ? -w : w);
  }
  if (tid < 32) coins[tid] = (tab.any_coin && tid < K) ? (int)tab.coin[tid] : -1;
  if (lane == 0) {
    for (int s = 0; s < S; ++s) p_mbar_init(p_smem_u32(full + s), 1);
    p_fence_init();
  }
  __syncthreads();

  // items are dealt to the warps of the whole grid round-robin: neighbouring warps work on neighbouring memory
  const int64_t first = (int64_t)blockIdx.x * plan.warps + warp, stride = (int64_t)gridDim.x * plan.warps;
  const int64_t my_items = first < plan.n_items ? (plan.n_items - first + stride - 1) / stride : 0;

  // lane = (group s of the item, query tile jt, word lane ch)
  const int nch = SIMPLE ? 1 : plan.nch, JT = plan.jt;
  const int sj = lane / nch, ch = lane - sj * nch;
  const int s = sj / JT, jt = sj - s * JT;
  const int j0 = jt * 2;
  const int Cw = C >> 1;
  const bool exact = SIMPLE || NW * nch == Cw;  // no lane has a word beyond the end of the row
  const bool literal = (a.flags & kFlagSignWorkerIndex) != 0;
  const uint32_t y_off = (uint32_t)s * plan.y_group_step + (uint32_t)ch * 8u;
  const uint32_t o_off = (uint32_t)(s * K + j0) * plan.row_bytes + (uint32_t)ch * 8u;
  const uint32_t u_step = (uint32_t)nch * 8u;
  // Where register slot u's word sits in a row.  With one lane per row (SIMPLE) the groups whose rows start in the
  // same banks as an earlier group's take their words in rotated order (slot u holds word (u + 1) mod NW), so
  // that the lanes of a warp, which all load slot u at once, touch different banks.
  const bool rot = ROT && ((plan.rot_groups >> s) & 1u);
  const uint32_t rot8 = rot ? 8u : 0u, last_off = rot ? 0u : (uint32_t)(NW - 1) * 8u;
  auto woff = [&](int u) -> uint32_t {
    if constexpr (SIMPLE && ROT) return u < NW - 1 ? (uint32_t)u * 8u + rot8 : last_off;
    else if constexpr (SIMPLE) return (uint32_t)u * 8u;
    else return (uint32_t)u * u_step;
  };
  const int c0 = (j0 < K) ? coins[j0] : -1, c1 = (j0 + 1 < K) ? coins[j0 + 1] : -1;
  const unsigned char* wrow0 = reinterpret_cast<const unsigned char*>(wtab) + (uint32_t)j0 * 8u;

  // Start the copies of the item whose first group is g0 into ring slot `slot`.  Group-major predictions (called
  // by lane 0): one copy of the whole block; a ragged last item may end on an 8-byte boundary: the copy takes the
  // whole 16-byte columns and the last two floats go by hand.  Worker-major (WM; called by the whole warp): lane 0
  // announces the bytes, lane i starts the copy of worker i's rows of the item's groups, which land worker by
  // worker, GW rows apart; a last item whose pieces are not whole 16-byte columns goes by hand.
  // (worker-major: where this lane's worker's batch starts, looked up once -- a per-lane index into the offset
  // table in the parameter bank is a serialised load)
  const float* my_batch = a.Yt;
  if constexpr (WM) my_batch += a.rows.on ? a.rows.off[lane < W ? lane : 0] : (int64_t)lane * a.y_rs;
  auto issue = [&](int64_t g0, int slot) {
    const int ng = (int)min((int64_t)GW, a.G - g0);
    unsigned char* dst = slots + (size_t)slot * plan.in_bytes;
    const uint32_t bar = p_smem_u32(full + slot);
    // (test hook: the item that holds one chosen group is never fetched, so the wait for it runs out)
    if (a.tune.withhold_group >= g0 && a.tune.withhold_group < g0 + ng) return;
    // the item's masks travel the same way: the whole 16-byte columns of the mask array that hold them (group g's
    // mask lands at word (g0 & 3) + g - g0 of the slot's mask area); by hand where those would end beyond the array
    const int64_t m0 = g0 & ~int64_t(3), m1 = (g0 + ng + 3) & ~int64_t(3);
    const uint32_t mask_bytes = m1 <= a.G ? (uint32_t)(m1 - m0) * 4u : 0u;
    if (lane == 0 && mask_bytes == 0)
      for (int q = 0; q < ng; ++q) reinterpret_cast<uint32_t*>(dst + plan.mask_off)[(int)(g0 & 3) + q] = a.mask[g0 + q];
    if constexpr (!WM) {
      const uint32_t bytes = (uint32_t)ng * plan.group_bytes, bytes16 = bytes & ~15u;
      const unsigned char* src = reinterpret_cast<const unsigned char*>(a.Yt) + g0 * (int64_t)plan.group_bytes;
      if (bytes16 != bytes) *reinterpret_cast<float2*>(dst + bytes16) = *reinterpret_cast<const float2*>(src + bytes16);
      // (release: what was written by hand above is visible to whoever sees the phase complete)
      p_arrive_expect_tx(bar, bytes16 + mask_bytes);
      if (bytes16) p_bulk_g2s(p_smem_u32(dst), src, bytes16, bar);
      if (mask_bytes) p_bulk_g2s(p_smem_u32(dst + plan.mask_off), a.mask + m0, mask_bytes, bar);
    } else {
      const uint32_t piece = (uint32_t)ng * plan.row_bytes;  // one worker's rows of the item's groups
      const bool whole = (piece & 15u) == 0;
      const float* src = my_batch + g0 * (int64_t)C;
      unsigned char* mine_dst = dst + (uint32_t)lane * plan.y_row_step;
      if (!whole && lane < W)
        for (uint32_t f = 0; f < piece / 4u; ++f) reinterpret_cast<float*>(mine_dst)[f] = src[f];
      __syncwarp();  // (what the lanes wrote by hand is ordered before lane 0's release below)
      if (lane == 0) {
        p_arrive_expect_tx(bar, (whole ? (uint32_t)W * piece : 0u) + mask_bytes);
        if (mask_bytes) p_bulk_g2s(p_smem_u32(dst + plan.mask_off), a.mask + m0, mask_bytes, bar);
      }
      if (whole && lane < W) p_bulk_g2s(p_smem_u32(mine_dst), src, piece, bar);
    }
  };

  const bool probe = plan.probe != 0;  // (test hook: a short limit, counted in non-blocking probes)
  // prologue: one item in flight
  const int64_t g_stride = stride * GW;
  int left = (int)my_items;  // items this warp has still to reduce (the launch keeps this below 2^31)
  int64_t g0 = first * GW;   // first group of the item being reduced
  if ((WM || lane == 0) && left > 0) issue(g0, 0);

  int slot = 0;  // ring slot of the item being reduced; the item started in the same iteration goes to the other
  uint32_t parity = 0;
  bool failed = false;
  for (; left > 0; --left, g0 += g_stride) {
    const int ng = (int)min((int64_t)GW, a.G - g0);
    // the slot that the previous item occupied is free (its results were copied out of it before the __syncwarp
    // that ended the previous iteration): refill it with the next item
    if ((WM || lane == 0) && left > 1) issue(g0 + g_stride, slot ^ 1);
    // wait for this item's bytes (bounded)
    {
      const uint32_t addr = p_smem_u32(full + slot);
      bool ok = false;
      for (uint32_t it = 0; it < plan.wait_limit && !ok; ++it) ok = probe ? p_test_wait(addr, parity) : p_try_wait(addr, parity);
      if (!__all_sync(kFullMask, ok)) {
        if (lane == 0) atomicAdd(&g_pack_wait_timeouts, 1u);
        failed = true;
        // this warp's items from here on are not written: say so in their groups' status words
        if (a.status != nullptr) {
          int64_t q = g0;
          for (int c = left; c > 0; --c, q += g_stride)
            if (s < GW && q + s < a.G) a.status[q + s] = kStTimeout;
        }
        break;
      }
    }
    const unsigned char* slot_base = slots + (size_t)slot * plan.in_bytes;
    const uint32_t mask =
        (s < ng) ? (reinterpret_cast<const uint32_t*>(slot_base + plan.mask_off)[(int)(g0 & 3) + s] & wb) : 0u;
    const unsigned char* yg = slot_base + y_off;
    uint64_t acc0[NW], acc1[NW];  // numerators of this lane's two queries, a pair of classes per word
    float inv0 = 0.f, inv1 = 0.f;
    bool pin0 = false, pin1 = false;
    int n = 0;
    if (s < ng) {
#pragma unroll
      for (int u = 0; u < NW; ++u) acc0[u] = acc1[u] = 0ull;
      float den0 = 0.f, den1 = 0.f;
      uint32_t r = 0;  // present workers so far = rank of the next one
      const unsigned char* yr = yg;
      const unsigned char* wr = wrow0;
      // one worker's row (an absent worker's row may be loaded; it is only used under `present`)
      auto row = [&](int i) {
        uint64_t y[NW];
#pragma unroll
        for (int u = 0; u < NW; ++u)
          y[u] = (exact || u * nch + ch < Cw) ? *reinterpret_cast<const uint64_t*>(yr + woff(u)) : 0ull;
        if ((mask >> i) & 1u) {
          // the signed, duplicated weights of this lane's two queries
          const uint32_t odd = (literal ? (uint32_t)i : r) & 1u;
          const ulonglong2 w2 = *reinterpret_cast<const ulonglong2*>(wr + odd * plan.sign_bytes);
          den0 = __fadd_rn(den0, p_lo(w2.x));
          den1 = __fadd_rn(den1, p_lo(w2.y));
#pragma unroll
          for (int u = 0; u < NW; ++u) {
            acc0[u] = p_ffma2(w2.x, y[u], acc0[u]);
            acc1[u] = p_ffma2(w2.y, y[u], acc1[u]);
          }
          ++r;
        }
        yr += plan.y_row_step, wr += plan.wrow_bytes;
      };
      // (DEEP: unrolled by four where a group has three or more lanes, K >= 5: measured 1.00-1.14x there, 0.93x
      // with one or two lanes per group; a kernel of its own, since the two loops side by side cost the shapes
      // that take the short one 6-10 %)
      if constexpr (DEEP) {
#pragma unroll 4
        for (int i = 0; i < W; ++i) row(i);
      } else {
#pragma unroll 2
        for (int i = 0; i < W; ++i) row(i);
      }
      n = (int)r;
      // alpha_j == beta_i for a present worker i: the interpolant takes that worker's value
      pin0 = c0 >= 0 && ((mask >> c0) & 1u), pin1 = c1 >= 0 && ((mask >> c1) & 1u);
      inv0 = __frcp_rn(den0), inv1 = __frcp_rn(den1);
      if (pin0 || pin1) {
#pragma unroll
        for (int u = 0; u < NW; ++u) {
          if (exact || u * nch + ch < Cw) {
            if (pin0) acc0[u] = *reinterpret_cast<const uint64_t*>(yg + (uint32_t)c0 * plan.y_row_step + woff(u));
            if (pin1) acc1[u] = *reinterpret_cast<const uint64_t*>(yg + (uint32_t)c1 * plan.y_row_step + woff(u));
          }
        }
      }
    }
    __syncwarp();  // every lane has finished reading the slot: the results take its place
    unsigned char* ob = slots + (size_t)slot * plan.in_bytes;
    if (s < ng) {
      unsigned char* orow = ob + o_off;
#pragma unroll
      for (int u = 0; u < NW; ++u) {
        if (exact || u * nch + ch < Cw) {
          float2 v0 = pin0 ? make_float2(p_lo(acc0[u]), p_hi(acc0[u])) : make_float2(p_lo(acc0[u]) * inv0, p_hi(acc0[u]) * inv0);
          float2 v1 = pin1 ? make_float2(p_lo(acc1[u]), p_hi(acc1[u])) : make_float2(p_lo(acc1[u]) * inv1, p_hi(acc1[u]) * inv1);
          if (n == 0) v0 = v1 = make_float2(0.f, 0.f);
          if (j0 < K) *reinterpret_cast<float2*>(orow + woff(u)) = v0;
          if (j0 + 1 < K) *reinterpret_cast<float2*>(orow + plan.row_bytes + woff(u)) = v1;
        }
      }
      if (jt == 0 && ch == 0) {
        if (a.n_used) a.n_used[g0 + s] = n;
        if (a.status) a.status[g0 + s] = (n == 0 ? kStNoWorkers : 0u) | (n < K ? kStFewWorkers : 0u);
      }
    }
    __syncwarp();  // all results are in place
    {
      // the item's results are one contiguous range: the warp streams it out in whole 16-byte columns (a ragged
      // last item may end on an 8-byte boundary)
      const uint32_t bytes = (uint32_t)ng * plan.result_bytes, n16 = bytes >> 4;
      unsigned char* dst = reinterpret_cast<unsigned char*>(a.Yh) + g0 * (int64_t)plan.result_bytes;
      for (uint32_t q = lane; q < n16; q += 32)
        st_stream(reinterpret_cast<float4*>(dst) + q, reinterpret_cast<const float4*>(ob)[q]);
      if (lane == 0 && (bytes & 15u))
        __stcs(reinterpret_cast<float2*>(dst + (n16 << 4)), *reinterpret_cast<const float2*>(ob + (n16 << 4)));
    }
    __syncwarp();  // the slot may be refilled
    parity ^= (uint32_t)slot;  // (a slot's phase flips every second item)
    slot ^= 1;
  }
  if (lane == 0 && failed) {
    // the copies of the failed item and of the one after it have been started: they must land before the CTA's
    // shared memory is given up (bounded)
    for (int d = 0; d < S && d < left; ++d) {
      const uint32_t addr = p_smem_u32(full + slot);
      for (uint32_t it = 0; it < plan.wait_limit; ++it)
        if (probe ? p_test_wait(addr, parity) : p_try_wait(addr, parity)) break;
      parity ^= (uint32_t)slot;
      slot ^= 1;
    }
  }
}

struct PackChoice {
  int nw = 0, nch = 0, jt = 0, gw = 0, warps = 0;
  uint32_t rot_groups = 0;
  bool worker_major = false;
  int in_bytes = 0, mask_off = 0, table_bytes = 0, smem = 0;
};

// How the words of a row are dealt to lanes: NW <= 5 words per lane (more would need more registers than 24 warps
// per SM leave), nch lanes per (group, query tile).  The largest NW that pads the row by at most an eighth, else the
// one that pads it least.
void choose_words(int Cw, int* nw, int* nch) {
  int best_nw = 1, best_waste = 1 << 30;
  for (int w = kPackMaxNW; w >= 1; --w) {
    const int n = (Cw + w - 1) / w;
    const int waste = n * w - Cw;
    if (waste * 8 <= Cw) {
      best_nw = w;
      break;
    }
    if (waste < best_waste) best_nw = w, best_waste = waste;
  }
  *nw = best_nw;
  *nch = (Cw + best_nw - 1) / best_nw;
}

// Shared-memory cost of an item, in passes of the 32 banks ("wavefronts"), for a given set of rotated groups.
// The rules are measured ones (64-bit accesses, cycles per instruction with the memory pipe saturated):
//   loads:  the whole warp at once; lanes reading the same word share it; the cost is the largest number of
//           different words that fall into one bank;
//   stores: one half-warp after the other, each costing the largest number of different words in one bank.
// A row's words are 8-byte aligned, so banks are counted in pairs.  Counted: the W x NW loads of the worker loop
// (every lane of group s reads word slot u of its row: bytes s * group_bytes + off(u)) and the 2 x NW stores of
// the results (lane (s, jt): bytes s * result_bytes + jt * 2 * row_bytes + off(u); the second query's row is a
// uniform shift).  What the rotation cannot change (weights, copy-out) is left out.
// Returned: passes * 4096 + the number of words beyond the first in every bank (a tie-break that lets a search
// move across sets with the same number of passes).  A pass of a store counts twice: the stores sit in the
// dependent tail of an item, between two warp barriers, and measured about that much dearer than the loads of
// the pipelined worker loop.
// in_step: bytes between two groups' rows of one worker in a ring slot (W C 4 group-major, C 4 worker-major).
int64_t rotation_cost(int K, int W, int C, int gw, int jt, uint32_t in_step, uint32_t rot_groups, int* passes = nullptr) {
  const int NW = C / 2;
  const uint32_t row_bytes = (uint32_t)C * 4u, group_bytes = in_step, result_bytes = (uint32_t)K * row_bytes;
  int loads = 0, stores = 0, excess_loads = 0, excess_stores = 0;
  for (int u = 0; u < NW; ++u) {
    uint32_t seen[16][32];  // the different words met so far in each bank pair
    int n_seen[16];
    auto reset = [&]() {
      for (int b = 0; b < 16; ++b) n_seen[b] = 0;
    };
    auto touch = [&](uint32_t byte) {
      const uint32_t word = byte / 8u, b = word % 16u;
      for (int q = 0; q < n_seen[b]; ++q)
        if (seen[b][q] == word) return;
      seen[b][n_seen[b]++] = word;
    };
    auto worst = [&]() {
      int m = 0;
      for (int b = 0; b < 16; ++b) m = n_seen[b] > m ? n_seen[b] : m;
      return m;
    };
    auto excess = [&]() {
      int e = 0;
      for (int b = 0; b < 16; ++b) e += n_seen[b] > 1 ? n_seen[b] - 1 : 0;
      return e;
    };
    auto off = [&](int s) -> uint32_t {
      const bool rot = (rot_groups >> s) & 1u;
      return (uint32_t)((u + (rot ? 1 : 0)) % NW) * 8u;
    };
    reset();
    for (int s = 0; s < gw; ++s) touch((uint32_t)s * group_bytes + off(s));
    loads += worst();
    excess_loads += excess();
    for (int half = 0; half < 2; ++half) {
      reset();
      for (int lane = half * 16; lane < half * 16 + 16 && lane < gw * jt; ++lane) {
        const int s = lane / jt, t = lane - s * jt;
        touch((uint32_t)s * result_bytes + (uint32_t)t * 2u * row_bytes + off(s));
      }
      stores += worst();
      excess_stores += excess();
    }
  }
  if (passes != nullptr) *passes = W * loads + 2 * stores;
  return (int64_t)(W * loads + 4 * stores) * 4096 + W * excess_loads + 4 * excess_stores;
}

// Which groups of an item keep the words of their rows rotated by one (kernels with one lane per row): the best of
// the sets "groups whose index has odd parity under a bit mask", improved by a few rounds of
// flip-one-group-if-it-helps.  Whether it is used follows what was measured on 18 shapes (K = 2 .. 16,
// C = 6, 8, 10; 2-3 GB each): with three or more lanes per group (K >= 5) every set the model prefers gained
// (6-55 %); with one or two lanes per group (K <= 4) it gained (28 %) only where shared memory is what bounds the
// kernel -- more than one pass per 25 bytes moved -- and cost 5-10 % elsewhere (those shapes already run at the
// DRAM rate, and the rotated code has a few more instructions); rows of fewer than 8 classes lost either way.
// The answer depends on the shape alone and is remembered per shape.  mode (tuning): 1 never, 2 whenever the
// model prefers a set.
uint32_t choose_rotation(int K, int W, int C, int gw, int jt, uint32_t in_step, int mode) {
  if (mode == 1 || gw < 2) return 0u;
  struct Entry {
    int K, W, C, gw, mode;
    uint32_t in_step, rot;
  };
  static std::mutex mu;
  static std::vector<Entry> memo;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : memo)
      if (e.K == K && e.W == W && e.C == C && e.gw == gw && e.mode == mode && e.in_step == in_step) return e.rot;
  }
  int plain_passes = 0;
  const int64_t plain = rotation_cost(K, W, C, gw, jt, in_step, 0u, &plain_passes);
  uint32_t best = 0u;
  int64_t best_cost = plain;
  for (uint32_t m = 1; m < 32; ++m) {
    uint32_t cand = 0u;
    for (int s = 0; s < gw; ++s)
      if (__builtin_popcount((uint32_t)s & m) & 1) cand |= 1u << s;
    const int64_t c = rotation_cost(K, W, C, gw, jt, in_step, cand);
    if (c < best_cost) best = cand, best_cost = c;
  }
  for (int round = 0; round < 3; ++round) {
    bool changed = false;
    for (int s = 0; s < gw; ++s) {
      const uint32_t cand = best ^ (1u << s);
      const int64_t c = rotation_cost(K, W, C, gw, jt, in_step, cand);
      if (c < best_cost) best = cand, best_cost = c, changed = true;
    }
    if (!changed) break;
  }
  // all passes of an item: the counted ones, the weights (about 1.5 per worker) and the copy-out (a load and a
  // store of every 128 result bytes)
  const int64_t result_bytes = (int64_t)gw * K * C * 4, moved = (int64_t)gw * W * C * 4 + result_bytes;
  const int64_t all_passes = plain_passes + (3 * W) / 2 + 2 * (result_bytes / 128);
  const bool bound_by_shared = all_passes * 25 >= moved;
  const bool use = best_cost < plain && (mode == 2 || (C >= 8 && (jt >= 3 || bound_by_shared)));
  const uint32_t rot = use ? best : 0u;
  std::lock_guard<std::mutex> lock(mu);
  if (memo.size() < 256) memo.push_back(Entry{K, W, C, gw, mode, in_step, rot});
  return rot;
}

// One batch per worker: rows of a worker C apart from group to group, the workers' batches anywhere (a table of
// offsets, or a stride that keeps them apart), all on 16-byte boundaries.
bool pack_worker_major(const DecodeArgs& a) {
  if (a.y_gs != a.C) return false;
  if (a.rows.on) {
    for (int i = 0; i < a.W; ++i)
      if (a.rows.off[i] % 4 != 0) return false;
    return true;
  }
  return a.y_rs % 4 == 0 && a.y_rs >= a.G * a.C;
}

bool plan_pack(const DecodeArgs& a, int smem_per_sm, PackChoice* out) {
  PackChoice p;
  const int K = a.K, W = a.W, C = (int)a.C;
  p.worker_major = !(a.y_rs == a.C && a.y_gs == (int64_t)a.W * a.C && !a.rows.on) && pack_worker_major(a);
  if (C < 2 || C > kPackMaxC || (C & 1)) return false;
  p.jt = (K + 1) / 2;
  choose_words(C / 2, &p.nw, &p.nch);
  const int lpg = p.jt * p.nch;  // lanes per group
  if (lpg > 32) return false;
  int gw = 32 / lpg;
  if (a.tune.cols > 0 && a.tune.cols < gw) gw = a.tune.cols;  // (tuning: upper bound on the groups per item)
  if ((int64_t)gw > a.G) gw = (int)a.G;
  // every item, and its block of results, starts on a 16-byte boundary
  // (worker-major: every worker's piece of an item)
  const int in_unit = p.worker_major ? C : W * C;
  while (gw >= 1 && (int64_t)gw < a.G && (((int64_t)gw * in_unit) % 4 != 0 || ((int64_t)gw * K * C) % 4 != 0)) --gw;
  if (gw < 1) return false;
  p.gw = gw;
  if (K > W) return false;  // (the results of an item are staged in the slot of its predictions)
  if ((a.G + gw - 1) / gw > (int64_t)INT32_MAX) return false;  // (a warp counts its items in 32 bits)
  p.mask_off = (gw * W * C * 4 + 127) & ~127;
  p.in_bytes = p.mask_off + kPackMaskBytes;
  const int KP = (K + 1) & ~1;
  p.table_bytes = (2 * W * KP * 8 + 128 + 128 + 127) & ~127;  // two copies, up to 120 B between them, coin[32]
  const int budget = smem_per_sm - 1024 - p.table_bytes;
  // Two slots per warp: one item in flight while one is reduced.  What hides the latency of the loads is the
  // number of warps (each with an item in flight), not the depth of a warp's ring: measured, 22 warps with two
  // slots beat 16 with three and 12 with four.
  const int per_warp = 64 + kPackStages * p.in_bytes;
  int warps = budget / per_warp;
  if (warps > pack_max_warps(p.nw)) warps = pack_max_warps(p.nw);
  if (a.tune.ctas_per_sm > 0 && a.tune.ctas_per_sm < warps) warps = a.tune.ctas_per_sm;  // (tuning: warps per CTA)
  if (warps < 4) return false;
  p.warps = warps;
  // (worker-major items hold a worker's rows of consecutive groups back to back, C floats apart; there the
  // sets the model prefers measured 0.91-0.93x -- what bounds that form is the W small copies per item, not
  // shared memory -- so nothing is rotated)
  if (p.nch == 1 && p.nw * 2 == C && !p.worker_major)
    p.rot_groups = choose_rotation(K, W, C, gw, p.jt, (uint32_t)(W * C * 4), a.tune.split);
  p.smem = p.table_bytes + warps * per_warp;
  *out = p;
  return true;
}

template <int NW, bool SIMPLE, bool ROT, bool WM, bool DEEP>
cudaError_t launch_pack(const DecodeArgs& a, const DecodeTables& tab, const PackChoice& c, const DeviceInfo& di,
                        cudaStream_t stream) {
  PackPlan plan;
  plan.gw = c.gw, plan.nch = c.nch, plan.jt = c.jt, plan.warps = c.warps;
  plan.in_bytes = c.in_bytes, plan.mask_off = c.mask_off, plan.table_bytes = c.table_bytes;
  plan.n_items = (a.G + c.gw - 1) / c.gw;
  const int KP = (a.K + 1) & ~1;
  plan.row_bytes = (uint32_t)a.C * 4u;
  plan.group_bytes = (uint32_t)a.W * plan.row_bytes;
  plan.y_group_step = c.worker_major ? plan.row_bytes : plan.group_bytes;
  plan.y_row_step = c.worker_major ? (uint32_t)c.gw * plan.row_bytes : plan.row_bytes;
  plan.result_bytes = (uint32_t)a.K * plan.row_bytes;
  plan.wrow_bytes = (uint32_t)KP * 8u;
  plan.sign_bytes = (uint32_t)a.W * plan.wrow_bytes;
  plan.sign_bytes += (64u + 128u - plan.sign_bytes % 128u) % 128u;  // (64 mod 128; a multiple of 8 stays one)
  plan.coin_off = plan.sign_bytes + (uint32_t)a.W * plan.wrow_bytes;
  plan.rot_groups = c.rot_groups;
  plan.probe = a.tune.wait_limit != 0;
  plan.wait_limit = plan.probe ? a.tune.wait_limit : kPackWaitLimit;
  struct Tag {};
  cudaError_t e = ensure_dynamic_smem<Tag>(decode_pack_kernel<NW, SIMPLE, ROT, WM, DEEP>, di.ordinal, c.smem);
  if (e != cudaSuccess) return e;
  int64_t grid = di.sms;
  const int64_t need = (plan.n_items + c.warps - 1) / c.warps;
  if (grid > need) grid = need;
  decode_pack_kernel<NW, SIMPLE, ROT, WM, DEEP><<<(unsigned)grid, c.warps * 32, c.smem, stream>>>(a, tab, plan);
  count_launch();
  return cudaGetLastError();
}

template <int NW = 1>
cudaError_t dispatch_nw(const DecodeArgs& a, const DecodeTables& tab, const PackChoice& c, const DeviceInfo& di,
                        cudaStream_t stream) {
  if constexpr (NW > kPackMaxNW) {
    return cudaErrorInvalidValue;
  } else {
    if (c.nw == NW) {
      const bool deep = c.jt >= 3;  // K >= 5
      if (c.nch == 1 && NW * 2 == a.C) {
        if (c.worker_major)
          return deep ? launch_pack<NW, true, false, true, true>(a, tab, c, di, stream)
                      : launch_pack<NW, true, false, true, false>(a, tab, c, di, stream);
        if (c.rot_groups != 0)
          return deep ? launch_pack<NW, true, true, false, true>(a, tab, c, di, stream)
                      : launch_pack<NW, true, true, false, false>(a, tab, c, di, stream);
        return deep ? launch_pack<NW, true, false, false, true>(a, tab, c, di, stream)
                    : launch_pack<NW, true, false, false, false>(a, tab, c, di, stream);
      }
      if (c.worker_major)
        return deep ? launch_pack<NW, false, false, true, true>(a, tab, c, di, stream)
                    : launch_pack<NW, false, false, true, false>(a, tab, c, di, stream);
      return deep ? launch_pack<NW, false, false, false, true>(a, tab, c, di, stream)
                  : launch_pack<NW, false, false, false, false>(a, tab, c, di, stream);
    }
    return dispatch_nw<NW + 1>(a, tab, c, di, stream);
  }
}

}  // namespace

// Dense buffers (rows and groups back to back, or one dense batch per worker), 16-byte aligned, an even number of
// classes up to 62.  Chosen
// automatically where it is the fastest of the decoders (measured on 3 GB problems, K = 4 .. 16: 1.1-1.5x the
// thread-per-(query, chunk) kernel at C = 10): rows of 6 .. 10 classes, which one lane covers whole, and at
// least 32 MB of predictions (K = 8, W = 12, C = 10: equal and launch-bound up to 65,536 groups, 1.10x at
// 131,072, 1.26x at 524,288).  Other even C up to 62 run correctly when asked for (tuning kernel = 4); there the
// other kernels are as fast or faster except at isolated C (32, 40, 62 with K <= 8).
bool decode_pack_eligible(const DecodeArgs& a) {
  if (a.tune.kernel != 0 && a.tune.kernel != 4) return false;
  if (a.tune.kernel == 0 && (a.C < 6 || a.C > 2 * kPackMaxNW || a.G * (int64_t)a.W * a.C * 4 < (int64_t(32) << 20))) return false;
  const bool group_major = a.y_rs == a.C && a.y_gs == (int64_t)a.W * a.C && !a.rows.on;
  if (!(group_major || pack_worker_major(a)) || a.o_rs != a.C || a.o_gs != (int64_t)a.K * a.C) return false;
  if (!aligned16(a.Yt) || !aligned16(a.Yh) || !aligned16(a.mask)) return false;
  const DeviceInfo* di = nullptr;
  if (current_device_info(&di) != cudaSuccess) return false;
  PackChoice c;
  return plan_pack(a, di->smem_per_sm, &c);
}

// The plan's host-side choices for a shape, without a device: groups per item, the rotated groups, and the model's
// shared-memory passes per item (loads of the worker loop + stores of the results) without and with them.
bool pack_rotation_info(int K, int W, int64_t C, int mode, int* groups_per_item, uint32_t* rotated_groups,
                        int* passes_plain, int* passes_chosen) {
  DecodeArgs a{};
  a.K = K, a.W = W, a.C = C, a.G = int64_t(1) << 30;
  a.tune.split = mode;
  PackChoice c;
  if (!plan_pack(a, 227 * 1024, &c)) return false;
  *groups_per_item = c.gw;
  *rotated_groups = c.rot_groups;
  *passes_plain = *passes_chosen = 0;
  if (c.nch == 1 && c.nw * 2 == C) {
    (void)rotation_cost(K, W, (int)C, c.gw, c.jt, (uint32_t)(W * C * 4), 0u, passes_plain);
    (void)rotation_cost(K, W, (int)C, c.gw, c.jt, (uint32_t)(W * C * 4), c.rot_groups, passes_chosen);
  }
  return true;
}

cudaError_t reset_pack_wait_timeouts() {
  const unsigned int zero = 0;
  return cudaMemcpyToSymbol(g_pack_wait_timeouts, &zero, sizeof(unsigned int));
}

cudaError_t read_pack_wait_timeouts(unsigned int* out) {
  return cudaMemcpyFromSymbol(out, g_pack_wait_timeouts, sizeof(unsigned int));
}

cudaError_t launch_decode_pack(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream) {
  const DeviceInfo* di = nullptr;
  cudaError_t e = current_device_info(&di);
  if (e != cudaSuccess) return e;
  PackChoice c;
  if (!plan_pack(a, di->smem_per_sm, &c)) return cudaErrorInvalidConfiguration;
  return dispatch_nw<>(a, tab, c, *di, stream);
}

}  // namespace approxifer

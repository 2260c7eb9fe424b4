// Shared declarations of the ApproxIFER CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "tables.h"

namespace approxifer {

// status[g] bits (mirrors approxifer.h)
constexpr uint32_t kStNoWorkers = 1u;
constexpr uint32_t kStFewWorkers = 2u;
constexpr uint32_t kStLocateUnderdetermined = 4u;
constexpr uint32_t kStNonfinite = 8u;
constexpr uint32_t kStTimeout = 16u;

constexpr uint32_t kFlagSignWorkerIndex = 1u;
constexpr uint32_t kFlagLocateHomogeneous = 2u;

// Rows of a group that are not a fixed stride apart: off[i] = element offset of worker i's row of group 0 from the
// base pointer (the rows of one worker for consecutive groups are still `gstride` apart).  Used by the scatter /
// gather entry points, where every worker's batch is a buffer of its own.
struct RowOffsets {
  int64_t off[kMaxW];
  int32_t on = 0;
};

struct EncodeArgs {
  const float* X;  // (bfloat16 payloads: really const uint16_t*, see `bf16`)
  float* Xt;
  int64_t x_gs, x_rs, o_gs, o_rs;  // element strides
  int64_t G, D;
  int32_t K, W;
  int32_t bf16 = 0;  // payload elements are bfloat16 (2 bytes) instead of fp32; weights and sums stay fp32
  RowOffsets rows;   // (scatter) where the W coded rows go, instead of o_rs apart
};

// Test / tuning choices of one decode call (all zero = automatic); see approxifer_debug_decode.
struct DecodeTuning {
  int32_t kernel = 0;       // 0 automatic; 1 per-column register-staged, 2 thread-per-(query, chunk), 3 bulk-copy
                            // staged, 4 packed-groups kernel (2..4: only where the kernel takes the shape)
  int32_t stages = 0;       // bulk-copy staged kernel: upper bound on the ring depth
  int32_t ctas_per_sm = 0;  // ... upper bound on resident CTAs per SM
  int32_t cols = 0;         // ... 16-byte columns per work item
  int32_t split = 0;        // ... thread groups sharing the K queries of a column
  // exercising the bounded waits (tests only): a poll limit (0 = the built-in one; polls are then non-blocking
  // probes) and a group whose staged data is never announced to the threads that wait for it (-1 = none)
  uint32_t wait_limit = 0;
  int64_t withhold_group = -1;
};

struct DecodeArgs {
  const float* Yt;
  const uint32_t* mask;
  float* Yh;
  int32_t* n_used;
  uint32_t* status;
  int64_t y_gs, y_rs, o_gs, o_rs;
  int64_t G, C;
  int32_t K, W;
  uint32_t flags;
  DecodeTuning tune = {};
  int32_t bf16 = 0;  // Yt and Yh hold bfloat16 elements (2 bytes); weights and sums stay fp32
  RowOffsets rows;   // (gather) where the W coded rows are, instead of y_rs apart
};

struct LocateArgs {
  const float* Yt;
  const uint32_t* mask;
  int32_t* adv;
  uint32_t* trusted;
  uint32_t* status;
  int64_t y_gs, y_rs;
  int64_t G, C;
  int32_t K, W, E;
  uint32_t flags;
  // Algorithm 3 (rational decoding) only: where r(alpha_j) goes; NULL for the locator proper
  float* Yh = nullptr;
  int64_t o_gs = 0, o_rs = 0;
  int32_t force_warp_kernel = 0;  // test hook: the warp-per-group kernel also where the thread-per-class one would run
  // locate and decode in one pass (Yh, o_gs, o_rs above receive the decoded predictions instead of Algorithm 3's)
  int32_t fuse_decode = 0;
  int32_t* n_used = nullptr;          // decode's optional outputs
  uint32_t* decode_status = nullptr;
  RowOffsets rows;                    // (gather) where the W coded rows are, instead of y_rs apart
};

// Each returns a cudaError_t from the launch (cudaSuccess if nothing to do).
cudaError_t launch_encode(const EncodeArgs& a, cudaStream_t stream);
cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream);
cudaError_t launch_locate(const LocateArgs& a, cudaStream_t stream);
cudaError_t launch_fma_peak(int iters, int blocks, float* sink, cudaStream_t stream);
cudaError_t launch_debug_weights(int K, int W, uint32_t flags, uint32_t mask, int which, float* w, int32_t* idx,
                                 int32_t* n, cudaStream_t stream);

// Wide-payload decoder (bulk-copy staged); see decode_staged.cu.
bool decode_staged_eligible(const DecodeArgs& a);
cudaError_t launch_decode_staged(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream);
cudaError_t read_decode_wait_timeouts(unsigned int* out);

// Short- and medium-payload decoder for dense buffers (groups packed into work items); see decode_pack.cu.
bool decode_pack_eligible(const DecodeArgs& a);
cudaError_t launch_decode_pack(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream);
cudaError_t read_pack_wait_timeouts(unsigned int* out);
bool pack_rotation_info(int K, int W, int64_t C, int mode, int* groups_per_item, uint32_t* rotated_groups,
                        int* passes_plain, int* passes_chosen);
cudaError_t reset_decode_wait_timeouts();
cudaError_t reset_pack_wait_timeouts();

// Short-payload decoder (C <= 32, dense buffers); see decode_small.cu.
bool decode_small_eligible(const DecodeArgs& a);
cudaError_t launch_decode_small(const DecodeArgs& a, const DecodeTables& tab, cudaStream_t stream);

// Thread-per-class locator for K+E <= kLocateRowsMaxM (locate_rows_impl.cuh); the warp-per-group kernel covers the rest.
constexpr int kLocateRowsMaxM = 15;
// ... and its alternative last steps (Algorithm 1's homogeneous system, Algorithm 3) for K+E <= kLocateAltMaxM
constexpr int kLocateAltMaxM = 13;
// ... and the one-pass locate + decode for K+E <= kLocateFuseMaxM and at most kLocateFuseMaxC classes
constexpr int kLocateFuseMaxM = 10;
constexpr int kLocateFuseMaxC = 128;
bool locate_fuse_eligible(const LocateArgs& a);
cudaError_t launch_locate_rows(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream);

void count_launch(int n = 1);

// What the launch planners need to know about the current device, asked once per device and process.
constexpr int kMaxDevices = 64;
struct DeviceInfo {
  int ordinal = -1;
  int sms = 0;          // multiprocessors
  int smem_per_sm = 0;  // shared memory per multiprocessor, bytes
};
cudaError_t current_device_info(const DeviceInfo** out);

// Raises a kernel's dynamic shared-memory limit to `bytes` on device `dev` unless an earlier call already
// did (one cache per kernel: instantiate with the kernel's own tag type).
template <typename KernelTag, typename Kernel>
cudaError_t ensure_dynamic_smem(Kernel kernel, int dev, int bytes) {
  static std::atomic<int> granted[kMaxDevices];
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (bytes <= 48 * 1024 || bytes <= granted[dev].load(std::memory_order_acquire)) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) granted[dev].store(bytes, std::memory_order_release);
  return e;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }

#ifdef __CUDACC__
// Streaming (evict-first) 128-bit and 32-bit global accesses: every payload
// byte is touched exactly once.
__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(float* p, float v) { __stcs(p, v); }

// How a payload is stored and how a thread sees it: Store = what one access moves, Vec = its fp32 lanes.
//   PayloadF32x4 / PayloadF32: fp32 elements, 16-byte / 4-byte columns
//   PayloadBf16x4 / PayloadBf16: bfloat16 elements (the upper half of a binary32), 8-byte / 2-byte columns;
//   widening is exact, narrowing rounds to nearest, ties to even (cvt.rn)
struct PayloadF32x4 {
  using Store = float4;
  using Vec = float4;
  static constexpr int kLanes = 4, kElemBytes = 4;
  static __device__ __forceinline__ Vec load(const Store* p) { return __ldcs(p); }
  static __device__ __forceinline__ void store(Store* p, Vec v) { __stcs(p, v); }
};
struct PayloadF32 {
  using Store = float;
  using Vec = float;
  static constexpr int kLanes = 1, kElemBytes = 4;
  static __device__ __forceinline__ Vec load(const Store* p) { return __ldcs(p); }
  static __device__ __forceinline__ void store(Store* p, Vec v) { __stcs(p, v); }
};
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
struct PayloadBf16x4 {
  using Store = uint2;
  using Vec = float4;
  static constexpr int kLanes = 4, kElemBytes = 2;
  static __device__ __forceinline__ Vec load(const Store* p) {
    const uint2 u = __ldcs(p);
    return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xffff0000u));
  }
  static __device__ __forceinline__ void store(Store* p, Vec v) { __stcs(p, make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w))); }
};
// eight bfloat16 elements as one 16-byte column (the encoder's choice when alignment and K allow: twice the bytes
// in flight per thread of the 8-byte path)
struct float8 {
  float4 lo, hi;
};
struct PayloadBf16x8 {
  using Store = uint4;
  using Vec = float8;
  static constexpr int kLanes = 8, kElemBytes = 2;
  static __device__ __forceinline__ Vec load(const Store* p) {
    const uint4 u = __ldcs(p);
    Vec v;
    v.lo = make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                       __uint_as_float(u.y & 0xffff0000u));
    v.hi = make_float4(__uint_as_float(u.z << 16), __uint_as_float(u.z & 0xffff0000u), __uint_as_float(u.w << 16),
                       __uint_as_float(u.w & 0xffff0000u));
    return v;
  }
  static __device__ __forceinline__ void store(Store* p, Vec v) {
    __stcs(p, make_uint4(pack_bf16x2(v.lo.x, v.lo.y), pack_bf16x2(v.lo.z, v.lo.w), pack_bf16x2(v.hi.x, v.hi.y), pack_bf16x2(v.hi.z, v.hi.w)));
  }
};
struct PayloadBf16 {
  using Store = unsigned short;
  using Vec = float;
  static constexpr int kLanes = 1, kElemBytes = 2;
  static __device__ __forceinline__ Vec load(const Store* p) { return __uint_as_float((uint32_t)__ldcs(p) << 16); }
  static __device__ __forceinline__ void store(Store* p, Vec v) { __stcs(p, (unsigned short)(pack_bf16x2(v, 0.f) & 0xffffu)); }
};

__device__ __forceinline__ uint32_t worker_bits(int W) { return W >= 32 ? 0xffffffffu : ((1u << W) - 1u); }
#endif

}  // namespace approxifer

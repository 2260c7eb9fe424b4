// C ABI of the ApproxIFER library: argument validation and dispatch.
// The declarations and their contracts are in include/approxifer.h.
#include <atomic>

#include "../../include/approxifer.h"
#include "common.cuh"

namespace approxifer {

namespace {
std::atomic<long long> g_launches{0};
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

cudaError_t current_device_info(const DeviceInfo** out) {
  static DeviceInfo info[kMaxDevices];
  static std::atomic<int> ready[kMaxDevices];
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (!ready[dev].load(std::memory_order_acquire)) {
    // (two threads may both fill the entry: they write the same values)
    DeviceInfo d;
    d.ordinal = dev;
    if ((e = cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev)) != cudaSuccess) return e;
    info[dev] = d;
    ready[dev].store(1, std::memory_order_release);
  }
  *out = &info[dev];
  return cudaSuccess;
}

namespace {

int check_kw(const approxifer_params* p) {
  if (p == nullptr) return APPROXIFER_E_NULL;
  if (p->K < 1 || p->K > APPROXIFER_MAX_K || p->W < 2 || p->W > APPROXIFER_MAX_W) return APPROXIFER_E_RANGE;
  if (p->flags & ~(APPROXIFER_SIGN_WORKER_INDEX | APPROXIFER_LOCATE_HOMOGENEOUS | APPROXIFER_ONE_PASS | APPROXIFER_TWO_LAUNCHES))
    return APPROXIFER_E_PARAM;
  return APPROXIFER_OK;
}

// [G][rows][len] with element strides gs, rs: rows must not overlap.
int check_layout(int64_t G, int64_t len, int64_t rs) {
  if (G < 0 || len < 1 || len > (int64_t(1) << 31)) return APPROXIFER_E_RANGE;
  if (rs < len) return APPROXIFER_E_RANGE;
  return APPROXIFER_OK;
}

int from_cuda(cudaError_t e) { return e == cudaSuccess ? APPROXIFER_OK : APPROXIFER_E_CUDA; }

}  // namespace
}  // namespace approxifer

using namespace approxifer;

namespace {
int decode_checked(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                   int64_t yt_rstride, const uint32_t* mask, float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                   int32_t* n_used, uint32_t* status, const DecodeTuning& tune, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, C, yt_rstride))) return rc;
  if ((rc = check_layout(G, C, yh_rstride))) return rc;
  if (yt_gstride < 0 || yh_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (Yt == nullptr || Yhat == nullptr || mask == nullptr) return APPROXIFER_E_NULL;
  DecodeArgs a{Yt,         mask,       Yhat,       n_used, status, yt_gstride, yt_rstride,
               yh_gstride, yh_rstride, G,          C,      params->K, params->W, params->flags, tune};
  return from_cuda(launch_decode(a, static_cast<cudaStream_t>(cuda_stream)));
}

int locate_checked(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                   int64_t yt_rstride, const uint32_t* mask, int32_t* adv, uint32_t* trusted_mask, uint32_t* status,
                   int force_warp_kernel, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if (params->E < 0) return APPROXIFER_E_RANGE;
  if (params->E < 1 || 2 * (params->K + params->E) > params->W) return APPROXIFER_E_PARAM;
  if ((params->flags & APPROXIFER_LOCATE_HOMOGENEOUS) && params->K + params->E > kLocateAltMaxM) return APPROXIFER_E_PARAM;
  if ((rc = check_layout(G, C, yt_rstride))) return rc;
  if (yt_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (Yt == nullptr || mask == nullptr || adv == nullptr || trusted_mask == nullptr) return APPROXIFER_E_NULL;
  LocateArgs a{Yt, mask, adv, trusted_mask, status, yt_gstride, yt_rstride, G, C, params->K, params->W, params->E, params->flags};
  a.force_warp_kernel = force_warp_kernel;
  return from_cuda(launch_locate(a, static_cast<cudaStream_t>(cuda_stream)));
}
}  // namespace

extern "C" {


int approxifer_encode(const approxifer_params* params, int64_t G, int64_t D, const float* X, int64_t x_gstride,
                      int64_t x_rstride, float* Xt, int64_t xt_gstride, int64_t xt_rstride, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, D, x_rstride))) return rc;
  if ((rc = check_layout(G, D, xt_rstride))) return rc;
  if (x_gstride < 0 || xt_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (X == nullptr || Xt == nullptr) return APPROXIFER_E_NULL;
  EncodeArgs a{X, Xt, x_gstride, x_rstride, xt_gstride, xt_rstride, G, D, params->K, params->W};
  return from_cuda(launch_encode(a, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_decode(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                      int64_t yt_rstride, const uint32_t* mask, float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                      int32_t* n_used, uint32_t* status, void* cuda_stream) {
  return decode_checked(params, G, C, Yt, yt_gstride, yt_rstride, mask, Yhat, yh_gstride, yh_rstride, n_used, status,
                        DecodeTuning{}, cuda_stream);
}

int approxifer_encode_bf16(const approxifer_params* params, int64_t G, int64_t D, const uint16_t* X, int64_t x_gstride,
                           int64_t x_rstride, uint16_t* Xt, int64_t xt_gstride, int64_t xt_rstride, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, D, x_rstride))) return rc;
  if ((rc = check_layout(G, D, xt_rstride))) return rc;
  if (x_gstride < 0 || xt_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (X == nullptr || Xt == nullptr) return APPROXIFER_E_NULL;
  EncodeArgs a{reinterpret_cast<const float*>(X), reinterpret_cast<float*>(Xt), x_gstride, x_rstride, xt_gstride, xt_rstride,
               G, D, params->K, params->W, 1};
  return from_cuda(launch_encode(a, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_decode_bf16(const approxifer_params* params, int64_t G, int64_t C, const uint16_t* Yt, int64_t yt_gstride,
                           int64_t yt_rstride, const uint32_t* mask, uint16_t* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                           int32_t* n_used, uint32_t* status, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, C, yt_rstride))) return rc;
  if ((rc = check_layout(G, C, yh_rstride))) return rc;
  if (yt_gstride < 0 || yh_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (Yt == nullptr || Yhat == nullptr || mask == nullptr) return APPROXIFER_E_NULL;
  DecodeArgs a{reinterpret_cast<const float*>(Yt), mask, reinterpret_cast<float*>(Yhat), n_used, status, yt_gstride, yt_rstride,
               yh_gstride, yh_rstride, G, C, params->K, params->W, params->flags, DecodeTuning{}, 1};
  return from_cuda(launch_decode(a, static_cast<cudaStream_t>(cuda_stream)));
}

namespace {
// Element offsets of W row pointers from the first one (same address space: device memory of this GPU or of a
// peer); false if a pointer is missing or not a whole number of elements away.
bool row_offsets(const float* const* rows, int W, RowOffsets* out) {
  if (rows == nullptr) return false;
  for (int i = 0; i < W; ++i) {
    if (rows[i] == nullptr) return false;
    const intptr_t diff = reinterpret_cast<intptr_t>(rows[i]) - reinterpret_cast<intptr_t>(rows[0]);
    if (diff % (intptr_t)sizeof(float) != 0) return false;
    out->off[i] = (int64_t)(diff / (intptr_t)sizeof(float));
  }
  for (int i = W; i < kMaxW; ++i) out->off[i] = 0;
  out->on = 1;
  return true;
}
}  // namespace

int approxifer_encode_scatter(const approxifer_params* params, int64_t G, int64_t D, const float* X, int64_t x_gstride,
                              int64_t x_rstride, float* const* Xt_rows, int64_t xt_gstride, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, D, x_rstride))) return rc;
  if (x_gstride < 0 || xt_gstride < D) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (X == nullptr || Xt_rows == nullptr) return APPROXIFER_E_NULL;
  EncodeArgs a{X, Xt_rows[0], x_gstride, x_rstride, xt_gstride, D, G, D, params->K, params->W};
  if (!row_offsets(Xt_rows, params->W, &a.rows)) return APPROXIFER_E_NULL;
  return from_cuda(launch_encode(a, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_decode_gather(const approxifer_params* params, int64_t G, int64_t C, const float* const* Yt_rows,
                             int64_t yt_gstride, const uint32_t* mask, float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                             int32_t* n_used, uint32_t* status, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, C, yh_rstride))) return rc;
  if (G < 0 || C < 1 || yt_gstride < C || yh_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (Yt_rows == nullptr || Yhat == nullptr || mask == nullptr) return APPROXIFER_E_NULL;
  DecodeArgs a{Yt_rows[0], mask, Yhat, n_used, status, yt_gstride, C, yh_gstride, yh_rstride, G, C, params->K, params->W, params->flags};
  if (!row_offsets(Yt_rows, params->W, &a.rows)) return APPROXIFER_E_NULL;
  return from_cuda(launch_decode(a, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_locate_gather(const approxifer_params* params, int64_t G, int64_t C, const float* const* Yt_rows,
                             int64_t yt_gstride, const uint32_t* mask, int32_t* adv, uint32_t* trusted_mask, uint32_t* status,
                             void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if (params->E < 0) return APPROXIFER_E_RANGE;
  if (params->E < 1 || 2 * (params->K + params->E) > params->W) return APPROXIFER_E_PARAM;
  if ((params->flags & APPROXIFER_LOCATE_HOMOGENEOUS) && params->K + params->E > kLocateAltMaxM) return APPROXIFER_E_PARAM;
  if (G < 0 || C < 1 || C > (int64_t(1) << 31) || yt_gstride < C) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (Yt_rows == nullptr || mask == nullptr || adv == nullptr || trusted_mask == nullptr) return APPROXIFER_E_NULL;
  LocateArgs a{Yt_rows[0], mask, adv, trusted_mask, status, yt_gstride, C, G, C, params->K, params->W, params->E, params->flags};
  if (!row_offsets(Yt_rows, params->W, &a.rows)) return APPROXIFER_E_NULL;
  return from_cuda(launch_locate(a, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_debug_decode(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                            int64_t yt_rstride, const uint32_t* mask, float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                            int32_t* n_used, uint32_t* status, const approxifer_decode_tuning* tuning, void* cuda_stream) {
  DecodeTuning t{};
  if (tuning != nullptr) {
    const int cols = tuning->cols, split = tuning->split;
    if (tuning->kernel < 0 || tuning->kernel > 4 || tuning->stages < 0 || tuning->stages == 1 || tuning->ctas_per_sm < 0 ||
        cols < 0 || (tuning->kernel != 4 && cols != 0 && cols != 16 && cols != 32 && cols != 64 && cols != 128 && cols != 256) ||
        (split != 0 && split != 1 && split != 2 && split != 4))
      return APPROXIFER_E_PARAM;
    if (tuning->wait_limit != 0 && tuning->wait_limit < 65536u) return APPROXIFER_E_PARAM;  // started copies need time to land
    if (tuning->withhold_group_plus1 < 0) return APPROXIFER_E_PARAM;
    t.kernel = tuning->kernel, t.stages = tuning->stages, t.ctas_per_sm = tuning->ctas_per_sm, t.cols = cols, t.split = split;
    t.wait_limit = tuning->wait_limit;
    t.withhold_group = tuning->withhold_group_plus1 - 1;
  }
  return decode_checked(params, G, C, Yt, yt_gstride, yt_rstride, mask, Yhat, yh_gstride, yh_rstride, n_used, status, t,
                        cuda_stream);
}

int approxifer_locate(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                      int64_t yt_rstride, const uint32_t* mask, int32_t* adv, uint32_t* trusted_mask, uint32_t* status,
                      void* cuda_stream) {
  return locate_checked(params, G, C, Yt, yt_gstride, yt_rstride, mask, adv, trusted_mask, status, 0, cuda_stream);
}

int approxifer_debug_locate(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                            int64_t yt_rstride, const uint32_t* mask, int32_t* adv, uint32_t* trusted_mask, uint32_t* status,
                            int force_warp_kernel, void* cuda_stream) {
  return locate_checked(params, G, C, Yt, yt_gstride, yt_rstride, mask, adv, trusted_mask, status, force_warp_kernel != 0,
                        cuda_stream);
}

int approxifer_decode_rational(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                               int64_t yt_rstride, const uint32_t* mask, float* Yhat, int64_t yh_gstride, int64_t yh_rstride,
                               uint32_t* status, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if (params->E < 0) return APPROXIFER_E_RANGE;
  const int m = params->K + params->E;
  if (m < 2 || m > kLocateAltMaxM || 2 * m > params->W) return APPROXIFER_E_PARAM;
  if ((rc = check_layout(G, C, yt_rstride))) return rc;
  if ((rc = check_layout(G, C, yh_rstride))) return rc;
  if (yt_gstride < 0 || yh_gstride < 0) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (Yt == nullptr || mask == nullptr || Yhat == nullptr) return APPROXIFER_E_NULL;
  LocateArgs a{Yt, mask, nullptr, nullptr, status, yt_gstride, yt_rstride, G, C, params->K, params->W, params->E, 0u,
               Yhat, yh_gstride, yh_rstride};
  return from_cuda(launch_locate(a, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_locate_decode(const approxifer_params* params, int64_t G, int64_t C, const float* Yt, int64_t yt_gstride,
                             int64_t yt_rstride, const uint32_t* mask, int32_t* adv, uint32_t* trusted_mask, float* Yhat,
                             int64_t yh_gstride, int64_t yh_rstride, int32_t* n_used, uint32_t* locate_status,
                             uint32_t* decode_status, void* cuda_stream) {
  // validate both steps before anything is enqueued
  if (G > 0 && Yhat == nullptr) return APPROXIFER_E_NULL;
  int rc = check_kw(params);
  if (rc) return rc;
  if ((rc = check_layout(G, C, yh_rstride))) return rc;
  if (yh_gstride < 0) return APPROXIFER_E_RANGE;
  // one pass where the thread-per-class locator can carry the decoding as its tail (all classes of a group in one
  // CTA, a small factor), else the two kernels back to back; the results are bit-identical
  if (params->E >= 1 && 2 * (params->K + params->E) <= params->W && yt_gstride >= 0 && G > 0 && Yt != nullptr && mask != nullptr &&
      adv != nullptr && trusted_mask != nullptr && check_layout(G, C, yt_rstride) == APPROXIFER_OK) {
    LocateArgs a{Yt, mask, adv, trusted_mask, locate_status, yt_gstride, yt_rstride, G, C, params->K, params->W, params->E, params->flags};
    const bool want = (params->flags & APPROXIFER_TWO_LAUNCHES) ? false
                      : (params->flags & APPROXIFER_ONE_PASS)   ? true
                                                                : G <= APPROXIFER_ONE_PASS_MAX_GROUPS;
    if (want && locate_fuse_eligible(a)) {
      a.Yh = Yhat, a.o_gs = yh_gstride, a.o_rs = yh_rstride;
      a.fuse_decode = 1, a.n_used = n_used, a.decode_status = decode_status;
      return from_cuda(launch_locate(a, static_cast<cudaStream_t>(cuda_stream)));
    }
  }
  rc = approxifer_locate(params, G, C, Yt, yt_gstride, yt_rstride, mask, adv, trusted_mask, locate_status, cuda_stream);
  if (rc) return rc;
  return approxifer_decode(params, G, C, Yt, yt_gstride, yt_rstride, trusted_mask, Yhat, yh_gstride, yh_rstride, n_used,
                           decode_status, cuda_stream);
}

int approxifer_debug_weights(const approxifer_params* params, uint32_t mask, int which, float* w, int32_t* idx,
                             int32_t* n, void* cuda_stream) {
  int rc = check_kw(params);
  if (rc) return rc;
  if (which != 0 && which != 1) return APPROXIFER_E_PARAM;
  if (w == nullptr || (which == 1 && (idx == nullptr || n == nullptr))) return APPROXIFER_E_NULL;
  return from_cuda(launch_debug_weights(params->K, params->W, params->flags, mask, which, w, idx, n,
                                        static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_debug_pack_rotation(int32_t K, int32_t W, int64_t C, int32_t mode, int32_t* groups_per_item,
                                   uint32_t* rotated_groups, int32_t* passes_plain, int32_t* passes_chosen) {
  if (groups_per_item == nullptr || rotated_groups == nullptr || passes_plain == nullptr || passes_chosen == nullptr)
    return APPROXIFER_E_PARAM;
  if (K < 1 || W < 2 || K > W || W > kMaxW || C < 1 || mode < 0 || mode > 2) return APPROXIFER_E_PARAM;
  int gw = 0, plain = 0, chosen = 0;
  uint32_t rot = 0;
  if (!pack_rotation_info(K, W, C, mode, &gw, &rot, &plain, &chosen)) gw = 0, rot = 0, plain = 0, chosen = 0;
  *groups_per_item = gw, *rotated_groups = rot, *passes_plain = plain, *passes_chosen = chosen;
  return APPROXIFER_OK;
}

int approxifer_debug_fma_peak(int iters, int blocks, float* sink, void* cuda_stream) {
  if (iters < 1 || blocks < 1 || blocks > (1 << 20)) return APPROXIFER_E_RANGE;
  if (sink == nullptr) return APPROXIFER_E_NULL;
  return from_cuda(launch_fma_peak(iters, blocks, sink, static_cast<cudaStream_t>(cuda_stream)));
}

int approxifer_reset_device_wait_timeouts(void) {
  return (reset_decode_wait_timeouts() == cudaSuccess && reset_pack_wait_timeouts() == cudaSuccess) ? APPROXIFER_OK : APPROXIFER_E_CUDA;
}

int64_t approxifer_device_wait_timeouts(void) {
  unsigned int n = 0, m = 0;
  if (read_decode_wait_timeouts(&n) != cudaSuccess || read_pack_wait_timeouts(&m) != cudaSuccess) return -1;
  return (int64_t)n + (int64_t)m;
}

const char* approxifer_strerror(int code) {
  switch (code) {
    case APPROXIFER_OK: return "ok";
    case APPROXIFER_E_NULL: return "a required pointer is NULL";
    case APPROXIFER_E_RANGE: return "argument out of range (K in 1..32, W in 2..32, E >= 0, G >= 0, 1 <= D <= 2^31, row stride >= row length)";
    case APPROXIFER_E_PARAM: return "inconsistent parameters (locate needs E >= 1 and 2(K+E) <= W; unknown flag bits)";
    case APPROXIFER_E_CUDA: return "the CUDA runtime reported an error at kernel launch";
    case APPROXIFER_E_WORKSPACE: return "the device workspace is too small to stage a single group";
    case APPROXIFER_E_TOO_LARGE: return "the batch is larger than the built-in staging area (APPROXIFER_STATIC_WORKSPACE_BYTES); split it or use approxifer_encode_host";
    default: return "unknown error code";
  }
}

int approxifer_version(void) { return APPROXIFER_VERSION; }

int64_t approxifer_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

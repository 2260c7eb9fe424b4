// approxifer_encode_host_static: the host-buffer encoder for callers that cannot obtain device memory.
//
// approxifer_encode_host needs a device workspace from its caller.  Some callers have none to give and no
// way to get one: an encoder front-end that runs beside a model server which reserved the whole device
// memory pool at start-up, or a request handler that is forbidden to call cudaMalloc because the
// allocation call takes a device-wide lock and synchronises, stalling the other streams of the process.
// For them the staging area is this file's fixed array in device memory.  It is part of the library's
// image: every GPU on which the library is used holds these bytes from the first use until the process
// exits, whether or not this entry point is ever called.
//
// The staging area keeps whatever the previous call left in it.  Nothing in it has to start at zero: the
// host-to-device copy writes every query element the kernel reads, and the kernel writes every element of the
// coded-query part that the device-to-host copy then reads.  (When D is not a multiple of 4 the rows are
// padded to whole 16-byte columns; the pad elements are neither written nor read by anyone.)
#include <atomic>
#include <mutex>

#include "../../include/approxifer.h"
#include "common.cuh"

namespace approxifer {
namespace {

static __device__ __align__(256) unsigned char g_static_workspace[APPROXIFER_STATIC_WORKSPACE_BYTES];

std::mutex g_setup_mutex;
unsigned char* g_workspace_ptr[kMaxDevices] = {};  // device address of g_static_workspace, per device

// In host code `g_static_workspace` is only a handle for the runtime, not an address a kernel or a copy
// could use; the real device address is asked for once per device, with that device current.
cudaError_t static_workspace(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_workspace_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_workspace);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_workspace_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_workspace_ptr[dev];
  return cudaSuccess;
}

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace
}  // namespace approxifer

using namespace approxifer;

extern "C" int approxifer_encode_host_static(const approxifer_params* params, int64_t G, int64_t D, const float* hX,
                                             float* hXt, void* cuda_stream) {
  if (params == nullptr) return APPROXIFER_E_NULL;
  if (params->K < 1 || params->K > APPROXIFER_MAX_K || params->W < 2 || params->W > APPROXIFER_MAX_W) return APPROXIFER_E_RANGE;
  if (params->flags & ~(APPROXIFER_SIGN_WORKER_INDEX | APPROXIFER_LOCATE_HOMOGENEOUS | APPROXIFER_ONE_PASS | APPROXIFER_TWO_LAUNCHES)) return APPROXIFER_E_PARAM;
  if (G < 0 || D < 1 || D > (int64_t(1) << 31)) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (hX == nullptr || hXt == nullptr) return APPROXIFER_E_NULL;
  const int K = params->K, W = params->W;
  // staging layout: [G][K][Dp] queries, then (256-byte aligned) [G][W][Dp] coded queries; Dp = D rounded up to
  // a multiple of 4 so that every row starts on a 16-byte boundary
  const int64_t Dp = (D + 3) & ~int64_t(3);
  // bound G by a division first, so that none of the products below can wrap (Dp <= 2^31 + 3, K + W <= 64)
  if ((unsigned long long)G > APPROXIFER_STATIC_WORKSPACE_BYTES / (4ull * (unsigned long long)Dp * (unsigned long long)(K + W)))
    return APPROXIFER_E_TOO_LARGE;
  const unsigned long long in_bytes = (unsigned long long)G * K * Dp * 4, out_bytes = (unsigned long long)G * W * Dp * 4;
  if (align256((size_t)in_bytes) + out_bytes > APPROXIFER_STATIC_WORKSPACE_BYTES) return APPROXIFER_E_TOO_LARGE;

  unsigned char* base = nullptr;
  if (static_workspace(&base) != cudaSuccess) return APPROXIFER_E_CUDA;
  float* dX = reinterpret_cast<float*>(base);
  float* dXt = reinterpret_cast<float*>(base + align256((size_t)in_bytes));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (Dp == D)
    e = cudaMemcpyAsync(dX, hX, (size_t)in_bytes, cudaMemcpyHostToDevice, st);
  else
    e = cudaMemcpy2DAsync(dX, (size_t)Dp * 4, hX, (size_t)D * 4, (size_t)D * 4, (size_t)G * K, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return APPROXIFER_E_CUDA;
  EncodeArgs a{dX, dXt, (int64_t)K * Dp, Dp, (int64_t)W * Dp, Dp, G, D, K, W};
  if (launch_encode(a, st) != cudaSuccess) return APPROXIFER_E_CUDA;
  if (Dp == D)
    e = cudaMemcpyAsync(hXt, dXt, (size_t)out_bytes, cudaMemcpyDeviceToHost, st);
  else
    e = cudaMemcpy2DAsync(hXt, (size_t)D * 4, dXt, (size_t)Dp * 4, (size_t)D * 4, (size_t)G * W, cudaMemcpyDeviceToHost, st);
  return e == cudaSuccess ? APPROXIFER_OK : APPROXIFER_E_CUDA;
}

// Host-buffer entry points: the same encode / decode / locate kernels, fed from and drained to HOST memory
// through a caller-provided device workspace.  The batch is cut into chunks of whole groups; chunk c runs
// on stream c % n_streams as  H2D copy -> kernel -> D2H copy,  so with two or more streams the two copy
// directions and the kernels of neighbouring chunks overlap.  Each stream owns one slice of the workspace,
// and work within a stream is ordered, which is what makes the reuse of a slice by the stream's next chunk
// safe.  Nothing is allocated and nothing is synchronised here.
#include "../../include/approxifer.h"
#include "common.cuh"

namespace approxifer {
namespace {

constexpr int kMaxStreams = 8;

struct ChunkPlan {
  int n_streams;
  int64_t groups_per_chunk;
  size_t slice_bytes;
};

// bytes_per_group: device bytes one group needs in a slice (inputs + outputs, each part 256-byte aligned
// at the slice level by the callers' layout helpers).
int plan_chunks(int64_t G, size_t bytes_per_group, size_t fixed_per_slice, size_t workspace_bytes, int n_streams,
                ChunkPlan* plan) {
  if (n_streams < 1 || n_streams > kMaxStreams) return APPROXIFER_E_RANGE;
  // no more slices than chunks are useful; each slice must hold at least one group
  size_t slice = (workspace_bytes / (size_t)n_streams) & ~(size_t)255;
  while (n_streams > 1 && slice < fixed_per_slice + bytes_per_group) {
    --n_streams;
    slice = (workspace_bytes / (size_t)n_streams) & ~(size_t)255;
  }
  if (slice < fixed_per_slice + bytes_per_group) return APPROXIFER_E_WORKSPACE;
  int64_t per = (int64_t)((slice - fixed_per_slice) / bytes_per_group);
  // balance: do not leave some streams idle when the batch would fit in fewer, larger chunks
  const int64_t want = (G + n_streams - 1) / n_streams;
  if (per > want) per = want > 0 ? want : 1;
  plan->n_streams = n_streams;
  plan->groups_per_chunk = per;
  plan->slice_bytes = slice;
  return APPROXIFER_OK;
}

inline size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace
}  // namespace approxifer

using namespace approxifer;

extern "C" {

int approxifer_encode_host(const approxifer_params* params, int64_t G, int64_t D, const float* hX, float* hXt,
                           void* workspace, size_t workspace_bytes, void* const* cuda_streams, int n_streams) {
  if (params == nullptr) return APPROXIFER_E_NULL;
  if (params->K < 1 || params->K > APPROXIFER_MAX_K || params->W < 2 || params->W > APPROXIFER_MAX_W) return APPROXIFER_E_RANGE;
  if (G < 0 || D < 1 || D > (int64_t(1) << 31)) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (hX == nullptr || hXt == nullptr || workspace == nullptr || cuda_streams == nullptr) return APPROXIFER_E_NULL;
  const int K = params->K, W = params->W;
  // slice layout: [chunk][K][D] queries, then [chunk][W][D] coded queries; D is padded so rows stay 16-byte aligned
  const int64_t Dp = (D + 3) & ~int64_t(3);
  const size_t in_g = (size_t)K * Dp * 4, out_g = (size_t)W * Dp * 4;
  ChunkPlan plan;
  int rc = plan_chunks(G, in_g + out_g, 512, workspace_bytes, n_streams, &plan);
  if (rc) return rc;
  int64_t g0 = 0;
  for (int64_t c = 0; g0 < G; ++c, g0 += plan.groups_per_chunk) {
    const int64_t ng = (G - g0 < plan.groups_per_chunk) ? G - g0 : plan.groups_per_chunk;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_streams[c % plan.n_streams]);
    char* slice = static_cast<char*>(workspace) + (size_t)(c % plan.n_streams) * plan.slice_bytes;
    float* dX = reinterpret_cast<float*>(slice);
    float* dXt = reinterpret_cast<float*>(slice + align256((size_t)ng * in_g));
    cudaError_t e;
    if (Dp == D) {
      e = cudaMemcpyAsync(dX, hX + g0 * K * D, (size_t)ng * K * D * 4, cudaMemcpyHostToDevice, st);
    } else {
      e = cudaMemcpy2DAsync(dX, (size_t)Dp * 4, hX + g0 * K * D, (size_t)D * 4, (size_t)D * 4, (size_t)ng * K,
                            cudaMemcpyHostToDevice, st);
    }
    if (e != cudaSuccess) return APPROXIFER_E_CUDA;
    EncodeArgs a{dX, dXt, (int64_t)K * Dp, Dp, (int64_t)W * Dp, Dp, ng, D, K, W};
    if (launch_encode(a, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (Dp == D) {
      e = cudaMemcpyAsync(hXt + g0 * W * D, dXt, (size_t)ng * W * D * 4, cudaMemcpyDeviceToHost, st);
    } else {
      e = cudaMemcpy2DAsync(hXt + g0 * W * D, (size_t)D * 4, dXt, (size_t)Dp * 4, (size_t)D * 4, (size_t)ng * W,
                            cudaMemcpyDeviceToHost, st);
    }
    if (e != cudaSuccess) return APPROXIFER_E_CUDA;
  }
  return APPROXIFER_OK;
}

int approxifer_decode_host(const approxifer_params* params, int64_t G, int64_t C, const float* hYt, const uint32_t* hmask,
                           float* hYhat, int32_t* hn_used, uint32_t* hstatus, void* workspace, size_t workspace_bytes,
                           void* const* cuda_streams, int n_streams) {
  if (params == nullptr) return APPROXIFER_E_NULL;
  if (params->K < 1 || params->K > APPROXIFER_MAX_K || params->W < 2 || params->W > APPROXIFER_MAX_W) return APPROXIFER_E_RANGE;
  if (params->flags & ~(APPROXIFER_SIGN_WORKER_INDEX | APPROXIFER_LOCATE_HOMOGENEOUS | APPROXIFER_ONE_PASS | APPROXIFER_TWO_LAUNCHES)) return APPROXIFER_E_PARAM;
  if (G < 0 || C < 1 || C > (int64_t(1) << 31)) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (hYt == nullptr || hmask == nullptr || hYhat == nullptr || workspace == nullptr || cuda_streams == nullptr)
    return APPROXIFER_E_NULL;
  const int K = params->K, W = params->W;
  // staged rows are padded to whole float4s for the 128-bit kernels; short rows (C <= 32) stay dense, which is
  // what the short-payload decoder takes and turns both copies into plain contiguous ones
  const int64_t Cp = (C <= 32) ? C : ((C + 3) & ~int64_t(3));
  const size_t in_g = (size_t)W * Cp * 4, out_g = (size_t)K * Cp * 4, small_g = 12;  // mask, n_used, status
  ChunkPlan plan;
  int rc = plan_chunks(G, in_g + out_g + small_g, 1280, workspace_bytes, n_streams, &plan);
  if (rc) return rc;
  int64_t g0 = 0;
  for (int64_t c = 0; g0 < G; ++c, g0 += plan.groups_per_chunk) {
    const int64_t ng = (G - g0 < plan.groups_per_chunk) ? G - g0 : plan.groups_per_chunk;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_streams[c % plan.n_streams]);
    char* slice = static_cast<char*>(workspace) + (size_t)(c % plan.n_streams) * plan.slice_bytes;
    size_t off = 0;
    float* dYt = reinterpret_cast<float*>(slice + off);
    off += align256((size_t)ng * in_g);
    float* dYh = reinterpret_cast<float*>(slice + off);
    off += align256((size_t)ng * out_g);
    uint32_t* dmask = reinterpret_cast<uint32_t*>(slice + off);
    off += align256((size_t)ng * 4);
    int32_t* dn = reinterpret_cast<int32_t*>(slice + off);
    off += align256((size_t)ng * 4);
    uint32_t* dst = reinterpret_cast<uint32_t*>(slice + off);
    cudaError_t e;
    if (Cp == C)
      e = cudaMemcpyAsync(dYt, hYt + g0 * W * C, (size_t)ng * W * C * 4, cudaMemcpyHostToDevice, st);
    else
      e = cudaMemcpy2DAsync(dYt, (size_t)Cp * 4, hYt + g0 * W * C, (size_t)C * 4, (size_t)C * 4, (size_t)ng * W,
                            cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return APPROXIFER_E_CUDA;
    if (cudaMemcpyAsync(dmask, hmask + g0, (size_t)ng * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    DecodeArgs a{dYt, dmask, dYh, dn, dst, (int64_t)W * Cp, Cp, (int64_t)K * Cp, Cp, ng, C, K, W, params->flags};
    if (launch_decode(a, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (Cp == C)
      e = cudaMemcpyAsync(hYhat + g0 * K * C, dYh, (size_t)ng * K * C * 4, cudaMemcpyDeviceToHost, st);
    else
      e = cudaMemcpy2DAsync(hYhat + g0 * K * C, (size_t)C * 4, dYh, (size_t)Cp * 4, (size_t)C * 4, (size_t)ng * K,
                            cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return APPROXIFER_E_CUDA;
    if (hn_used && cudaMemcpyAsync(hn_used + g0, dn, (size_t)ng * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (hstatus && cudaMemcpyAsync(hstatus + g0, dst, (size_t)ng * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return APPROXIFER_E_CUDA;
  }
  return APPROXIFER_OK;
}

int approxifer_locate_host(const approxifer_params* params, int64_t G, int64_t C, const float* hYt, const uint32_t* hmask,
                           int32_t* hadv, uint32_t* htrusted, uint32_t* hstatus, void* workspace, size_t workspace_bytes,
                           void* const* cuda_streams, int n_streams) {
  if (params == nullptr) return APPROXIFER_E_NULL;
  if (params->K < 1 || params->K > APPROXIFER_MAX_K || params->W < 2 || params->W > APPROXIFER_MAX_W || params->E < 0)
    return APPROXIFER_E_RANGE;
  if (params->E < 1 || 2 * (params->K + params->E) > params->W) return APPROXIFER_E_PARAM;
  if (params->flags & ~(APPROXIFER_SIGN_WORKER_INDEX | APPROXIFER_LOCATE_HOMOGENEOUS | APPROXIFER_ONE_PASS | APPROXIFER_TWO_LAUNCHES)) return APPROXIFER_E_PARAM;
  if ((params->flags & APPROXIFER_LOCATE_HOMOGENEOUS) && params->K + params->E > kLocateAltMaxM) return APPROXIFER_E_PARAM;
  if (G < 0 || C < 1 || C > (int64_t(1) << 31)) return APPROXIFER_E_RANGE;
  if (G == 0) return APPROXIFER_OK;
  if (hYt == nullptr || hmask == nullptr || hadv == nullptr || htrusted == nullptr || workspace == nullptr ||
      cuda_streams == nullptr)
    return APPROXIFER_E_NULL;
  const int K = params->K, W = params->W, E = params->E;
  const size_t in_g = (size_t)W * C * 4, small_g = 12 + (size_t)E * 4;
  ChunkPlan plan;
  int rc = plan_chunks(G, in_g + small_g, 1280, workspace_bytes, n_streams, &plan);
  if (rc) return rc;
  int64_t g0 = 0;
  for (int64_t c = 0; g0 < G; ++c, g0 += plan.groups_per_chunk) {
    const int64_t ng = (G - g0 < plan.groups_per_chunk) ? G - g0 : plan.groups_per_chunk;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_streams[c % plan.n_streams]);
    char* slice = static_cast<char*>(workspace) + (size_t)(c % plan.n_streams) * plan.slice_bytes;
    size_t off = 0;
    float* dYt = reinterpret_cast<float*>(slice + off);
    off += align256((size_t)ng * in_g);
    uint32_t* dmask = reinterpret_cast<uint32_t*>(slice + off);
    off += align256((size_t)ng * 4);
    int32_t* dadv = reinterpret_cast<int32_t*>(slice + off);
    off += align256((size_t)ng * E * 4);
    uint32_t* dtr = reinterpret_cast<uint32_t*>(slice + off);
    off += align256((size_t)ng * 4);
    uint32_t* dst = reinterpret_cast<uint32_t*>(slice + off);
    if (cudaMemcpyAsync(dYt, hYt + g0 * W * C, (size_t)ng * W * C * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (cudaMemcpyAsync(dmask, hmask + g0, (size_t)ng * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    LocateArgs a{dYt, dmask, dadv, dtr, dst, (int64_t)W * C, C, ng, C, K, W, E, params->flags};
    if (launch_locate(a, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (cudaMemcpyAsync(hadv + g0 * E, dadv, (size_t)ng * E * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (cudaMemcpyAsync(htrusted + g0, dtr, (size_t)ng * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return APPROXIFER_E_CUDA;
    if (hstatus && cudaMemcpyAsync(hstatus + g0, dst, (size_t)ng * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return APPROXIFER_E_CUDA;
  }
  return APPROXIFER_OK;
}

}  // extern "C"

// Thread-per-class locator: dispatch on the number of workers to the translation units that hold the kernels
// (locate_rows_n8.cu .. locate_rows_n32.cu, all generated from locate_rows_impl.cuh).
#include "common.cuh"

namespace approxifer {

cudaError_t launch_locate_rows_8(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream);
cudaError_t launch_locate_rows_16(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream);
cudaError_t launch_locate_rows_24(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream);
cudaError_t launch_locate_rows_32(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream);

cudaError_t launch_locate_rows(const LocateArgs& a, const LocateTables& tab, cudaStream_t stream) {
  if (a.W <= 8) return launch_locate_rows_8(a, tab, stream);
  if (a.W <= 16) return launch_locate_rows_16(a, tab, stream);
  if (a.W <= 24) return launch_locate_rows_24(a, tab, stream);
  return launch_locate_rows_32(a, tab, stream);
}

}  // namespace approxifer

#include "kernels_row.cuh"

namespace dnnf {
int launch_row_e(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 408011: launch_one<4, 8, 1, 1, true>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

#include "kernels_row.cuh"

namespace dnnf {
int launch_row_c(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 404011: launch_one<4, 4, 1, 1, true>(L, st); break;
    case 116011: launch_one<1, 16, 1, 1, false>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

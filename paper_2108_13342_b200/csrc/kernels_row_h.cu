#include "kernels_row.cuh"

namespace dnnf {
int launch_row_h(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 401041: launch_one<4, 1, 4, 1, true>(L, st); break;
    case 402041: launch_one<4, 2, 4, 1, true>(L, st); break;
    case 401081: launch_one<4, 1, 8, 1, true>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

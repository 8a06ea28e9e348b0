#include "kernels_row.cuh"

namespace dnnf {
int launch_row_a(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 401014: launch_one<4, 1, 1, 4, true>(L, st); break;
    case 401012: launch_one<4, 1, 1, 2, true>(L, st); break;
    case 401011: launch_one<4, 1, 1, 1, true>(L, st); break;
    case 101014: launch_one<1, 1, 1, 4, false>(L, st); break;
    case 101011: launch_one<1, 1, 1, 1, false>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

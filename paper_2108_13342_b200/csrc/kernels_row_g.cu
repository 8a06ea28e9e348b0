#include "kernels_row.cuh"

namespace dnnf {
int launch_row_g(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 401021: launch_one<4, 1, 2, 1, true>(L, st); break;
    case 402021: launch_one<4, 2, 2, 1, true>(L, st); break;
    case 403021: launch_one<4, 3, 2, 1, true>(L, st); break;
    case 404021: launch_one<4, 4, 2, 1, true>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

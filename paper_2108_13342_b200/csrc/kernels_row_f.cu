#include "kernels_row.cuh"

namespace dnnf {
int launch_row_f(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 402081: launch_one<4, 2, 8, 1, false>(L, st); break;
    case 404081: launch_one<4, 4, 8, 1, false>(L, st); break;
    case 408081: launch_one<4, 8, 8, 1, false>(L, st); break;
    case 108081: launch_one<1, 8, 8, 1, false>(L, st); break;
    case 132081: launch_one<1, 32, 8, 1, false>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

#include "kernels_row.cuh"

namespace dnnf {
int launch_row_b(const Launch& L, cudaStream_t st) {
  switch (L.variant) {
    case 402012: launch_one<4, 2, 1, 2, true>(L, st); break;
    case 402011: launch_one<4, 2, 1, 1, true>(L, st); break;
    case 104011: launch_one<1, 4, 1, 1, false>(L, st); break;
    default: return 2;
  }
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
}  // namespace dnnf

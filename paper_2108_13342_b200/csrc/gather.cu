// Gather along axis 0 (Table 2, One-to-Many): y[r, :] = table[indices[r], :] for every element r of the index tensor.
//
// A pure data movement bound by HBM: the result is written once, the rows it names are read once each time they are
// named.  One warp copies one row, 128 bits per lane where the row length and the addresses allow; an index outside
// [0, V) is clamped to the nearest row, so that no index value can make the kernel read outside the table.
#include <cuda_runtime.h>

#include <set>

#include "ir.h"
#include "launch_util.h"
#include "lower.h"

namespace dnnf {

struct GatherParams {
  const void* table;
  const float* indices;
  void* out;
  int32_t V, D, rows;
  int32_t elt;             // bytes per element (4 or 2)
  int32_t vec;             // 16-byte pieces per row when rows are 16-byte aligned, else 0
};

__global__ void __launch_bounds__(256) gather_rows_kernel(const __grid_constant__ GatherParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (r >= p.rows) return;
  int i = __float2int_rn(__ldg(p.indices + r));
  i = min(max(i, 0), p.V - 1);
  const size_t row_bytes = (size_t)p.D * p.elt;
  const char* src = reinterpret_cast<const char*>(p.table) + (size_t)i * row_bytes;
  char* dst = reinterpret_cast<char*>(p.out) + (size_t)r * row_bytes;
  if (p.vec) {
    for (int v = lane; v < p.vec; v += 32) reinterpret_cast<uint4*>(dst)[v] = __ldg(reinterpret_cast<const uint4*>(src) + v);
  } else if (p.elt == 4) {
    for (int v = lane; v < p.D; v += 32) reinterpret_cast<uint32_t*>(dst)[v] = __ldg(reinterpret_cast<const uint32_t*>(src) + v);
  } else {
    for (int v = lane; v < p.D; v += 32) reinterpret_cast<uint16_t*>(dst)[v] = __ldg(reinterpret_cast<const uint16_t*>(src) + v);
  }
}

int gather_launch(const Launch& L, cudaStream_t st) {
  const GatherParams& p = *reinterpret_cast<const GatherParams*>(L.blob.data());
  launch_pdl(gather_rows_kernel, L.grid, 256, 0, st, p);
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}

void gather_patch(Launch& L, const std::vector<void*>& ip, const std::vector<void*>& op) {
  GatherParams& p = *reinterpret_cast<GatherParams*>(L.blob.data());
  p.table = ip[0]; p.indices = reinterpret_cast<const float*>(ip[1]); p.out = op[0];
}

int lower_gather(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why) {
  if (ops.size() != 1) { why = "a Gather runs as a block of its own"; return DNNF_ERR_UNSUPPORTED_OP; }
  const Op& A = g.ops[anchor];
  const Tensor& T = g.tensors[A.in[0]];
  const Tensor& I = g.tensors[A.in[1]];
  const Tensor& Y = g.tensors[A.out[0]];
  if (I.numel() >= (1ll << 31) / 8 || T.dims[0] >= (1ll << 31) || T.dims[1] >= (1ll << 31)) { why = "tensor too large"; return DNNF_ERR_UNSUPPORTED_OP; }
  Launch& L = out.launch;
  L = Launch{};
  L.blob.assign(sizeof(GatherParams), 0);
  GatherParams& p = *reinterpret_cast<GatherParams*>(L.blob.data());
  p.V = (int)T.dims[0]; p.D = (int)T.dims[1]; p.rows = (int)I.numel();
  p.elt = T.dtype == DNNF_BF16 ? 2 : 4;
  const int64_t row_bytes = (int64_t)p.D * p.elt;
  p.vec = row_bytes % 16 == 0 ? (int)(row_bytes / 16) : 0;      // tensors start on 256-byte boundaries
  L.in_tensors = {A.in[0], A.in[1]};
  L.out_tensors = {A.out[0]};
  out.inputs = {A.in[0], A.in[1]};
  out.outputs = {A.out[0]};
  L.family = DNNF_FAMILY_GATHER;
  L.grid = (p.rows + 7) / 8;
  L.threads = 256;
  L.flops = 0;
  L.ew.prog = Program{};
  (void)Y;
  out.lowered = true;
  return DNNF_OK;
}

}  // namespace dnnf

// dnnf_run: resolve device pointers and launch one kernel per block on the
// caller's stream.  Nothing here allocates or synchronises.
#include <cuda_runtime.h>

#include "ir.h"

namespace dnnf {

int launch_ew(const Launch& L, cudaStream_t st);
int launch_row(const Launch& L, cudaStream_t st);
int launch_contraction(const Launch& L, void* status_words, int block_index, cudaStream_t st, std::string& err);
void patch_contraction(Launch& L, const std::vector<void*>& in_ptrs, const std::vector<void*>& out_ptrs, std::string& err);

static void* resolve(Graph& g, int t) {
  while (g.tensors[t].alias_of >= 0) t = g.tensors[t].alias_of;
  Tensor& T = g.tensors[t];
  if (T.external || T.is_output) return T.bound;
  if (T.ws_offset < 0 || !g.ws_ptr) return nullptr;
  return (char*)g.ws_ptr + T.ws_offset;
}

int run_blocks(Graph& g, int only, void* stream) {
  if (!g.planned) { g.err = "graph is not planned (or the plan is not runnable)"; return DNNF_ERR_STATE; }
  if (g.ws_bytes > 256 && !g.ws_ptr) { g.err = "workspace not bound"; return DNNF_ERR_WORKSPACE; }
  cudaStream_t st = (cudaStream_t)stream;
  // Resolve every pointer first so that a failure launches nothing.
  for (int bi : g.run_order) {
    if (only >= 0 && bi != only) continue;
    Block& b = g.blocks[bi];
    Launch& L = b.launch;
    if (L.family == DNNF_FAMILY_ALIAS) continue;
    std::vector<void*> ip, op;
    for (int t : L.in_tensors) { void* p = resolve(g, t); if (!p) { g.err = "tensor '" + g.tensors[t].name + "' is not bound"; return DNNF_ERR_UNBOUND; } ip.push_back(p); }
    for (int t : L.out_tensors) { void* p = resolve(g, t); if (!p) { g.err = "output tensor is not bound"; return DNNF_ERR_UNBOUND; } op.push_back(p); }
    if (L.family == DNNF_FAMILY_ROW) {
      for (size_t i = 0; i < ip.size(); ++i) L.row.in[i].ptr = ip[i];
      for (size_t i = 0; i < op.size(); ++i) L.row.out[i].ptr = op[i];
    } else if (L.family == DNNF_FAMILY_ELEMENTWISE || L.family == DNNF_FAMILY_TRANSPOSE) {
      for (size_t i = 0; i < ip.size(); ++i) L.ew.in[i].ptr = ip[i];
      for (size_t i = 0; i < op.size(); ++i) L.ew.out[i].ptr = op[i];
    } else {
      std::string err;
      patch_contraction(L, ip, op, err);
      if (!err.empty()) { g.err = err; return DNNF_ERR_CUDA; }
    }
  }
  for (int bi : g.run_order) {
    if (only >= 0 && bi != only) continue;
    Block& b = g.blocks[bi];
    Launch& L = b.launch;
    int rc = 0;
    switch (L.family) {
      case DNNF_FAMILY_ALIAS: break;
      case DNNF_FAMILY_ELEMENTWISE: case DNNF_FAMILY_TRANSPOSE: rc = launch_ew(L, st); break;
      case DNNF_FAMILY_ROW: rc = launch_row(L, st); break;
      default: { std::string err; rc = launch_contraction(L, g.ws_ptr, bi, st, err); if (rc) g.err = err; break; }
    }
    if (rc) {
      if (g.err.empty()) g.err = "kernel launch failed";
      g.err += std::string(" (") + cudaGetErrorString(cudaGetLastError()) + ")";
      return DNNF_ERR_CUDA;
    }
  }
  return DNNF_OK;
}

int read_status(Graph& g, int* status, int* block) {
  *status = 0;
  if (block) *block = -1;
  if (!g.ws_ptr) return DNNF_OK;
  int words[2] = {0, 0};
  if (cudaMemcpy(words, g.ws_ptr, sizeof words, cudaMemcpyDeviceToHost) != cudaSuccess) { g.err = "status read failed"; return DNNF_ERR_CUDA; }
  *status = words[0];
  if (block) *block = words[0] ? words[1] : -1;
  return DNNF_OK;
}

}  // namespace dnnf

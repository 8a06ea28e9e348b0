// dnnf_run_static_ws: run a planned graph with its between-block intermediates in a
// fixed device array owned by the library, for callers that must not allocate.
#include <cuda_runtime.h>

#include <mutex>

#include "ir.h"

namespace dnnf {
int run_blocks(Graph& g, int only_block, void* stream);
}

// One copy per GPU that loads this library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_ws[DNNF_STATIC_WS_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_ws_addr[kMaxDevices];        // device address of g_static_ws, per device ordinal
bool g_ws_known[kMaxDevices];
std::mutex g_ws_mutex;

// In host code `g_static_ws` is only a handle for the runtime, not a device address:
// the address has to be asked for, once per device, with that device current.
int static_ws_address(void** out, std::string& err) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { err = "cannot identify the current device"; return DNNF_ERR_CUDA; }
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  if (!g_ws_known[dev]) {
    void* p = nullptr;
    cudaError_t rc = cudaGetSymbolAddress(&p, g_static_ws);
    if (rc != cudaSuccess || !p) { err = std::string("cudaGetSymbolAddress failed: ") + cudaGetErrorString(rc); return DNNF_ERR_CUDA; }
    g_ws_addr[dev] = p;
    g_ws_known[dev] = true;
  }
  *out = g_ws_addr[dev];
  return DNNF_OK;
}
}  // namespace

extern "C" DNNF_API int dnnf_run_static_ws(dnnf_graph* g, void* cuda_stream) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  dnnf::Graph& G = g->g;
  try {
    if (!G.planned) { G.err = "graph is not planned"; return DNNF_ERR_STATE; }
    if (G.ws_bytes > (size_t)DNNF_STATIC_WS_BYTES) {
      G.err = "plan needs " + std::to_string(G.ws_bytes) + " bytes of workspace; the built-in array holds " +
              std::to_string((size_t)DNNF_STATIC_WS_BYTES) + ": use dnnf_run with a caller-provided workspace";
      return DNNF_ERR_WORKSPACE;
    }
    void* ws = nullptr;
    int rc = static_ws_address(&ws, G.err);
    if (rc != DNNF_OK) return rc;
    // the status words and the kernels' arrival counters must start at zero; everything else is written before it is read
    if (cudaMemsetAsync(ws, 0, G.ws_zero_bytes, (cudaStream_t)cuda_stream) != cudaSuccess) { G.err = "cannot clear the status words"; return DNNF_ERR_CUDA; }
    void* saved_ptr = G.ws_ptr;
    size_t saved_bytes = G.ws_bound_bytes;
    G.ws_ptr = ws; G.ws_bound_bytes = DNNF_STATIC_WS_BYTES;
    rc = dnnf::run_blocks(G, -1, cuda_stream);
    G.ws_ptr = saved_ptr; G.ws_bound_bytes = saved_bytes;
    return rc;
  } catch (...) {
    G.err = "unexpected exception";
    return DNNF_ERR_INVALID_ARG;
  }
}

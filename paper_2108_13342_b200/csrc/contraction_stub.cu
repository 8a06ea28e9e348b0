#include "lower.h"
#include <cuda_runtime.h>
namespace dnnf {
int lower_contraction(const Graph&, const std::vector<int>&, uint32_t, int, Block&, std::string& why) { why = "contraction kernels not built"; return DNNF_ERR_UNSUPPORTED_OP; }
int launch_contraction(const Launch&, void*, int, cudaStream_t, std::string& err) { err = "no contraction kernel"; return 1; }
void patch_contraction(Launch&, const std::vector<void*>&, const std::vector<void*>&, std::string&) {}
}

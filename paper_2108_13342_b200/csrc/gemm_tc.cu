// Tensor-core GEMM path (tcgen05 + TMA + TMEM).  Placeholder until the kernel lands:
// nothing is eligible, so every contraction takes the CUDA-core kernel.
#include "gemm_params.h"
#include "ir.h"
namespace dnnf {
bool tc_gemm_eligible(const GemmParams&) { return false; }
bool tc_gemm_prepare(Launch&, std::string&) { return true; }
int tc_gemm_launch(const Launch&, cudaStream_t) { return 1; }
void tc_gemm_plan(Launch&) {}
}

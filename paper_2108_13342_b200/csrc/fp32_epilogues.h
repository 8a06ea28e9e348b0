// Compile-time epilogue programs of the fp32 contraction kernels (split-TF32 tensor-core kernel and the FMA kernel for
// skinny pointwise convolutions): the chains that follow a pointwise convolution or an fp32 matrix product in practice.
#pragma once
#include "chain.cuh"
#include "static_programs.h"

namespace dnnf {
namespace tf32 {

// ---- static epilogue programs ------------------------------------------------------------------
#define MO(o, s, i) MicroOp{o, s, i, 0}
DNNF_SP_BEGIN(FP_Store, 2) MO(M_MOV, S_ANCHOR, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(FP_Bias, 3) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(FP_ScaleShiftClip, 5)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_CLIP, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(FP_ScaleShiftResidual, 5)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(FP_ScaleShiftClipResidual, 6)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_CLIP, S_CONST, 0), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
// the later slices of a contraction that the planner split along K: the partial sum arrives as a residual
DNNF_SP_BEGIN(FP_Residual, 3) MO(M_MOV, S_IN, 0), MO(M_ADD, S_ANCHOR, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(FP_ResidualScaleShiftClip, 6)
  MO(M_MOV, S_IN, 0), MO(M_ADD, S_ANCHOR, 0), MO(M_MUL, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_CLIP, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
// a projection without a residual (the channel count changes), alone or as the last K slice
DNNF_SP_BEGIN(FP_ScaleShift, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(FP_ResidualScaleShift, 5)
  MO(M_MOV, S_IN, 0), MO(M_ADD, S_ANCHOR, 0), MO(M_MUL, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
// the last layer of an image decoder: bias, Tanh
DNNF_SP_BEGIN(FP_BiasTanh, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_TANH, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
#undef MO
using Static = TypeList<FP_Store, FP_Bias, FP_ScaleShiftClip, FP_ScaleShiftResidual, FP_ScaleShiftClipResidual, FP_Residual,
                        FP_ResidualScaleShiftClip, FP_ScaleShift, FP_ResidualScaleShift, FP_BiasTanh>;


}  // namespace tf32
}  // namespace dnnf

// Parameter block, epilogue IO and compile-time epilogue programs shared by the convolution kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "chain.cuh"
#include "ir.h"
#include "static_programs.h"

namespace dnnf {

struct DwParams {
  int32_t N, H, W, C;
  const float* x;
  const float* k;          // [3][3][C]
  int32_t n_in, n_out;
  TensorArg in[kMaxIn];    // strides over (c, w, h, n), innermost first
  TensorArg out[kMaxOut];
  Program prog;
};

struct DwIO {
  const DwParams& p;
  float accv[4];
  uint32_t n, h, w, c;
  __device__ __forceinline__ uint32_t off(const TensorArg& a) const {
    return (uint32_t)a.base + c * (uint32_t)a.stride[0] + w * (uint32_t)a.stride[1] + h * (uint32_t)a.stride[2] + n * (uint32_t)a.stride[3];
  }
  __device__ __forceinline__ void load(int idx, float (&dst)[4]) const {
    const TensorArg& a = p.in[idx];
    if (a.stride[0] == 0) { float x = load_scalar<true>(a, off(a)); dst[0] = dst[1] = dst[2] = dst[3] = x; }
    else load_vec4<true>(a, off(a), dst);
  }
  __device__ __forceinline__ void anchor(float (&dst)[4]) const {
#pragma unroll
    for (int v = 0; v < 4; ++v) dst[v] = accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[4]) const { store_vec4<true>(p.out[idx], off(p.out[idx]), val, false); }
  __device__ __forceinline__ void row_reduce(int, float (&)[4]) const {}
};

// P results of a kernel's own IO side by side: one pass of the chain serves 4 * P values, so an interpreted chain pays
// its dispatch once per 4 * P values instead of once per 4 (and the P loads of an operand are in flight together).
template <class IO, int P>
struct BatchIO {
  static constexpr int VV = 4 * P;
  IO io[P];
  bool on[P];
  __device__ __forceinline__ void load(int idx, float (&dst)[VV]) const {
#pragma unroll
    for (int u = 0; u < P; ++u) {
      float (&d)[4] = *reinterpret_cast<float (*)[4]>(&dst[4 * u]);
      if (on[u]) io[u].load(idx, d);
      else d[0] = d[1] = d[2] = d[3] = 0.0f;
    }
  }
  __device__ __forceinline__ void anchor(float (&dst)[VV]) const {
#pragma unroll
    for (int u = 0; u < P; ++u)
#pragma unroll
      for (int v = 0; v < 4; ++v) dst[4 * u + v] = io[u].accv[v];
  }
  __device__ __forceinline__ void store(int idx, const float (&val)[VV]) const {
#pragma unroll
    for (int u = 0; u < P; ++u)
      if (on[u]) io[u].store(idx, *reinterpret_cast<const float (*)[4]>(&val[4 * u]));
  }
  __device__ __forceinline__ void row_reduce(int, float (&)[VV]) const {}
};

#define MO(o, s, i) MicroOp{o, s, i, 0}
DNNF_SP_BEGIN(CP_ScaleShiftClip, 5)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_CLIP, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(CP_ScaleShiftResidual, 5)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(CP_Store, 2) MO(M_MOV, S_ANCHOR, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(CP_ScaleShiftClipResidual, 6)
  MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_CLIP, S_CONST, 0), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(CP_Relu, 3) MO(M_MOV, S_ANCHOR, 0), MO(M_RELU, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(CP_Residual, 3) MO(M_MOV, S_ANCHOR, 0), MO(M_ADD, S_IN, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(CP_ScaleShift, 4) MO(M_MOV, S_ANCHOR, 0), MO(M_MUL, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
#undef MO
using ConvStatic = TypeList<CP_ScaleShiftClip, CP_ScaleShiftResidual, CP_Store, CP_ScaleShiftClipResidual, CP_Relu, CP_Residual, CP_ScaleShift>;


}  // namespace dnnf

// Device-side micro-op interpreter shared by every kernel family.
//
// One call evaluates the block's whole element-wise program on VV values per
// thread (a few 128-bit vectors), so the per-op dispatch -- a warp-uniform
// branch on data held in the constant bank -- is amortised over VV elements and
// no intermediate of the fused chain ever leaves registers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "microop.h"

namespace dnnf {

struct FastDiv {
  uint32_t m, s, d;
  __device__ __forceinline__ uint32_t div(uint32_t n) const { return d == 1 ? n : (__umulhi(n, m) >> s); }
};

__device__ __forceinline__ float op_sigmoid(float x) { return __fdividef(1.0f, 1.0f + __expf(-x)); }
__device__ __forceinline__ float op_gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
// 0.5*x*(1+tanh(u)) == x*sigmoid(2u), u = sqrt(2/pi)*(x + 0.044715 x^3)
__device__ __forceinline__ float op_gelu_tanh(float x) {
  float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return x * op_sigmoid(2.0f * u);
}

template <int VV>
__device__ __forceinline__ void apply_op(int op, float (&acc)[VV], const float (&src)[VV], float c0, float c1) {
  switch (op) {
    case M_MOV:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = src[v];
      break;
    case M_ADD:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] + src[v];
      break;
    case M_SUB:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] - src[v];
      break;
    case M_RSUB:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = src[v] - acc[v];
      break;
    case M_MUL:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] * src[v];
      break;
    case M_DIV:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] / src[v];
      break;
    case M_RDIV:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = src[v] / acc[v];
      break;
    case M_MAX:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = fmaxf(acc[v], src[v]);
      break;
    case M_MIN:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = fminf(acc[v], src[v]);
      break;
    case M_NEG:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = -acc[v];
      break;
    case M_ABS:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = fabsf(acc[v]);
      break;
    case M_RECIP:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = 1.0f / acc[v];
      break;
    case M_SQUARE:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] * acc[v];
      break;
    case M_SQRT:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = sqrtf(acc[v]);
      break;
    case M_EXP:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = __expf(acc[v]);
      break;
    case M_LOG:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = logf(acc[v]);
      break;
    case M_TANH:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = tanhf(acc[v]);
      break;
    case M_ERF:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = erff(acc[v]);
      break;
    case M_SIGMOID:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = op_sigmoid(acc[v]);
      break;
    case M_RELU:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = fmaxf(acc[v], 0.0f);
      break;
    case M_GELU_ERF:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = op_gelu_erf(acc[v]);
      break;
    case M_GELU_TANH:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = op_gelu_tanh(acc[v]);
      break;
    case M_CLIP:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = fminf(fmaxf(acc[v], c0), c1);
      break;
    case M_POW:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = powf(acc[v], c0);
      break;
    default: break;
  }
}

// IO concept:
//   void load(int in_idx, float (&dst)[VV]);     external input at this thread's elements
//   void anchor(float (&dst)[VV]);               contraction result (S_ANCHOR)
//   void store(int out_idx, const float (&v)[VV]);
//   void row_reduce(int op, float (&acc)[VV]);   M_ROW* (row kernels only)
template <int VV, int NT, class IO>
__device__ __forceinline__ void run_program(const Program& prog, IO& io) {
  // Saved values sit in separately named arrays selected by a switch, so that they
  // stay in registers (an array indexed by the slot number would go to local memory).
  float acc[VV], t0[VV], t1[VV], t2[VV], t3[VV];
#pragma unroll
  for (int v = 0; v < VV; ++v) { acc[v] = 0.0f; t0[v] = 0.0f; t1[v] = 0.0f; t2[v] = 0.0f; t3[v] = 0.0f; }
  const int n = prog.n;
#pragma unroll 1
  for (int pc = 0; pc < n; ++pc) {
    const MicroOp m = prog.ops[pc];
    if (m.op == M_SAVE) {
      switch (m.idx) {
        case 0:
#pragma unroll
          for (int v = 0; v < VV; ++v) t0[v] = acc[v];
          break;
        case 1:
          if (NT > 1) {
#pragma unroll
            for (int v = 0; v < VV; ++v) t1[v] = acc[v];
          }
          break;
        case 2:
          if (NT > 2) {
#pragma unroll
            for (int v = 0; v < VV; ++v) t2[v] = acc[v];
          }
          break;
        default:
          if (NT > 3) {
#pragma unroll
            for (int v = 0; v < VV; ++v) t3[v] = acc[v];
          }
          break;
      }
      continue;
    }
    if (m.op == M_STORE) { io.store(m.idx, acc); continue; }
    if (m.op >= M_ROWSUM) { io.row_reduce(m.op, acc); continue; }
    float c0 = 0.0f, c1 = 0.0f;
    if (m.src == S_IN) {
      float src[VV];
      io.load(m.idx, src);
      apply_op<VV>(m.op, acc, src, c0, c1);
    } else if (m.src == S_TMP) {
      switch (m.idx) {
        case 0: apply_op<VV>(m.op, acc, t0, c0, c1); break;
        case 1: if (NT > 1) apply_op<VV>(m.op, acc, t1, c0, c1); break;
        case 2: if (NT > 2) apply_op<VV>(m.op, acc, t2, c0, c1); break;
        default: if (NT > 3) apply_op<VV>(m.op, acc, t3, c0, c1); break;
      }
    } else if (m.src == S_ANCHOR) {
      float src[VV];
      io.anchor(src);
      apply_op<VV>(m.op, acc, src, c0, c1);
    } else {
      float src[VV];
      if (m.src == S_CONST) {
        c0 = prog.consts[m.idx];
        c1 = prog.consts[m.idx + 1 < kMaxConst ? m.idx + 1 : m.idx];
      }
#pragma unroll
      for (int v = 0; v < VV; ++v) src[v] = c0;
      apply_op<VV>(m.op, acc, src, c0, c1);
    }
  }
}

// ---- element loads / stores with dtype conversion --------------------------------

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f, bool exact) {
  if (exact) return (uint16_t)(__float_as_uint(f) >> 16);      // value came from a bf16: low bits are zero
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

__device__ __forceinline__ float load_scalar(const TensorArg& a, int64_t off) {
  if (a.dtype == 0) return __ldg(reinterpret_cast<const float*>(a.ptr) + off);
  return bf16_bits_to_float(__ldg(reinterpret_cast<const uint16_t*>(a.ptr) + off));
}
__device__ __forceinline__ void load_vec4(const TensorArg& a, int64_t off, float* dst) {
  if (a.dtype == 0) {
    float4 v = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(a.ptr) + off));
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  } else {
    uint2 v = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(a.ptr) + off));
    dst[0] = __uint_as_float(v.x << 16); dst[1] = __uint_as_float(v.x & 0xffff0000u);
    dst[2] = __uint_as_float(v.y << 16); dst[3] = __uint_as_float(v.y & 0xffff0000u);
  }
}
__device__ __forceinline__ void store_scalar(const TensorArg& a, int64_t off, float v, bool exact) {
  if (a.dtype == 0) reinterpret_cast<float*>(a.ptr)[off] = v;
  else reinterpret_cast<uint16_t*>(a.ptr)[off] = float_to_bf16_bits(v, exact);
}
__device__ __forceinline__ void store_vec4(const TensorArg& a, int64_t off, const float* v, bool exact) {
  if (a.dtype == 0) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(a.ptr) + off) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
    uint32_t lo = (uint32_t)float_to_bf16_bits(v[0], exact) | ((uint32_t)float_to_bf16_bits(v[1], exact) << 16);
    uint32_t hi = (uint32_t)float_to_bf16_bits(v[2], exact) | ((uint32_t)float_to_bf16_bits(v[3], exact) << 16);
    *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.ptr) + off) = make_uint2(lo, hi);
  }
}

}  // namespace dnnf

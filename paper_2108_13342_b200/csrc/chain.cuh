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

#include "launch_util.h"
#include "microop.h"
#include "static_programs.h"

namespace dnnf {

// exp through ex2.approx (2 ulp) with flush-to-zero: relative error about |x| * 6e-8 from
// the rounding of x*log2(e), far inside the 1e-5 budget for the |x| < 100 that matter.
__device__ __forceinline__ float fast_exp(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x * 1.4426950408889634f));
  return y;
}
__device__ __forceinline__ float fast_rcp(float x) {
  float y;
  asm("rcp.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Flush-to-zero form for operands known to be >= 1 (the erf polynomial).  Measured, not deduced: it takes 13 %
// of the instructions out of the LayerNorm+GELU block, while the same form inside the sigmoid made the
// swish+transpose block 7 % slower.
__device__ __forceinline__ float fast_rcp_ftz(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float op_sigmoid(float x) { return fast_rcp(1.0f + fast_exp(-x)); }
__device__ __forceinline__ float op_gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
// 0.5*x*(1+tanh(u)) == x*sigmoid(2u), u = sqrt(2/pi)*(x + 0.044715 x^3)
__device__ __forceinline__ float op_gelu_tanh(float x) {
  float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return x * op_sigmoid(2.0f * u);
}

// tanh.approx: 2^-11 relative error -- for epilogues whose result is rounded to bf16 anyway
__device__ __forceinline__ float fast_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float op_gelu_tanh_fast(float x) {
  float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  float h = 0.5f * x;
  return fmaf(h, fast_tanh(u), h);
}

// erf by the rational/exponential form of Abramowitz & Stegun 7.1.26 (absolute error 1.5e-7):
// a dozen instructions against the library routine's ~30; used where the result is rounded to bf16.
// Abramowitz-Stegun 7.1.26 (|error| <= 1.5e-7 plus a few 1e-8 from the MUFU reciprocal and exponential).
// Used inside GELU in every precision: 0.5 |x| * 2e-7 is far below the fp32 chains' 1e-5 bar; a bare Erf
// operator in an fp32 chain keeps erff().
__device__ __forceinline__ float fast_erf(float x) {
  const float ax = fabsf(x);
  const float t = fast_rcp_ftz(fmaf(0.3275911f, ax, 1.0f));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  const float y = 1.0f - poly * t * fast_exp(-ax * ax);
  return copysignf(y, x);
}

// kFast: the caller rounds results to bf16 (2e-2 budget), so MUFU-approximate forms are used.
template <int VV, bool kFast = false>
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
      for (int v = 0; v < VV; ++v) acc[v] = __fdividef(acc[v], src[v]);
      break;
    case M_RDIV:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = __fdividef(src[v], acc[v]);
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
      for (int v = 0; v < VV; ++v) acc[v] = fast_rcp(acc[v]);
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
      for (int v = 0; v < VV; ++v) acc[v] = fast_exp(acc[v]);
      break;
    case M_LOG:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = logf(acc[v]);
      break;
    case M_TANH:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = kFast ? fast_tanh(acc[v]) : tanhf(acc[v]);
      break;
    case M_ERF:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = kFast ? fast_erf(acc[v]) : erff(acc[v]);
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
      for (int v = 0; v < VV; ++v) acc[v] = 0.5f * acc[v] * (1.0f + fast_erf(acc[v] * 0.70710678118654752f));
      break;
    case M_GELU_TANH:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = kFast ? op_gelu_tanh_fast(acc[v]) : op_gelu_tanh(acc[v]);
      break;
    case M_CLIP:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = fminf(fmaxf(acc[v], c0), c1);
      break;
    case M_POW:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = powf(acc[v], c0);
      break;
    case M_SIN:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = sinf(acc[v]);
      break;
    case M_COS:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = cosf(acc[v]);
      break;
    case M_ASIN:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = asinf(acc[v]);
      break;
    case M_CEIL:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = ceilf(acc[v]);
      break;
    case M_FLOOR:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = floorf(acc[v]);
      break;
    case M_ROUND:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = rintf(acc[v]);
      break;
    case M_NOT:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] == 0.0f ? 1.0f : 0.0f;
      break;
    case M_LEAKY:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] > 0.0f ? acc[v] : c0 * acc[v];
      break;
    case M_GT:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] > src[v] ? 1.0f : 0.0f;
      break;
    case M_LT:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] < src[v] ? 1.0f : 0.0f;
      break;
    case M_PRELU:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = acc[v] > 0.0f ? acc[v] : src[v] * acc[v];
      break;
    case M_RPRELU:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = src[v] > 0.0f ? src[v] : acc[v] * src[v];
      break;
    case M_BF16R:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = __bfloat162float(__float2bfloat16_rn(acc[v]));
      break;
    case M_TRUNC:
#pragma unroll
      for (int v = 0; v < VV; ++v) acc[v] = truncf(acc[v]);
      break;
    default: break;
  }
}

// IO concept:
//   void load(int in_idx, float (&dst)[VV]);     external input at this thread's elements
//   void anchor(float (&dst)[VV]);               contraction result (S_ANCHOR)
//   void store(int out_idx, const float (&v)[VV]);
//   void row_reduce(int op, float (&acc)[VV]);   M_ROW* (row kernels only)
//
// Saved values sit in separately named arrays selected by a switch, so that they stay
// in registers (an array indexed by the slot number would go to local memory).
template <int VV>
struct ChainState {
  float acc[VV], t0[VV], t1[VV];
};

template <int VV, bool kFast, class IO>
__device__ __forceinline__ void exec_one(const MicroOp m, ChainState<VV>& st, IO& io, const Program& prog) {
  if (m.op == M_SAVE) {
    if (m.idx == 0) {
#pragma unroll
      for (int v = 0; v < VV; ++v) st.t0[v] = st.acc[v];
    } else {
#pragma unroll
      for (int v = 0; v < VV; ++v) st.t1[v] = st.acc[v];
    }
    return;
  }
  if (m.op == M_STORE) { io.store(m.idx, st.acc); return; }
  if (m.op >= M_ROWSUM) { io.row_reduce(m.op, st.acc); return; }
  if (m.op == M_SELECT || m.op == M_RSELECT) {       // acc = condition (saved value number m.pad) ? acc : operand, or the reverse
    float src[VV];
    if (m.src == S_IN) io.load(m.idx, src);
    else if (m.src == S_ANCHOR) io.anchor(src);
    else {
      const float c = m.src == S_CONST ? prog.consts[m.idx] : 0.0f;
#pragma unroll
      for (int v = 0; v < VV; ++v) src[v] = m.src == S_TMP ? (m.idx == 0 ? st.t0[v] : st.t1[v]) : c;
    }
#pragma unroll
    for (int v = 0; v < VV; ++v) {
      const bool take_acc = ((m.pad == 0 ? st.t0[v] : st.t1[v]) != 0.0f) == (m.op == M_SELECT);
      st.acc[v] = take_acc ? st.acc[v] : src[v];
    }
    return;
  }
  float c0 = 0.0f, c1 = 0.0f;
  if (m.src == S_IN) {
    float src[VV];
    io.load(m.idx, src);
    apply_op<VV, kFast>(m.op, st.acc, src, c0, c1);
  } else if (m.src == S_TMP) {
    if (m.idx == 0) apply_op<VV, kFast>(m.op, st.acc, st.t0, c0, c1);
    else apply_op<VV, kFast>(m.op, st.acc, st.t1, c0, c1);
  } else if (m.src == S_ANCHOR) {
    float src[VV];
    io.anchor(src);
    apply_op<VV, kFast>(m.op, st.acc, src, c0, c1);
  } else {
    float src[VV];
    if (m.src == S_CONST) {
      c0 = prog.consts[m.idx];
      c1 = prog.consts[m.idx + 1 < kMaxConst ? m.idx + 1 : m.idx];
    }
#pragma unroll
    for (int v = 0; v < VV; ++v) src[v] = c0;
    apply_op<VV, kFast>(m.op, st.acc, src, c0, c1);
  }
}

template <class SP, int I, int VV, bool kFast, class IO>
__device__ __forceinline__ void static_step(ChainState<VV>& st, IO& io, const Program& prog) {
  constexpr MicroOp m = SP::op(I);
  exec_one<VV, kFast>(m, st, io, prog);
}
template <class SP, int VV, bool kFast, class IO, int... I>
__device__ __forceinline__ void run_static(ChainState<VV>& st, IO& io, const Program& prog, std::integer_sequence<int, I...>) {
  (static_step<SP, I, VV, kFast>(st, io, prog), ...);
}

// SP = DynProg: interpret prog at run time.  Otherwise SP is a compile-time table with
// the same opcodes as prog (the host checked), and the whole chain is straight-line code.
template <int VV, class SP, bool kFast = false, class IO>
__device__ __forceinline__ void run_program(const Program& prog, IO& io) {
  ChainState<VV> st;
#pragma unroll
  for (int v = 0; v < VV; ++v) { st.acc[v] = 0.0f; st.t0[v] = 0.0f; st.t1[v] = 0.0f; }
  if constexpr (SP::n == 0) {
    const int n = prog.n;
#pragma unroll 1
    for (int pc = 0; pc < n; ++pc) exec_one<VV, kFast>(prog.ops[pc], st, io, prog);
  } else {
    run_static<SP, VV, kFast>(st, io, prog, std::make_integer_sequence<int, SP::n>{});
  }
}

// ---- element loads / stores with dtype conversion --------------------------------

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }
__device__ __forceinline__ uint16_t float_to_bf16_bits(float f, bool exact) {
  if (exact) return (uint16_t)(__float_as_uint(f) >> 16);      // value came from a bf16: low bits are zero
  return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}

// F32: every tensor of the block is fp32 (decided on the host), so the dtype test folds.
template <bool F32>
__device__ __forceinline__ float load_scalar(const TensorArg& a, uint32_t off) {
  if (F32 || a.dtype == 0) return __ldg(reinterpret_cast<const float*>(a.ptr) + off);
  return bf16_bits_to_float(__ldg(reinterpret_cast<const uint16_t*>(a.ptr) + off));
}
template <bool F32>
__device__ __forceinline__ void load_vec4(const TensorArg& a, uint32_t off, float* dst) {
  if (F32 || a.dtype == 0) {
    float4 v = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(a.ptr) + off));
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  } else {
    uint2 v = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(a.ptr) + off));
    dst[0] = __uint_as_float(v.x << 16); dst[1] = __uint_as_float(v.x & 0xffff0000u);
    dst[2] = __uint_as_float(v.y << 16); dst[3] = __uint_as_float(v.y & 0xffff0000u);
  }
}
template <bool F32>
__device__ __forceinline__ void store_scalar(const TensorArg& a, uint32_t off, float v, bool exact) {
  if (F32 || a.dtype == 0) reinterpret_cast<float*>(a.ptr)[off] = v;
  else reinterpret_cast<uint16_t*>(a.ptr)[off] = float_to_bf16_bits(v, exact);
}
template <bool F32>
__device__ __forceinline__ void store_vec4(const TensorArg& a, uint32_t off, const float* v, bool exact) {
  if (F32 || a.dtype == 0) {
    *reinterpret_cast<float4*>(reinterpret_cast<float*>(a.ptr) + off) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
    uint32_t lo, hi;
    if (exact) {
      lo = (uint32_t)float_to_bf16_bits(v[0], true) | ((uint32_t)float_to_bf16_bits(v[1], true) << 16);
      hi = (uint32_t)float_to_bf16_bits(v[2], true) | ((uint32_t)float_to_bf16_bits(v[3], true) << 16);
    } else {                                   // one packed conversion per pair (full-rate pipe)
      __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
      lo = *reinterpret_cast<uint32_t*>(&p0); hi = *reinterpret_cast<uint32_t*>(&p1);
    }
    *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(a.ptr) + off) = make_uint2(lo, hi);
  }
}

}  // namespace dnnf

// Compile-time copies of the micro-op programs that recur in practice.
//
// The host lowers every block to a micro-op program.  When that program's opcode
// and operand pattern equals one of the tables below, the block runs in a kernel
// instantiated on the table: the interpreter loop unrolls, every dispatch branch
// folds, loads hoist to the top and the chain becomes straight-line code -- the
// analogue of the paper's "once a fused operator's code is generated it is reused
// for the same pattern in this and other models" (Section 4.4).  Any other program
// still runs, through the same interpreter driven by the runtime table.
// Constants (scales, eps, clip bounds) stay runtime values in both cases.
#pragma once
#include <utility>

#include "microop.h"

namespace dnnf {

struct DynProg { static constexpr int n = 0; };

#define DNNF_SP_BEGIN(NAME, N)                                                     \
  struct NAME {                                                                    \
    static constexpr int n = N;                                                    \
    __host__ __device__ static constexpr MicroOp op(int i) {                       \
      constexpr MicroOp t[N] = {
#define DNNF_SP_END                                                                \
      };                                                                           \
      return t[i];                                                                 \
    }                                                                              \
  };
#define MO(o, s, i) MicroOp{o, s, i, 0}

// ---- element-wise / transpose families -------------------------------------------------
DNNF_SP_BEGIN(SP_Move, 2) MO(M_MOV, S_IN, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_BiasScaleSwish, 7)
  MO(M_MOV, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_MUL, S_CONST, 0), MO(M_SAVE, S_TMP, 0), MO(M_SIGMOID, S_NONE, 0),
  MO(M_MUL, S_TMP, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_AddIn, 3) MO(M_MOV, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_MulIn, 3) MO(M_MOV, S_IN, 0), MO(M_MUL, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_MulC, 3) MO(M_MOV, S_IN, 0), MO(M_MUL, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Sigmoid, 3) MO(M_MOV, S_IN, 0), MO(M_SIGMOID, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_GeluErf, 3) MO(M_MOV, S_IN, 0), MO(M_GELU_ERF, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_ScaleShiftClip, 5)
  MO(M_MOV, S_IN, 0), MO(M_MUL, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_CLIP, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
// the same chains with the value stored twice (itself and through an index map: SpaceToDepth / DepthToSpace / a Concat part)
DNNF_SP_BEGIN(SP_ScaleShiftClip2, 6)
  MO(M_MOV, S_IN, 0), MO(M_MUL, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_CLIP, S_CONST, 0), MO(M_STORE, S_NONE, 0), MO(M_STORE, S_NONE, 1) DNNF_SP_END
DNNF_SP_BEGIN(SP_SigmoidMul2, 5)
  MO(M_MOV, S_IN, 0), MO(M_SIGMOID, S_NONE, 0), MO(M_MUL, S_IN, 1), MO(M_STORE, S_NONE, 0), MO(M_STORE, S_NONE, 1) DNNF_SP_END
// x * 0.5 * (1 + erf(x / sqrt 2)) spelled as five primitive operators
DNNF_SP_BEGIN(SP_GeluPrimitives, 8)
  MO(M_MOV, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_MUL, S_CONST, 0), MO(M_ERF, S_NONE, 0), MO(M_ADD, S_CONST, 1),
  MO(M_MUL, S_TMP, 0), MO(M_MUL, S_CONST, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END

// single operators (the one-kernel-per-operator baseline must not be handicapped by the interpreter)
DNNF_SP_BEGIN(SP_ScaleShift, 4) MO(M_MOV, S_IN, 0), MO(M_MUL, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Clip, 3) MO(M_MOV, S_IN, 0), MO(M_CLIP, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_AddC, 3) MO(M_MOV, S_IN, 0), MO(M_ADD, S_CONST, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Erf, 3) MO(M_MOV, S_IN, 0), MO(M_ERF, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_GeluTanh, 3) MO(M_MOV, S_IN, 0), MO(M_GELU_TANH, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_SubIn, 3) MO(M_MOV, S_IN, 0), MO(M_SUB, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_DivIn, 3) MO(M_MOV, S_IN, 0), MO(M_DIV, S_IN, 1), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Square, 3) MO(M_MOV, S_IN, 0), MO(M_SQUARE, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Sqrt, 3) MO(M_MOV, S_IN, 0), MO(M_SQRT, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Relu, 3) MO(M_MOV, S_IN, 0), MO(M_RELU, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END

// ---- row family --------------------------------------------------------------------------
DNNF_SP_BEGIN(SP_ScaleMaskSoftmax, 12)
  MO(M_MOV, S_IN, 0), MO(M_MUL, S_CONST, 0), MO(M_ADD, S_IN, 1), MO(M_SAVE, S_TMP, 0), MO(M_ROWMAX, S_NONE, 0),
  MO(M_RSUB, S_TMP, 0), MO(M_EXP, S_NONE, 0), MO(M_SAVE, S_TMP, 0), MO(M_ROWSUM, S_NONE, 0), MO(M_RECIP, S_NONE, 0), MO(M_MUL, S_TMP, 0),
  MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_Softmax, 10)
  MO(M_MOV, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_ROWMAX, S_NONE, 0), MO(M_RSUB, S_TMP, 0), MO(M_EXP, S_NONE, 0),
  MO(M_SAVE, S_TMP, 0), MO(M_ROWSUM, S_NONE, 0), MO(M_RECIP, S_NONE, 0), MO(M_MUL, S_TMP, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_AddLayerNormGelu, 16)
  MO(M_MOV, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_SAVE, S_TMP, 0), MO(M_ROWMEAN, S_NONE, 0), MO(M_RSUB, S_TMP, 0),
  MO(M_SAVE, S_TMP, 0), MO(M_SQUARE, S_NONE, 0), MO(M_ROWMEAN, S_NONE, 0), MO(M_ADD, S_CONST, 0), MO(M_SQRT, S_NONE, 0),
  MO(M_RECIP, S_NONE, 0), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_IN, 2), MO(M_ADD, S_IN, 3), MO(M_GELU_ERF, S_NONE, 0), MO(M_STORE, S_NONE, 0) DNNF_SP_END
DNNF_SP_BEGIN(SP_LayerNorm, 14)
  MO(M_MOV, S_IN, 0), MO(M_SAVE, S_TMP, 0), MO(M_ROWMEAN, S_NONE, 0), MO(M_RSUB, S_TMP, 0), MO(M_SAVE, S_TMP, 0),
  MO(M_SQUARE, S_NONE, 0), MO(M_ROWMEAN, S_NONE, 0), MO(M_ADD, S_CONST, 0), MO(M_SQRT, S_NONE, 0), MO(M_RECIP, S_NONE, 0), MO(M_MUL, S_TMP, 0),
  MO(M_MUL, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0) DNNF_SP_END
// bias + residual + LayerNorm (the transformer's post-attention / post-FFN block)
DNNF_SP_BEGIN(SP_BiasResidualLayerNorm, 16)
  MO(M_MOV, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_SAVE, S_TMP, 0), MO(M_ROWMEAN, S_NONE, 0),
  MO(M_RSUB, S_TMP, 0), MO(M_SAVE, S_TMP, 0), MO(M_SQUARE, S_NONE, 0), MO(M_ROWMEAN, S_NONE, 0), MO(M_ADD, S_CONST, 0),
  MO(M_SQRT, S_NONE, 0), MO(M_RECIP, S_NONE, 0), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_IN, 3), MO(M_ADD, S_IN, 4), MO(M_STORE, S_NONE, 0) DNNF_SP_END
// the same with the sum also stored (pre-LayerNorm blocks keep the residual stream): outputs 0 = sum, 1 = normalised
DNNF_SP_BEGIN(SP_BiasResidualStoreLayerNorm, 17)
  MO(M_MOV, S_IN, 0), MO(M_ADD, S_IN, 1), MO(M_ADD, S_IN, 2), MO(M_STORE, S_NONE, 0), MO(M_SAVE, S_TMP, 0), MO(M_ROWMEAN, S_NONE, 0),
  MO(M_RSUB, S_TMP, 0), MO(M_SAVE, S_TMP, 0), MO(M_SQUARE, S_NONE, 0), MO(M_ROWMEAN, S_NONE, 0), MO(M_ADD, S_CONST, 0),
  MO(M_SQRT, S_NONE, 0), MO(M_RECIP, S_NONE, 0), MO(M_MUL, S_TMP, 0), MO(M_MUL, S_IN, 3), MO(M_ADD, S_IN, 4), MO(M_STORE, S_NONE, 1) DNNF_SP_END

#undef MO

template <class... T> struct TypeList {};
using EwStatic = TypeList<SP_Move, SP_BiasScaleSwish, SP_AddIn, SP_MulIn, SP_MulC, SP_Sigmoid, SP_GeluErf, SP_ScaleShiftClip,
                          SP_GeluPrimitives, SP_ScaleShift, SP_Clip, SP_AddC, SP_Erf, SP_GeluTanh, SP_SubIn, SP_DivIn, SP_Square, SP_Sqrt,
                          SP_Relu, SP_ScaleShiftClip2, SP_SigmoidMul2>;
using TrStatic = TypeList<SP_Move, SP_BiasScaleSwish>;
using RowStatic = TypeList<SP_ScaleMaskSoftmax, SP_Softmax, SP_AddLayerNormGelu, SP_LayerNorm, SP_BiasResidualLayerNorm,
                           SP_BiasResidualStoreLayerNorm>;

template <class SP>
inline bool program_matches(const Program& p) {
  if (p.n != SP::n) return false;
  for (int i = 0; i < SP::n; ++i) {
    MicroOp a = SP::op(i), b = p.ops[i];
    if (a.op != b.op || a.idx != b.idx) return false;
    bool has_src = !(a.op == M_SAVE || a.op == M_STORE);
    if (has_src && a.src != b.src) return false;
  }
  return true;
}

template <class List> struct StaticSet;
template <class... SP>
struct StaticSet<TypeList<SP...>> {
  // 1-based index of the matching table, 0 if none
  static int find(const Program& p) {
    int i = 0, r = 0;
    ((++i, (r == 0 && program_matches<SP>(p)) ? (r = i) : 0), ...);
    return r;
  }
  // calls f.template run<SP>() for the table with 1-based index `id`
  template <class F>
  static bool dispatch(int id, F&& f) {
    int i = 0;
    bool done = false;
    ((++i, (i == id && !done) ? (f.template run<SP>(), done = true) : false), ...);
    return done;
  }
};

}  // namespace dnnf

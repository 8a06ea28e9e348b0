// Micro-op programs and kernel parameter blocks shared by the host lowering and
// the device kernels.
//
// A fused block's per-element work (the data-flow tree of Section 4.4 after
// common-sub-tree elimination) is linearised by the host into a short program
// for an accumulator machine: one running value `acc`, a few saved values
// `tmp[k]`, operands taken from external inputs, constants or saved values.
// Every lane of a warp executes the same program, so dispatch is a uniform
// branch.  Programs whose opcode sequence matches a compile-time table run in a
// kernel instantiation where the dispatch folds away.
#pragma once
#include <stdint.h>

namespace dnnf {

constexpr int kMaxDims = 6;      // iteration-space rank after refinement
constexpr int kMaxIn = 8;        // external inputs of a block
constexpr int kMaxOut = 4;       // external outputs of a block
constexpr int kMaxOps = 40;      // micro-ops per program
constexpr int kMaxConst = 12;
constexpr int kMaxTmp = 2;      // saved values live in registers: two per element

enum MOp : uint8_t {
  M_END = 0,
  M_MOV,        // acc = src
  M_SAVE,       // tmp[idx] = acc
  M_STORE,      // out[idx] = acc
  M_ADD, M_SUB, M_RSUB, M_MUL, M_DIV, M_RDIV, M_MAX, M_MIN,   // acc = acc (op) src ; R*: src (op) acc
  M_NEG, M_ABS, M_RECIP, M_SQUARE, M_SQRT, M_EXP, M_LOG, M_TANH, M_ERF, M_SIGMOID, M_RELU,
  M_GELU_ERF, M_GELU_TANH,
  M_CLIP,       // acc = min(max(acc, const[idx]), const[idx+1])
  M_POW,        // acc = pow(acc, const[idx])
  M_SIN, M_COS, M_ASIN, M_CEIL, M_FLOOR, M_ROUND,
  M_NOT,        // acc = acc == 0 ? 1 : 0
  M_LEAKY,      // acc = acc > 0 ? acc : const[idx] * acc
  M_GT, M_LT,   // acc = acc > src ? 1 : 0 ; acc = acc < src ? 1 : 0
  M_PRELU, M_RPRELU,   // acc = acc > 0 ? acc : src * acc ; acc = src > 0 ? src : acc * src
  M_SELECT,     // acc = tmp[pad] != 0 ? acc : src   (Where: the condition waits in a saved value)
  M_RSELECT,    // acc = tmp[pad] != 0 ? src : acc
  M_BF16R,      // acc = nearest bfloat16 (ties to even) of acc
  M_TRUNC,      // acc = the integer toward zero
  M_ROWSUM, M_ROWMEAN, M_ROWMAX, M_ROWPROD,   // row kernels only: acc = reduce over the row, broadcast
  M_ROWSCAN, M_ROWSCAN_X, M_ROWSCAN_R, M_ROWSCAN_RX,   // row kernels only: running sum along the row; X exclusive, R from the far end
  M__COUNT
};

enum MSrc : uint8_t { S_NONE = 0, S_TMP, S_IN, S_CONST, S_ANCHOR };

struct MicroOp {
  uint8_t op, src, idx, pad;
};

struct Program {
  int32_t n;
  int32_t flags;                 // bit 0: pure data movement (bit-exact copies)
  MicroOp ops[kMaxOps];
  float consts[kMaxConst];
};
constexpr int kProgPureMove = 1;

// One external tensor as seen from the block's iteration space: element offset
//   off = base + sum_d idx[d] * stride[d]
// (element counts below 2^31 per tensor are checked at lowering time, so 32-bit
// offsets are enough on the device.)
struct TensorArg {
  void* ptr;
  int32_t base;
  int32_t stride[kMaxDims];
  int32_t dtype;       // 0 f32, 1 bf16
  int32_t mode;        // 0 direct; 2 element-wise gather; 1 / 3 staged through shared-memory slot 0 / 1
};

// Iteration space: extent[0] is the OUTERMOST dim, extent[ndim-1] the innermost.
struct IterSpace {
  int32_t ndim;
  uint32_t extent[kMaxDims];
  uint32_t div_m[kMaxDims], div_s[kMaxDims];   // n / extent[d] == umulhi(n, div_m[d]) >> div_s[d] for n < 2^31
};

// Division by a run-time constant as multiply-high and shift (valid for n < 2^31): a hardware-less integer
// divide is some 40 dependent instructions, which a single issuing thread feels on every tile.
struct FastDiv { uint32_t d, m, s; };
inline FastDiv make_fastdiv(uint32_t d) {
  FastDiv f{d, 0, 0};
  if (d <= 1) return f;
  uint32_t lg = 0;
  while ((1ull << lg) < d) ++lg;
  const uint64_t p = 31 + lg;
  f.m = (uint32_t)(((1ull << p) + d - 1) / d);
  f.s = (uint32_t)(p - 32);
  return f;
}
#ifdef __CUDACC__
__device__ __forceinline__ uint32_t fd_div(uint32_t n, const FastDiv& f) { return f.d <= 1 ? n : (__umulhi(n, f.m) >> f.s); }
#endif

inline void set_fastdiv(IterSpace& it) {
  for (int d = 0; d < it.ndim; ++d) {
    uint32_t e = it.extent[d];
    if (e <= 1) { it.div_m[d] = 0; it.div_s[d] = 0; continue; }
    uint32_t lg = 0;
    while ((1ull << lg) < e) ++lg;
    uint64_t p = 31 + lg;
    it.div_m[d] = (uint32_t)(((1ull << p) + e - 1) / e);
    it.div_s[d] = (uint32_t)(p - 32);
  }
}

struct EwParams {
  IterSpace it;
  int32_t n_in, n_out;
  TensorArg in[kMaxIn];
  TensorArg out[kMaxOut];
  Program prog;
  int32_t vec;          // elements per vector along the innermost dim (4 or 1)
  int32_t tdim;         // transpose family: iteration dim along which staged inputs are contiguous
  int64_t total;        // product of extents
  int32_t tiles_t, tiles_i;   // transpose family: tiles along tdim / innermost dim
  FastDiv fd_tiles_t, fd_tiles_i;
  uint32_t inner_vecs, inner_m, inner_s;   // vectors along the innermost dim and its fast divisor
};

inline void fastdiv_for(uint32_t e, uint32_t& m, uint32_t& s) {
  if (e <= 1) { m = 0; s = 0; return; }
  uint32_t lg = 0;
  while ((1ull << lg) < e) ++lg;
  uint64_t p = 31 + lg;
  m = (uint32_t)(((1ull << p) + e - 1) / e);
  s = (uint32_t)(p - 32);
}

struct RowParams {
  IterSpace it;         // outer dims ...; innermost = row length L
  int32_t n_in, n_out;
  TensorArg in[kMaxIn];
  TensorArg out[kMaxOut];
  Program prog;
  int64_t rows;
  int32_t L;
  int32_t vec;          // 4 if L % 4 == 0 and all accesses 16B-aligned, else 1
  float inv_L;          // 1 / L (row means multiply by it)
};

}  // namespace dnnf

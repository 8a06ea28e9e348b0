// Block lowering internals shared by lower.cpp and the contraction lowering.
#pragma once
#include <map>
#include <set>
#include <string>
#include <vector>

#include "ir.h"

namespace dnnf {

// Element offset of a tensor as a linear form over the block's iteration dims.
struct View {
  std::vector<int64_t> coef;
  int64_t c0 = 0;
  bool operator==(const View& o) const { return coef == o.coef && c0 == o.c0; }
};

struct SplitRequest { int dim = -1; int64_t inner = 0; };

// Result of aligning a view with a tensor's dims: which tensor dim each
// iteration dim walks along, and with what multiplier.
struct Aligned {
  std::vector<int> tdim;        // per iteration dim: tensor dim, -1 if coef == 0
  std::vector<int64_t> mult;    // per iteration dim
  std::vector<int64_t> cst;     // per tensor dim: constant coordinate
};

struct ExtArg { int tensor; View view; };

struct LowerCtx {
  const Graph& g;
  std::vector<int> ops;                 // topological
  std::set<int> in_block;
  std::vector<int64_t> ext;             // iteration extents, outermost first
  std::map<int, View> views;            // in-block tensors (and the reference)
  std::vector<ExtArg> ins, outs;        // external args in first-use order
  Program prog{};
  std::string why;
  SplitRequest split;
  explicit LowerCtx(const Graph& gg) : g(gg) {}
};

std::vector<int64_t> contiguous_strides(const std::vector<int64_t>& dims);
bool align_view(LowerCtx& cx, const View& v, const std::vector<int64_t>& dims, Aligned& out);
// Derive all views reachable from `ref` (identity view over ref's dims), refining
// the iteration space as needed.  `stop_at` ops are not crossed (the anchor).
bool derive_views(LowerCtx& cx, int ref_tensor, const std::set<int>& stop_ops);
bool backward_views(LowerCtx& cx, const Op& op, const View& vout, std::vector<View>& vin);
bool forward_view(LowerCtx& cx, const Op& op, int slot, const View& vin, View& vout);
// Emit the accumulator program for the block's element-wise work.  `anchor_out`
// (or -1) is the tensor whose value enters as S_ANCHOR.
bool emit_program(LowerCtx& cx, int anchor_out, int max_tmp);
int find_or_add_arg(std::vector<ExtArg>& v, int tensor, const View& view);

int lower_contraction(const Graph& g, const std::vector<int>& ops, uint32_t flags, int anchor, Block& out, std::string& why);
// MatMul -> [scale] -> [+ mask] -> Softmax -> MatMul as one kernel (beyond Table 3)
int lower_attention(const Graph& g, const std::vector<int>& ops, uint32_t flags, Block& out, std::string& why);
// Conv1x1 + chain -> DwConv3x3 + chain -> Conv1x1 + chain as one kernel (beyond Table 3)
int lower_mbconv(const Graph& g, const std::vector<int>& ops, uint32_t flags, Block& out, std::string& why);

}  // namespace dnnf

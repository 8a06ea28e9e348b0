// ECG construction: shape inference, mapping types (Table 2), Table 3 lookup.
#include "ir.h"

#include <algorithm>
#include <functional>

namespace dnnf {

int Graph::add_tensor(const std::string& name, int dtype, const std::vector<int64_t>& dims) {
  Tensor t;
  t.id = (int)tensors.size();
  t.name = name;
  t.dtype = dtype;
  t.dims = dims;
  tensors.push_back(t);
  return t.id;
}

void Graph::relink() {
  for (auto& t : tensors) { t.consumers.clear(); if (!t.external) t.producer = -1; }
  for (auto& o : ops) {
    if (!o.alive) continue;
    for (int t : o.in) tensors[t].consumers.push_back(o.id);
    for (int t : o.out) tensors[t].producer = o.id;
  }
}

std::vector<int> Graph::topo_order() const {
  // Operators are appended in a valid order and rewriting appends replacements
  // after their operands' producers, but not necessarily before their consumers:
  // do a real sort (Kahn), stable in op id.
  int n = (int)ops.size();
  std::vector<int> indeg(n, 0), order;
  for (auto& o : ops) {
    if (!o.alive) continue;
    for (int t : o.in) { int p = tensors[t].producer; if (p >= 0 && ops[p].alive) indeg[o.id]++; }
  }
  std::vector<int> ready;
  for (auto& o : ops) if (o.alive && indeg[o.id] == 0) ready.push_back(o.id);
  std::make_heap(ready.begin(), ready.end(), std::greater<int>());
  while (!ready.empty()) {
    std::pop_heap(ready.begin(), ready.end(), std::greater<int>());
    int id = ready.back(); ready.pop_back();
    order.push_back(id);
    for (int t : ops[id].out)
      for (int c : tensors[t].consumers) {
        if (!ops[c].alive) continue;
        // one decrement per (edge): an op consuming the same tensor twice has two edges
        int edges = (int)std::count(ops[c].in.begin(), ops[c].in.end(), t);
        // consumers list holds c once per edge, so decrement once here
        (void)edges;
        if (--indeg[c] == 0) { ready.push_back(c); std::push_heap(ready.begin(), ready.end(), std::greater<int>()); }
      }
  }
  return order;
}

const char* op_name(int k) {
  static const char* names[] = {"?", "Add", "Sub", "Mul", "Div", "MulC", "AddC", "Sigmoid", "Tanh", "Erf", "Exp", "Log",
    "Sqrt", "Abs", "Neg", "Recip", "Square", "Relu", "Clip", "Pow", "Gelu", "ScaleShift", "Transpose", "Reshape",
    "Flatten", "Squeeze", "Unsqueeze", "Split", "Slice", "MatMul", "Conv1x1", "DwConv3x3", "Softmax", "LayerNorm",
    "ReduceSum", "ReduceMean", "ReduceMax", "ReduceProd", "Expand", "BitShift", "DepthToSpace", "SpaceToDepth", "Resize", "Concat", "MaxPool", "AveragePool", "Sin", "Cos", "Asin", "Ceil", "Floor",
    "Round", "LeakyRelu", "Not", "Greater", "PRelu", "ConvTranspose", "Gather", "Where", "Cast", "CumSum", "InstanceNorm", "Einsum", "Col2Im", "ConcatPart"};
  if (k <= 0 || k >= DNNF_OP__COUNT) return "?";
  return names[k];
}

bool is_index_only(int k) {
  return k == DNNF_OP_TRANSPOSE || k == DNNF_OP_RESHAPE || k == DNNF_OP_FLATTEN || k == DNNF_OP_SQUEEZE ||
         k == DNNF_OP_UNSQUEEZE || k == DNNF_OP_SLICE || k == DNNF_OP_SPLIT || k == DNNF_OP_EXPAND || k == DNNF_OP_CONCATPART;
}
bool is_elementwise(int k) {
  return (k >= DNNF_OP_ADD && k <= DNNF_OP_SCALESHIFT) || k == DNNF_OP_BITSHIFT || (k >= DNNF_OP_SIN && k <= DNNF_OP_PRELU) ||
         k == DNNF_OP_WHERE || k == DNNF_OP_CAST;
}
bool is_broadcasting_elementwise(int k) { return is_binary_elementwise(k) || k == DNNF_OP_WHERE; }
bool is_binary_elementwise(int k) {
  return k == DNNF_OP_ADD || k == DNNF_OP_SUB || k == DNNF_OP_MUL || k == DNNF_OP_DIV || k == DNNF_OP_GREATER || k == DNNF_OP_PRELU;
}
bool is_row_anchor(int k) {
  return k == DNNF_OP_SOFTMAX || k == DNNF_OP_LAYERNORM || (k >= DNNF_OP_REDUCESUM && k <= DNNF_OP_REDUCEPROD) || k == DNNF_OP_CUMSUM;
}
bool is_contraction(int k) {      // anchors that take an epilogue chain and nothing in front
  return k == DNNF_OP_MATMUL || k == DNNF_OP_CONV1X1 || k == DNNF_OP_DWCONV3X3 || k == DNNF_OP_MAXPOOL || k == DNNF_OP_AVGPOOL || k == DNNF_OP_COL2IM || k == DNNF_OP_INSTANCENORM ||
         k == DNNF_OP_GATHER;
}

// Associative / commutative / distributive flags (Section 3.2).  Operators with
// none of them are the partition points of the rewriting pass (Section 4.2).
uint32_t math_props(int k) {
  switch (k) {
    case DNNF_OP_ADD: return P_ASSOC | P_COMM | P_DIST;
    case DNNF_OP_MUL: return P_ASSOC | P_COMM | P_DIST;
    case DNNF_OP_SUB: return P_DIST;
    case DNNF_OP_DIV: return P_DIST;
    case DNNF_OP_MULC: case DNNF_OP_ADDC: return P_ASSOC | P_COMM | P_DIST;
    case DNNF_OP_RECIP: case DNNF_OP_SQUARE: case DNNF_OP_SQRT: case DNNF_OP_ABS: case DNNF_OP_POW:
      return P_DIST;                       // distribute over products: f(a*b) = f(a)*f(b)
    case DNNF_OP_NEG: return P_DIST | P_COMM;
    case DNNF_OP_EXP: case DNNF_OP_LOG: return P_COMM;   // exchange with ReduceSum/ReduceProd
    case DNNF_OP_BITSHIFT: return P_COMM | P_DIST;
    case DNNF_OP_REDUCESUM: case DNNF_OP_REDUCEPROD: return P_COMM | P_ASSOC;
    default: return 0;
  }
}

static bool same_shape(const Tensor& a, const Tensor& b) { return a.dims == b.dims; }

// Mapping type of ONE (input, output) pair of an operator (Section 3.1 defines
// the types "between one input and one output").
int edge_mapping(const Graph& g, const Op& op, int slot) {
  const Tensor& in = g.tensors[op.in[slot]];
  const Tensor& out = g.tensors[op.out[0]];
  int k = op.kind;
  if (is_broadcasting_elementwise(k))
    return same_shape(in, out) ? DNNF_ONE_TO_ONE : DNNF_ONE_TO_MANY;     // "elementwise w/ broadcast"
  if (k == DNNF_OP_SCALESHIFT) return slot == 0 ? DNNF_ONE_TO_ONE : DNNF_ONE_TO_MANY;
  if (k == DNNF_OP_LAYERNORM || k == DNNF_OP_INSTANCENORM) return slot == 0 ? DNNF_MANY_TO_MANY : DNNF_ONE_TO_MANY;
  return node_mapping(g, op);
}

int node_mapping(const Graph& g, const Op& op) {
  int k = op.kind;
  switch (k) {
    case DNNF_OP_ADD: case DNNF_OP_SUB: case DNNF_OP_MUL: case DNNF_OP_DIV: case DNNF_OP_GREATER: case DNNF_OP_PRELU: case DNNF_OP_WHERE: {
      // most complex pair decides (Section 3.1)
      int m = DNNF_ONE_TO_ONE;
      for (int s = 0; s < (int)op.in.size(); ++s) m = std::max(m, edge_mapping(g, op, s));
      return m;
    }
    case DNNF_OP_SCALESHIFT: return DNNF_ONE_TO_ONE;     // BatchNormalization is listed One-to-One
    case DNNF_OP_TRANSPOSE: return DNNF_SHUFFLE;
    case DNNF_OP_RESHAPE: case DNNF_OP_FLATTEN: case DNNF_OP_SQUEEZE: case DNNF_OP_UNSQUEEZE: return DNNF_REORGANIZE;
    case DNNF_OP_SPLIT: case DNNF_OP_SLICE: case DNNF_OP_CONCAT: case DNNF_OP_CONCATPART: return DNNF_ONE_TO_ONE;
    case DNNF_OP_EXPAND: case DNNF_OP_GATHER: return DNNF_ONE_TO_MANY;
    case DNNF_OP_MATMUL: case DNNF_OP_CONV1X1: case DNNF_OP_DWCONV3X3: case DNNF_OP_SOFTMAX: case DNNF_OP_LAYERNORM:
    case DNNF_OP_REDUCESUM: case DNNF_OP_REDUCEMEAN: case DNNF_OP_REDUCEMAX: case DNNF_OP_REDUCEPROD:
    case DNNF_OP_MAXPOOL: case DNNF_OP_AVGPOOL: case DNNF_OP_CUMSUM: case DNNF_OP_COL2IM: case DNNF_OP_INSTANCENORM:
      return DNNF_MANY_TO_MANY;
    default: return DNNF_ONE_TO_ONE;
  }
}

// Table 3.  The printed table is an image; this is its reconstruction from the
// text of Section 3.2: One-to-One takes the other operand's type (green);
// Reorganize/Shuffle turn One-to-One into their type and combine among
// themselves (green), and need profiling against One-to-Many / Many-to-Many
// (yellow); One-to-Many -> Many-to-Many and Many-to-Many -> Many-to-Many are
// unprofitable (red); Many-to-Many -> One-to-Many needs profiling (yellow).
// 23 green+yellow cells and 2 red ones, matching the 23 code-generation rules
// of Section 4.4.
void table3(int a, int b, int* fused, int* colour) {
  const int OO = DNNF_ONE_TO_ONE, RE = DNNF_REORGANIZE, SH = DNNF_SHUFFLE, OM = DNNF_ONE_TO_MANY, MM = DNNF_MANY_TO_MANY;
  const int G = DNNF_FUSE_THROUGH, Y = DNNF_FUSE_DEPEND, R = DNNF_FUSE_BREAK;
  int f, c;
  if (a == OO) { f = b; c = G; }
  else if (b == OO) { f = a; c = G; }
  else if ((a == RE || a == SH) && (b == RE || b == SH)) { f = (a == SH && b == SH) ? SH : RE; c = G; }
  else if ((a == RE || a == SH)) { f = b; c = Y; }              // then b is OM or MM
  else if (a == OM && b == MM) { f = MM; c = R; }
  else if (a == MM && b == MM) { f = MM; c = R; }
  else { f = a; c = Y; }                                        // a in {OM, MM}, b in {OM, RE, SH}; MM->OM
  *fused = f; *colour = c;
}

// ---------------------------------------------------------------------------
// Shape inference
// ---------------------------------------------------------------------------
static bool broadcast_dims(const std::vector<int64_t>& a, const std::vector<int64_t>& b, std::vector<int64_t>& out) {
  size_t r = std::max(a.size(), b.size());
  out.assign(r, 1);
  for (size_t i = 0; i < r; ++i) {
    int64_t da = i < r - a.size() ? 1 : a[i - (r - a.size())];
    int64_t db = i < r - b.size() ? 1 : b[i - (r - b.size())];
    if (da != db && da != 1 && db != 1) return false;
    out[i] = std::max(da, db);
  }
  return true;
}

int infer_shapes(Graph& g, Op& op, std::string& err) {
  auto in = [&](int i) -> const Tensor& { return g.tensors[op.in[i]]; };
  auto need = [&](size_t n) { if (op.in.size() != n) { err = std::string(op_name(op.kind)) + ": wrong number of inputs"; return false; } return true; };
  std::vector<std::vector<int64_t>> outs;
  int k = op.kind;
  auto norm_axis = [&](int64_t a, int rank) { return a < 0 ? a + rank : a; };
  if (is_binary_elementwise(k)) {
    if (!need(2)) return DNNF_ERR_INVALID_ARG;
    std::vector<int64_t> o;
    if (!broadcast_dims(in(0).dims, in(1).dims, o)) { err = "broadcast mismatch"; return DNNF_ERR_SHAPE; }
    outs.push_back(o);
  } else if (k == DNNF_OP_SCALESHIFT) {
    if (!need(3)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    int ax = (int)norm_axis(op.at.axis, rank);
    if (ax < 0 || ax >= rank || in(1).numel() != in(0).dims[ax] || in(2).numel() != in(0).dims[ax]) { err = "ScaleShift: parameter length"; return DNNF_ERR_SHAPE; }
    op.at.axis = ax;
    outs.push_back(in(0).dims);
  } else if (k == DNNF_OP_LAYERNORM) {
    if (op.in.size() != 1 && !need(3)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    if (norm_axis(op.at.axis, rank) != rank - 1) { err = "LayerNorm: last axis only"; return DNNF_ERR_UNSUPPORTED_OP; }
    if (op.in.size() == 3 && (in(1).numel() != in(0).dims.back() || in(2).numel() != in(0).dims.back())) { err = "LayerNorm: parameter length"; return DNNF_ERR_SHAPE; }
    outs.push_back(in(0).dims);
  } else if (k == DNNF_OP_WHERE) {
    if (!need(3)) return DNNF_ERR_INVALID_ARG;
    std::vector<int64_t> ab, o;
    if (!broadcast_dims(in(1).dims, in(2).dims, ab) || !broadcast_dims(in(0).dims, ab, o)) { err = "broadcast mismatch"; return DNNF_ERR_SHAPE; }
    outs.push_back(o);
  } else if (k == DNNF_OP_CAST) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    if (op.at.to < DNNF_CAST_F32 || op.at.to > DNNF_CAST_BOOL) { err = "Cast: unknown target type"; return DNNF_ERR_INVALID_ARG; }
    outs.push_back(in(0).dims);
  } else if (k == DNNF_OP_CUMSUM) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    if (norm_axis(op.at.axis, rank) != rank - 1) { err = "CumSum: last axis only"; return DNNF_ERR_UNSUPPORTED_OP; }
    outs.push_back(in(0).dims);
  } else if (is_elementwise(k)) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    outs.push_back(in(0).dims);
  } else if (k == DNNF_OP_SOFTMAX) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    if (norm_axis(op.at.axis, rank) != rank - 1) { err = "Softmax: last axis only"; return DNNF_ERR_UNSUPPORTED_OP; }
    outs.push_back(in(0).dims);
  } else if (k >= DNNF_OP_REDUCESUM && k <= DNNF_OP_REDUCEPROD) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    if (norm_axis(op.at.axis, rank) != rank - 1) { err = "Reduce: last axis only"; return DNNF_ERR_UNSUPPORTED_OP; }
    auto d = in(0).dims;
    if (op.at.keepdims) d.back() = 1; else d.pop_back();
    outs.push_back(d);
  } else if (k == DNNF_OP_TRANSPOSE) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    size_t r = in(0).dims.size();
    if (op.at.perm.size() != r) { err = "Transpose: perm rank"; return DNNF_ERR_SHAPE; }
    std::vector<int> seen(r, 0);
    std::vector<int64_t> d(r);
    for (size_t i = 0; i < r; ++i) {
      int64_t p = op.at.perm[i];
      if (p < 0 || p >= (int64_t)r || seen[p]) { err = "Transpose: bad perm"; return DNNF_ERR_SHAPE; }
      seen[p] = 1; d[i] = in(0).dims[p];
    }
    outs.push_back(d);
  } else if (k == DNNF_OP_RESHAPE) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    auto d = op.at.shape;
    int64_t known = 1; int neg = -1;
    for (size_t i = 0; i < d.size(); ++i) { if (d[i] == -1) { if (neg >= 0) { err = "Reshape: two -1"; return DNNF_ERR_SHAPE; } neg = (int)i; } else known *= d[i]; }
    if (neg >= 0) { if (known == 0 || in(0).numel() % known) { err = "Reshape: size"; return DNNF_ERR_SHAPE; } d[neg] = in(0).numel() / known; known *= d[neg]; }
    if (known != in(0).numel()) { err = "Reshape: element count differs"; return DNNF_ERR_SHAPE; }
    op.at.shape = d;
    outs.push_back(d);
  } else if (k == DNNF_OP_FLATTEN) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    int ax = (int)norm_axis(op.at.axis, rank);
    int64_t lead = 1, tail = 1;
    for (int i = 0; i < rank; ++i) (i < ax ? lead : tail) *= in(0).dims[i];
    outs.push_back({lead, tail});
  } else if (k == DNNF_OP_SQUEEZE) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    std::vector<int64_t> d;
    for (int i = 0; i < rank; ++i) {
      bool drop = false;
      for (auto a : op.at.axes) if (norm_axis(a, rank) == i) drop = true;
      if (drop && in(0).dims[i] != 1) { err = "Squeeze: dim is not 1"; return DNNF_ERR_SHAPE; }
      if (!drop) d.push_back(in(0).dims[i]);
    }
    outs.push_back(d);
  } else if (k == DNNF_OP_UNSQUEEZE) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)(in(0).dims.size() + op.at.axes.size());
    std::vector<int64_t> axes;
    for (auto a : op.at.axes) axes.push_back(norm_axis(a, rank));
    std::sort(axes.begin(), axes.end());
    auto d = in(0).dims;
    for (auto a : axes) { if (a > (int64_t)d.size()) { err = "Unsqueeze: axis"; return DNNF_ERR_SHAPE; } d.insert(d.begin() + a, 1); }
    outs.push_back(d);
  } else if (k == DNNF_OP_SLICE) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    int rank = (int)in(0).dims.size();
    int ax = (int)norm_axis(op.at.axis, rank);
    if (ax < 0 || ax >= rank || op.at.start < 0 || op.at.end > in(0).dims[ax] || op.at.start >= op.at.end) { err = "Slice: range"; return DNNF_ERR_SHAPE; }
    op.at.axis = ax;
    auto d = in(0).dims; d[ax] = op.at.end - op.at.start;
    outs.push_back(d);
  } else if (k == DNNF_OP_MAXPOOL || k == DNNF_OP_AVGPOOL) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    if (in(0).dims.size() != 4) { err = "pooling takes an NHWC tensor"; return DNNF_ERR_SHAPE; }
    const int64_t kk = op.at.kernel, st = op.at.stride, pd = op.at.pad;
    if (kk < 1 || st < 1 || pd < 0 || pd >= kk || kk > in(0).dims[1] + 2 * pd || kk > in(0).dims[2] + 2 * pd) { err = "pooling: kernel, stride or pad"; return DNNF_ERR_SHAPE; }
    auto d = in(0).dims;
    d[1] = (d[1] + 2 * pd - kk) / st + 1;
    d[2] = (d[2] + 2 * pd - kk) / st + 1;
    outs.push_back(d);
  } else if (k == DNNF_OP_INSTANCENORM) {
    if (!need(3)) return DNNF_ERR_INVALID_ARG;
    if (in(0).dims.size() != 4) { err = "InstanceNorm takes an NHWC tensor"; return DNNF_ERR_SHAPE; }
    if (in(1).numel() != in(0).dims[3] || in(2).numel() != in(0).dims[3]) { err = "InstanceNorm: parameter length"; return DNNF_ERR_SHAPE; }
    outs.push_back(in(0).dims);
  } else if (k == DNNF_OP_COL2IM) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    const int64_t kk = op.at.kernel, st = op.at.stride, pd = op.at.pad;
    if (in(0).dims.size() != 4 || kk < 1 || st < 1 || st > kk || pd < 0 || pd >= kk || in(0).dims[3] % (kk * kk)) { err = "Col2Im: patch tensor, kernel, stride or pad"; return DNNF_ERR_SHAPE; }
    auto d = in(0).dims;
    d[1] = (d[1] - 1) * st + kk - 2 * pd;
    d[2] = (d[2] - 1) * st + kk - 2 * pd;
    d[3] = d[3] / (kk * kk);
    outs.push_back(d);
  } else if (k == DNNF_OP_GATHER) {
    if (!need(2)) return DNNF_ERR_INVALID_ARG;
    if (in(0).dims.size() != 2 || in(1).dtype != DNNF_F32 || in(1).dims.size() + 1 > (size_t)kMaxDims) { err = "Gather: table [V,D] and fp32 indices"; return DNNF_ERR_SHAPE; }
    if (op.at.axis != 0 && op.at.axis != -2) { err = "Gather: axis 0 only"; return DNNF_ERR_UNSUPPORTED_OP; }
    auto d = in(1).dims; d.push_back(in(0).dims[1]);
    outs.push_back(d);
  } else if (k == DNNF_OP_CONCATPART) {
    if (op.in.size() != 1 && op.in.size() != 2) { err = "ConcatPart: operand count"; return DNNF_ERR_INVALID_ARG; }
    int rank = (int)in(0).dims.size();
    int ax = (int)op.at.axis;
    if ((int)op.at.shape.size() != rank || ax < 0 || ax >= rank) { err = "Concat: rank or axis"; return DNNF_ERR_SHAPE; }
    for (int d = 0; d < rank; ++d) if (d != ax && in(0).dims[d] != op.at.shape[d]) { err = "Concat: inputs differ off the axis"; return DNNF_ERR_SHAPE; }
    if (op.at.start < 0 || op.at.start + in(0).dims[ax] > op.at.shape[ax]) { err = "Concat: range"; return DNNF_ERR_SHAPE; }
    if (op.in.size() == 2 && (in(1).dims != op.at.shape || in(1).dtype != in(0).dtype)) { err = "Concat: inputs differ in type"; return DNNF_ERR_SHAPE; }
    outs.push_back(op.at.shape);
  } else if (k == DNNF_OP_EXPAND) {
    if (!need(1)) return DNNF_ERR_INVALID_ARG;
    std::vector<int64_t> o;
    if (!broadcast_dims(in(0).dims, op.at.shape, o) || o != op.at.shape) { err = "Expand: shape"; return DNNF_ERR_SHAPE; }
    outs.push_back(o);
  } else if (k == DNNF_OP_MATMUL) {
    if (!need(2)) return DNNF_ERR_INVALID_ARG;
    auto a = in(0).dims, b = in(1).dims;
    if (a.size() < 2 || b.size() < 2 || a.back() != b[b.size() - 2]) { err = "MatMul: inner dimensions differ"; return DNNF_ERR_SHAPE; }
    std::vector<int64_t> ba(a.begin(), a.end() - 2), bb(b.begin(), b.end() - 2), bo;
    if (!broadcast_dims(ba, bb, bo)) { err = "MatMul: batch dims"; return DNNF_ERR_SHAPE; }
    bo.push_back(a[a.size() - 2]); bo.push_back(b.back());
    outs.push_back(bo);
  } else if (k == DNNF_OP_CONV1X1) {
    if (!need(2)) return DNNF_ERR_INVALID_ARG;
    if (in(0).dims.size() != 4 || in(1).dims.size() != 2 || in(0).dims[3] != in(1).dims[0]) { err = "Conv1x1: NHWC x [Cin,Cout]"; return DNNF_ERR_SHAPE; }
    auto d = in(0).dims; d[3] = in(1).dims[1];
    outs.push_back(d);
  } else if (k == DNNF_OP_DWCONV3X3) {
    if (!need(2)) return DNNF_ERR_INVALID_ARG;
    if (in(0).dims.size() != 4 || in(1).dims != std::vector<int64_t>{3, 3, in(0).dims[3]}) { err = "DwConv3x3: NHWC x [3,3,C]"; return DNNF_ERR_SHAPE; }
    outs.push_back(in(0).dims);
  } else {
    err = "unknown operator kind";
    return DNNF_ERR_UNSUPPORTED_OP;
  }
  for (auto& d : outs) {
    if (d.size() > (size_t)kMaxDims) { err = "rank above 6"; return DNNF_ERR_SHAPE; }
    for (auto v : d) if (v <= 0) { err = "empty dimension"; return DNNF_ERR_SHAPE; }
    int dt = in(0).dtype;
    if (k == DNNF_OP_WHERE) dt = in(1).dtype;
    if (k == DNNF_OP_CAST) dt = op.at.to == DNNF_CAST_BF16 ? DNNF_BF16 : DNNF_F32;
    int t = g.add_tensor("", dt, d);
    g.tensors[t].producer = op.id;
    op.out.push_back(t);
  }
  return DNNF_OK;
}

}  // namespace dnnf

// C ABI: argument checking, state machine, error messages.  No exception leaves
// this file.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <exception>

#include "ir.h"

using namespace dnnf;

namespace dnnf {
int run_blocks(Graph& g, int only_block, void* stream);
int read_status(Graph& g, int* status, int* block);
int profile_measure(Graph& g, void* scratch, size_t scratch_bytes, void* stream, int iters, int* n_measured);
}

#define DNNF_TRY try {
#define DNNF_CATCH(gptr)                                                              \
  } catch (const std::exception& e) { if (gptr) (gptr)->g.err = e.what(); return DNNF_ERR_INVALID_ARG; } \
    catch (...) { if (gptr) (gptr)->g.err = "unknown exception"; return DNNF_ERR_INVALID_ARG; }

static int fail(dnnf_graph* g, int code, const char* msg) { if (g) g->g.err = msg; return code; }

namespace dnnf { int selftest_wait_expiry(Graph& g, unsigned long long limit_ns, void* stream); }

extern "C" {

const char* dnnf_version(void) { return "dnnf-b200 0.1"; }

int dnnf_graph_create(dnnf_graph** out) {
  if (!out) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  *out = new dnnf_graph();
  return DNNF_OK;
  DNNF_CATCH((dnnf_graph*)nullptr)
}

int dnnf_graph_destroy(dnnf_graph* g) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  delete g;
  return DNNF_OK;
}

const char* dnnf_last_error(const dnnf_graph* g) { return g ? g->g.err.c_str() : "null graph"; }

int dnnf_add_tensor(dnnf_graph* g, const char* name, int dtype, int rank, const int64_t* dims, int kind, int* tensor_id) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  if (g->g.planned || !g->g.blocks.empty()) return fail(g, DNNF_ERR_STATE, "graph is already planned");
  if (!dims || !tensor_id || rank < 0 || rank > kMaxDims) return fail(g, DNNF_ERR_INVALID_ARG, "bad rank or null pointer");
  if (dtype != DNNF_F32 && dtype != DNNF_BF16) return fail(g, DNNF_ERR_INVALID_ARG, "unknown dtype");
  std::vector<int64_t> d(dims, dims + rank);
  for (auto v : d) if (v <= 0) return fail(g, DNNF_ERR_SHAPE, "dimensions must be positive");
  int id = g->g.add_tensor(name ? name : "", dtype, d);
  g->g.tensors[id].external = true;
  g->g.tensors[id].weight = (kind == DNNF_WEIGHT);
  *tensor_id = id;
  return DNNF_OK;
  DNNF_CATCH(g)
}

static int parse_attrs(const dnnf_attr* a, int n, Attrs& at, std::string& err) {
  for (int i = 0; i < n; ++i) {
    const dnnf_attr& x = a[i];
    if (x.n < 0 || x.n > 8) { err = "attribute length"; return DNNF_ERR_INVALID_ARG; }
    std::vector<int64_t> v(x.i, x.i + x.n);
    switch (x.key) {
      case DNNF_ATTR_C: at.c = x.f; break;
      case DNNF_ATTR_LO: at.lo = x.f; break;
      case DNNF_ATTR_HI: at.hi = x.f; break;
      case DNNF_ATTR_P: at.p = x.f; break;
      case DNNF_ATTR_EPS: at.eps = x.f; break;
      case DNNF_ATTR_APPROX: at.approx = x.i[0]; break;
      case DNNF_ATTR_AXIS: at.axis = x.i[0]; break;
      case DNNF_ATTR_KEEPDIMS: at.keepdims = x.i[0]; break;
      case DNNF_ATTR_START: at.start = x.i[0]; break;
      case DNNF_ATTR_END: at.end = x.i[0]; break;
      case DNNF_ATTR_BITS: at.bits = x.i[0]; break;
      case DNNF_ATTR_PERM: at.perm = v; break;
      case DNNF_ATTR_SHAPE: at.shape = v; break;
      case DNNF_ATTR_SIZES: at.sizes = v; break;
      case DNNF_ATTR_AXES: at.axes = v; break;
      case DNNF_ATTR_BLOCK: at.block = x.i[0]; break;
      case DNNF_ATTR_SCALE: at.scale = x.i[0]; break;
      case DNNF_ATTR_KERNEL: at.kernel = x.i[0]; break;
      case DNNF_ATTR_STRIDE: at.stride = x.i[0]; break;
      case DNNF_ATTR_PAD: at.pad = x.i[0]; break;
      case DNNF_ATTR_TO: at.to = x.i[0]; break;
      case DNNF_ATTR_EXCLUSIVE: at.exclusive = x.i[0] != 0; break;
      case DNNF_ATTR_REVERSE: at.reverse = x.i[0] != 0; break;
      case DNNF_ATTR_LABELS_A: at.perm = v; break;          // an Einsum has no other use for these three lists
      case DNNF_ATTR_LABELS_B: at.sizes = v; break;
      case DNNF_ATTR_LABELS_OUT: at.axes = v; break;
      default: err = "unknown attribute key"; return DNNF_ERR_INVALID_ARG;
    }
  }
  return DNNF_OK;
}

int dnnf_add_op(dnnf_graph* g, int op_kind, int n_in, const int* in_ids, const dnnf_attr* attrs, int n_attrs,
                int max_out, int* out_ids, int* n_out) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  Graph& G = g->g;
  if (G.planned || !G.blocks.empty()) return fail(g, DNNF_ERR_STATE, "graph is already planned");
  if (op_kind <= 0 || op_kind >= DNNF_OP__COUNT) return fail(g, DNNF_ERR_UNSUPPORTED_OP, "unknown operator kind");
  if (n_in <= 0 || n_in > 4 || !in_ids || !out_ids || !n_out || (n_attrs > 0 && !attrs)) return fail(g, DNNF_ERR_INVALID_ARG, "bad argument");
  for (int i = 0; i < n_in; ++i) if (in_ids[i] < 0 || in_ids[i] >= (int)G.tensors.size()) return fail(g, DNNF_ERR_INVALID_ARG, "input id out of range");
  Attrs at;
  std::string err;
  int rc = parse_attrs(attrs, n_attrs, at, err);
  if (rc) { G.err = err; return rc; }
  size_t n_tensors_before = G.tensors.size(), n_ops_before = G.ops.size();
  auto rollback = [&]() { G.tensors.resize(n_tensors_before); G.ops.resize(n_ops_before); };
  int source = G.n_source_ops;
  std::vector<int> outs;
  if (op_kind == DNNF_OP_SPLIT) {
    // A Split is n Slices of one tensor (Table 2 lists both as One-to-One); the ECG holds the Slices.
    const Tensor& X = G.tensors[in_ids[0]];
    int rank = (int)X.dims.size();
    int64_t ax = at.axis < 0 ? at.axis + rank : at.axis;
    if (ax < 0 || ax >= rank || at.sizes.empty()) return fail(g, DNNF_ERR_SHAPE, "Split: axis or sizes");
    int64_t tot = 0;
    for (auto s : at.sizes) tot += s;
    if (tot != X.dims[ax]) return fail(g, DNNF_ERR_SHAPE, "Split: sizes do not sum to the axis length");
    int64_t start = 0;
    for (auto s : at.sizes) {
      Op o; o.id = (int)G.ops.size(); o.kind = DNNF_OP_SLICE; o.source_id = source; o.in = {in_ids[0]};
      o.at.axis = ax; o.at.start = start; o.at.end = start + s;
      rc = infer_shapes(G, o, err);
      if (rc) { rollback(); G.err = err; return rc; }
      outs.push_back(o.out[0]);
      G.ops.push_back(o);
      start += s;
    }
  } else if (op_kind == DNNF_OP_CONCATPART) {
    return fail(g, DNNF_ERR_UNSUPPORTED_OP, "ConcatPart is made by Concat only");
  } else if (op_kind == DNNF_OP_CONCAT) {
    // One ConcatPart per input, chained through the result they fill in place.
    if (n_in < 2) return fail(g, DNNF_ERR_INVALID_ARG, "Concat takes 2 to 4 inputs");
    const Tensor& X0 = G.tensors[in_ids[0]];
    int rank = (int)X0.dims.size();
    int64_t ax = at.axis < 0 ? at.axis + rank : at.axis;
    if (ax < 0 || ax >= rank) return fail(g, DNNF_ERR_SHAPE, "Concat: axis");
    std::vector<int64_t> full = X0.dims;
    full[ax] = 0;
    for (int i = 0; i < n_in; ++i) {
      const Tensor& Xi = G.tensors[in_ids[i]];
      if ((int)Xi.dims.size() != rank || Xi.dtype != X0.dtype) return fail(g, DNNF_ERR_SHAPE, "Concat: inputs differ in rank or type");
      full[ax] += Xi.dims[ax];
    }
    int64_t start = 0;
    int carrier = -1;
    for (int i = 0; i < n_in; ++i) {
      Op o; o.id = (int)G.ops.size(); o.kind = DNNF_OP_CONCATPART; o.source_id = source;
      o.in = {in_ids[i]};
      if (carrier >= 0) o.in.push_back(carrier);
      o.at.axis = ax; o.at.start = start; o.at.shape = full;
      rc = infer_shapes(G, o, err);
      if (rc) { rollback(); G.err = err; return rc; }
      carrier = o.out[0];
      start += G.tensors[in_ids[i]].dims[ax];
      G.ops.push_back(o);
    }
    outs = {carrier};
  } else if (op_kind == DNNF_OP_CONVTRANSPOSE) {
    // stride = kernel: every output element receives one term per input channel, so the operator is a pointwise
    // convolution onto k*k*Cout channels followed by the DepthToSpace that spreads them over the k x k cell
    if (n_in != 2) return fail(g, DNNF_ERR_INVALID_ARG, "ConvTranspose takes (x, W)");
    const std::vector<int64_t> xd = G.tensors[in_ids[0]].dims, wd = G.tensors[in_ids[1]].dims;
    const int64_t k = at.kernel;
    if (xd.size() != 4 || wd.size() != 4 || k < 1 || wd[0] != xd[3] || wd[1] != k || wd[2] != k)
      return fail(g, DNNF_ERR_SHAPE, "ConvTranspose: NHWC x [Cin,k,k,Cout] with stride = kernel = k");
    // STRIDE defaults to 1 in the attribute block; a ConvTranspose without the attribute means stride = kernel
    bool has_stride = false;
    for (int i = 0; i < n_attrs; ++i) if (attrs[i].key == DNNF_ATTR_STRIDE) has_stride = true;
    const int64_t st = has_stride ? at.stride : k, pd = at.pad;
    if (st < 1 || st > k || pd < 0 || pd >= k) return fail(g, DNNF_ERR_SHAPE, "ConvTranspose: 1 <= stride <= kernel and 0 <= pad < kernel");
    if ((xd[1] - 1) * st + k - 2 * pd < 1 || (xd[2] - 1) * st + k - 2 * pd < 1) return fail(g, DNNF_ERR_SHAPE, "ConvTranspose: empty result");
    const bool overlap = st != k || pd != 0;
    int cur = -1;
    auto emit = [&](int kind, std::vector<int> ins, const Attrs& a) -> int {
      Op o; o.id = (int)G.ops.size(); o.kind = kind; o.source_id = source; o.in = ins; o.at = a;
      int r = infer_shapes(G, o, err);
      if (r) return r;
      cur = o.out[0];
      G.ops.push_back(o);
      return DNNF_OK;
    };
    Attrs a1, a2, a3, a4, a5;
    a1.shape = {wd[0], k * k * wd[3]};
    rc = emit(DNNF_OP_RESHAPE, {in_ids[1]}, a1);
    if (!rc) rc = emit(DNNF_OP_CONV1X1, {in_ids[0], cur}, a2);
    a3.shape = {xd[0], xd[1], xd[2], k, k, wd[3]}; a4.perm = {0, 1, 3, 2, 4, 5}; a5.shape = {xd[0], xd[1] * k, xd[2] * k, wd[3]};
    if (overlap) {
      // patches overlap (or are cropped): every output element adds the patch values that land on it
      Attrs a6; a6.kernel = k; a6.stride = st; a6.pad = pd;
      if (!rc) rc = emit(DNNF_OP_COL2IM, {cur}, a6);
    } else {
      if (!rc) rc = emit(DNNF_OP_RESHAPE, {cur}, a3);
      if (!rc) rc = emit(DNNF_OP_TRANSPOSE, {cur}, a4);
      if (!rc) rc = emit(DNNF_OP_RESHAPE, {cur}, a5);
    }
    if (rc) { rollback(); G.err = err; return rc; }
    outs = {cur};
  } else if (op_kind == DNNF_OP_GATHER && n_in == 2 &&
             (G.tensors[in_ids[0]].dims.size() != 2 || !(at.axis == 0 || at.axis == -2))) {
    // Gather along any axis of a table of any rank: the axis moves to the front, the other axes merge into the row of a
    // [V, D] table, rows are gathered, and the index axes move to where the gathered axis was.
    const std::vector<int64_t> d = G.tensors[in_ids[0]].dims, qd = G.tensors[in_ids[1]].dims;
    const int r = (int)d.size(), nq = (int)qd.size();
    const int a = (int)(at.axis < 0 ? at.axis + r : at.axis);
    if (r < 1 || a < 0 || a >= r) return fail(g, DNNF_ERR_SHAPE, "Gather: axis");
    if (r - 1 + nq > kMaxDims || r - 1 + nq < 1) return fail(g, DNNF_ERR_SHAPE, "Gather: rank of the result");
    int cur = in_ids[0];
    auto emit = [&](int kind, std::vector<int> ins, const Attrs& at2) -> int {
      Op o; o.id = (int)G.ops.size(); o.kind = kind; o.source_id = source; o.in = ins; o.at = at2;
      int rr = infer_shapes(G, o, err);
      if (rr) return rr;
      cur = o.out[0];
      G.ops.push_back(o);
      return DNNF_OK;
    };
    int64_t rest = 1;
    std::vector<int64_t> others;
    for (int i = 0; i < r; ++i) if (i != a) { rest *= d[i]; others.push_back(d[i]); }
    Attrs a1, a2, a3, a4, a5;
    a1.perm.push_back(a);
    for (int i = 0; i < r; ++i) if (i != a) a1.perm.push_back(i);
    rc = DNNF_OK;
    if (a != 0) rc = emit(DNNF_OP_TRANSPOSE, {cur}, a1);
    a2.shape = {d[a], rest};
    if (!rc && G.tensors[cur].dims != a2.shape) rc = emit(DNNF_OP_RESHAPE, {cur}, a2);
    a3.axis = 0;
    if (!rc) rc = emit(DNNF_OP_GATHER, {cur, in_ids[1]}, a3);
    a4.shape = qd;
    a4.shape.insert(a4.shape.end(), others.begin(), others.end());
    if (!rc && G.tensors[cur].dims != a4.shape) rc = emit(DNNF_OP_RESHAPE, {cur}, a4);
    if (!rc && a != 0) {
      for (int i = 0; i < a; ++i) a5.perm.push_back(nq + i);
      for (int i = 0; i < nq; ++i) a5.perm.push_back(i);
      for (int i = a; i < r - 1; ++i) a5.perm.push_back(nq + i);
      rc = emit(DNNF_OP_TRANSPOSE, {cur}, a5);
    }
    if (rc) { rollback(); G.err = err; return rc; }
    outs = {cur};
  } else if (op_kind == DNNF_OP_EINSUM) {
    // Labels of both operands and of the result: batch.  Of both operands only: summed.  Of one operand and the
    // result: that operand's free axes.  With the operands permuted to [batch, free, summed] and [batch, summed, free]
    // and each group merged into one axis the operator is a batched matrix product.
    if (n_in != 2) return fail(g, DNNF_ERR_INVALID_ARG, "Einsum takes two operands");
    const std::vector<int64_t>& la = at.perm, & lb = at.sizes, & lo = at.axes;
    const std::vector<int64_t> da = G.tensors[in_ids[0]].dims, db = G.tensors[in_ids[1]].dims;
    if (la.size() != da.size() || lb.size() != db.size()) return fail(g, DNNF_ERR_SHAPE, "Einsum: one label per axis");
    auto pos = [](const std::vector<int64_t>& l, int64_t x) { for (size_t i = 0; i < l.size(); ++i) if (l[i] == x) return (int)i; return -1; };
    auto repeats = [](const std::vector<int64_t>& l) { for (size_t i = 0; i < l.size(); ++i) for (size_t j = i + 1; j < l.size(); ++j) if (l[i] == l[j]) return true; return false; };
    if (repeats(la) || repeats(lb) || repeats(lo)) return fail(g, DNNF_ERR_UNSUPPORTED_OP, "Einsum: a label repeats inside one operand");
    std::vector<int64_t> batch, fa, fb, sum;       // labels, in the order of the result (batch, free) or of A (summed)
    for (auto x : lo) {
      const int ia = pos(la, x), ib = pos(lb, x);
      if (ia < 0 && ib < 0) return fail(g, DNNF_ERR_SHAPE, "Einsum: a result label is in no operand");
      if (ia >= 0 && ib >= 0) { if (da[ia] != db[ib]) return fail(g, DNNF_ERR_SHAPE, "Einsum: extents of a label differ"); batch.push_back(x); }
      else (ia >= 0 ? fa : fb).push_back(x);
    }
    for (auto x : la) if (pos(lo, x) < 0) {
      const int ib = pos(lb, x);
      if (ib < 0) return fail(g, DNNF_ERR_UNSUPPORTED_OP, "Einsum: a label of one operand only is summed away (use ReduceSum)");
      if (da[pos(la, x)] != db[ib]) return fail(g, DNNF_ERR_SHAPE, "Einsum: extents of a label differ");
      sum.push_back(x);
    }
    for (auto x : lb) if (pos(lo, x) < 0 && pos(la, x) < 0) return fail(g, DNNF_ERR_UNSUPPORTED_OP, "Einsum: a label of one operand only is summed away (use ReduceSum)");
    if (sum.empty()) return fail(g, DNNF_ERR_UNSUPPORTED_OP, "Einsum without a summed label (an element-wise or outer product: use Mul)");
    int cur = -1;
    auto emit = [&](int kind, std::vector<int> ins, const Attrs& a) -> int {
      Op o; o.id = (int)G.ops.size(); o.kind = kind; o.source_id = source; o.in = ins; o.at = a;
      int r = infer_shapes(G, o, err);
      if (r) return r;
      cur = o.out[0];
      G.ops.push_back(o);
      return DNNF_OK;
    };
    auto identity = [](const std::vector<int64_t>& p) { for (size_t i = 0; i < p.size(); ++i) if (p[i] != (int64_t)i) return false; return true; };
    auto prod = [&](const std::vector<int64_t>& labels, const std::vector<int64_t>& l, const std::vector<int64_t>& d) { int64_t n = 1; for (auto x : labels) n *= d[pos(l, x)]; return n; };
    const int64_t Bt = prod(batch, la, da), M = prod(fa, la, da), K = prod(sum, la, da), Nn = prod(fb, lb, db);
    // operand: permute to the group order, merge the groups
    auto arrange = [&](int t, const std::vector<int64_t>& l, const std::vector<std::vector<int64_t>>& groups, const std::vector<int64_t>& shape) -> int {
      Attrs ap, ar;
      for (auto& grp : groups) for (auto x : grp) ap.perm.push_back(pos(l, x));
      cur = t;
      int r = DNNF_OK;
      if (!identity(ap.perm)) r = emit(DNNF_OP_TRANSPOSE, {cur}, ap);
      ar.shape = shape;
      if (!r && G.tensors[cur].dims != shape) r = emit(DNNF_OP_RESHAPE, {cur}, ar);
      return r;
    };
    const bool batched = !batch.empty();
    std::vector<int64_t> sa = batched ? std::vector<int64_t>{Bt, M, K} : std::vector<int64_t>{M, K};
    std::vector<int64_t> sb = batched ? std::vector<int64_t>{Bt, K, Nn} : std::vector<int64_t>{K, Nn};
    rc = arrange(in_ids[0], la, {batch, fa, sum}, sa);
    const int ta = cur;
    if (!rc) rc = arrange(in_ids[1], lb, {batch, sum, fb}, sb);
    const int tb = cur;
    if (!rc) rc = emit(DNNF_OP_MATMUL, {ta, tb}, Attrs{});
    if (!rc) {
      // [batch, free of A, free of B] -> the separate axes -> the result's order
      std::vector<int64_t> have = batch;
      have.insert(have.end(), fa.begin(), fa.end());
      have.insert(have.end(), fb.begin(), fb.end());
      Attrs ar, ap;
      for (auto x : have) ar.shape.push_back(pos(la, x) >= 0 ? da[pos(la, x)] : db[pos(lb, x)]);
      if (ar.shape.empty()) ar.shape = {1};
      if (G.tensors[cur].dims != ar.shape) rc = emit(DNNF_OP_RESHAPE, {cur}, ar);
      for (auto x : lo) ap.perm.push_back(pos(have, x));
      if (!rc && !lo.empty() && !identity(ap.perm)) rc = emit(DNNF_OP_TRANSPOSE, {cur}, ap);
    }
    if (rc) { rollback(); G.err = err; return rc; }
    outs = {cur};
  } else if (op_kind == DNNF_OP_DEPTHTOSPACE || op_kind == DNNF_OP_SPACETODEPTH || op_kind == DNNF_OP_RESIZE) {
    // Index maps of an NHWC tensor, recorded as the Reorganize / Shuffle / One-to-Many operators they consist of.
    const Tensor& X = G.tensors[in_ids[0]];
    if (X.dims.size() != 4) return fail(g, DNNF_ERR_SHAPE, "DepthToSpace / SpaceToDepth / Resize take an NHWC tensor");
    const int64_t N = X.dims[0], H = X.dims[1], W = X.dims[2], Cc = X.dims[3];
    const int64_t b = op_kind == DNNF_OP_RESIZE ? at.scale : at.block;
    if (b < 1) return fail(g, DNNF_ERR_INVALID_ARG, "block size / scale must be a positive integer");
    int cur = in_ids[0];
    auto emit = [&](int kind, const Attrs& a) -> int {
      Op o; o.id = (int)G.ops.size(); o.kind = kind; o.source_id = source; o.in = {cur}; o.at = a;
      int r = infer_shapes(G, o, err);
      if (r) return r;
      cur = o.out[0];
      G.ops.push_back(o);
      return DNNF_OK;
    };
    Attrs a1, a2, a3;
    int k2 = DNNF_OP_TRANSPOSE;
    if (op_kind == DNNF_OP_DEPTHTOSPACE) {
      if (Cc % (b * b)) return fail(g, DNNF_ERR_SHAPE, "DepthToSpace: channels are not a multiple of block^2");
      a1.shape = {N, H, W, b, b, Cc / (b * b)}; a2.perm = {0, 1, 3, 2, 4, 5}; a3.shape = {N, H * b, W * b, Cc / (b * b)};
    } else if (op_kind == DNNF_OP_SPACETODEPTH) {
      if (H % b || W % b) return fail(g, DNNF_ERR_SHAPE, "SpaceToDepth: height or width is not a multiple of block");
      a1.shape = {N, H / b, b, W / b, b, Cc}; a2.perm = {0, 1, 3, 2, 4, 5}; a3.shape = {N, H / b, W / b, b * b * Cc};
    } else {
      a1.shape = {N, H, 1, W, 1, Cc}; k2 = DNNF_OP_EXPAND; a2.shape = {N, H, b, W, b, Cc}; a3.shape = {N, H * b, W * b, Cc};
    }
    rc = emit(DNNF_OP_RESHAPE, a1);
    if (!rc) rc = emit(k2, a2);
    if (!rc) rc = emit(DNNF_OP_RESHAPE, a3);
    if (rc) { rollback(); G.err = err; return rc; }
    outs = {cur};
  } else {
    Op o; o.id = (int)G.ops.size(); o.kind = op_kind; o.source_id = source; o.in.assign(in_ids, in_ids + n_in); o.at = at;
    rc = infer_shapes(G, o, err);
    if (rc) { rollback(); G.err = err; return rc; }
    outs = o.out;
    G.ops.push_back(o);
  }
  if ((int)outs.size() > max_out) { rollback(); return fail(g, DNNF_ERR_INVALID_ARG, "out_ids capacity too small"); }
  for (size_t i = n_ops_before; i < G.ops.size(); ++i) { G.ops[i].mapping = node_mapping(G, G.ops[i]); G.ops[i].props = math_props(G.ops[i].kind); }
  for (size_t i = 0; i < outs.size(); ++i) out_ids[i] = outs[i];
  *n_out = (int)outs.size();
  G.n_source_ops++;
  return DNNF_OK;
  DNNF_CATCH(g)
}

int dnnf_mark_output(dnnf_graph* g, int t) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  if (g->g.planned || !g->g.blocks.empty()) return fail(g, DNNF_ERR_STATE, "graph is already planned");
  if (t < 0 || t >= (int)g->g.tensors.size()) return fail(g, DNNF_ERR_INVALID_ARG, "tensor id out of range");
  if (g->g.tensors[t].external) return fail(g, DNNF_ERR_INVALID_ARG, "an external tensor cannot be an output");
  g->g.tensors[t].is_output = true;
  return DNNF_OK;
}

int dnnf_tensor_info(const dnnf_graph* g, int t, int* dtype, int* rank, int64_t* dims) {
  if (!g || t < 0 || t >= (int)g->g.tensors.size()) return DNNF_ERR_INVALID_ARG;
  const Tensor& T = g->g.tensors[t];
  if (dtype) *dtype = T.dtype;
  if (rank) *rank = (int)T.dims.size();
  if (dims) for (size_t i = 0; i < T.dims.size(); ++i) dims[i] = T.dims[i];
  return DNNF_OK;
}

int dnnf_op_mapping(const dnnf_graph* g, int op, int* mapping) {
  if (!g || !mapping || op < 0 || op >= (int)g->g.ops.size()) return DNNF_ERR_INVALID_ARG;
  *mapping = node_mapping(g->g, g->g.ops[op]);
  return DNNF_OK;
}

int dnnf_mapping_check(int first, int second, int* fused, int* colour) {
  if (first < 0 || first > 4 || second < 0 || second > 4 || !fused || !colour) return DNNF_ERR_INVALID_ARG;
  table3(first, second, fused, colour);
  return DNNF_OK;
}

int dnnf_rewrite(dnnf_graph* g, uint32_t flags, dnnf_rewrite_stats* st) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  if (g->g.planned || !g->g.blocks.empty()) return fail(g, DNNF_ERR_STATE, "rewrite must come before plan");
  return rewrite_graph(g->g, flags, st);
  DNNF_CATCH(g)
}

int dnnf_plan(dnnf_graph* g, uint32_t flags, dnnf_plan_stats* st) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  if (g->g.ops.empty()) return fail(g, DNNF_ERR_STATE, "empty graph");
  bool any_out = false;
  for (auto& t : g->g.tensors) any_out |= t.is_output;
  if (!any_out) return fail(g, DNNF_ERR_STATE, "no output marked");
  int rc = plan_graph(g->g, flags);
  if (rc == DNNF_OK && st) *st = g->g.pstats;
  return rc;
  DNNF_CATCH(g)
}

int dnnf_block_count(const dnnf_graph* g, int* n) {
  if (!g || !n) return DNNF_ERR_INVALID_ARG;
  *n = (int)g->g.blocks.size();
  return DNNF_OK;
}

int dnnf_block_info(const dnnf_graph* g, int bi, dnnf_block_desc* out) {
  if (!g || !out || bi < 0 || bi >= (int)g->g.blocks.size()) return DNNF_ERR_INVALID_ARG;
  const Graph& G = g->g;
  const Block& b = G.blocks[bi];
  std::memset(out, 0, sizeof *out);
  out->family = b.launch.family;
  out->mapping = b.mapping;
  out->n_ops = (int)b.ops.size();
  for (size_t i = 0; i < b.ops.size() && i < 48; ++i) out->op_kinds[i] = G.ops[b.ops[i]].kind;
  out->n_inputs = (int)b.inputs.size();
  out->n_outputs = (int)b.outputs.size();
  for (int t : b.inputs) out->bytes_in += G.tensors[t].bytes();
  for (int t : b.outputs) out->bytes_out += written_bytes(G, t);
  out->flops = b.launch.flops;
  { const Program* pr = program_of(b.launch); out->n_microops = pr ? pr->n : 0; }
  out->grid = b.launch.grid;
  out->threads = b.launch.threads;
  out->variant = b.launch.variant;
  return DNNF_OK;
}

int dnnf_selftest_wait_expiry(dnnf_graph* g, uint64_t limit_ns, void* stream) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  return dnnf::selftest_wait_expiry(g->g, limit_ns, stream);
}

int dnnf_block_tensors(const dnnf_graph* g, int bi, int* in_ids, int cap_in, int* n_in, int* out_ids, int cap_out, int* n_out) {
  if (!g || !n_in || !n_out || bi < 0 || bi >= (int)g->g.blocks.size()) return DNNF_ERR_INVALID_ARG;
  const Block& b = g->g.blocks[bi];
  *n_in = (int)b.inputs.size(); *n_out = (int)b.outputs.size();
  for (int i = 0; in_ids && i < cap_in && i < *n_in; ++i) in_ids[i] = b.inputs[i];
  for (int i = 0; out_ids && i < cap_out && i < *n_out; ++i) out_ids[i] = b.outputs[i];
  return DNNF_OK;
}

int dnnf_tensor_location(const dnnf_graph* g, int tensor_id, int* where, int64_t* workspace_offset) {
  if (!g || !where || tensor_id < 0 || tensor_id >= (int)g->g.tensors.size()) return DNNF_ERR_INVALID_ARG;
  const Graph& G = g->g;
  if (!G.planned) return DNNF_ERR_STATE;
  int t = tensor_id;
  while (G.tensors[t].alias_of >= 0) t = G.tensors[t].alias_of;
  const Tensor& T = G.tensors[t];
  if (workspace_offset) *workspace_offset = -1;
  if (T.external || T.is_output) { *where = t == tensor_id ? 0 : 3; if (workspace_offset && t != tensor_id) *workspace_offset = t; return DNNF_OK; }
  if (T.ws_offset >= 0) { *where = 1; if (workspace_offset) *workspace_offset = T.ws_offset; return DNNF_OK; }
  *where = 2;
  return DNNF_OK;
}

int dnnf_block_program(const dnnf_graph* g, int bi, char* buf, size_t cap) {
  if (!g || !buf || cap == 0 || bi < 0 || bi >= (int)g->g.blocks.size()) return DNNF_ERR_INVALID_ARG;
  static const char* on[] = {"END", "MOV", "SAVE", "STORE", "ADD", "SUB", "RSUB", "MUL", "DIV", "RDIV", "MAX", "MIN", "NEG", "ABS",
    "RECIP", "SQUARE", "SQRT", "EXP", "LOG", "TANH", "ERF", "SIGMOID", "RELU", "GELU_ERF", "GELU_TANH", "CLIP", "POW",
    "SIN", "COS", "ASIN", "CEIL", "FLOOR", "ROUND", "NOT", "LEAKY", "GT", "LT", "PRELU", "RPRELU", "SELECT", "RSELECT", "BF16R", "TRUNC", "ROWSUM", "ROWMEAN", "ROWMAX", "ROWPROD",
    "ROWSCAN", "ROWSCAN_X", "ROWSCAN_R", "ROWSCAN_RX"};
  static_assert(sizeof(on) / sizeof(on[0]) == M__COUNT, "one name per micro-op");
  const Block& b = g->g.blocks[bi];
  const Program* pr = program_of(b.launch);
  std::string s;
  if (pr) for (int i = 0; i < pr->n; ++i) {
    const MicroOp& m = pr->ops[i];
    if (i) s += "; ";
    s += on[m.op < M__COUNT ? m.op : 0];
    char t[48] = "";
    if (m.op == M_SAVE) snprintf(t, sizeof t, " t%d", m.idx);
    else if (m.op == M_STORE) snprintf(t, sizeof t, " out%d", m.idx);
    else if (m.src == S_IN) snprintf(t, sizeof t, " in%d", m.idx);
    else if (m.src == S_TMP) snprintf(t, sizeof t, " t%d", m.idx);
    else if (m.src == S_CONST) snprintf(t, sizeof t, " c%d=%g", m.idx, pr->consts[m.idx]);
    else if (m.src == S_ANCHOR) snprintf(t, sizeof t, " anchor");
    s += t;
  }
  snprintf(buf, cap, "%s", s.c_str());
  return DNNF_OK;
}

int dnnf_op_block(const dnnf_graph* g, int op, int* block) {
  if (!g || !block || op < 0 || op >= (int)g->g.ops.size()) return DNNF_ERR_INVALID_ARG;
  *block = g->g.ops[op].block;
  return DNNF_OK;
}

int dnnf_op_count(const dnnf_graph* g, int* n) {
  if (!g || !n) return DNNF_ERR_INVALID_ARG;
  *n = (int)g->g.ops.size();
  return DNNF_OK;
}

int dnnf_op_kind(const dnnf_graph* g, int op, int* kind, int* alive) {
  if (!g || op < 0 || op >= (int)g->g.ops.size()) return DNNF_ERR_INVALID_ARG;
  if (kind) *kind = g->g.ops[op].kind;
  if (alive) *alive = g->g.ops[op].alive ? 1 : 0;
  return DNNF_OK;
}

int dnnf_workspace_size(const dnnf_graph* g, size_t* bytes) {
  if (!g || !bytes) return DNNF_ERR_INVALID_ARG;
  if (!g->g.planned) return DNNF_ERR_STATE;
  *bytes = g->g.ws_bytes;
  return DNNF_OK;
}

int dnnf_bind(dnnf_graph* g, int t, void* dev_ptr) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  Graph& G = g->g;
  if (t < 0 || t >= (int)G.tensors.size()) return fail(g, DNNF_ERR_INVALID_ARG, "tensor id out of range");
  if (!dev_ptr || ((uintptr_t)dev_ptr & 15)) return fail(g, DNNF_ERR_INVALID_ARG, "device pointer must be non-null and 16-byte aligned");
  if (!G.tensors[t].external && !G.tensors[t].is_output) return fail(g, DNNF_ERR_INVALID_ARG, "only external tensors and marked outputs can be bound");
  G.tensors[t].bound = dev_ptr;
  return DNNF_OK;
}

int dnnf_profile_db_set(const char* signature, double microseconds) {
  if (!signature || !(microseconds > 0)) return DNNF_ERR_INVALID_ARG;
  profile_db_set(signature, microseconds);
  return DNNF_OK;
}
int dnnf_profile_db_get(const char* signature, double* microseconds) {
  if (!signature || !microseconds) return DNNF_ERR_INVALID_ARG;
  return profile_db_get(signature, microseconds) ? DNNF_OK : DNNF_ERR_INVALID_ARG;
}
int dnnf_profile_db_size(size_t* n_entries) {
  if (!n_entries) return DNNF_ERR_INVALID_ARG;
  *n_entries = profile_db_size();
  return DNNF_OK;
}
int dnnf_profile_db_clear(void) { profile_db_clear(); return DNNF_OK; }
int dnnf_profile_db_save(const char* path) { return path ? profile_db_save(path) : DNNF_ERR_INVALID_ARG; }
int dnnf_profile_db_load(const char* path, int* n_loaded) { return path ? profile_db_load(path, n_loaded) : DNNF_ERR_INVALID_ARG; }

static int copy_out(const std::string& s, char* buf, size_t cap) {
  if (!buf || cap == 0) return DNNF_ERR_INVALID_ARG;
  size_t n = std::min(cap - 1, s.size());
  memcpy(buf, s.data(), n);
  buf[n] = 0;
  return DNNF_OK;
}
int dnnf_block_signature(const dnnf_graph* g, int block, char* host_buf, size_t capacity) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  const Graph& G = g->g;
  if (!G.planned && G.blocks.empty()) return DNNF_ERR_STATE;
  if (block < 0 || block >= (int)G.blocks.size()) return DNNF_ERR_INVALID_ARG;
  return copy_out(block_signature(G, G.blocks[block]), host_buf, capacity);
}
int dnnf_profile_miss_count(const dnnf_graph* g, int* n) {
  if (!g || !n) return DNNF_ERR_INVALID_ARG;
  *n = (int)g->g.profile_misses.size();
  return DNNF_OK;
}
int dnnf_profile_miss(const dnnf_graph* g, int index, char* host_buf, size_t capacity) {
  if (!g || index < 0 || index >= (int)g->g.profile_misses.size()) return DNNF_ERR_INVALID_ARG;
  return copy_out(g->g.profile_misses[index].signature, host_buf, capacity);
}
int dnnf_profile_measure(dnnf_graph* g, void* scratch, size_t scratch_bytes, void* cuda_stream, int iters, int* n_measured) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  return profile_measure(g->g, scratch, scratch_bytes, cuda_stream, iters, n_measured);
  DNNF_CATCH(g)
}

int dnnf_workspace_zero_bytes(const dnnf_graph* g, size_t* bytes) {
  if (!g || !bytes) return DNNF_ERR_INVALID_ARG;
  if (!g->g.planned) return DNNF_ERR_STATE;
  *bytes = g->g.ws_zero_bytes;
  return DNNF_OK;
}

int dnnf_bind_workspace(dnnf_graph* g, void* dev_ptr, size_t bytes) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  Graph& G = g->g;
  if (!G.planned) return fail(g, DNNF_ERR_STATE, "plan first");
  if (!dev_ptr || ((uintptr_t)dev_ptr & 255)) return fail(g, DNNF_ERR_INVALID_ARG, "workspace must be non-null and 256-byte aligned");
  if (bytes < G.ws_bytes) return fail(g, DNNF_ERR_WORKSPACE, "workspace too small");
  G.ws_ptr = dev_ptr; G.ws_bound_bytes = bytes;
  G.last_status_base = nullptr;      // no run yet on this workspace: dnnf_status reads the new one
  return DNNF_OK;
}

int dnnf_run(dnnf_graph* g, void* stream) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  return run_blocks(g->g, -1, stream);
  DNNF_CATCH(g)
}

int dnnf_run_block(dnnf_graph* g, int block, void* stream) {
  if (!g) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  if (block < 0 || block >= (int)g->g.blocks.size()) return fail(g, DNNF_ERR_INVALID_ARG, "block index out of range");
  return run_blocks(g->g, block, stream);
  DNNF_CATCH(g)
}

int dnnf_status(dnnf_graph* g, int* status, int* block) {
  if (!g || !status) return DNNF_ERR_INVALID_ARG;
  DNNF_TRY
  return read_status(g->g, status, block);
  DNNF_CATCH(g)
}

int dnnf_launch_count(const dnnf_graph* g, int* n) {
  if (!g || !n) return DNNF_ERR_INVALID_ARG;
  if (!g->g.planned) return DNNF_ERR_STATE;
  *n = g->g.pstats.n_kernels;
  return DNNF_OK;
}

const char* dnnf_rule_name(int i) {
  static const char* names[] = {"assoc:recip-recip-mul", "assoc:sqrt-sqrt", "assoc:abs-abs", "assoc:reducesum-square",
                                "dist:common-factor", "dist:a-plus-a-mul-b", "dist:square-minus-product",
                                "comm:swap-operands", "comm:reducesum-bitshift", "comm:reduceprod-exp",
                                "strength:pow-to-square-sqrt", "fold:constant", "canon:layernorm"};
  if (i < 0 || i >= (int)(sizeof names / sizeof names[0])) return "";
  return names[i];
}

}  // extern "C"

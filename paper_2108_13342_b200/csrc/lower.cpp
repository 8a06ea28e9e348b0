// Lowering of a fusion block to one kernel launch (Section 4.4).
//
// The paper walks a data-flow tree from the block's output back to its inputs,
// fusing one operator pair at a time with a rule chosen by the pair's mapping
// types, and shares common sub-trees.  Here the same walk has two products:
//   1. index maps: every tensor of the block is expressed as a linear form over
//      ONE iteration space, so Reorganize / Shuffle / Slice operators and
//      broadcasts become strides and offsets of the loads and stores ("operations
//      that have a changed data index", Section 4.4.2) and cost nothing;
//   2. a micro-op program for the arithmetic, each value computed once.
#include "lower.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <deque>

namespace dnnf {

void finalize_ew(Launch& L);
bool finalize_row(Launch& L);

std::vector<int64_t> contiguous_strides(const std::vector<int64_t>& dims) {
  std::vector<int64_t> s(dims.size(), 1);
  for (int i = (int)dims.size() - 2; i >= 0; --i) s[i] = s[i + 1] * dims[i + 1];
  return s;
}

int find_or_add_arg(std::vector<ExtArg>& v, int tensor, const View& view) {
  for (size_t i = 0; i < v.size(); ++i)
    if (v[i].tensor == tensor && v[i].view == view) return (int)i;
  v.push_back({tensor, view});
  return (int)v.size() - 1;
}

bool align_view(LowerCtx& cx, const View& v, const std::vector<int64_t>& dims, Aligned& out) {
  int nd = (int)cx.ext.size(), r = (int)dims.size();
  auto ts = contiguous_strides(dims);
  out.tdim.assign(nd, -1);
  out.mult.assign(nd, 0);
  out.cst.assign(r, 0);
  if (v.c0 < 0) { cx.why = "negative view offset"; return false; }
  for (int k = 0; k < r; ++k) {
    int64_t q = v.c0 / ts[k];
    out.cst[k] = (k == 0) ? q : q % dims[k];
  }
  for (int d = 0; d < nd; ++d) {
    int64_t c = v.coef[d];
    if (c == 0 || cx.ext[d] == 1) continue;
    if (c < 0) { cx.why = "negative stride"; return false; }
    int k = -1;
    for (int j = 0; j < r; ++j) if (dims[j] > 1 && ts[j] <= c) { k = j; break; }
    if (k < 0 || c % ts[k]) { cx.why = "view does not align with tensor dims"; return false; }
    out.tdim[d] = k;
    out.mult[d] = c / ts[k];
  }
  for (int k = 0; k < r; ++k) {
    int64_t hi = out.cst[k];
    int worst = -1; int64_t worst_span = 0;
    for (int d = 0; d < nd; ++d) if (out.tdim[d] == k) {
      hi += out.mult[d] * (cx.ext[d] - 1);
      int64_t span = out.mult[d] * cx.ext[d];
      if (span > worst_span) { worst_span = span; worst = d; }
    }
    if (hi <= dims[k] - 1) continue;
    // an iteration dim runs across several tensor dims: split it at the boundary
    if (worst >= 0 && out.cst[k] == 0) {
      int64_t m = out.mult[worst];
      if (dims[k] % m == 0) {
        int64_t q = dims[k] / m;
        if (q >= 1 && q < cx.ext[worst] && cx.ext[worst] % q == 0) {
          cx.split.dim = worst; cx.split.inner = q;
          cx.why = "refine";
          return false;
        }
      }
    }
    cx.why = "index map is not expressible as strides";
    return false;
  }
  return true;
}

// View of a (possibly broadcast) operand given the output's alignment.
static View broadcast_view(const LowerCtx& cx, const Aligned& al, const std::vector<int64_t>& in_dims, int rank_out) {
  View v; v.coef.assign(cx.ext.size(), 0);
  auto is = contiguous_strides(in_dims);
  int shift = rank_out - (int)in_dims.size();
  for (size_t d = 0; d < cx.ext.size(); ++d) {
    int k = al.tdim[d];
    if (k < 0) continue;
    int ki = k - shift;
    if (ki < 0 || in_dims[ki] == 1) continue;
    v.coef[d] = al.mult[d] * is[ki];
  }
  for (int k = 0; k < rank_out; ++k) {
    int ki = k - shift;
    if (ki < 0 || in_dims[ki] == 1) continue;
    v.c0 += al.cst[k] * is[ki];
  }
  return v;
}

bool backward_views(LowerCtx& cx, const Op& op, const View& vout, std::vector<View>& vin) {
  const Graph& g = cx.g;
  const Tensor& out = g.tensors[op.out[0]];
  vin.assign(op.in.size(), View{});
  int k = op.kind;
  auto in = [&](int i) -> const Tensor& { return g.tensors[op.in[i]]; };
  if (k == DNNF_OP_RESHAPE || k == DNNF_OP_FLATTEN || k == DNNF_OP_SQUEEZE || k == DNNF_OP_UNSQUEEZE) {
    vin[0] = vout;                      // same flat order
    return true;
  }
  if (is_broadcasting_elementwise(k) || k == DNNF_OP_EXPAND) {
    bool need_align = false;
    for (size_t i = 0; i < op.in.size(); ++i) if (in(i).dims != out.dims) need_align = true;
    Aligned al;
    if (need_align && !align_view(cx, vout, out.dims, al)) return false;
    for (size_t i = 0; i < op.in.size(); ++i)
      vin[i] = (in(i).dims == out.dims) ? vout : broadcast_view(cx, al, in(i).dims, (int)out.dims.size());
    return true;
  }
  if (k == DNNF_OP_SCALESHIFT || k == DNNF_OP_LAYERNORM) {
    vin[0] = vout;
    Aligned al;
    if (!align_view(cx, vout, out.dims, al)) return false;
    int ax = k == DNNF_OP_SCALESHIFT ? (int)op.at.axis : (int)out.dims.size() - 1;
    for (int s = 1; s < (int)op.in.size(); ++s) {
      View v; v.coef.assign(cx.ext.size(), 0);
      for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] == ax) v.coef[d] = al.mult[d];
      v.c0 = al.cst[ax];
      vin[s] = v;
    }
    return true;
  }
  if (k == DNNF_OP_TRANSPOSE) {
    Aligned al;
    if (!align_view(cx, vout, out.dims, al)) return false;
    auto is = contiguous_strides(in(0).dims);
    View v; v.coef.assign(cx.ext.size(), 0);
    for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] >= 0) v.coef[d] = al.mult[d] * is[op.at.perm[al.tdim[d]]];
    for (size_t j = 0; j < out.dims.size(); ++j) v.c0 += al.cst[j] * is[op.at.perm[j]];
    vin[0] = v;
    return true;
  }
  if (k == DNNF_OP_SLICE) {
    Aligned al;
    if (!align_view(cx, vout, out.dims, al)) return false;
    auto is = contiguous_strides(in(0).dims);
    View v; v.coef.assign(cx.ext.size(), 0);
    for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] >= 0) v.coef[d] = al.mult[d] * is[al.tdim[d]];
    for (size_t j = 0; j < out.dims.size(); ++j) v.c0 += al.cst[j] * is[j];
    v.c0 += op.at.start * is[op.at.axis];
    vin[0] = v;
    return true;
  }
  if (k == DNNF_OP_CONCATPART) {
    // the iteration space is the part's: the result's view starts inside the part's range of the axis
    Aligned al;
    if (!align_view(cx, vout, out.dims, al)) return false;
    auto is = contiguous_strides(in(0).dims);
    View v; v.coef.assign(cx.ext.size(), 0);
    for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] >= 0) v.coef[d] = al.mult[d] * is[al.tdim[d]];
    for (size_t j = 0; j < out.dims.size(); ++j) v.c0 += al.cst[j] * is[j];
    v.c0 -= op.at.start * is[op.at.axis];
    if (v.c0 < 0) { cx.why = "Concat: view outside the part"; return false; }
    vin[0] = v;                         // the result so far (second operand) is extended in place, never read
    return true;
  }
  if (k == DNNF_OP_SOFTMAX || k == DNNF_OP_CUMSUM) { vin[0] = vout; return true; }
  if (k >= DNNF_OP_REDUCESUM && k <= DNNF_OP_REDUCEPROD) {
    cx.why = "cannot derive a reduction's input from its output";
    return false;
  }
  if (is_elementwise(k)) { vin[0] = vout; return true; }
  cx.why = std::string("no index map through ") + op_name(k);
  return false;
}

// 1 = derived, 0 = not derivable from this operand (try another), -1 = error
static int forward_view_i(LowerCtx& cx, const Op& op, int slot, const View& vi, View& vo) {
  const Graph& g = cx.g;
  const Tensor& in = g.tensors[op.in[slot]];
  const Tensor& out = g.tensors[op.out[0]];
  int k = op.kind;
  if (k == DNNF_OP_RESHAPE || k == DNNF_OP_FLATTEN || k == DNNF_OP_SQUEEZE || k == DNNF_OP_UNSQUEEZE) { vo = vi; return 1; }
  if (k == DNNF_OP_TRANSPOSE) {
    Aligned al;
    if (!align_view(cx, vi, in.dims, al)) return -1;
    auto os = contiguous_strides(out.dims);
    std::vector<int> inv(in.dims.size());
    for (size_t j = 0; j < in.dims.size(); ++j) inv[op.at.perm[j]] = (int)j;
    vo.coef.assign(cx.ext.size(), 0); vo.c0 = 0;
    for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] >= 0) vo.coef[d] = al.mult[d] * os[inv[al.tdim[d]]];
    for (size_t j = 0; j < in.dims.size(); ++j) vo.c0 += al.cst[j] * os[inv[j]];
    return 1;
  }
  if (k >= DNNF_OP_REDUCESUM && k <= DNNF_OP_REDUCEPROD) {
    Aligned al;
    if (!align_view(cx, vi, in.dims, al)) return -1;
    int last = (int)in.dims.size() - 1;
    std::vector<int64_t> od(in.dims.begin(), in.dims.end() - 1);
    auto os = contiguous_strides(od);
    vo.coef.assign(cx.ext.size(), 0); vo.c0 = 0;
    for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] >= 0 && al.tdim[d] != last) vo.coef[d] = al.mult[d] * os[al.tdim[d]];
    for (int j = 0; j < last; ++j) vo.c0 += al.cst[j] * os[j];
    return 1;
  }
  if (k == DNNF_OP_CONCATPART) {
    if (slot != 0) { cx.why = "a Concat's result so far cannot be produced in the block that extends it"; return -1; }
    Aligned al;
    if (!align_view(cx, vi, in.dims, al)) return -1;
    auto os = contiguous_strides(out.dims);
    vo.coef.assign(cx.ext.size(), 0); vo.c0 = 0;
    for (size_t d = 0; d < cx.ext.size(); ++d) if (al.tdim[d] >= 0) vo.coef[d] = al.mult[d] * os[al.tdim[d]];
    for (size_t j = 0; j < in.dims.size(); ++j) vo.c0 += al.cst[j] * os[j];
    vo.c0 += op.at.start * os[op.at.axis];
    return 1;
  }
  if (k == DNNF_OP_SLICE || k == DNNF_OP_EXPAND) { cx.why = "partial iteration space"; return -1; }
  if (k == DNNF_OP_SOFTMAX || k == DNNF_OP_CUMSUM) { vo = vi; return 1; }
  if (k == DNNF_OP_LAYERNORM || k == DNNF_OP_SCALESHIFT) { if (slot != 0) return 0; vo = vi; return 1; }
  if (is_elementwise(k)) {
    if (in.dims == out.dims) { vo = vi; return 1; }
    // Coming from a broadcast operand (e.g. a per-row statistic): the result covers the whole
    // iteration space.  Accept the identity map if walking it back reproduces this operand's view.
    int64_t tot = 1, no = 1;
    for (auto e : cx.ext) tot *= e;
    for (auto e : out.dims) no *= e;
    if (tot != no) return 0;
    View cand; cand.coef = contiguous_strides(cx.ext);
    std::vector<View> vin;
    SplitRequest keep = cx.split;
    if (!backward_views(cx, op, cand, vin)) { if (cx.split.dim >= 0) return -1; cx.split = keep; cx.why.clear(); return 0; }
    if (!(vin[slot] == vi)) return 0;
    vo = cand; return 1;
  }
  cx.why = std::string("no index map through ") + op_name(k);
  return -1;
}

bool forward_view(LowerCtx& cx, const Op& op, int slot, const View& vin, View& vout) {
  return forward_view_i(cx, op, slot, vin, vout) == 1;
}

static bool derive_once(LowerCtx& cx, int ref, const std::set<int>& stop_ops) {
  const Graph& g = cx.g;
  cx.views.clear();
  View id; id.coef = contiguous_strides(cx.ext);
  cx.views[ref] = id;
  std::deque<int> q{ref};
  auto set_view = [&](int t, const View& v) -> bool {
    auto it = cx.views.find(t);
    if (it == cx.views.end()) { cx.views[t] = v; q.push_back(t); return true; }
    if (!(it->second == v)) { cx.why = "one value is needed under two different index maps"; return false; }
    return true;
  };
  while (!q.empty()) {
    int t = q.front(); q.pop_front();
    const Tensor& T = g.tensors[t];
    int p = T.producer;
    const bool p_is_reduce = p >= 0 && g.ops[p].kind >= DNNF_OP_REDUCESUM && g.ops[p].kind <= DNNF_OP_REDUCEPROD;
    if (p >= 0 && cx.in_block.count(p) && !stop_ops.count(p) && !p_is_reduce) {   // a reduction's input is the reference
      std::vector<View> vin;
      if (!backward_views(cx, g.ops[p], cx.views[t], vin)) return false;
      for (size_t s = 0; s < vin.size(); ++s) {
        int it = g.ops[p].in[s];
        int pp = g.tensors[it].producer;
        if (pp >= 0 && cx.in_block.count(pp)) { if (!set_view(it, vin[s])) return false; }
      }
    }
    for (int c : T.consumers) {
      if (!cx.in_block.count(c) || stop_ops.count(c)) continue;
      const Op& C = g.ops[c];
      if (cx.views.count(C.out[0])) continue;
      for (size_t s = 0; s < C.in.size(); ++s) {
        if (C.in[s] != t) continue;
        View vo;
        int r = forward_view_i(cx, C, (int)s, cx.views[t], vo);
        if (r < 0) return false;
        if (r == 1) { if (!set_view(C.out[0], vo)) return false; break; }
      }
    }
  }
  return true;
}

bool derive_views(LowerCtx& cx, int ref, const std::set<int>& stop_ops) {
  for (int iter = 0; iter < 24; ++iter) {
    cx.split = SplitRequest{};
    cx.why.clear();
    if (derive_once(cx, ref, stop_ops)) return true;
    if (cx.split.dim < 0) return false;
    int d = cx.split.dim; int64_t q = cx.split.inner;
    if ((int)cx.ext.size() >= kMaxDims + 2) { cx.why = "iteration space rank too high"; return false; }
    int64_t e = cx.ext[d];
    cx.ext[d] = e / q;
    cx.ext.insert(cx.ext.begin() + d + 1, q);
  }
  cx.why = "iteration-space refinement did not converge";
  return false;
}

// ---------------------------------------------------------------------------
// Accumulator-program emission
// ---------------------------------------------------------------------------
namespace {

struct Val { int kind = 0; int id = -1; };   // kind 0: in-block tensor id, 1: external arg index, 2: the anchor's result
inline bool operator<(const Val& a, const Val& b) { return a.kind != b.kind ? a.kind < b.kind : a.id < b.id; }
inline bool operator==(const Val& a, const Val& b) { return a.kind == b.kind && a.id == b.id; }

struct Emitter {
  LowerCtx& cx;
  int max_tmp;
  std::map<Val, int> uses;          // remaining arithmetic uses
  std::map<Val, int> tmp_of;        // value -> tmp slot
  bool tmp_busy[kMaxTmp] = {false, false};
  Val acc{-1, -1};
  bool acc_valid = false;
  std::map<int, Val> root_of;       // in-block tensor -> value
  std::map<Val, std::vector<int>> stores;   // value -> out arg indices
  bool fail = false;

  Emitter(LowerCtx& c, int mt) : cx(c), max_tmp(mt) {}

  bool push(uint8_t op, uint8_t src = S_NONE, uint8_t idx = 0, uint8_t pad = 0) {
    if (cx.prog.n >= kMaxOps) { cx.why = "fused chain is longer than the micro-op budget"; fail = true; return false; }
    cx.prog.ops[cx.prog.n++] = MicroOp{op, src, idx, pad};
    return true;
  }
  int cst(float v) {
    for (int n = 0; n < used_const; ++n) if (std::memcmp(&cx.prog.consts[n], &v, 4) == 0) return n;
    if (used_const >= kMaxConst) { cx.why = "too many constants"; fail = true; return 0; }
    cx.prog.consts[used_const] = v;
    return used_const++;
  }
  int cst2(float a, float b) {      // two adjacent constants
    if (used_const + 2 > kMaxConst) { cx.why = "too many constants"; fail = true; return 0; }
    cx.prog.consts[used_const] = a; cx.prog.consts[used_const + 1] = b;
    used_const += 2;
    return used_const - 2;
  }
  int used_const = 0;

  int alloc_tmp() {
    for (int i = 0; i < max_tmp; ++i) if (!tmp_busy[i]) { tmp_busy[i] = true; return i; }
    cx.why = "fused chain needs more live values than the register budget allows";
    fail = true;
    return 0;
  }
  void release(const Val& v) {
    auto it = tmp_of.find(v);
    if (it != tmp_of.end()) { tmp_busy[it->second] = false; tmp_of.erase(it); }
  }
  // keep the value now in acc alive across an overwrite
  void spill_acc_if_live() {
    if (!acc_valid) return;
    if (acc.kind != 0) return;                       // external / anchor: can be re-read
    if (uses[acc] <= 0) return;
    if (tmp_of.count(acc)) return;
    int t = alloc_tmp();
    if (fail) return;
    tmp_of[acc] = t;
    push(M_SAVE, S_TMP, (uint8_t)t);
  }
  // operand descriptor of a value that is NOT in acc
  bool src_of(const Val& v, uint8_t& src, uint8_t& idx) {
    if (v.kind == 1) { src = S_IN; idx = (uint8_t)v.id; return true; }
    if (v.kind == 2) { src = S_ANCHOR; idx = 0; return true; }
    auto it = tmp_of.find(v);
    if (it == tmp_of.end()) { cx.why = "internal: value lost"; fail = true; return false; }
    src = S_TMP; idx = (uint8_t)it->second;
    return true;
  }
  bool in_acc(const Val& v) const { return acc_valid && acc == v; }
  void load_acc(const Val& v) {
    if (in_acc(v)) return;
    spill_acc_if_live();
    uint8_t s, i;
    if (!src_of(v, s, i)) return;
    push(M_MOV, s, i);
    acc = v; acc_valid = true;
  }
  void consume(const Val& v) {
    if (v.kind != 0) return;
    if (--uses[v] <= 0) release(v);
  }
  void produced(int tensor) {
    Val v{0, tensor};
    acc = v; acc_valid = true;
    auto it = stores.find(v);
    if (it != stores.end()) for (int o : it->second) push(M_STORE, S_NONE, (uint8_t)o);
  }
  // acc holds operand a; it will be overwritten by the result: save it first if needed later
  void protect_operand_in_acc(const Val& a, int uses_by_this_op) {
    if (a.kind != 0) return;
    if (uses[a] - uses_by_this_op > 0 && !tmp_of.count(a)) {
      int t = alloc_tmp();
      if (fail) return;
      tmp_of[a] = t;
      push(M_SAVE, S_TMP, (uint8_t)t);
    }
  }
  void unary(const Val& a, uint8_t op, uint8_t src = S_NONE, uint8_t idx = 0) {
    load_acc(a);
    protect_operand_in_acc(a, 1);
    push(op, src, idx);
    consume(a);
  }
  // Where: the condition is parked in a saved value, a goes to acc, b is the operand of the selection
  void select(const Val& c, const Val& a, const Val& b) {
    bool parked_here = false;
    if (!tmp_of.count(c)) {
      load_acc(c);
      if (fail) return;
      int t = alloc_tmp();
      if (fail) return;
      tmp_of[c] = t;
      push(M_SAVE, S_TMP, (uint8_t)t);
      parked_here = true;
    }
    const int tc = tmp_of[c];
    if (in_acc(b) && !(a == b)) {                    // b is at hand: select the other way round
      protect_operand_in_acc(b, 1);
      if (fail) return;
      uint8_t s, i;
      if (!src_of(a, s, i)) return;
      push(M_RSELECT, s, i, (uint8_t)tc);
      consume(a); consume(b);
      if (c.kind == 0) { if (--uses[c] <= 0) release(c); }
      else if (parked_here) { tmp_busy[tc] = false; tmp_of.erase(c); }
      return;
    }
    if (!in_acc(a)) {
      // the value now in acc (the condition, or an operand that lives only there) is kept if still needed
      if (acc_valid && !(acc == c)) spill_acc_if_live();
      if (fail) return;
      uint8_t s, i;
      if (!src_of(a, s, i)) return;
      push(M_MOV, s, i);
      acc = a; acc_valid = true;
    }
    if (!(a == b)) {
      protect_operand_in_acc(a, 1);
      if (fail) return;
      uint8_t s, i;
      if (!src_of(b, s, i)) return;
      push(M_SELECT, s, i, (uint8_t)tc);
    }
    consume(a); consume(b);
    // the condition leaves its slot unless an in-block value that is still needed sits there
    if (c.kind == 0) {
      if (--uses[c] <= 0) release(c);
    } else if (parked_here) {
      tmp_busy[tc] = false; tmp_of.erase(c);
    }
  }
  void binary(const Val& a, const Val& b, uint8_t op, uint8_t rop, bool commutative) {
    if (a == b) {
      load_acc(a);
      protect_operand_in_acc(a, 2);
      if (op == M_MUL) push(M_SQUARE);
      else if (op == M_ADD) push(M_MUL, S_CONST, (uint8_t)cst(2.0f));
      else {   // a-a, a/a, max(a,a): go through a tmp
        int t;
        if (tmp_of.count(a)) t = tmp_of[a]; else { t = alloc_tmp(); if (fail) return; push(M_SAVE, S_TMP, (uint8_t)t); tmp_busy[t] = false; }
        push(op, S_TMP, (uint8_t)t);
      }
      consume(a); consume(a);
      return;
    }
    uint8_t s, i;
    if (in_acc(a)) {
      protect_operand_in_acc(a, 1);
      if (!src_of(b, s, i)) return;
      push(op, s, i);
    } else if (in_acc(b)) {
      protect_operand_in_acc(b, 1);
      if (!src_of(a, s, i)) return;
      push(commutative ? op : rop, s, i);
    } else {
      // prefer loading an in-block value (it may live only in a tmp) and reading the other as operand
      load_acc(a);
      if (fail) return;
      protect_operand_in_acc(a, 1);
      if (!src_of(b, s, i)) return;
      push(op, s, i);
    }
    consume(a); consume(b);
  }
};

}  // namespace

bool emit_program(LowerCtx& cx, int anchor_out, int max_tmp) {
  const Graph& g = cx.g;
  Emitter E(cx, max_tmp);
  cx.prog = Program{};
  cx.ins.clear(); cx.outs.clear();

  // Pass 1: resolve every in-block tensor to the value it carries and count uses.
  // Index-only operators forward their operand's value (they only change indexing).
  std::map<int, std::vector<View>> in_views;     // op id -> views of its inputs
  auto ext_value = [&](int tensor, const View& v) -> Val {
    return Val{1, find_or_add_arg(cx.ins, tensor, v)};
  };
  auto is_in_block_tensor = [&](int t) { int p = g.tensors[t].producer; return p >= 0 && cx.in_block.count(p) > 0; };
  bool any_arith = false;
  std::vector<std::pair<int, std::vector<Val>>> work;   // arithmetic ops with operand values
  for (int oid : cx.ops) {
    const Op& op = g.ops[oid];
    if (op.out[0] == anchor_out) {           // the anchor itself: its value arrives from the contraction
      E.root_of[op.out[0]] = Val{2, 0};
      continue;
    }
    if (is_contraction(op.kind)) { cx.why = "second contraction in block"; return false; }
    auto vit = cx.views.find(op.out[0]);
    if (vit == cx.views.end()) { cx.why = "operator is not connected to the block's reference tensor"; return false; }
    std::vector<View> vin;
    if (!backward_views(cx, op, vit->second, vin)) {
      // reductions cannot be walked backwards; their input view is already known
      if (op.kind >= DNNF_OP_REDUCESUM && op.kind <= DNNF_OP_REDUCEPROD && cx.views.count(op.in[0])) { vin.assign(1, cx.views[op.in[0]]); cx.why.clear(); }
      else return false;
    }
    std::vector<Val> vals;
    for (size_t s = 0; s < op.in.size(); ++s) {
      int t = op.in[s];
      if (op.kind == DNNF_OP_CONCATPART && s > 0) break;      // extended in place, not an operand of the kernel
      if (is_in_block_tensor(t)) {
        auto r = E.root_of.find(t);
        if (r == E.root_of.end()) { cx.why = "internal: operand before producer"; return false; }
        vals.push_back(r->second);
      } else {
        vals.push_back(ext_value(t, vin[s]));
      }
    }
    if (is_index_only(op.kind)) {
      E.root_of[op.out[0]] = vals[0];
    } else {
      any_arith = true;
      E.root_of[op.out[0]] = Val{0, op.out[0]};
      for (auto& v : vals) if (v.kind == 0) E.uses[v]++;
      work.push_back({oid, vals});
    }
  }
  if ((int)cx.ins.size() > kMaxIn) { cx.why = "block reads more external tensors than a kernel takes"; return false; }

  // Block outputs: produced here and visible outside (graph output or outside consumer).
  for (int oid : cx.ops) {
    const Op& op = g.ops[oid];
    for (int t : op.out) {
      const Tensor& T = g.tensors[t];
      bool outside = T.is_output;
      for (int c : T.consumers) if (!cx.in_block.count(c)) outside = true;
      if (!outside) continue;
      auto vit = cx.views.find(t);
      if (vit == cx.views.end()) { cx.why = "output not reachable"; return false; }
      // A tensor that leaves the block must be written completely: the iteration space has to cover all of it.
      // (With a Slice further down the block the space is the slice's, and a tensor in front of the Slice that
      // is also read outside would be written only in part.)
      {
        int64_t covered = 1;
        for (size_t d = 0; d < vit->second.coef.size() && d < cx.ext.size(); ++d) if (vit->second.coef[d] != 0) covered *= cx.ext[d];
        const bool part = T.producer >= 0 && g.ops[T.producer].kind == DNNF_OP_CONCATPART;   // writes its own range only
        if (part ? covered != g.tensors[g.ops[T.producer].in[0]].numel() : (covered != T.numel() || vit->second.c0 != 0)) { cx.why = "a tensor that is read outside the block would be written only in part"; return false; }
      }
      int oi = find_or_add_arg(cx.outs, t, vit->second);
      E.stores[E.root_of[t]].push_back(oi);
    }
  }
  if (cx.outs.empty()) { cx.why = "block has no output"; return false; }
  if ((int)cx.outs.size() > kMaxOut) { cx.why = "block writes more tensors than a kernel takes"; return false; }
  if (!any_arith) cx.prog.flags |= kProgPureMove;

  // Pass 2: emit.
  // external inputs (or the anchor's result) stored straight to outputs
  for (auto& kv : E.stores) {
    if (kv.first.kind == 0) continue;
    E.load_acc(kv.first);
    for (int o : kv.second) E.push(M_STORE, S_NONE, (uint8_t)o);
  }
  for (auto& w : work) {
    const Op& op = g.ops[w.first];
    auto& v = w.second;
    switch (op.kind) {
      case DNNF_OP_ADD: E.binary(v[0], v[1], M_ADD, M_ADD, true); break;
      case DNNF_OP_MUL: E.binary(v[0], v[1], M_MUL, M_MUL, true); break;
      case DNNF_OP_SUB: E.binary(v[0], v[1], M_SUB, M_RSUB, false); break;
      case DNNF_OP_DIV: E.binary(v[0], v[1], M_DIV, M_RDIV, false); break;
      case DNNF_OP_MULC: E.unary(v[0], M_MUL, S_CONST, (uint8_t)E.cst((float)op.at.c)); break;
      case DNNF_OP_ADDC: E.unary(v[0], M_ADD, S_CONST, (uint8_t)E.cst((float)op.at.c)); break;
      case DNNF_OP_SIGMOID: E.unary(v[0], M_SIGMOID); break;
      case DNNF_OP_TANH: E.unary(v[0], M_TANH); break;
      case DNNF_OP_ERF: E.unary(v[0], M_ERF); break;
      case DNNF_OP_EXP: E.unary(v[0], M_EXP); break;
      case DNNF_OP_LOG: E.unary(v[0], M_LOG); break;
      case DNNF_OP_SQRT: E.unary(v[0], M_SQRT); break;
      case DNNF_OP_ABS: E.unary(v[0], M_ABS); break;
      case DNNF_OP_SIN: E.unary(v[0], M_SIN); break;
      case DNNF_OP_COS: E.unary(v[0], M_COS); break;
      case DNNF_OP_ASIN: E.unary(v[0], M_ASIN); break;
      case DNNF_OP_CEIL: E.unary(v[0], M_CEIL); break;
      case DNNF_OP_FLOOR: E.unary(v[0], M_FLOOR); break;
      case DNNF_OP_ROUND: E.unary(v[0], M_ROUND); break;
      case DNNF_OP_NOT: E.unary(v[0], M_NOT); break;
      case DNNF_OP_LEAKYRELU: E.unary(v[0], M_LEAKY, S_CONST, (uint8_t)E.cst((float)op.at.c)); break;
      case DNNF_OP_GREATER: E.binary(v[0], v[1], M_GT, M_LT, false); break;
      case DNNF_OP_PRELU: E.binary(v[0], v[1], M_PRELU, M_RPRELU, false); break;
      case DNNF_OP_NEG: E.unary(v[0], M_NEG); break;
      case DNNF_OP_RECIP: E.unary(v[0], M_RECIP); break;
      case DNNF_OP_SQUARE: E.unary(v[0], M_SQUARE); break;
      case DNNF_OP_RELU: E.unary(v[0], M_RELU); break;
      case DNNF_OP_CLIP: E.unary(v[0], M_CLIP, S_CONST, (uint8_t)E.cst2((float)op.at.lo, (float)op.at.hi)); break;
      case DNNF_OP_POW:
        if (op.at.p == 2.0) E.unary(v[0], M_SQUARE);
        else if (op.at.p == 0.5) E.unary(v[0], M_SQRT);
        else if (op.at.p == -1.0) E.unary(v[0], M_RECIP);
        else E.unary(v[0], M_POW, S_CONST, (uint8_t)E.cst((float)op.at.p));
        break;
      case DNNF_OP_GELU: E.unary(v[0], op.at.approx ? M_GELU_TANH : M_GELU_ERF); break;
      case DNNF_OP_SCALESHIFT: {
        E.load_acc(v[0]); E.protect_operand_in_acc(v[0], 1);
        uint8_t s, i;
        if (!E.src_of(v[1], s, i)) break; E.push(M_MUL, s, i);
        if (!E.src_of(v[2], s, i)) break; E.push(M_ADD, s, i);
        E.consume(v[0]);
        break;
      }
      case DNNF_OP_WHERE: E.select(v[0], v[1], v[2]); break;
      case DNNF_OP_CAST:
        if (op.at.to == DNNF_CAST_BF16) E.unary(v[0], M_BF16R);
        else if (op.at.to == DNNF_CAST_I32) E.unary(v[0], M_TRUNC);
        else if (op.at.to == DNNF_CAST_BOOL) { E.unary(v[0], M_NOT); E.push(M_NOT); }
        else { E.load_acc(v[0]); E.protect_operand_in_acc(v[0], 1); E.consume(v[0]); }
        break;
      case DNNF_OP_CUMSUM: E.unary(v[0], (uint8_t)(M_ROWSCAN + (op.at.exclusive ? 1 : 0) + (op.at.reverse ? 2 : 0))); break;
      case DNNF_OP_SOFTMAX: {
        E.load_acc(v[0]); E.protect_operand_in_acc(v[0], 1);
        int t = E.alloc_tmp(); if (E.fail) break;
        E.push(M_SAVE, S_TMP, (uint8_t)t); E.push(M_ROWMAX); E.push(M_RSUB, S_TMP, (uint8_t)t); E.push(M_EXP);
        E.push(M_SAVE, S_TMP, (uint8_t)t); E.push(M_ROWSUM); E.push(M_RECIP); E.push(M_MUL, S_TMP, (uint8_t)t);
        E.tmp_busy[t] = false;
        E.consume(v[0]);
        break;
      }
      case DNNF_OP_LAYERNORM: {
        E.load_acc(v[0]); E.protect_operand_in_acc(v[0], 1);
        int t = E.alloc_tmp(); if (E.fail) break;
        // two-pass statistics on the register-resident row: mean, then mean of squared deviations
        E.push(M_SAVE, S_TMP, (uint8_t)t); E.push(M_ROWMEAN); E.push(M_RSUB, S_TMP, (uint8_t)t);
        E.push(M_SAVE, S_TMP, (uint8_t)t); E.push(M_SQUARE); E.push(M_ROWMEAN);
        E.push(M_ADD, S_CONST, (uint8_t)E.cst((float)op.at.eps)); E.push(M_SQRT); E.push(M_RECIP); E.push(M_MUL, S_TMP, (uint8_t)t);
        E.tmp_busy[t] = false;
        if (v.size() >= 3) {
          uint8_t s, i;
          if (!E.src_of(v[1], s, i)) break; E.push(M_MUL, s, i);
          if (!E.src_of(v[2], s, i)) break; E.push(M_ADD, s, i);
        }
        E.consume(v[0]);
        break;
      }
      case DNNF_OP_REDUCESUM: E.unary(v[0], M_ROWSUM); break;
      case DNNF_OP_REDUCEMEAN: E.unary(v[0], M_ROWMEAN); break;
      case DNNF_OP_REDUCEMAX: E.unary(v[0], M_ROWMAX); break;
      case DNNF_OP_REDUCEPROD: E.unary(v[0], M_ROWPROD); break;
      default:
        cx.why = std::string("no device code for ") + op_name(op.kind);
        return false;
    }
    if (E.fail) return false;
    E.produced(op.out[0]);
    if (E.fail) return false;
  }
  if (E.fail) return false;
  if (cx.prog.n == 0) { cx.why = "empty program"; return false; }
  // Number the external inputs in the order the program first reads them: the same chain then gives the same
  // program whatever order its operators were declared in, and finds its compile-time table.
  {
    const int n_in = (int)cx.ins.size();
    std::vector<int> map(n_in, -1);
    int next = 0;
    for (int i = 0; i < cx.prog.n; ++i) {
      const MicroOp& m = cx.prog.ops[i];
      if (m.src == S_IN && m.idx < n_in && map[m.idx] < 0) map[m.idx] = next++;
    }
    for (int k = 0; k < n_in; ++k) if (map[k] < 0) map[k] = next++;
    std::vector<ExtArg> ins(n_in);
    for (int k = 0; k < n_in; ++k) ins[map[k]] = cx.ins[k];
    cx.ins.swap(ins);
    for (int i = 0; i < cx.prog.n; ++i) if (cx.prog.ops[i].src == S_IN && cx.prog.ops[i].idx < n_in) cx.prog.ops[i].idx = (uint8_t)map[cx.prog.ops[i].idx];
  }
  return true;
}

// ---------------------------------------------------------------------------
// Packaging into kernel parameters
// ---------------------------------------------------------------------------
namespace {

struct Packed {
  std::vector<int64_t> ext;
  std::vector<std::vector<int64_t>> coefs;   // per arg (ins then outs)
};

// Drop extent-1 dims and merge adjacent dims that every argument walks contiguously.
void collapse(Packed& p) {
  size_t na = p.coefs.size();
  for (int d = (int)p.ext.size() - 1; d >= 0; --d) {
    if (p.ext[d] == 1 && p.ext.size() > 1) {
      p.ext.erase(p.ext.begin() + d);
      for (auto& c : p.coefs) c.erase(c.begin() + d);
    }
  }
  bool changed = true;
  while (changed) {
    changed = false;
    for (size_t d = 0; d + 1 < p.ext.size(); ++d) {
      bool ok = true;
      for (size_t a = 0; a < na; ++a) if (p.coefs[a][d] != p.coefs[a][d + 1] * p.ext[d + 1]) { ok = false; break; }
      if (!ok) continue;
      p.ext[d + 1] *= p.ext[d];
      p.ext.erase(p.ext.begin() + d);
      for (auto& c : p.coefs) c.erase(c.begin() + d);
      changed = true;
      break;
    }
  }
}

bool fill_arg(TensorArg& a, const Graph& g, const ExtArg& e, const std::vector<int64_t>& coef) {
  a.ptr = nullptr;
  if (g.tensors[e.tensor].numel() >= (1ll << 31)) return false;
  a.base = (int32_t)e.view.c0;
  for (int d = 0; d < kMaxDims; ++d) a.stride[d] = d < (int)coef.size() ? (int32_t)coef[d] : 0;
  a.dtype = g.tensors[e.tensor].dtype;
  a.mode = 0;
  return true;
}

}  // namespace

static int lower_elementwise_or_row(const Graph& g, const std::vector<int>& ops, int anchor, Block& out, std::string& why) {
  LowerCtx cx(g);
  cx.ops = ops;
  for (int o : ops) cx.in_block.insert(o);

  int ref = -1;
  if (anchor >= 0) {
    const Op& A = g.ops[anchor];
    ref = A.in[0];                         // the rows being reduced define the iteration space
  } else {
    for (int oid : ops) {
      for (int t : g.ops[oid].out) {
        const Tensor& T = g.tensors[t];
        bool outside = T.is_output;
        for (int c : T.consumers) if (!cx.in_block.count(c)) outside = true;
        if (outside) ref = t;              // the last one in topological order wins
      }
    }
    for (int oid : ops) if (g.ops[oid].kind == DNNF_OP_CONCATPART) ref = g.ops[oid].in[0];   // the part, not the whole result
  }
  if (ref < 0) { why = "block has no output"; return DNNF_ERR_UNSUPPORTED_OP; }
  cx.ext = g.tensors[ref].dims;
  if (cx.ext.empty()) cx.ext.push_back(1);
  const int64_t row_len = cx.ext.back();
  if (!derive_views(cx, ref, {})) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }
  // Aligning the views may split iteration dims (a Reshape across a Slice, say).  The reduced axis has to stay one
  // dim: the row kernels reduce over the innermost dim only.
  if (anchor >= 0 && cx.ext.back() != row_len) { why = "the reduced axis is not a single run of elements in every operand"; return DNNF_ERR_UNSUPPORTED_OP; }
  if (!emit_program(cx, -1, anchor >= 0 ? 2 : kMaxTmp)) { why = cx.why; return DNNF_ERR_UNSUPPORTED_OP; }

  Packed p;
  p.ext = cx.ext;
  for (auto& a : cx.ins) p.coefs.push_back(a.view.coef);
  for (auto& a : cx.outs) p.coefs.push_back(a.view.coef);
  int64_t L = 0;
  if (anchor >= 0) {
    // keep the row dim separate: collapse only the outer dims
    L = p.ext.back();
    Packed q; q.ext.assign(p.ext.begin(), p.ext.end() - 1);
    if (q.ext.empty()) q.ext.push_back(1);
    for (auto& c : p.coefs) { q.coefs.emplace_back(c.begin(), c.begin() + (long)q.ext.size()); if (p.ext.size() == 1) q.coefs.back().assign(1, 0); }
    std::vector<int64_t> inner;
    for (auto& c : p.coefs) inner.push_back(c.back());
    collapse(q);
    p.ext = q.ext; p.ext.push_back(L);
    for (size_t a = 0; a < p.coefs.size(); ++a) { p.coefs[a] = q.coefs[a]; p.coefs[a].push_back(inner[a]); }
  } else {
    collapse(p);
  }
  if ((int)p.ext.size() > kMaxDims) { why = "iteration space rank too high"; return DNNF_ERR_UNSUPPORTED_OP; }
  for (auto e : p.ext) if (e > 0x7fffffffLL) { why = "dimension too large"; return DNNF_ERR_UNSUPPORTED_OP; }

  Launch& L_ = out.launch;
  L_ = Launch{};
  out.inputs.clear(); out.outputs.clear();
  for (auto& a : cx.ins) { L_.in_tensors.push_back(a.tensor); if (std::find(out.inputs.begin(), out.inputs.end(), a.tensor) == out.inputs.end()) out.inputs.push_back(a.tensor); }
  for (auto& a : cx.outs) { L_.out_tensors.push_back(a.tensor); out.outputs.push_back(a.tensor); }
  int nd = (int)p.ext.size();
  int n_in = (int)cx.ins.size(), n_out = (int)cx.outs.size();
  int64_t total = 1;
  for (auto e : p.ext) total *= e;

  auto vec_ok = [&](const TensorArg& a, int inner, bool is_out) {
    // vector access needs unit (or, for inputs, zero) inner stride and 4-element-aligned everything else
    if (a.stride[inner] == 0 && !is_out) return true;
    if (a.stride[inner] != 1) return false;
    if (a.base % 4) return false;
    for (int d = 0; d < nd; ++d) if (d != inner && a.stride[d] % 4) return false;
    return true;
  };

  if (anchor >= 0) {
    RowParams& rp = L_.row;
    rp.it.ndim = nd;
    for (int d = 0; d < nd; ++d) rp.it.extent[d] = (uint32_t)p.ext[d];
    rp.n_in = n_in; rp.n_out = n_out;
    bool fits = true;
    for (int i = 0; i < n_in; ++i) fits &= fill_arg(rp.in[i], g, cx.ins[i], p.coefs[i]);
    for (int i = 0; i < n_out; ++i) fits &= fill_arg(rp.out[i], g, cx.outs[i], p.coefs[n_in + i]);
    if (!fits) { why = "tensor with 2^31 or more elements"; return DNNF_ERR_UNSUPPORTED_OP; }
    rp.prog = cx.prog;
    rp.L = (int)L; rp.rows = total / L;
    int inner = nd - 1;
    bool v4 = (L % 4 == 0);
    for (int i = 0; i < n_in; ++i) {
      if (rp.in[i].stride[inner] != 0 && rp.in[i].stride[inner] != 1) { why = "row block input is not contiguous along the row"; return DNNF_ERR_UNSUPPORTED_OP; }
      if (!vec_ok(rp.in[i], inner, false)) v4 = false;
    }
    for (int i = 0; i < n_out; ++i) {
      if (rp.out[i].stride[inner] != 0 && rp.out[i].stride[inner] != 1) { why = "row block output is not contiguous along the row"; return DNNF_ERR_UNSUPPORTED_OP; }
      if (rp.out[i].stride[inner] == 1 && !vec_ok(rp.out[i], inner, true)) v4 = false;
    }
    rp.vec = v4 ? 4 : 1;
    if (L > 8192) { why = "row longer than a CTA's registers hold"; return DNNF_ERR_UNSUPPORTED_OP; }
    L_.family = DNNF_FAMILY_ROW;
    if (!finalize_row(L_)) { why = "row length has no kernel variant"; return DNNF_ERR_UNSUPPORTED_OP; }
    out.lowered = true;
    return DNNF_OK;
  }

  EwParams& ep = L_.ew;
  ep.it.ndim = nd;
  for (int d = 0; d < nd; ++d) ep.it.extent[d] = (uint32_t)p.ext[d];
  ep.n_in = n_in; ep.n_out = n_out;
  bool fits = true;
  for (int i = 0; i < n_in; ++i) fits &= fill_arg(ep.in[i], g, cx.ins[i], p.coefs[i]);
  for (int i = 0; i < n_out; ++i) fits &= fill_arg(ep.out[i], g, cx.outs[i], p.coefs[n_in + i]);
  if (!fits) { why = "tensor with 2^31 or more elements"; return DNNF_ERR_UNSUPPORTED_OP; }
  ep.prog = cx.prog;
  ep.total = total;
  int inner = nd - 1;
  // A pure Reorganize block whose output walks its input in the same flat order is a zero-copy alias.
  if ((cx.prog.flags & kProgPureMove) && n_in == 1 && n_out == 1 && nd == 1 && ep.in[0].stride[0] == 1 && ep.out[0].stride[0] == 1 &&
      ep.in[0].base == 0 && ep.out[0].base == 0 && !g.tensors[cx.outs[0].tensor].is_output &&
      g.tensors[cx.ins[0].tensor].numel() == g.tensors[cx.outs[0].tensor].numel() &&
      g.tensors[cx.ins[0].tensor].dtype == g.tensors[cx.outs[0].tensor].dtype) {
    L_.family = DNNF_FAMILY_ALIAS;
    out.lowered = true;
    return DNNF_OK;
  }
  // Inputs that run contiguously along another iteration dim are staged through shared memory.
  int tdim = -1, n_staged = 0;
  bool gather = false;
  for (int i = 0; i < n_in; ++i) {
    int64_t s = ep.in[i].stride[inner];
    if (s == 0 || s == 1) continue;
    int td = -1;
    for (int d = 0; d < nd - 1; ++d) if (ep.in[i].stride[d] == 1) td = d;
    if (td < 0) { ep.in[i].mode = 2; gather = true; continue; }    // strided everywhere: element-wise gather
    if (tdim >= 0 && td != tdim) { ep.in[i].mode = 2; gather = true; continue; }
    tdim = td; ep.in[i].mode = 1; n_staged++;
  }
  if (n_staged > 2) {
    int kept = 0;
    for (int i = 0; i < n_in; ++i) if (ep.in[i].mode == 1 && ++kept > 2) { ep.in[i].mode = 2; gather = true; }
    n_staged = 2;
  }
  for (int i = 0; i < n_out; ++i) if (ep.out[i].stride[inner] != 1) { ep.out[i].mode = 2; gather = true; }
  (void)gather;
  bool v4 = (p.ext[inner] % 4 == 0);
  for (int i = 0; i < n_in; ++i) if (ep.in[i].mode == 0 && !vec_ok(ep.in[i], inner, false)) v4 = false;
  for (int i = 0; i < n_out; ++i) if (ep.out[i].mode == 0 && !vec_ok(ep.out[i], inner, true)) v4 = false;
  ep.vec = v4 ? 4 : 1;
  ep.tdim = tdim;
  L_.family = n_staged > 0 ? DNNF_FAMILY_TRANSPOSE : DNNF_FAMILY_ELEMENTWISE;
  if (total >= (1ll << 31)) { why = "more than 2^31 elements in one block"; return DNNF_ERR_UNSUPPORTED_OP; }
  finalize_ew(L_);
  out.lowered = true;
  return DNNF_OK;
}

const Program* program_of(const Launch& L) {
  if (L.family == DNNF_FAMILY_ALIAS) return nullptr;
  if (L.family == DNNF_FAMILY_ROW) return &L.row.prog;
  return &L.ew.prog;     // contraction families keep their epilogue program here too
}

int lower_block(const Graph& g, const std::vector<int>& ops_in, uint32_t flags, Block& out, std::string& why) {
  tl_plan_flags = flags;
  // topological order inside the block
  std::vector<int> ops = ops_in;
  {
    auto order = g.topo_order();
    std::map<int, int> pos;
    for (size_t i = 0; i < order.size(); ++i) pos[order[i]] = (int)i;
    std::sort(ops.begin(), ops.end(), [&](int a, int b) { return pos[a] < pos[b]; });
  }
  out.ops = ops;
  int n_anchor = 0, anchor = -1;
  for (int o : ops) {
    int k = g.ops[o].kind;
    if (is_row_anchor(k) || is_contraction(k)) { n_anchor++; anchor = o; }
    if (k == DNNF_OP_BITSHIFT) { why = "BitShift has no device code"; return DNNF_ERR_UNSUPPORTED_OP; }
  }
  if (n_anchor == 3 && (flags & DNNF_PLAN_BEYOND_TABLE3)) {
    out.mapping = DNNF_MANY_TO_MANY;
    bool conv = false;
    for (int o : ops) if (g.ops[o].kind == DNNF_OP_DWCONV3X3) conv = true;
    return conv ? lower_mbconv(g, ops, flags, out, why) : lower_attention(g, ops, flags, out, why);
  }
  if (n_anchor > 1) { why = "more than one Many-to-Many operator in a block"; return DNNF_ERR_UNSUPPORTED_OP; }
  // A ConcatPart ends its block: it stores the block's values into its range of the Concat's result.  The
  // operators that read the whole result, and the one that produced the result so far, run in other blocks.
  {
    int parts = 0;
    for (int o : ops) {
      const Op& P = g.ops[o];
      if (P.kind != DNNF_OP_CONCATPART) continue;
      if (++parts > 1) { why = "two parts of a Concat in one block"; return DNNF_ERR_UNSUPPORTED_OP; }
      for (int c : g.tensors[P.out[0]].consumers) if (std::find(ops.begin(), ops.end(), c) != ops.end()) { why = "a Concat's result is complete only after its last part's block"; return DNNF_ERR_UNSUPPORTED_OP; }
      if (P.in.size() > 1) { int pp = g.tensors[P.in[1]].producer; if (pp >= 0 && std::find(ops.begin(), ops.end(), pp) != ops.end()) { why = "two parts of a Concat in one block"; return DNNF_ERR_UNSUPPORTED_OP; } }
    }
  }
  // fused mapping type of the block: fold Table 3 along the topological order
  int m = g.ops[ops[0]].mapping;
  for (size_t i = 1; i < ops.size(); ++i) { int f, c; table3(m, g.ops[ops[i]].mapping, &f, &c); m = f; }
  out.mapping = m;
  if (anchor >= 0 && is_contraction(g.ops[anchor].kind)) return lower_contraction(g, ops, flags, anchor, out, why);
  return lower_elementwise_or_row(g, ops, anchor, out, why);
}

}  // namespace dnnf

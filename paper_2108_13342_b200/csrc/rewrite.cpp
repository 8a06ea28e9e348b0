// Mathematical-property graph rewriting (Section 4.2, Table 4).
//
// The pass works on the ECG before planning.  Operators with none of the
// associative / commutative / distributive properties are partition points; the
// rules below only ever touch property-bearing operators, so a match never crosses
// a partition.  Each round collects every match in the graph, applies the one with
// the largest #FLOPS reduction (ties: lowest operator id) and repeats until no rule
// reduces #FLOPS any more -- the greedy scheme of Section 4.2.  Rules whose #FLOPS are
// unchanged but which load an operand once instead of twice (Table 4, footnote) are
// applied once per site.
//
// #FLOPS model (the one that reproduces every count printed in Table 4): an
// element-wise operator costs its number of output elements, a reduction over the
// innermost axis its number of input elements, index-only operators nothing.
//
// Only the ten rules printed in Table 4 exist here (the paper states 149 but prints
// ten), plus common-subexpression merging, Pow(x,2)/Pow(x,0.5) strength reduction and,
// behind a flag, the folding of the 9-operator LayerNorm expansion.
#include <algorithm>
#include <cstring>
#include <functional>
#include <map>
#include <set>

#include "ir.h"

namespace dnnf {

namespace {

enum Rule { R_ASSOC_RECIP = 0, R_ASSOC_SQRT, R_ASSOC_ABS, R_ASSOC_SQUARE, R_DIST_FACTOR, R_DIST_A_PLUS_AB, R_DIST_SQUARE_MINUS,
            R_COMM_SWAP, R_COMM_SUM_SHIFT, R_COMM_PROD_EXP, R_STRENGTH_POW, R_FOLD_CONST, R_CANON_LN, R__COUNT };

int64_t op_flops(const Graph& g, const Op& o) {
  if (!o.alive) return 0;
  if (is_index_only(o.kind)) return 0;
  if (o.kind >= DNNF_OP_REDUCESUM && o.kind <= DNNF_OP_REDUCEPROD) return g.tensors[o.in[0]].numel();
  if (o.kind == DNNF_OP_SOFTMAX) return 5 * g.tensors[o.in[0]].numel();
  if (o.kind == DNNF_OP_LAYERNORM || o.kind == DNNF_OP_INSTANCENORM) return 7 * g.tensors[o.in[0]].numel();
  if (o.kind == DNNF_OP_MATMUL) { const Tensor& a = g.tensors[o.in[0]]; return 2 * g.tensors[o.out[0]].numel() * a.dims.back(); }
  if (o.kind == DNNF_OP_CONV1X1) return 2 * g.tensors[o.out[0]].numel() * g.tensors[o.in[1]].dims[0];
  if (o.kind == DNNF_OP_DWCONV3X3) return 18 * g.tensors[o.out[0]].numel();
  if (o.kind == DNNF_OP_COL2IM) return g.tensors[o.in[0]].numel();
  if (o.kind == DNNF_OP_SCALESHIFT) return 2 * g.tensors[o.out[0]].numel();
  return g.tensors[o.out[0]].numel();
}

struct Rewriter {
  Graph& g;
  dnnf_rewrite_stats st{};
  std::set<std::pair<int, int>> zero_gain_done;      // (rule, root tensor)

  explicit Rewriter(Graph& gg) : g(gg) {}

  const Op* producer(int t) const { int p = g.tensors[t].producer; return (p >= 0 && g.ops[p].alive) ? &g.ops[p] : nullptr; }
  int uses(int t) const { return (int)g.tensors[t].consumers.size() + (g.tensors[t].is_output ? 1 : 0); }
  bool is(int t, int kind) const { const Op* p = producer(t); return p && p->kind == kind; }

  // Append an operator; if `reuse_out` >= 0 the operator writes that existing tensor
  // (so the ids the caller holds for outputs / later operators stay valid).
  int add_op(int kind, std::vector<int> in, const Attrs& at = Attrs{}, int reuse_out = -1) {
    Op o; o.id = (int)g.ops.size(); o.kind = kind; o.in = std::move(in); o.at = at; o.source_id = g.n_source_ops++;
    std::string err;
    size_t nt = g.tensors.size();
    if (infer_shapes(g, o, err) != DNNF_OK) { g.tensors.resize(nt); return -1; }
    if (reuse_out >= 0) {
      if (g.tensors[o.out[0]].dims != g.tensors[reuse_out].dims) { g.tensors.resize(nt); return -1; }
      g.tensors.resize(nt);
      o.out[0] = reuse_out;
      int old = g.tensors[reuse_out].producer;
      if (old >= 0) g.ops[old].alive = false;
      g.tensors[reuse_out].producer = o.id;
    }
    o.mapping = node_mapping(g, o);
    o.props = math_props(kind);
    g.ops.push_back(o);
    return o.out[0];
  }

  void dce() {
    bool changed = true;
    while (changed) {
      changed = false;
      g.relink();
      for (auto& o : g.ops) {
        if (!o.alive) continue;
        bool used = false;
        for (int t : o.out) if (g.tensors[t].is_output || !g.tensors[t].consumers.empty()) used = true;
        if (!used) { o.alive = false; changed = true; }
      }
    }
    g.relink();
  }

  int64_t flops() const { int64_t f = 0; for (auto& o : g.ops) f += op_flops(g, o); return f; }

  // ---- common subexpressions: identical operators on identical inputs are one node ------------
  bool cse() {
    bool any = false;
    std::map<std::string, int> seen;
    for (int oid : g.topo_order()) {
      Op& o = g.ops[oid];
      if (o.out.size() != 1 || g.tensors[o.out[0]].is_output) continue;
      if (o.kind == DNNF_OP_CONCATPART) continue;      // a part extends its Concat's result in place: not a value of its own
      std::string key = std::to_string(o.kind) + ":";
      std::vector<int> ins = o.in;
      if ((o.kind == DNNF_OP_ADD || o.kind == DNNF_OP_MUL) && ins.size() == 2 && ins[0] > ins[1]) std::swap(ins[0], ins[1]);
      for (int t : ins) key += std::to_string(t) + ",";
      char buf[160];
      snprintf(buf, sizeof buf, "|%a|%a|%a|%a|%a|%lld|%lld|%lld|%lld|%lld|%lld", o.at.c, o.at.lo, o.at.hi, o.at.p, o.at.eps, (long long)o.at.approx,
               (long long)o.at.axis, (long long)o.at.keepdims, (long long)o.at.start, (long long)o.at.end, (long long)o.at.bits);
      key += buf;
      snprintf(buf, sizeof buf, "|%lld|%lld|%lld|%lld|%lld", (long long)o.at.block, (long long)o.at.scale, (long long)o.at.kernel,
               (long long)o.at.stride, (long long)o.at.pad);
      key += buf;
      snprintf(buf, sizeof buf, "|%lld|%lld|%lld", (long long)o.at.to, (long long)o.at.exclusive, (long long)o.at.reverse);
      key += buf;
      for (auto v : o.at.perm) key += "p" + std::to_string(v);
      for (auto v : o.at.shape) key += "s" + std::to_string(v);
      for (auto v : o.at.axes) key += "a" + std::to_string(v);
      auto it = seen.find(key);
      if (it == seen.end()) { seen[key] = o.out[0]; continue; }
      // redirect consumers of the duplicate to the first occurrence
      int keep = it->second, dup = o.out[0];
      for (auto& c : g.ops) if (c.alive) for (int& t : c.in) if (t == dup) t = keep;
      o.alive = false;
      any = true;
      g.relink();
    }
    return any;
  }

  // ---- layout selection (Section 4.4.2, "inter-block optimization") -----------------------------
  // The operators whose speed depends on the data layout -- convolutions, pools, GEMMs, Softmax and the
  // other last-axis operators -- exist here in one layout each, so a graph written in another layout
  // (a channels-first network) reaches them through Transposes: those Transposes state the layout the
  // dominant operator of the coming block wants.  Element-wise operators and batch normalisation are
  // indifferent to layout, so they take the dominant operator's: a Transpose is moved from the output
  // of such an operator to its operands (f(x)^T = f(x^T), a per-channel operand follows its axis),
  // and moved again, until it meets the Transpose that brought the tensor into the other layout; the
  // two compose, to nothing when they are inverses.  What remains are Transposes of graph inputs and
  // outputs.  The pass is kept only if the graph has fewer Transposes and no more #FLOPS than before.
  static std::vector<int64_t> compose_perm(const std::vector<int64_t>& first, const std::vector<int64_t>& then) {
    std::vector<int64_t> r(then.size());
    for (size_t i = 0; i < then.size(); ++i) r[i] = first[then[i]];
    return r;
  }
  static bool identity_perm(const std::vector<int64_t>& p) {
    for (size_t i = 0; i < p.size(); ++i) if (p[i] != (int64_t)i) return false;
    return true;
  }
  bool layout_indifferent(const Op& o) const {
    if (!is_elementwise(o.kind) || o.out.size() != 1) return false;
    return true;
  }
  // Can a Transpose by `perm` of tensor t be expressed without a new data movement?
  bool transposable(int t, const std::vector<int64_t>& perm, int out_numel, std::map<int, bool>& memo, int depth = 0) {
    auto it = memo.find(t);
    if (it != memo.end()) return it->second;
    bool ok = false;
    const Tensor& T = g.tensors[t];
    const Op* p = producer(t);
    if (T.dims.size() != perm.size()) ok = false;
    else if (p && p->kind == DNNF_OP_TRANSPOSE) ok = true;
    else if (T.numel() < out_numel && !p) ok = true;               // a broadcast constant: permuting it costs no pass over the data
    else if (p && layout_indifferent(*p) && depth < 64) {
      ok = true;
      for (size_t i = 0; i < p->in.size() && ok; ++i) {
        if (p->kind == DNNF_OP_SCALESHIFT && i > 0) continue;
        const Tensor& a = g.tensors[p->in[i]];
        if (a.numel() == 1) continue;
        ok = transposable(p->in[i], perm, out_numel, memo, depth + 1);
      }
    } else {
      // some other consumer already reads this tensor through the same Transpose
      for (int c : T.consumers) if (g.ops[c].alive && g.ops[c].kind == DNNF_OP_TRANSPOSE && g.ops[c].at.perm == perm) ok = true;
      if (ok && depth == 0) ok = false;
    }
    memo[t] = ok;
    return ok;
  }
  // Transposes of feature maps; one of a (broadcast) weight moves no data worth counting
  int count_transposes() const {
    int n = 0;
    for (auto& o : g.ops) if (o.alive && o.kind == DNNF_OP_TRANSPOSE && !g.tensors[o.in[0]].weight) n++;
    return n;
  }

  int crossings = 0;      // Transposes moved across a layout-indifferent operator
  bool move_transposes_once() {
    g.relink();
    for (int oid : g.topo_order()) {
      const Op T = g.ops[oid];
      if (!T.alive || T.kind != DNNF_OP_TRANSPOSE) continue;
      const int x = T.in[0], y = T.out[0];
      const Op* P = producer(x);
      if (!P) continue;
      if (P->kind == DNNF_OP_TRANSPOSE) {
        std::vector<int64_t> r = compose_perm(P->at.perm, T.at.perm);
        const int src = P->in[0];
        if (identity_perm(r)) {
          if (g.tensors[y].is_output) continue;
          for (auto& c : g.ops) if (c.alive) for (int& t : c.in) if (t == y) t = src;
          g.ops[oid].alive = false;
        } else {
          Attrs at; at.perm = r;
          if (add_op(DNNF_OP_TRANSPOSE, {src}, at, y) < 0) continue;
        }
        return true;
      }
      if (!layout_indifferent(*P)) continue;
      std::map<int, bool> memo;
      const int out_numel = (int)std::min<int64_t>(g.tensors[x].numel(), INT32_MAX);
      if (!transposable(x, T.at.perm, out_numel, memo)) continue;
      const Op Pc = *P;
      std::vector<int> ins;
      bool ok = true;
      for (size_t i = 0; i < Pc.in.size() && ok; ++i) {
        const Tensor& a = g.tensors[Pc.in[i]];
        if ((Pc.kind == DNNF_OP_SCALESHIFT && i > 0) || a.numel() == 1) { ins.push_back(Pc.in[i]); continue; }
        Attrs at; at.perm = T.at.perm;
        int t = add_op(DNNF_OP_TRANSPOSE, {Pc.in[i]}, at);
        if (t < 0) ok = false;
        ins.push_back(t);
      }
      if (!ok) continue;
      Attrs at = Pc.at;
      if (Pc.kind == DNNF_OP_SCALESHIFT) {
        const int64_t rank = (int64_t)T.at.perm.size();
        const int64_t axis = Pc.at.axis < 0 ? Pc.at.axis + rank : Pc.at.axis;
        for (int64_t i = 0; i < rank; ++i) if (T.at.perm[i] == axis) at.axis = i;
      }
      if (add_op(Pc.kind, ins, at, y) < 0) continue;
      ++crossings;
      return true;
    }
    return false;
  }

  void select_layouts() {
    if (count_transposes() < 2) return;
    Graph saved = g;
    const int n_before = count_transposes();
    const int64_t f_before = flops();
    int moves = 0;
    crossings = 0;
    while (moves < 100000 && move_transposes_once()) { ++moves; }
    while (cse()) {}
    dce();
    const int n_after = count_transposes();
    // Back-to-back Transposes alone (the head split followed by K^T in attention) are left as the graph has them:
    // they already share a block and compose there as index maps.
    if (crossings == 0 || n_after >= n_before || flops() > f_before) { g = saved; g.relink(); return; }
    st.layout_transposes_removed = n_before - n_after;
  }

  // ---- product trees: flatten, simplify the multiset of factors, rebuild -----------------------
  void collect_factors(int t, int root, std::vector<int>& leaves, std::vector<int>& inner) {
    const Op* p = producer(t);
    if (p && p->kind == DNNF_OP_MUL && (t == root || uses(t) == 1)) {
      inner.push_back(p->id);
      collect_factors(p->in[0], root, leaves, inner);
      collect_factors(p->in[1], root, leaves, inner);
    } else {
      leaves.push_back(t);
    }
  }

  struct Candidate { int rule; int root_op; int64_t gain; std::function<bool()> apply; };

  // Returns the factor list after one simplification step, or empty if none applies.
  bool simplify_factors(std::vector<int>& f, int& rule, std::vector<std::function<int()>>& make) {
    // two Sqrt of the same tensor -> that tensor                          (Table 4, Associative row 2)
    // (a negative entry stands for a node that an earlier step of this simplification will create)
    for (size_t i = 0; i < f.size(); ++i) for (size_t j = i + 1; j < f.size(); ++j) {
      if (f[i] < 0 || f[j] < 0) continue;
      const Op *a = producer(f[i]), *b = producer(f[j]);
      if (a && b && a->kind == DNNF_OP_SQRT && b->kind == DNNF_OP_SQRT && a->in[0] == b->in[0] && uses(f[i]) <= (f[i] == f[j] ? 2 : 1) && uses(f[j]) <= (f[i] == f[j] ? 2 : 1)) {
        int x = a->in[0];
        f.erase(f.begin() + j); f.erase(f.begin() + i); f.push_back(x);
        rule = R_ASSOC_SQRT;
        return true;
      }
    }
    // the same factor twice -> Square(factor)                               (row 4)
    for (size_t i = 0; i < f.size(); ++i) for (size_t j = i + 1; j < f.size(); ++j) {
      if (f[i] >= 0 && f[i] == f[j] && !g.tensors[f[i]].external) {
        int x = f[i];
        f.erase(f.begin() + j); f.erase(f.begin() + i);
        f.push_back(-(int)make.size() - 1);
        make.push_back([this, x]() { return add_op(DNNF_OP_SQUARE, {x}); });
        rule = R_ASSOC_SQUARE;
        return true;
      }
    }
    // Abs(X) and Abs(Y) -> Abs(X * Y)                                       (row 3, after a commutative swap)
    for (size_t i = 0; i < f.size(); ++i) for (size_t j = i + 1; j < f.size(); ++j) {
      if (f[i] < 0 || f[j] < 0) continue;
      const Op *a = producer(f[i]), *b = producer(f[j]);
      if (a && b && a->kind == DNNF_OP_ABS && b->kind == DNNF_OP_ABS && uses(f[i]) == 1 && uses(f[j]) == 1 &&
          g.tensors[a->in[0]].dims == g.tensors[b->in[0]].dims) {
        int x = a->in[0], y = b->in[0];
        f.erase(f.begin() + j); f.erase(f.begin() + i);
        f.push_back(-(int)make.size() - 1);
        make.push_back([this, x, y]() { int m = add_op(DNNF_OP_MUL, {x, y}); return m < 0 ? -1 : add_op(DNNF_OP_ABS, {m}); });
        rule = R_ASSOC_ABS;
        return true;
      }
    }
    return false;
  }

  void product_candidates(std::vector<Candidate>& out) {
    for (auto& o : g.ops) {
      if (!o.alive || o.kind != DNNF_OP_MUL) continue;
      // only roots: the product is not itself a single-use factor of another product
      bool is_root = true;
      int t = o.out[0];
      if (uses(t) == 1 && !g.tensors[t].is_output)
        for (int c : g.tensors[t].consumers) if (g.ops[c].kind == DNNF_OP_MUL) is_root = false;
      if (!is_root) continue;
      std::vector<int> leaves, inner;
      collect_factors(t, t, leaves, inner);
      if (leaves.size() < 3) continue;
      int root_op = o.id;
      out.push_back({-1, root_op, 0, [this, t, root_op]() {
        // re-collect (the graph may have changed since the scan) and rewrite in place
        std::vector<int> f, in;
        collect_factors(t, t, f, in);
        std::vector<std::function<int()>> make;
        int rule = -1, applied = 0, last_rule = -1;
        while (simplify_factors(f, rule, make)) { applied++; last_rule = rule; st.applied_by_rule[rule]++; }
        if (!applied) return false;
        // materialise new unary nodes, then rebuild the product smallest factors first
        std::vector<int> made;
        for (auto& m : make) { int r = m(); if (r < 0) return false; made.push_back(r); }
        for (int& x : f) if (x < 0) x = made[-x - 1];
        std::stable_sort(f.begin(), f.end(), [&](int a, int b) { return g.tensors[a].numel() < g.tensors[b].numel(); });
        if (f.size() == 1) return false;       // a bare copy: leave such degenerate products alone
        int acc = f[0];
        for (size_t i = 1; i < f.size(); ++i) {
          acc = add_op(DNNF_OP_MUL, {acc, f[i]}, Attrs{}, i + 1 == f.size() ? t : -1);
          if (acc < 0) return false;
        }
        (void)last_rule; (void)root_op;
        return true;
      }});
    }
  }

  // ---- the remaining printed rules ------------------------------------------------------------
  void local_candidates(std::vector<Candidate>& out, uint32_t flags) {
    for (auto& o : g.ops) {
      if (!o.alive) continue;
      const int t = o.out.empty() ? -1 : o.out[0];
      const int id = o.id;
      if (o.kind == DNNF_OP_POW && (o.at.p == 2.0 || o.at.p == 0.5)) {
        int x = o.in[0]; double p = o.at.p;
        out.push_back({R_STRENGTH_POW, id, 0, [this, t, x, p]() { return add_op(p == 2.0 ? DNNF_OP_SQUARE : DNNF_OP_SQRT, {x}, Attrs{}, t) >= 0; }});
        continue;
      }
      if (o.kind == DNNF_OP_ADD) {
        const Op *a = producer(o.in[0]), *b = producer(o.in[1]);
        // X*F + Y*F -> (X+Y)*F                                              (Distributive row 1; the common factor
        // is the one kept outside the sum -- the row as printed, A.C + A.B -> (A+B).C, is not an identity)
        if (a && b && a != b && a->kind == DNNF_OP_MUL && b->kind == DNNF_OP_MUL && uses(o.in[0]) == 1 && uses(o.in[1]) == 1) {
          for (int i = 0; i < 2; ++i) for (int j = 0; j < 2; ++j) {
            if (a->in[i] != b->in[j]) continue;
            int f = a->in[i], x = a->in[1 - i], y = b->in[1 - j];
            if (g.tensors[x].dims != g.tensors[y].dims) continue;
            int64_t gain = g.tensors[o.in[0]].numel() + g.tensors[o.in[1]].numel() + g.tensors[t].numel() - 2 * g.tensors[t].numel();
            out.push_back({R_DIST_FACTOR, id, gain, [this, t, f, x, y]() {
              int s = add_op(DNNF_OP_ADD, {x, y});
              return s >= 0 && add_op(DNNF_OP_MUL, {s, f}, Attrs{}, t) >= 0;
            }});
            i = j = 2;
          }
        }
        // A + A*B -> A*(B+1)                                                (Distributive row 2: same #FLOPS, A loaded once)
        for (int s = 0; s < 2; ++s) {
          const Op* m = producer(o.in[s]);
          int a_t = o.in[1 - s];
          if (!m || m->kind != DNNF_OP_MUL || uses(o.in[s]) != 1) continue;
          for (int i = 0; i < 2; ++i) {
            if (m->in[i] != a_t) continue;
            int b_t = m->in[1 - i];
            if (g.tensors[b_t].dims != g.tensors[t].dims) continue;
            out.push_back({R_DIST_A_PLUS_AB, id, 0, [this, t, a_t, b_t]() {
              Attrs at; at.c = 1.0;
              int s1 = add_op(DNNF_OP_ADDC, {b_t}, at);
              return s1 >= 0 && add_op(DNNF_OP_MUL, {a_t, s1}, Attrs{}, t) >= 0;
            }});
            break;
          }
        }
      }
      if (o.kind == DNNF_OP_SUB) {
        // Square(S) - S*C -> S*(S - C)                                      (Distributive row 3)
        const Op *a = producer(o.in[0]), *b = producer(o.in[1]);
        if (a && b && a->kind == DNNF_OP_SQUARE && b->kind == DNNF_OP_MUL && uses(o.in[0]) == 1 && uses(o.in[1]) == 1) {
          int s = a->in[0];
          for (int i = 0; i < 2; ++i) {
            if (b->in[i] != s) continue;
            int c = b->in[1 - i];
            int64_t gain = g.tensors[t].numel();
            out.push_back({R_DIST_SQUARE_MINUS, id, gain, [this, t, s, c]() {
              int d = add_op(DNNF_OP_SUB, {s, c});
              return d >= 0 && add_op(DNNF_OP_MUL, {s, d}, Attrs{}, t) >= 0;
            }});
            break;
          }
        }
      }
      if (o.kind == DNNF_OP_MUL) {
        // Recip(A) * Recip(A*B) -> Square(Recip(A)) * Recip(B)              (Associative row 1: same #FLOPS, A loaded once)
        for (int s = 0; s < 2; ++s) {
          const Op *r1 = producer(o.in[s]), *r2 = producer(o.in[1 - s]);
          if (!r1 || !r2 || r1->kind != DNNF_OP_RECIP || r2->kind != DNNF_OP_RECIP || uses(o.in[1 - s]) != 1) continue;
          const Op* m = producer(r2->in[0]);
          if (!m || m->kind != DNNF_OP_MUL || uses(r2->in[0]) != 1) continue;
          int a_t = r1->in[0];
          for (int i = 0; i < 2; ++i) {
            if (m->in[i] != a_t) continue;
            int b_t = m->in[1 - i], ra = o.in[s];
            out.push_back({R_ASSOC_RECIP, id, 0, [this, t, ra, b_t]() {
              int sq = add_op(DNNF_OP_SQUARE, {ra});
              int rb = add_op(DNNF_OP_RECIP, {b_t});
              return sq >= 0 && rb >= 0 && add_op(DNNF_OP_MUL, {sq, rb}, Attrs{}, t) >= 0;
            }});
            break;
          }
          break;
        }
      }
      if (o.kind == DNNF_OP_REDUCESUM) {
        // ReduceSum(BitShift(A)) -> BitShift(ReduceSum(A))                  (Commutative row 2; left shifts only: exact on integers)
        const Op* sh = producer(o.in[0]);
        if (sh && sh->kind == DNNF_OP_BITSHIFT && uses(o.in[0]) == 1) {
          int a_t = sh->in[0]; Attrs red = o.at, sat = sh->at;
          int64_t gain = g.tensors[a_t].numel() - g.tensors[t].numel();
          out.push_back({R_COMM_SUM_SHIFT, id, gain, [this, t, a_t, red, sat]() {
            int r = add_op(DNNF_OP_REDUCESUM, {a_t}, red);
            return r >= 0 && add_op(DNNF_OP_BITSHIFT, {r}, sat, t) >= 0;
          }});
        }
      }
      if (o.kind == DNNF_OP_REDUCEPROD) {
        // ReduceProd(Exp(A)) -> Exp(ReduceSum(A))                           (Commutative row 3)
        const Op* ex = producer(o.in[0]);
        if (ex && ex->kind == DNNF_OP_EXP && uses(o.in[0]) == 1) {
          int a_t = ex->in[0]; Attrs red = o.at;
          int64_t gain = g.tensors[a_t].numel() - g.tensors[t].numel();
          out.push_back({R_COMM_PROD_EXP, id, gain, [this, t, a_t, red]() {
            int r = add_op(DNNF_OP_REDUCESUM, {a_t}, red);
            return r >= 0 && add_op(DNNF_OP_EXP, {r}, Attrs{}, t) >= 0;
          }});
        }
      }
      if ((flags & DNNF_REWRITE_CANON_MACRO) && o.kind == DNNF_OP_ADD) {
        // y = ((x - mean(x)) / sqrt(mean((x - mean(x))^2) + eps)) * gamma + beta  ->  LayerNorm(x, gamma, beta)
        for (int s = 0; s < 2; ++s) {
          const Op* mul = producer(o.in[s]);
          int beta = o.in[1 - s];
          if (!mul || mul->kind != DNNF_OP_MUL || uses(o.in[s]) != 1) continue;
          for (int i = 0; i < 2; ++i) {
            const Op* div = producer(mul->in[i]);
            int gamma = mul->in[1 - i];
            if (!div || div->kind != DNNF_OP_DIV || uses(mul->in[i]) != 1) continue;
            int xc = div->in[0];
            const Op* sub = producer(xc);
            const Op* sq = producer(div->in[1]);
            if (!sub || sub->kind != DNNF_OP_SUB || !sq || sq->kind != DNNF_OP_SQRT || uses(div->in[1]) != 1) continue;
            const Op* addc = producer(sq->in[0]);
            if (!addc || addc->kind != DNNF_OP_ADDC || uses(sq->in[0]) != 1) continue;
            const Op* var = producer(addc->in[0]);
            if (!var || var->kind != DNNF_OP_REDUCEMEAN || !var->at.keepdims || uses(addc->in[0]) != 1) continue;
            const Op* sqr = producer(var->in[0]);
            if (!sqr || !(sqr->kind == DNNF_OP_SQUARE || (sqr->kind == DNNF_OP_POW && sqr->at.p == 2.0)) || sqr->in[0] != xc || uses(var->in[0]) != 1) continue;
            if (uses(xc) != 2) continue;
            int x = sub->in[0];
            const Op* mean = producer(sub->in[1]);
            if (!mean || mean->kind != DNNF_OP_REDUCEMEAN || !mean->at.keepdims || mean->in[0] != x || uses(sub->in[1]) != 1) continue;
            const int hidden = (int)g.tensors[x].dims.back();
            if (g.tensors[gamma].numel() != hidden || g.tensors[beta].numel() != hidden) continue;
            double eps = addc->at.c;
            out.push_back({R_CANON_LN, id, 1, [this, t, x, gamma, beta, eps]() {
              Attrs at; at.axis = -1; at.eps = eps;
              return add_op(DNNF_OP_LAYERNORM, {x, gamma, beta}, at, t) >= 0;
            }});
            i = 2; s = 2;
          }
        }
      }
    }
  }

  int run(uint32_t flags) {
    g.relink();
    st.ops_before = 0;
    for (auto& o : g.ops) if (o.alive) st.ops_before++;
    st.flops_before = flops();
    if (!(flags & DNNF_REWRITE_KEEP_LAYOUT)) select_layouts();
    for (int round = 0; round < 100000; ++round) {
      if (cse()) dce();
      std::vector<Candidate> cands;
      local_candidates(cands, flags);
      product_candidates(cands);
      // evaluate every candidate's true #FLOPS change by trying it on a copy
      int best = -1; int64_t best_gain = 0; bool best_zero = false;
      for (size_t i = 0; i < cands.size(); ++i) {
        Candidate& c = cands[i];
        int root_t = g.ops[c.root_op].out[0];
        bool zero_rule = (c.rule == R_ASSOC_RECIP || c.rule == R_DIST_A_PLUS_AB || c.rule == R_STRENGTH_POW);
        if (zero_rule && zero_gain_done.count({c.rule, root_t})) continue;
        Graph saved = g;
        dnnf_rewrite_stats saved_st = st;
        int64_t before = flops();
        bool ok = c.apply();
        int64_t gain = 0;
        if (ok) { dce(); gain = before - flops(); }
        g = saved; st = saved_st;
        g.relink();
        if (!ok) continue;
        bool take = gain > 0 || (gain == 0 && zero_rule) || c.rule == R_CANON_LN;   // canonicalisation is structural
        if (c.rule == R_CANON_LN) gain = std::max<int64_t>(gain, 1);
        if (!take) continue;
        if (best < 0 || gain > best_gain) { best = (int)i; best_gain = gain; best_zero = zero_rule; }
      }
      if (best < 0) break;
      Candidate& c = cands[best];
      int root_t = g.ops[c.root_op].out[0];
      if (!c.apply()) break;
      if (c.rule >= 0) st.applied_by_rule[c.rule]++;
      if (best_zero) zero_gain_done.insert({c.rule, root_t});
      st.rules_applied++;
      dce();
    }
    st.ops_after = 0;
    for (auto& o : g.ops) if (o.alive) st.ops_after++;
    st.flops_after = flops();
    return DNNF_OK;
  }
};

}  // namespace

int64_t graph_flops(const Graph& g) { int64_t f = 0; for (auto& o : g.ops) f += op_flops(g, o); return f; }

int rewrite_graph(Graph& g, uint32_t flags, dnnf_rewrite_stats* stats) {
  Rewriter R(g);
  std::memset(&R.st, 0, sizeof R.st);
  if (flags & DNNF_REWRITE_NONE) {
    g.relink();
    for (auto& o : g.ops) if (o.alive) R.st.ops_before++;
    R.st.ops_after = R.st.ops_before;
    R.st.flops_before = R.st.flops_after = graph_flops(g);
    if (stats) *stats = R.st;
    return DNNF_OK;
  }
  int rc = R.run(flags);
  if (stats) *stats = R.st;
  return rc;
}

}  // namespace dnnf

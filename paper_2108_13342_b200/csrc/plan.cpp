// Fusion-plan generation (Section 4.3, Listing 1) and plan finalisation.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <map>
#include <set>
#include <string>

#include "gemm_params.h"
#include "ir.h"

namespace dnnf {

namespace {

struct Bits {
  std::vector<uint64_t> w;
  explicit Bits(int n = 0) : w((n + 63) / 64, 0) {}
  void set(int i) { w[i >> 6] |= 1ull << (i & 63); }
  bool get(int i) const { return (w[i >> 6] >> (i & 63)) & 1; }
  void or_with(const Bits& o) { for (size_t i = 0; i < w.size(); ++i) w[i] |= o.w[i]; }
};

struct Planner {
  Graph& g;
  uint32_t flags;
  std::vector<int> order;            // topological
  std::vector<int> pos;              // op id -> topological position
  std::vector<Bits> anc, desc;       // strict ancestors / descendants per op
  std::vector<int> block_of;         // op id -> block index or -1
  std::vector<std::vector<int>> blocks;
  std::vector<int> btype;
  int yellow = 0, yellow_fused = 0;
  bool debug = dev_env("DNNF_DEBUG_PLAN") != nullptr;

  Planner(Graph& gg, uint32_t f) : g(gg), flags(f) {}

  std::vector<int> successors(int o) const {
    std::vector<int> s;
    for (int t : g.ops[o].out) for (int c : g.tensors[t].consumers) if (std::find(s.begin(), s.end(), c) == s.end()) s.push_back(c);
    std::sort(s.begin(), s.end(), [&](int a, int b) { return pos[a] < pos[b]; });
    return s;
  }
  std::vector<int> predecessors(int o) const {
    std::vector<int> s;
    for (int t : g.ops[o].in) { int p = g.tensors[t].producer; if (p >= 0 && g.ops[p].alive && std::find(s.begin(), s.end(), p) == s.end()) s.push_back(p); }
    std::sort(s.begin(), s.end(), [&](int a, int b) { return pos[a] < pos[b]; });
    return s;
  }

  void reachability() {
    int n = (int)g.ops.size();
    anc.assign(n, Bits(n)); desc.assign(n, Bits(n));
    for (int o : order) for (int p : predecessors(o)) { anc[o].or_with(anc[p]); anc[o].set(p); }
    for (auto it = order.rbegin(); it != order.rend(); ++it) for (int s : successors(*it)) { desc[*it].or_with(desc[s]); desc[*it].set(s); }
  }

  // A block must stay convex: no path between two members may leave the block,
  // otherwise the fused kernel would have to run both before and after an
  // outside operator.  (The paper does not spell this legality rule out.)
  bool convex(const std::vector<int>& members) const {
    int n = (int)g.ops.size();
    Bits in(n), a(n), d(n);
    for (int m : members) { in.set(m); a.or_with(anc[m]); d.or_with(desc[m]); }
    for (size_t i = 0; i < a.w.size(); ++i) if (a.w[i] & d.w[i] & ~in.w[i]) return false;
    return true;
  }

  // Convexity looks at one block.  Two convex blocks can still need each other (a1 -> b1 and b2 -> a2 with b1, b2
  // joined only through a common consumer), so the block graph itself has to stay acyclic: starting from the
  // candidate block's successors and walking whole blocks at a time, no path may lead back into the candidate.
  bool no_cycle(const std::vector<int>& members) const {
    const int n = (int)g.ops.size();
    std::vector<char> in(n, 0), seen(n, 0);
    for (int m : members) in[m] = 1;
    std::vector<int> stack;
    auto visit = [&](int o) {
      if (seen[o] || in[o]) return;
      const int b = block_of[o];
      if (b >= 0) { for (int x : blocks[b]) if (!seen[x] && !in[x]) { seen[x] = 1; stack.push_back(x); } }
      if (!seen[o]) { seen[o] = 1; stack.push_back(o); }
    };
    for (int m : members) for (int s : successors(m)) visit(s);
    while (!stack.empty()) {
      int o = stack.back(); stack.pop_back();
      for (int s : successors(o)) {
        if (in[s]) return false;
        visit(s);
      }
    }
    return true;
  }

  // Mapping type of `op` as met along the edge from `from` (Section 3.1 defines
  // types per input/output pair).  With STRICT_TABLE3 the node type is used.
  int type_along(int op, int from_tensor) const {
    const Op& o = g.ops[op];
    if (flags & DNNF_PLAN_STRICT_TABLE3) return o.mapping;
    int best = -1;
    for (size_t s = 0; s < o.in.size(); ++s) if (o.in[s] == from_tensor) { int m = edge_mapping(g, o, (int)s); if (best < 0 || m < best) best = m; }
    return best < 0 ? o.mapping : best;
  }
  // Type of a predecessor as seen from its output: the simplest pair it offers.
  int type_as_pred(int op) const {
    const Op& o = g.ops[op];
    if (flags & DNNF_PLAN_STRICT_TABLE3) return o.mapping;
    int best = o.mapping;
    for (size_t s = 0; s < o.in.size(); ++s) best = std::min(best, edge_mapping(g, o, (int)s));
    return best;
  }
  bool seed_eligible(int op) const {
    const Op& o = g.ops[op];
    if (o.mapping == DNNF_ONE_TO_ONE) return true;
    if (flags & DNNF_PLAN_STRICT_TABLE3) return false;
    return is_elementwise(o.kind) && type_as_pred(op) == DNNF_ONE_TO_ONE;
  }
  int64_t irs_size(int op) const { int64_t b = 0; for (int t : g.ops[op].out) b += g.tensors[t].bytes(); return b; }

  bool lowers(const std::vector<int>& members, Block* out = nullptr) {
    Block tmp; std::string why;
    Block& b = out ? *out : tmp;
    bool ok = lower_block(g, members, flags, b, why) == DNNF_OK;
    if (ok) b.ops = members;
    if (!ok && debug) {
      fprintf(stderr, "[dnnf plan] cannot lower {");
      for (int m : members) fprintf(stderr, " %s#%d", op_name(g.ops[m].kind), m);
      fprintf(stderr, " }: %s\n", why.c_str());
    }
    return ok;
  }

  // Cost of a lowered candidate block: the profiling database's measured latency when it has the block's
  // signature (Section 4.3), else the analytic model -- and the miss is remembered so that it can be measured.
  std::map<std::string, std::vector<int>> misses;
  int hits = 0;
  double cost(const Block& b) {
    if (b.launch.family == DNNF_FAMILY_ALIAS) return 0.0;
    const std::string sig = block_signature(g, b);
    double us;
    if (profile_db_get(sig, &us)) { ++hits; return us; }
    misses.emplace(sig, b.ops);
    return block_cost_us(g, b);
  }

  // Step 2.2: the constraint check.  The paper's "empirically determined
  // threshold" (register pressure etc.) becomes: the merged block must lower
  // to one kernel within the register / argument / program-length budgets.
  bool check_constraint(const std::vector<int>& merged) {
    if (!convex(merged) || !no_cycle(merged)) return false;
    int anchors = 0;
    for (int m : merged) if (g.ops[m].mapping == DNNF_MANY_TO_MANY) anchors++;
    if (anchors > 1) return false;
    if (flags & DNNF_PLAN_ALLOW_PROLOGUE) return true;
    return lowers(merged);
  }

  // Step 2.3 for yellow cells.  The paper looks the combination up in a
  // profiling database; this build uses an analytic stand-in: HBM bytes over
  // bandwidth plus a launch cost per kernel.
  bool profitable(const std::vector<int>& cur, int cand, const std::vector<int>& merged) {
    yellow++;
    if (flags & DNNF_PLAN_ALLOW_PROLOGUE) { yellow_fused++; return true; }
    Block a, b, m;
    if (!lowers(merged, &m)) return false;
    if (!lowers(cur, &a) || !lowers({cand}, &b)) { yellow_fused++; return true; }
    bool ok = cost(m) <= cost(a) + cost(b);
    if (ok) yellow_fused++;
    return ok;
  }

  bool try_add(int bi, int cand, int first_type, int second_type, bool cand_is_second) {
    int fused, colour;
    table3(first_type, second_type, &fused, &colour);
    if (colour == DNNF_FUSE_BREAK) return false;
    std::vector<int> merged = blocks[bi];
    merged.push_back(cand);
    if (!check_constraint(merged)) return false;
    if (colour == DNNF_FUSE_DEPEND && !profitable(blocks[bi], cand, merged)) return false;
    (void)cand_is_second;
    blocks[bi] = merged;
    block_of[cand] = bi;
    btype[bi] = fused;
    return true;
  }

  void fuse_successor(int op, int succ, int bi) {
    if (block_of[succ] >= 0) return;
    int via = -1;
    for (int t : g.ops[op].out) if (std::find(g.ops[succ].in.begin(), g.ops[succ].in.end(), t) != g.ops[succ].in.end()) via = t;
    if (!try_add(bi, succ, btype[bi], type_along(succ, via), true)) return;
    for (int s : successors(succ)) fuse_successor(succ, s, bi);     // Step 2.4
  }
  void fuse_predecessor(int op, int pred, int bi) {
    (void)op;
    if (block_of[pred] >= 0) return;
    if (!try_add(bi, pred, type_as_pred(pred), btype[bi], false)) return;
    for (int p : predecessors(pred)) fuse_predecessor(pred, p, bi);
  }

  void run_listing1() {
    for (;;) {
      // Step 1: One-to-One operator with the smallest intermediate result; ties in graph order.
      int seed = -1;
      for (int o : order) {
        if (block_of[o] >= 0 || !seed_eligible(o)) continue;
        if (seed < 0 || irs_size(o) < irs_size(seed)) seed = o;
      }
      if (seed < 0) break;
      int bi = (int)blocks.size();
      blocks.push_back({seed});
      btype.push_back(flags & DNNF_PLAN_STRICT_TABLE3 ? g.ops[seed].mapping : DNNF_ONE_TO_ONE);
      block_of[seed] = bi;
      for (int s : successors(seed)) fuse_successor(seed, s, bi);       // Step 2
      for (int p : predecessors(seed)) fuse_predecessor(seed, p, bi);   // Step 3
    }
    for (int o : order) if (block_of[o] < 0) { block_of[o] = (int)blocks.size(); blocks.push_back({o}); btype.push_back(g.ops[o].mapping); }
  }

  // Intra-block optimisation of Section 4.4.2: a Reorganize/Shuffle operator with a
  // single consumer is replaced by changed indexing.  Operators of these types are
  // never seeds, so ones no seed reached are folded here into the block of their
  // producer (as store indexing) or else of their consumer (as load indexing).
  void absorb_index_ops() {
    bool changed = true;
    while (changed) {
      changed = false;
      for (int o : order) {
        int bi = block_of[o];
        if (blocks[bi].size() != 1 || !is_index_only(g.ops[o].kind)) continue;
        std::vector<int> targets;
        for (int p : predecessors(o)) targets.push_back(block_of[p]);
        auto succ = successors(o);
        if (succ.size() == 1) targets.push_back(block_of[succ[0]]);
        for (int tb : targets) {
          if (tb == bi) continue;
          std::vector<int> merged = blocks[tb];
          merged.push_back(o);
          if (!convex(merged) || !no_cycle(merged)) continue;
          Block m, a, b;
          if (!lowers(merged, &m)) continue;
          if (lowers(blocks[tb], &a) && lowers({o}, &b) && cost(m) > cost(a) + cost(b)) continue;
          blocks[tb] = merged; blocks[bi].clear(); block_of[o] = tb;
          changed = true;
          break;
        }
      }
    }
  }

  double cost_of(const std::vector<int>& members) {
    if (members.empty()) return 0.0;
    Block b;
    if (!lowers(members, &b)) return 1e30;
    return cost(b);
  }

  // Second half of the same intra-block optimisation: an index-only operator at the END of
  // a block whose result is read only by one other block moves into that block, where it
  // becomes the consumer's load indexing (for a GEMM: the operand's strides).
  void migrate_index_tails() {
    bool changed = true;
    int guard = 0;
    while (changed && guard++ < 10000) {
      changed = false;
      for (auto it = order.rbegin(); it != order.rend() && !changed; ++it) {
        int o = *it;
        if (!is_index_only(g.ops[o].kind)) continue;
        int x = block_of[o];
        int y = -1; bool ok = true;
        for (int t : g.ops[o].out) {
          if (g.tensors[t].is_output) ok = false;
          for (int c : g.tensors[t].consumers) { if (block_of[c] == x) ok = false; else if (y < 0) y = block_of[c]; else if (y != block_of[c]) ok = false; }
        }
        if (!ok || y < 0) continue;
        std::vector<int> xs, ys = blocks[y];
        for (int m : blocks[x]) if (m != o) xs.push_back(m);
        ys.push_back(o);
        if (!convex(ys) || (!xs.empty() && !convex(xs)) || !no_cycle(ys)) continue;
        double before = cost_of(blocks[x]) + cost_of(blocks[y]);
        double after = cost_of(xs) + cost_of(ys);
        if (after >= 1e30 || after > before) continue;
        blocks[x] = xs; blocks[y] = ys; block_of[o] = y;
        changed = true;
      }
    }
  }

  // Listing 1 applied once more with whole blocks as the operators: a producer block and a
  // consumer block merge when Table 3 allows the pair of block types, the union stays convex,
  // passes the constraint check and is not slower by the cost model.
  void merge_blocks() {
    bool changed = true;
    int guard = 0;
    while (changed && guard++ < 10000) {
      changed = false;
      for (int o : order) {
        int x = block_of[o];
        for (int s : successors(o)) {
          int y = block_of[s];
          if (y == x) continue;
          int fused, colour;
          table3(btype[x], btype[y], &fused, &colour);
          if (colour == DNNF_FUSE_BREAK) continue;
          std::vector<int> merged = blocks[x];
          merged.insert(merged.end(), blocks[y].begin(), blocks[y].end());
          if (!check_constraint(merged)) continue;
          if (cost_of(merged) > cost_of(blocks[x]) + cost_of(blocks[y])) continue;
          for (int m : blocks[y]) block_of[m] = x;
          blocks[x] = merged; blocks[y].clear(); btype[x] = fused;
          changed = true;
          break;
        }
        if (changed) break;
      }
    }
  }
};

}  // namespace

// Analytic block cost: algorithmic bytes over HBM bandwidth (element-wise gathers
// pay a sector per element), contraction flops over tensor/FMA peak, one launch.
double block_cost_us(const Graph& g, const Block& b) {
  const Launch& L = b.launch;
  if (L.family == DNNF_FAMILY_ALIAS) return 0.0;
  double bytes = 0;
  auto add = [&](int tensor, int mode, bool is_out = false) {
    const Tensor& T = g.tensors[tensor];
    double e = (double)(is_out ? written_bytes(g, tensor) : T.bytes());
    if (mode == 2) e = e / (T.dtype == DNNF_BF16 ? 2 : 4) * 32.0;
    bytes += e;
  };
  if (L.family == DNNF_FAMILY_ELEMENTWISE || L.family == DNNF_FAMILY_TRANSPOSE) {
    for (int i = 0; i < L.ew.n_in; ++i) add(L.in_tensors[i], L.ew.in[i].mode);
    for (int i = 0; i < L.ew.n_out; ++i) add(L.out_tensors[i], L.ew.out[i].mode, true);
  } else if (L.family == DNNF_FAMILY_GEMM || L.family == DNNF_FAMILY_CONV1X1) {
    // operands: what the contraction reads (a strided view may cover part of a larger tensor)
    const GemmParams& gp = *reinterpret_cast<const GemmParams*>(L.blob.data());
    double nb = (double)gp.batch_ext[0] * gp.batch_ext[1];
    bytes += nb * gp.M * gp.K * (gp.A.dtype ? 2 : 4) * ((gp.A.batch_stride[0] || gp.A.batch_stride[1] || nb == 1) ? 1.0 : 1.0 / nb);
    bytes += nb * gp.K * gp.N * (gp.B.dtype ? 2 : 4) * ((gp.B.batch_stride[0] || gp.B.batch_stride[1] || nb == 1) ? 1.0 : 1.0 / nb);
    for (size_t i = 2; i < L.in_tensors.size(); ++i) add(L.in_tensors[i], 0);
    for (int t : L.out_tensors) add(t, 0, true);
  } else {
    for (int t : b.inputs) add(t, 0);
    for (int t : b.outputs) add(t, 0, true);
  }
  double t_mem = bytes / 6.5e6;                       // us at 6.5 TB/s
  double t_cmp = (double)L.flops / 1.4e9;             // us at 1.4 PFLOP/s
  return std::max(t_mem, t_cmp) + 2.0;
}

bool tf32_shape_fits(int64_t M, int64_t N, int64_t K);
bool conv_small_shape_fits(int64_t M, int64_t N, int64_t K);

// Whether a split into parts x slices tensor-core kernels beats the kernel the contraction would otherwise run on.
// Both sides are rough models fitted to measurements on this GPU: the tiled FMA kernels reach about 10 TFLOP/s on
// such shapes; the one-tile-per-CTA mma.sync kernel (up to 65536 rows) takes about 4.7 ns + 0.044 ns x K per 16 x 32
// tile over the whole GPU (on 6272 pixels: 96 -> 576 channels 61 us, 64 -> 384 37 us, 576 -> 96 40 us, 576 -> 160
// 55 us), so it is the better choice for deep contractions and the worse one for wide ones; a split kernel costs about
// 9 us of launch, setup and tail, every part reads A again, every slice but the last writes a partial sum that a
// later one reads.
static bool split_pays(int64_t M, int64_t N, int64_t K, int64_t parts, int64_t slices) {
  if (plan_flag(DNNF_PLAN_SPLIT_ALWAYS)) return true;      // development switch: the tests use it to reach the split at small sizes
  const double unsplit_us = conv_small_shape_fits(M, N, K)
      ? (double)((M + 15) / 16) * (double)((N + 31) / 32) * (4.7 + 0.044 * (double)K) * 1e-3
      : 2.0 * (double)M * (double)N * (double)K / 1e7;
  const double bytes = 4.0 * (double)M * ((double)parts * (double)K + (double)N * (1.0 + 2.0 * (double)(slices - 1)));
  const double split_us = 9.0 * (double)(parts * slices) + bytes / 4e6;
  return split_us < unsplit_us;
}

// An fp32 pointwise convolution (or plain fp32 matrix product) too deep for the tensor-core kernel (its B images and a tile of whole A rows must
// fit in shared memory) would run on the FMA pipes at a quarter of the speed.  It is split along K into 2-8
// convolutions that fit, chained through Adds: sum_k = sum_{k < K/s} + ... .  The slices of x and W are views, the
// Add joins the next slice's epilogue, so the cost is one extra write and read of the partial sum.  (A lowering
// decision, not one of the paper's rewriting rules: it is applied to every plan, fused or not.)
static void split_deep_pointwise(Graph& g, const std::set<int>& decided) {
  if (plan_flag(DNNF_PLAN_NO_K_SLICES)) return;
  const size_t n_ops = g.ops.size();
  bool any = false;
  for (size_t oi = 0; oi < n_ops; ++oi) {
    if (!g.ops[oi].alive || (g.ops[oi].kind != DNNF_OP_CONV1X1 && g.ops[oi].kind != DNNF_OP_MATMUL)) continue;
    const int x = g.ops[oi].in[0], w = g.ops[oi].in[1], y = g.ops[oi].out[0];
    if (g.tensors[x].dtype != DNNF_F32 || g.tensors[w].dtype != DNNF_F32) continue;
    if (g.ops[oi].kind == DNNF_OP_MATMUL && (g.tensors[x].dims.size() != 2 || g.tensors[w].dims.size() != 2)) continue;   // plain matrix products only
    const int64_t K = g.tensors[w].dims[0], N = g.tensors[w].dims[1], M = g.tensors[x].numel() / K;
    if (tf32_shape_fits(M, N, K)) continue;
    int s = 0;
    for (int c : {2, 3, 4, 5, 6, 8}) if (K % (4 * c) == 0 && tf32_shape_fits(M, N, K / c)) { s = c; break; }
    if (!s || (!decided.count((int)oi) && !split_pays(M, N, K, 1, s))) continue;      // parts of a column split were costed as a whole
    const int source = g.ops[oi].source_id;
    auto add = [&](int kind, std::vector<int> in, const Attrs& at, int reuse_out) -> int {
      Op o; o.id = (int)g.ops.size(); o.kind = kind; o.in = std::move(in); o.at = at; o.source_id = source;
      std::string err;
      const size_t nt = g.tensors.size();
      if (infer_shapes(g, o, err) != DNNF_OK) { g.tensors.resize(nt); return -1; }
      if (reuse_out >= 0) { g.tensors.resize(nt); o.out[0] = reuse_out; g.tensors[reuse_out].producer = o.id; }
      o.mapping = node_mapping(g, o);
      o.props = math_props(kind);
      g.ops.push_back(o);
      return o.out[0];
    };
    // as matrix products over [pixels, K]: a MatMul takes its operands through Slice / Reshape views
    const int64_t ks = K / s;
    int wcol = -1; int64_t wc0 = 0, wc1 = 0;
    {
      const int pw = g.tensors[w].producer;
      if (pw >= 0 && g.ops[pw].alive && g.ops[pw].kind == DNNF_OP_SLICE && g.ops[pw].at.axis == 1 && g.tensors[g.ops[pw].in[0]].dims.size() == 2) {
        wcol = g.ops[pw].in[0]; wc0 = g.ops[pw].at.start; wc1 = g.ops[pw].at.end;
      }
    }
    Attrs r2; r2.shape = {M, K};
    const int x2 = g.tensors[x].dims == r2.shape ? x : add(DNNF_OP_RESHAPE, {x}, r2, -1);
    int acc = -1;
    bool ok = x2 >= 0;
    for (int i = 0; i < s && ok; ++i) {
      Attrs ax, aw;
      ax.axis = 1; ax.start = i * ks; ax.end = (i + 1) * ks;
      aw.axis = 0; aw.start = i * ks; aw.end = (i + 1) * ks;
      int ws;
      if (wcol >= 0) {                       // W is itself a column block of a wider matrix: rows first, then the columns
        Attrs ac; ac.axis = 1; ac.start = wc0; ac.end = wc1;
        const int wr = add(DNNF_OP_SLICE, {wcol}, aw, -1);
        ws = wr < 0 ? -1 : add(DNNF_OP_SLICE, {wr}, ac, -1);
      } else {
        ws = add(DNNF_OP_SLICE, {w}, aw, -1);
      }
      const int xs = add(DNNF_OP_SLICE, {x2}, ax, -1);
      if (xs < 0 || ws < 0) { ok = false; break; }
      const int c = add(DNNF_OP_MATMUL, {xs, ws}, Attrs{}, -1);
      if (c < 0) { ok = false; break; }
      acc = acc < 0 ? c : add(DNNF_OP_ADD, {c, acc}, Attrs{}, -1);
      if (acc < 0) ok = false;
    }
    if (ok) {
      Attrs r4; r4.shape = g.tensors[y].dims;
      if (add(DNNF_OP_RESHAPE, {acc}, r4, y) < 0) ok = false;
    }
    if (ok) { g.ops[oi].alive = false; any = true; }
  }
  if (any) g.relink();
}

// An fp32 pointwise convolution with more output channels than the tensor-core kernel's accumulators hold (N > 192),
// or whose B images do not fit its shared memory at any depth the K split can reach, becomes several convolutions over column blocks of W whose results are the parts of a Concat along the channel
// axis.  The One-to-One operators that follow the convolution and work channel by channel (folded BN, activations,
// bias, a residual of the same shape) are applied per part, with Slice views of their vector / tensor operands, so that
// they stay in the convolutions' epilogues and each part is stored straight into the result.  The part width is the one
// that needs the fewest kernels once the K split below has been applied to the parts as well (at most 32; every part
// reads x again, but the tiled FMA kernel such a convolution would otherwise run on is slower by an order of magnitude).
static void split_wide_pointwise(Graph& g, std::set<int>& decided) {
  if (plan_flag(DNNF_PLAN_NO_COLUMN_BLOCKS) || plan_flag(DNNF_PLAN_NO_TF32_GEMM)) return;
  g.relink();
  const size_t n_ops = g.ops.size();
  bool any = false;
  for (size_t oi = 0; oi < n_ops; ++oi) {
    if (!g.ops[oi].alive || g.ops[oi].kind != DNNF_OP_CONV1X1) continue;
    const int x = g.ops[oi].in[0], w = g.ops[oi].in[1], y = g.ops[oi].out[0];
    if (g.tensors[x].dtype != DNNF_F32 || g.tensors[w].dtype != DNNF_F32) continue;
    const int64_t K = g.tensors[w].dims[0], N = g.tensors[w].dims[1], M = g.tensors[x].numel() / K;
    if (M < 512 || N % 4 || tf32_shape_fits(M, N, K)) continue;
    // the widest part (a multiple of 16 columns) that the kernel takes at this depth; every part reads x again, so
    // only splits into a few parts are worth it (deeper or wider problems stay with the FMA kernel)
    int64_t nw = 0, best = 1 << 30;
    for (int64_t c = std::min<int64_t>(192, (N + 15) / 16 * 16); c >= 48; c -= 16)
      for (int sl : {1, 2, 3, 4, 5, 6, 8}) {
        if (K % (4 * sl) || !tf32_shape_fits(M, c, K / sl)) continue;
        const int64_t kernels = (N + c - 1) / c * sl;
        if (kernels < best) { best = kernels; nw = c; }
        break;                                                              // more slices at this width only cost more
      }
    if (!nw || best > 32) continue;
    const int64_t parts = (N + nw - 1) / nw;
    if (parts == 1) continue;                                              // the K split alone does it
    if (!split_pays(M, N, K, parts, best / parts)) continue;
    nw = ((N + parts - 1) / parts + 15) / 16 * 16;                        // even the parts out
    const std::vector<int64_t> ydims = g.tensors[y].dims;
    // the chain of channel-wise operators behind the convolution
    struct Link { int op; int other; int other_kind; };                   // other_kind: 0 none, 1 vector [N], 2 tensor like y; ScaleShift: two vectors
    std::vector<Link> chain;
    int t = y;
    for (;;) {
      const Tensor& T = g.tensors[t];
      if (T.is_output || T.consumers.size() != 1) break;
      const Op& c = g.ops[T.consumers[0]];
      if (!c.alive || c.out.size() != 1 || g.tensors[c.out[0]].dims != ydims) break;
      Link l{c.id, -1, 0};
      if (c.kind == DNNF_OP_SCALESHIFT) {
        if (c.in[0] != t || (c.at.axis != 3 && c.at.axis != -1)) break;
      } else if (is_binary_elementwise(c.kind)) {
        if (c.in[0] == c.in[1]) break;
        const int o = c.in[0] == t ? c.in[1] : c.in[0];
        const Tensor& O = g.tensors[o];
        if (O.dims == std::vector<int64_t>{N}) l.other_kind = 1;
        else if (O.dims == ydims) l.other_kind = 2;
        else break;
        l.other = o;
      } else if (!(is_elementwise(c.kind) && c.in.size() == 1)) {
        break;
      }
      chain.push_back(l);
      t = c.out[0];
    }
    const int result = t;                                                  // the tensor the Concat will write
    const int source = g.ops[oi].source_id;
    auto add = [&](int kind, std::vector<int> in, const Attrs& at, int src_id, int reuse_out) -> int {
      Op o; o.id = (int)g.ops.size(); o.kind = kind; o.in = std::move(in); o.at = at; o.source_id = src_id;
      std::string err;
      const size_t nt = g.tensors.size();
      if (infer_shapes(g, o, err) != DNNF_OK) { g.tensors.resize(nt); return -1; }
      if (reuse_out >= 0) { g.tensors.resize(nt); o.out[0] = reuse_out; g.tensors[reuse_out].producer = o.id; }
      o.mapping = node_mapping(g, o);
      o.props = math_props(kind);
      g.ops.push_back(o);
      return o.out[0];
    };
    auto slice = [&](int tensor, int axis, int64_t a, int64_t b, int src_id) {
      Attrs at; at.axis = axis; at.start = a; at.end = b;
      return add(DNNF_OP_SLICE, {tensor}, at, src_id, -1);
    };
    Attrs r2; r2.shape = {M, K};
    const int x2 = add(DNNF_OP_RESHAPE, {x}, r2, source, -1);
    bool ok = x2 >= 0;
    int carrier = -1;
    for (int64_t n0 = 0; n0 < N && ok; n0 += nw) {
      const int64_t n1 = std::min(N, n0 + nw);
      const int wj = slice(w, 1, n0, n1, source);
      if (wj < 0) { ok = false; break; }
      int v = add(DNNF_OP_MATMUL, {x2, wj}, Attrs{}, source, -1);
      if (v < 0) { ok = false; break; }
      decided.insert((int)g.ops.size() - 1);
      Attrs r4; r4.shape = ydims; r4.shape[3] = n1 - n0;
      v = add(DNNF_OP_RESHAPE, {v}, r4, source, -1);
      for (const Link& l : chain) {
        if (v < 0) break;
        const Op c = g.ops[l.op];                                          // copy: g.ops grows below
        if (c.kind == DNNF_OP_SCALESHIFT) {
          const int sc = slice(c.in[1], 0, n0, n1, c.source_id), sh = slice(c.in[2], 0, n0, n1, c.source_id);
          Attrs at = c.at; at.axis = 3;
          v = (sc < 0 || sh < 0) ? -1 : add(c.kind, {v, sc, sh}, at, c.source_id, -1);
        } else if (l.other_kind) {
          const int o = slice(l.other, l.other_kind == 1 ? 0 : 3, n0, n1, c.source_id);
          if (o < 0) { v = -1; break; }
          std::vector<int> in = c.in[0] == l.other ? std::vector<int>{o, v} : std::vector<int>{v, o};
          v = add(c.kind, in, c.at, c.source_id, -1);
        } else {
          v = add(c.kind, {v}, c.at, c.source_id, -1);
        }
      }
      if (v < 0) { ok = false; break; }
      Op part; part.id = (int)g.ops.size(); part.kind = DNNF_OP_CONCATPART; part.source_id = source;
      part.in = {v};
      if (carrier >= 0) part.in.push_back(carrier);
      part.at.axis = 3; part.at.start = n0; part.at.shape = ydims;
      std::string err;
      const size_t nt = g.tensors.size();
      if (infer_shapes(g, part, err) != DNNF_OK) { g.tensors.resize(nt); ok = false; break; }
      if (n1 == N) { g.tensors.resize(nt); part.out[0] = result; g.tensors[result].producer = part.id; }
      part.mapping = node_mapping(g, part);
      part.props = 0;
      carrier = part.out[0];
      g.ops.push_back(part);
    }
    if (!ok) continue;                       // what was added stays unused and is dropped as dead code below
    g.ops[oi].alive = false;
    for (const Link& l : chain) g.ops[l.op].alive = false;
    any = true;
    g.relink();
  }
  if (any) g.relink();
}

thread_local uint32_t tl_plan_flags = 0;

// Beyond Table 3: a block that ends in the scores of an attention head, the Softmax block behind it and the block of
// the product with V become one block where that lowers to the single-kernel form.  The scores have the Softmax as
// their only reader and the probabilities the second product, so the union is convex and depends on nothing that
// depends on it.
static void fuse_attention_blocks(const Graph& g, uint32_t flags, std::vector<std::vector<int>>& live) {
  std::vector<int> bo(g.ops.size(), -1);
  for (size_t i = 0; i < live.size(); ++i) for (int o : live[i]) bo[o] = (int)i;
  for (size_t r = 0; r < live.size(); ++r) {
    // the Softmax block: its one Many-to-Many operator is the Softmax (the scale / mask chain may sit in it or in
    // the block of the first product; lowering sorts that out)
    int smo = -1, anchors = 0;
    for (int o : live[r]) { const int k = g.ops[o].kind; if (is_row_anchor(k) || is_contraction(k)) { ++anchors; if (k == DNNF_OP_SOFTMAX) smo = o; } }
    if (anchors != 1 || smo < 0) continue;
    const Op& sm = g.ops[smo];
    const Tensor& pr = g.tensors[sm.out[0]];
    if (pr.is_output || pr.consumers.size() != 1) continue;
    // back along the chain in front of the Softmax to the tensor that enters this block
    int t = sm.in[0];
    while (g.tensors[t].producer >= 0 && bo[g.tensors[t].producer] == (int)r) t = g.ops[g.tensors[t].producer].in[0];
    const Tensor& sc = g.tensors[t];
    if (sc.producer < 0 || sc.is_output || sc.consumers.size() != 1) continue;
    const int a = bo[sc.producer], c = bo[pr.consumers[0]];
    if (a < 0 || c < 0 || a == c || a == (int)r || c == (int)r || live[a].empty() || live[c].empty()) continue;
    if (g.ops[pr.consumers[0]].kind != DNNF_OP_MATMUL) continue;
    std::vector<int> merged = live[a];
    merged.insert(merged.end(), live[r].begin(), live[r].end());
    merged.insert(merged.end(), live[c].begin(), live[c].end());
    Block trial; std::string why;
    if (lower_block(g, merged, flags, trial, why) != DNNF_OK || trial.launch.family != DNNF_FAMILY_ATTENTION) { if (dev_env("DNNF_DEBUG_PLAN")) fprintf(stderr, "attention not fused: %s\n", why.c_str()); continue; }
    for (int o : live[r]) bo[o] = a;
    for (int o : live[c]) bo[o] = a;
    live[a] = merged; live[r].clear(); live[c].clear();
  }
  std::vector<std::vector<int>> keep;
  for (auto& b : live) if (!b.empty()) keep.push_back(b);
  live.swap(keep);
}

// Beyond Table 3, second case: the block of a depthwise 3x3 convolution between the blocks of the pointwise convolution
// that makes its input and the one that reads its result (an inverted-residual block) becomes one block when the three
// lower to the single kernel.
static void fuse_mbconv_blocks(const Graph& g, uint32_t flags, std::vector<std::vector<int>>& live) {
  std::vector<int> bo(g.ops.size(), -1);
  for (size_t i = 0; i < live.size(); ++i) for (int o : live[i]) bo[o] = (int)i;
  auto one_anchor = [&](const std::vector<int>& b, int kind) {
    int n = 0, found = -1;
    for (int o : b) { const int k = g.ops[o].kind; if (is_row_anchor(k) || is_contraction(k)) { ++n; if (k == kind) found = o; } }
    return n == 1 ? found : -1;
  };
  for (size_t r = 0; r < live.size(); ++r) {
    const int dwo = one_anchor(live[r], DNNF_OP_DWCONV3X3);
    if (dwo < 0) continue;
    const Tensor& e = g.tensors[g.ops[dwo].in[0]];
    if (e.producer < 0 || e.is_output || e.consumers.size() != 1) continue;
    const int a = bo[e.producer];
    if (a < 0 || a == (int)r || live[a].empty() || one_anchor(live[a], DNNF_OP_CONV1X1) < 0) continue;
    // forward along the chain behind the depthwise filter to the tensor that leaves this block
    int t = g.ops[dwo].out[0];
    while (g.tensors[t].consumers.size() == 1 && bo[g.tensors[t].consumers[0]] == (int)r && !g.tensors[t].is_output) t = g.ops[g.tensors[t].consumers[0]].out[0];
    const Tensor& d = g.tensors[t];
    if (d.is_output || d.consumers.size() != 1) continue;
    const int c = bo[d.consumers[0]];
    if (c < 0 || c == (int)r || c == a || live[c].empty() || one_anchor(live[c], DNNF_OP_CONV1X1) != d.consumers[0]) continue;
    std::vector<int> merged = live[a];
    merged.insert(merged.end(), live[r].begin(), live[r].end());
    merged.insert(merged.end(), live[c].begin(), live[c].end());
    Block trial; std::string why;
    if (lower_block(g, merged, flags, trial, why) != DNNF_OK || trial.launch.family != DNNF_FAMILY_MBCONV) { if (dev_env("DNNF_DEBUG_PLAN")) fprintf(stderr, "inverted-residual block not fused: %s\n", why.c_str()); continue; }
    for (int o : live[r]) bo[o] = a;
    for (int o : live[c]) bo[o] = a;
    live[a] = merged; live[r].clear(); live[c].clear();
  }
  std::vector<std::vector<int>> keep;
  for (auto& b : live) if (!b.empty()) keep.push_back(b);
  live.swap(keep);
}

int plan_graph(Graph& g, uint32_t flags) {
  tl_plan_flags = flags;
  g.relink();
  {
    std::set<int> decided;                  // matrix products made by the column split: their K split is part of that decision
    split_wide_pointwise(g, decided);
    split_deep_pointwise(g, decided);
  }
  // Operators whose results nobody reads (not a graph output, no live consumer) are not planned: they would
  // form blocks without an output.  (The rewriting pass removes them as well; a graph planned without rewriting
  // may still carry some.)
  for (bool changed = true; changed;) {
    changed = false;
    for (auto& o : g.ops) {
      if (!o.alive) continue;
      bool used = false;
      for (int t : o.out) if (g.tensors[t].is_output || !g.tensors[t].consumers.empty()) used = true;
      if (!used) { o.alive = false; changed = true; }
    }
    if (changed) g.relink();
  }
  g.blocks.clear(); g.run_order.clear();
  g.planned = false;
  for (auto& o : g.ops) { o.block = -1; if (o.alive) o.mapping = node_mapping(g, o); }
  for (auto& t : g.tensors) { t.ws_offset = -1; t.alias_of = -1; t.removable = false; }

  Planner P(g, flags);
  P.order = g.topo_order();
  P.pos.assign(g.ops.size(), -1);
  for (size_t i = 0; i < P.order.size(); ++i) P.pos[P.order[i]] = (int)i;
  P.block_of.assign(g.ops.size(), -1);
  P.reachability();
  if (flags & DNNF_PLAN_UNFUSED) {
    for (int o : P.order) { P.block_of[o] = (int)P.blocks.size(); P.blocks.push_back({o}); P.btype.push_back(g.ops[o].mapping); }
  } else {
    P.run_listing1();
    if (!(flags & DNNF_PLAN_ALLOW_PROLOGUE)) { P.absorb_index_ops(); P.migrate_index_tails(); P.merge_blocks(); }
  }

  // Materialise blocks in an order that respects dependencies (first member's position
  // is not enough after predecessor fusion: sort blocks topologically).
  std::vector<std::vector<int>> live;
  for (auto& b : P.blocks) if (!b.empty()) live.push_back(b);
  if ((flags & DNNF_PLAN_BEYOND_TABLE3) && !(flags & (DNNF_PLAN_UNFUSED | DNNF_PLAN_ALLOW_PROLOGUE))) { fuse_attention_blocks(g, flags, live); fuse_mbconv_blocks(g, flags, live); }
  int nb = (int)live.size();
  std::vector<int> bo(g.ops.size(), -1);
  for (int i = 0; i < nb; ++i) for (int o : live[i]) bo[o] = i;
  std::vector<std::set<int>> deps(nb);
  for (int i = 0; i < nb; ++i)
    for (int o : live[i]) for (int t : g.ops[o].in) { int p = g.tensors[t].producer; if (p >= 0 && g.ops[p].alive && bo[p] != i) deps[i].insert(bo[p]); }
  std::vector<int> first_pos(nb, 1 << 30);
  for (int i = 0; i < nb; ++i) for (int o : live[i]) first_pos[i] = std::min(first_pos[i], P.pos[o]);
  std::vector<int> done(nb, 0), border;
  for (int round = 0; round < nb; ++round) {
    int pick = -1;
    for (int i = 0; i < nb; ++i) {
      if (done[i]) continue;
      bool ready = true;
      for (int d : deps[i]) if (!done[d]) ready = false;
      if (ready && (pick < 0 || first_pos[i] < first_pos[pick])) pick = i;
    }
    if (pick < 0) { g.err = "internal: cyclic block dependencies"; return DNNF_ERR_STATE; }
    done[pick] = 1; border.push_back(pick);
  }

  bool runnable = true;
  for (int bi : border) {
    Block b; std::string why;
    int rc = lower_block(g, live[bi], flags, b, why);
    if (rc != DNNF_OK) {
      if (flags & DNNF_PLAN_ALLOW_PROLOGUE) { b.ops = live[bi]; b.lowered = false; runnable = false; }
      else {
        g.err = "cannot lower block starting at " + std::string(op_name(g.ops[live[bi][0]].kind)) + ": " + why;
        return DNNF_ERR_UNSUPPORTED_OP;
      }
    }
    b.mapping = P.btype[P.block_of[live[bi][0]]];
    int idx = (int)g.blocks.size();
    for (int o : b.ops) g.ops[o].block = idx;
    g.blocks.push_back(std::move(b));
    g.run_order.push_back(idx);
  }

  // IR_removable (Section 3.2): an intermediate disappears iff every consumer sits in
  // its producer's block.  What remains is materialised in the workspace.
  int64_t irs_unfused = 0, irs_fused = 0;
  for (auto& t : g.tensors) {
    if (t.external || t.producer < 0 || !g.ops[t.producer].alive) continue;
    bool outside = false;
    for (int c : t.consumers) if (g.ops[c].block != g.ops[t.producer].block) outside = true;
    t.removable = !outside && !t.is_output;
    if (!t.is_output) { irs_unfused += t.bytes(); if (!t.removable) irs_fused += t.bytes(); }
  }
  // zero-copy aliases
  for (auto& b : g.blocks) if (b.lowered && b.launch.family == DNNF_FAMILY_ALIAS) {
    g.tensors[b.launch.out_tensors[0]].alias_of = b.launch.in_tensors[0];
    irs_fused -= g.tensors[b.launch.out_tensors[0]].bytes();
  }
  // A Concat's parts fill one result in place: the result so far shares storage with the extended one.
  for (auto& o : g.ops) if (o.alive && o.kind == DNNF_OP_CONCATPART && o.in.size() > 1) {
    g.tensors[o.in[1]].alias_of = o.out[0];
    irs_fused -= g.tensors[o.in[1]].bytes();
    irs_unfused -= g.tensors[o.in[1]].bytes();
  }
  // Workspace: first-fit over live ranges in block order.
  struct Range { int64_t off, size; int last_use; };
  std::vector<Range> active;
  int64_t ws = 256;                       // status words live in the first 256 bytes,
  for (auto& b : g.blocks)                // kernels' arrival counters right behind them (the zeroed header)
    if (b.lowered && b.launch.counter_bytes > 0) { b.launch.counter_off = ws; ws += (b.launch.counter_bytes + 255) / 256 * 256; }
  const int64_t header = ws;
  g.ws_zero_bytes = (size_t)header;
  auto root = [&](int t) { while (g.tensors[t].alias_of >= 0) t = g.tensors[t].alias_of; return t; };
  std::vector<int> last_use(g.tensors.size(), -1);
  for (size_t bi = 0; bi < g.blocks.size(); ++bi) {
    for (int t : g.blocks[bi].inputs) last_use[root(t)] = (int)bi;
    for (int t : g.blocks[bi].outputs) last_use[root(t)] = std::max(last_use[root(t)], (int)bi);
  }
  for (size_t bi = 0; bi < g.blocks.size(); ++bi) {
    Block& b = g.blocks[bi];
    if (!b.lowered || b.launch.family == DNNF_FAMILY_ALIAS) continue;
    for (int t0 : b.outputs) {
      const int t = root(t0);             // a Concat's parts: the shared result, placed when its first part runs
      Tensor& T = g.tensors[t];
      if (T.is_output) continue;          // bound by the caller
      if (T.ws_offset >= 0) continue;
      int64_t size = (T.bytes() + 255) / 256 * 256;
      // free ranges whose last use is before this block
      std::vector<Range> keep;
      for (auto& r : active) if (r.last_use >= (int)bi) keep.push_back(r);
      active.swap(keep);
      std::sort(active.begin(), active.end(), [](const Range& a, const Range& c) { return a.off < c.off; });
      int64_t off = header;
      for (auto& r : active) { if (off + size <= r.off) break; off = std::max(off, r.off + r.size); }
      active.push_back({off, size, std::max(last_use[t], (int)bi)});
      T.ws_offset = off;
      ws = std::max(ws, off + size);
    }
  }
  for (auto& b : g.blocks)                // kernels' own scratch (split-K partials) behind the tensors, never shared
    if (b.lowered && b.launch.scratch_bytes > 0) { b.launch.scratch_off = ws; ws += (b.launch.scratch_bytes + 255) / 256 * 256; }
  g.ws_bytes = (size_t)ws;
  g.plan_flags = flags;
  g.planned = runnable;

  dnnf_plan_stats& s = g.pstats;
  std::memset(&s, 0, sizeof s);
  std::set<int> src;
  for (auto& o : g.ops) if (o.alive) src.insert(o.source_id);
  s.n_ops = (int)src.size();
  s.n_blocks = (int)g.blocks.size();
  for (auto& b : g.blocks) if (!b.lowered || b.launch.family != DNNF_FAMILY_ALIAS) s.n_kernels++;
  s.fusion_rate = s.n_blocks ? (double)s.n_ops / s.n_blocks : 0.0;
  s.irs_bytes_unfused = irs_unfused;
  s.irs_bytes_fused = irs_fused;
  s.workspace_bytes = ws;
  s.n_yellow_decisions = P.yellow;
  s.n_yellow_fused = P.yellow_fused;
  s.n_profile_hits = P.hits;
  s.n_profile_misses = (int32_t)P.misses.size();
  g.profile_hits = P.hits;
  g.profile_misses.clear();
  for (auto& kv : P.misses) g.profile_misses.push_back({kv.first, kv.second});
  return DNNF_OK;
}

}  // namespace dnnf

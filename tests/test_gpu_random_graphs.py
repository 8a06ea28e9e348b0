"""Random operator graphs against the oracle.  A seeded generator strings bounded element-wise operators, broadcasts
against vectors and full tensors, transposes, reshapes, slices, last-axis reductions, Softmax / LayerNorm and
matrix products into DAGs with several outputs; every graph runs fused (and un-fused) with outputs and workspace
poisoned by NaN, and has to reproduce the oracle."""
import numpy as np
import pytest

from paper_2108_13342_b200 import binding as B
from paper_2108_13342_b200 import workloads as W
from paper_2108_13342_b200.runtime import Session
from oracle import interp as O
from util import RTOL_F32, close, graph

pytestmark = pytest.mark.gpu


class _Rng:
    """Counter-based draws from the shared input generator (no method arithmetic here)."""
    def __init__(self, seed):
        self.seed, self.n = seed, 0

    def u(self):
        self.n += 1
        return float(W.uniform(4242 + self.seed, self.n, (1,), 0.0, 1.0)[0])

    def pick(self, xs):
        return xs[min(int(self.u() * len(xs)), len(xs) - 1)]


def _build(seed, big=False, dtype="f32", extended=False, table2=False):
    r = _Rng(seed)
    bsz, rows, cols = r.pick([1, 2, 3]), r.pick([5, 8, 16, 33]), r.pick([8, 12, 32, 64])
    if big:      # sizes that reach the vectorised, multi-vector, multi-warp and tensor-core variants
        bsz, rows, cols = r.pick([1, 2, 4]), r.pick([96, 256, 520, 1024]), r.pick([128, 256, 768, 1000, 2048])
    g = graph("rand%d" % seed)
    ins = {}
    def data(a):
        return W.round_to_bf16(a) if dtype == "bf16" else a
    g.ext("X", (bsz, rows, cols), dtype); ins["X"] = data(W.uniform(777, 1000 + seed, (bsz, rows, cols), -1.0, 1.0))
    g.ext("X2", (bsz, rows, cols), dtype); ins["X2"] = data(W.uniform(777, 2000 + seed, (bsz, rows, cols), -1.0, 1.0))
    pool = [("X", (bsz, rows, cols)), ("X2", (bsz, rows, cols))]
    n_ext = [0]

    def vec(n, lo, hi):
        n_ext[0] += 1
        name = "v%d" % n_ext[0]
        g.ext(name, (n,)); ins[name] = W.uniform(777, 3000 + 10 * seed + n_ext[0], (n,), lo, hi)
        return name

    def vec_like(shape):
        n_ext[0] += 1
        name = "f%d" % n_ext[0]
        g.ext(name, shape, dtype); ins[name] = data(W.uniform(777, 6000 + 10 * seed + n_ext[0], shape, -1.0, 1.0))
        return name

    def mat(k, n):
        n_ext[0] += 1
        name = "m%d" % n_ext[0]
        g.ext(name, (k, n), dtype); ins[name] = data(W.uniform(777, 4000 + 10 * seed + n_ext[0], (k, n), -0.3, 0.3))
        return name

    n_ops = 4 + int(r.u() * (4 if dtype == "bf16" else 9))
    for _ in range(n_ops):
        t, shp = r.pick(pool[-4:]) if r.u() < 0.7 else r.pick(pool)      # mostly recent values (long chains), sometimes old ones (diamonds)
        kind = r.pick(["unary", "unary", "vec", "full", "transpose", "reshape", "slice", "reduce", "softmax", "layernorm", "matmul",
                       "rowvec", "exp", "div", "reduce0", "permute"] + (["concat", "concat", "concat"] if extended else [])
                      + (["where", "where", "cumsum", "cumsum", "where_vec"] if table2 else []))
        if kind in ("reduce", "reduce0", "softmax", "layernorm", "cumsum") and shp[-1] > 8192:
            continue                                    # longer rows than the row kernels take (the plan says so)
        if kind == "unary":
            op, at = r.pick([("Tanh", {}), ("Sigmoid", {}), ("Relu", {}), ("Abs", {}), ("Square", {}), ("Neg", {}),
                             ("MulC", {"c": 0.5}), ("AddC", {"c": 0.25}), ("Gelu", {"approx": "erf"}), ("Erf", {})])
            if op == "Square":
                t = g.add("Tanh", [t])                  # keep magnitudes bounded
            o = g.add(op, [t], **at)
        elif kind == "where":                          # the condition and both branches are values of the graph
            cands = [p for p in pool if p[1] == shp]
            a, b, c = r.pick(cands)[0], r.pick(cands)[0], r.pick(cands)[0]
            o = g.add("Where", [g.add("Greater", [t, a]), b, g.add("Neg", [c])])
        elif kind == "where_vec":                      # a broadcast condition and a broadcast branch
            o = g.add("Where", [g.add("Greater", [vec(shp[-1], -1.0, 1.0), vec(shp[-1], -1.0, 1.0)]), t, vec(shp[-1], -1.0, 1.0)])
        elif kind == "cumsum":
            o = g.add("CumSum", [g.add("Tanh", [t])], axis=-1, exclusive=int(r.u() < 0.3), reverse=int(r.u() < 0.3))
            o = g.add("MulC", [o], c=1.0 / max(1, shp[-1]) ** 0.5)
        elif kind == "exp":
            o = g.add("Exp", [g.add("MulC", [g.add("Tanh", [t])], c=0.5)])
        elif kind == "div":
            cands = [p for p in pool if p[1] == shp]
            den = g.add("AddC", [g.add("Abs", [g.add("Tanh", [r.pick(cands)[0]])])], c=1.5)
            o = g.add("Div", [g.add("Tanh", [t]), den])
        elif kind == "concat":
            cands = [p for p in pool if p[1] == shp]
            other = r.pick(cands)[0]
            ax = int(r.u() * len(shp))
            third = [vec_like(shp)] if r.u() < 0.3 else []
            o = g.add("Concat", [t, other] + third, axis=ax)
            shp = shp[:ax] + ((2 + len(third)) * shp[ax],) + shp[ax + 1:]
        elif kind == "rowvec":
            if len(shp) < 2:
                continue
            n_ext[0] += 1
            name = "c%d" % n_ext[0]
            cshape = shp[:-1] + (1,)
            g.ext(name, cshape); ins[name] = W.uniform(777, 5000 + 10 * seed + n_ext[0], cshape, 0.5, 1.5)
            o = g.add(r.pick(["Add", "Mul"]), [t, name])
        elif kind == "reduce0":
            if len(shp) < 2:
                continue
            o = g.add(r.pick(["ReduceSum", "ReduceMax"]), [g.add("Tanh", [t])], axis=-1, keepdims=0)
            shp = shp[:-1]
        elif kind == "permute":
            if len(shp) != 3:
                continue
            perm = r.pick([(0, 2, 1), (1, 0, 2), (2, 1, 0), (1, 2, 0), (2, 0, 1)])
            o = g.add("Transpose", [t], perm=perm)
            shp = tuple(shp[p] for p in perm)
        elif kind == "vec":
            o = g.add(r.pick(["Add", "Mul", "Sub"]), [t, vec(shp[-1], 0.5, 1.5)])
        elif kind == "full":
            cands = [p for p in pool if p[1] == shp and p[0] != t]
            if not cands:
                continue
            o = g.add(r.pick(["Add", "Mul", "Sub"]), [t, r.pick(cands)[0]])
            o = g.add("Tanh", [o])
        elif kind == "transpose":
            if len(shp) < 2:
                continue
            perm = list(range(len(shp)))
            i, j = len(shp) - 1, int(r.u() * (len(shp) - 1))
            perm[i], perm[j] = perm[j], perm[i]
            o = g.add("Transpose", [t], perm=tuple(perm))
            shp = tuple(shp[p] for p in perm)
        elif kind == "reshape":
            if len(shp) == 3:
                new = (shp[0] * shp[1], shp[2]) if r.u() < 0.5 else (shp[0], shp[1] * shp[2])
            elif len(shp) == 2 and shp[0] % 2 == 0:
                new = (2, shp[0] // 2, shp[1])
            else:
                continue
            o = g.add("Reshape", [t], shape=new)
            shp = new
        elif kind == "slice":
            ax = int(r.u() * len(shp))
            if shp[ax] < 4:
                continue
            a = int(r.u() * (shp[ax] // 2)); e = a + max(1, int(r.u() * (shp[ax] - a)))
            o = g.add("Slice", [t], axis=ax, start=a, end=e)
            shp = shp[:ax] + (e - a,) + shp[ax + 1:]
        elif kind == "reduce":
            o = g.add(r.pick(["ReduceSum", "ReduceMean", "ReduceMax"]), [t], axis=-1, keepdims=1)
            shp = shp[:-1] + (1,)
        elif kind == "softmax":
            o = g.add("Softmax", [t], axis=-1)
        elif kind == "layernorm":
            if shp[-1] < 4:
                continue
            o = g.add("LayerNorm", [t, vec(shp[-1], 0.8, 1.2), vec(shp[-1], -0.2, 0.2)], axis=-1, eps=1e-5)
        else:
            if len(shp) < 2:
                continue                                # MatMul takes a matrix on the left
            n = r.pick([8, 16, 24])
            o = g.add("MatMul", [t, mat(shp[-1], n)])
            shp = shp[:-1] + (n,)
        if kind not in ("transpose", "reshape", "slice", "reduce", "matmul"):
            pass
        pool.append((o, shp))
    outs = {pool[-1][0]}
    for _ in range(int(r.u() * 3)):
        cand = r.pick(pool[2:])
        outs.add(cand[0])
    for i, o in enumerate(sorted(outs)):
        g.mark_output(o)
    return W.Workload(g, ins)


def _random_db(wl, seed):
    """Pseudo-random latencies for every candidate block the planner asks about (odd seeds: growing with block size)."""
    from paper_2108_13342_b200.runtime import build_graph
    for rnd_ in range(4):
        g = build_graph(wl.graph)[0]
        g.rewrite(B.REWRITE_NONE)
        g.plan(B.PLAN_FUSED)
        misses = g.profile_misses()
        if not misses:
            break
        for i, sig in enumerate(misses):
            u = float(W.uniform(9100 + seed, 100 * rnd_ + i, (1,), 1.0, 20.0)[0])
            if seed % 2:
                u *= 1 + 3 * sig.split("|")[1].count("+")
            B.profile_db_set(sig, u)


@pytest.mark.parametrize("seed", [pytest.param(i, id=str(i)) for i in range(300)] + [pytest.param(-i - 1, id="big%d" % i) for i in range(60)])
def test_random_graph(seed):
    wl = _build(seed, False) if seed >= 0 else _build(1000 - seed, True)
    ref = O.run_graph(wl.graph, wl.inputs)
    for flags, rewrite, db in ((B.PLAN_FUSED, B.REWRITE_NONE, False), (B.PLAN_UNFUSED, B.REWRITE_NONE, False),
                               (B.PLAN_FUSED, B.REWRITE_DEFAULT, False), (B.PLAN_FUSED, B.REWRITE_NONE, True)):
        B.profile_db_clear()
        try:
            if db:
                _random_db(wl, seed)
            s = Session(wl, plan_flags=flags, rewrite_flags=rewrite)
            s.workspace[s.g.workspace_zero_bytes():].fill_(0xFF)
            for n in wl.graph.outputs:
                s.buffers[n].fill_(float("nan"))
            s.run()
            assert s.g.status()[0] == 0
            for n in wl.graph.outputs:
                got = s.output(n)
                assert np.isfinite(got).all(), (n, "unwritten elements", [b["ops"] for b in s.g.blocks()])
                try:
                    close(got, ref[n], 2e-5)
                except AssertionError as e:
                    raise AssertionError(f"{n} flags {flags} rewrite {rewrite} db {db} plan {[b['ops'] for b in s.g.blocks()]}: {e}") from None
        finally:
            B.profile_db_clear()


@pytest.mark.parametrize("seed", [pytest.param(i, id=str(i)) for i in list(range(120)) + [2334]]     # 2334: two convex blocks that needed each other
                         + [pytest.param(-i - 1, id="big%d" % i) for i in range(30)])
def test_random_graph_with_concat(seed):
    """The same generator with Concat among the operators: parts stored by producer blocks of every family,
    results read through views, nested and repeated inputs."""
    wl = _build(5000 + seed, False, extended=True) if seed >= 0 else _build(6000 - seed, True, extended=True)
    ref = O.run_graph(wl.graph, wl.inputs)
    for flags in (B.PLAN_FUSED, B.PLAN_UNFUSED):
        s = Session(wl, plan_flags=flags, rewrite_flags=B.REWRITE_NONE)
        s.workspace[s.g.workspace_zero_bytes():].fill_(0xFF)
        for n in wl.graph.outputs:
            s.buffers[n].fill_(float("nan"))
        s.run()
        assert s.g.status()[0] == 0
        for n in wl.graph.outputs:
            got = s.output(n)
            assert np.isfinite(got).all(), (n, "unwritten elements", [b["ops"] for b in s.g.blocks()])
            try:
                close(got, ref[n], 2e-4 if seed < 0 else 2e-5)
            except AssertionError as e:
                raise AssertionError(f"{n} plan {[b['ops'] for b in s.g.blocks()]}: {e}") from None


def _build_cnn(seed):
    """Random NHWC fp32 graphs over the convolution-side operators: pointwise / depthwise / transposed convolutions with
    folded-BN epilogues, pooling, SpaceToDepth / DepthToSpace, Resize, channel and spatial Concat, residual adds."""
    r = _Rng(seed)
    n, hw, c = r.pick([1, 2, 3]), r.pick([4, 8, 12, 16]), r.pick([4, 8, 16, 24])
    g = graph("cnn%d" % seed)
    ins = {}
    g.ext("X", (n, hw, hw, c)); ins["X"] = W.uniform(778, 1000 + seed, (n, hw, hw, c), -1.0, 1.0)
    pool = [("X", (n, hw, hw, c))]
    cnt = [0]

    def ext(shape, lo, hi, kind="weight"):
        cnt[0] += 1
        name = "w%d" % cnt[0]
        g.ext(name, shape, kind=kind); ins[name] = W.uniform(778, 3000 + 20 * seed + cnt[0], shape, lo, hi)
        return name

    def bn_act(t, ch):
        t = g.add("ScaleShift", [t, ext((ch,), 0.5, 1.5), ext((ch,), -0.5, 0.5)], axis=-1)
        act = r.pick(["clip", "relu", "leaky", "none", "sigmoid"])
        if act == "clip": t = g.add("Clip", [t], lo=0.0, hi=6.0)
        elif act == "relu": t = g.add("Relu", [t])
        elif act == "leaky": t = g.add("LeakyRelu", [t], alpha=0.1)
        elif act == "sigmoid": t = g.add("Sigmoid", [t])
        return t

    for _ in range(5 + int(r.u() * 8)):
        t, shp = r.pick(pool[-3:]) if r.u() < 0.7 else r.pick(pool)
        N, H, Wd, C = shp
        kind = r.pick(["conv", "conv", "dw", "maxpool", "avgpool", "gap", "s2d", "d2s", "resize", "catc", "cath", "add", "deconv", "unary"])
        if kind in ("dw", "maxpool", "avgpool", "gap") and C % 4:
            continue                                  # these kernels move four channels per thread
        if kind == "conv":
            co = r.pick([4, 8, 16, 24, 32])
            o = bn_act(g.add("Conv1x1", [t, ext((C, co), -0.4, 0.4)]), co); shp = (N, H, Wd, co)
        elif kind == "dw":
            o = bn_act(g.add("DwConv3x3", [t, ext((3, 3, C), -0.4, 0.4)]), C)
        elif kind in ("maxpool", "avgpool"):
            k, s_, p = r.pick([(2, 2, 0), (3, 2, 1), (3, 1, 1), (2, 1, 0)])
            if H + 2 * p < k or Wd + 2 * p < k:
                continue
            o = g.add("MaxPool" if kind == "maxpool" else "AveragePool", [t], kernel=k, stride=s_, pad=p)
            shp = (N, (H + 2 * p - k) // s_ + 1, (Wd + 2 * p - k) // s_ + 1, C)
            if r.u() < 0.5:
                o = bn_act(o, C)
        elif kind == "gap":
            if H != Wd or H < 2:
                continue
            o = g.add("AveragePool", [t], kernel=H, stride=1, pad=0)
            gate = g.add("Sigmoid", [g.add("Conv1x1", [o, ext((C, C), -0.4, 0.4)])])
            o = g.add("Mul", [t, gate])
        elif kind == "s2d":
            if H % 2 or Wd % 2 or C * 4 > 128:
                continue
            o = g.add("SpaceToDepth", [t], block=2); shp = (N, H // 2, Wd // 2, C * 4)
        elif kind == "d2s":
            if C % 4 or H * 2 > 48:
                continue
            o = g.add("DepthToSpace", [t], block=2); shp = (N, H * 2, Wd * 2, C // 4)
        elif kind == "resize":
            if H * 2 > 48:
                continue
            o = g.add("Resize", [t], scale=2); shp = (N, H * 2, Wd * 2, C)
        elif kind in ("catc", "cath"):
            ax = 3 if kind == "catc" else 1
            cands = [p for p in pool if all(p[1][d] == shp[d] for d in range(4) if d != ax) and p[1][ax] + shp[ax] <= 160]
            if not cands:
                continue
            other = r.pick(cands)
            o = g.add("Concat", [t, other[0]], axis=ax)
            shp = tuple(shp[d] + (other[1][d] if d == ax else 0) for d in range(4))
        elif kind == "add":
            cands = [p for p in pool if p[1] == shp and p[0] != t]
            if not cands:
                continue
            o = g.add("Add", [t, r.pick(cands)[0]])
        elif kind == "deconv":
            if H * 2 > 48:
                continue
            co = r.pick([4, 8, 16])
            o = bn_act(g.add("ConvTranspose", [t, ext((C, 2, 2, co), -0.4, 0.4)], kernel=2), co); shp = (N, H * 2, Wd * 2, co)
        else:
            o = g.add(r.pick(["Tanh", "Relu", "Abs", "Sin"]), [t])
        pool.append((o, shp))
    outs = {pool[-1][0]}
    for _ in range(int(r.u() * 3)):
        outs.add(r.pick(pool[1:])[0]) if len(pool) > 1 else None
    for o in sorted(outs):
        if o != "X":
            g.mark_output(o)
    if not g.outputs:
        g.mark_output(g.add("Relu", ["X"]))
    return W.Workload(g, ins)


@pytest.mark.parametrize("seed", range(160))
def test_random_cnn_graph(seed):
    wl = _build_cnn(7000 + seed)
    ref = O.run_graph(wl.graph, wl.inputs)
    for flags, rewrite in ((B.PLAN_FUSED, B.REWRITE_NONE), (B.PLAN_UNFUSED, B.REWRITE_NONE), (B.PLAN_FUSED, B.REWRITE_DEFAULT)):
        s = Session(wl, plan_flags=flags, rewrite_flags=rewrite)
        s.workspace[s.g.workspace_zero_bytes():].fill_(0xFF)
        for n in wl.graph.outputs:
            s.buffers[n].fill_(float("nan"))
        s.run()
        assert s.g.status()[0] == 0
        for n in wl.graph.outputs:
            got = s.output(n)
            assert np.isfinite(got).all(), (n, "unwritten elements", [b["ops"] for b in s.g.blocks()])
            try:
                close(got, ref[n], 1e-4)
            except AssertionError as e:
                raise AssertionError(f"{n} flags {flags} rewrite {rewrite} plan {[b['ops'] for b in s.g.blocks()]}: {e}") from None


@pytest.mark.parametrize("seed", range(80))
def test_random_graph_bf16(seed):
    """bf16 activations and weights (vectors stay fp32), short chains, fused plan: intermediates stay in fp32 inside a
    block, every stored tensor is rounded to bf16."""
    wl = _build(2000 + seed, seed % 4 == 3, "bf16")
    ref = O.run_graph(wl.graph, wl.inputs)
    s = Session(wl, plan_flags=B.PLAN_FUSED, rewrite_flags=B.REWRITE_NONE)
    s.workspace[s.g.workspace_zero_bytes():].fill_(0xFF)
    for n in wl.graph.outputs:
        s.buffers[n].fill_(float("nan"))
    s.run()
    assert s.g.status()[0] == 0
    for n in wl.graph.outputs:
        got = s.output(n)
        assert np.isfinite(got).all(), (n, "unwritten elements", [b["ops"] for b in s.g.blocks()])
        try:
            close(got, ref[n], 3e-2)
        except AssertionError as e:
            raise AssertionError(f"{n} plan {[b['ops'] for b in s.g.blocks()]}: {e}") from None


@pytest.mark.parametrize("seed", [pytest.param(i, id=str(i)) for i in range(100)] + [pytest.param(-i - 1, id="big%d" % i) for i in range(24)])
def test_random_graph_with_where_and_cumsum(seed):
    """The same generator with Where (conditions and branches computed in the graph, or broadcast) and CumSum (inclusive,
    exclusive, reverse) among the operators."""
    wl = _build(8000 + seed, False, table2=True) if seed >= 0 else _build(9000 - seed, True, table2=True)
    ref = O.run_graph(wl.graph, wl.inputs)
    for flags, rewrite in ((B.PLAN_FUSED, B.REWRITE_NONE), (B.PLAN_UNFUSED, B.REWRITE_NONE), (B.PLAN_FUSED, B.REWRITE_DEFAULT)):
        s = Session(wl, plan_flags=flags, rewrite_flags=rewrite)
        s.workspace[s.g.workspace_zero_bytes():].fill_(0xFF)
        for n in wl.graph.outputs:
            s.buffers[n].fill_(float("nan"))
        s.run()
        assert s.g.status()[0] == 0
        for n in wl.graph.outputs:
            got = s.output(n)
            assert np.isfinite(got).all(), (n, "unwritten elements", [b["ops"] for b in s.g.blocks()])
            try:
                close(got, ref[n], 2e-5)
            except AssertionError as e:
                raise AssertionError(f"{n} flags {flags} rewrite {rewrite} plan {[b['ops'] for b in s.g.blocks()]}: {e}") from None

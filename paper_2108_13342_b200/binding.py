"""ctypes binding of the C ABI in include/dnnf.h.

Argument marshalling only: every step of graph rewriting, planning and block
execution runs inside libdnnf.so.  The library is built in-tree by
paper_2108_13342_b200/build.py; if it is missing, importing this module raises --
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdnnf.so")


class DnnfError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"dnnf error {code}: {msg}")
        self.code = code


OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED_OP, ERR_STATE, ERR_UNBOUND, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(9)
F32, BF16 = 0, 1
INPUT, WEIGHT = 0, 1
ONE_TO_ONE, REORGANIZE, SHUFFLE, ONE_TO_MANY, MANY_TO_MANY = range(5)
GREEN, YELLOW, RED = range(3)
MAPPING_NAMES = ["One-to-One", "Reorganize", "Shuffle", "One-to-Many", "Many-to-Many"]
FAMILY_NAMES = ["alias", "elementwise", "transpose", "row", "gemm", "conv1x1", "dwconv", "pool", "gather", "attention", "mbconv", "instnorm"]

OP_NAMES = ["?", "Add", "Sub", "Mul", "Div", "MulC", "AddC", "Sigmoid", "Tanh", "Erf", "Exp", "Log", "Sqrt", "Abs",
            "Neg", "Recip", "Square", "Relu", "Clip", "Pow", "Gelu", "ScaleShift", "Transpose", "Reshape", "Flatten",
            "Squeeze", "Unsqueeze", "Split", "Slice", "MatMul", "Conv1x1", "DwConv3x3", "Softmax", "LayerNorm",
            "ReduceSum", "ReduceMean", "ReduceMax", "ReduceProd", "Expand", "BitShift", "DepthToSpace", "SpaceToDepth", "Resize", "Concat", "MaxPool", "AveragePool", "Sin", "Cos", "Asin", "Ceil",
            "Floor", "Round", "LeakyRelu", "Not", "Greater", "PRelu", "ConvTranspose", "Gather", "Where", "Cast", "CumSum", "InstanceNorm",
            "Einsum", "Col2Im", "ConcatPart"]
OP = {n: i for i, n in enumerate(OP_NAMES) if i}

ATTR = {"c": 1, "lo": 2, "hi": 3, "p": 4, "eps": 5, "approx": 6, "axis": 7, "keepdims": 8, "start": 9, "end": 10,
        "bits": 11, "perm": 12, "shape": 13, "sizes": 14, "axes": 15, "block": 16, "scale": 17, "kernel": 18, "stride": 19, "pad": 20,
        "to": 21, "exclusive": 22, "reverse": 23, "labels_a": 24, "labels_b": 25, "labels_out": 26,
        "alpha": 1}      # LeakyRelu's slope travels as attribute C
CAST_TO = {"f32": 0, "bf16": 1, "i32": 2, "bool": 3}
_FLOAT_ATTRS = {"c", "lo", "hi", "p", "eps", "alpha"}

REWRITE_DEFAULT, REWRITE_NONE, REWRITE_CANON_MACRO, REWRITE_KEEP_LAYOUT = 0, 1, 2, 4
PLAN_FUSED, PLAN_UNFUSED, PLAN_STRICT_TABLE3, PLAN_ALLOW_PROLOGUE, PLAN_BEYOND_TABLE3 = 0, 1, 2, 4, 8
# kernel-selection overrides (same blocks and results, another kernel of the family)
PLAN_SPLIT_ALWAYS, PLAN_NO_K_SLICES, PLAN_NO_COLUMN_BLOCKS, PLAN_NO_TF32_GEMM = 0x100, 0x200, 0x400, 0x800
PLAN_NO_PAIR_GEMM, PLAN_NO_SPLIT_K, PLAN_NO_TMA_DWCONV, PLAN_NO_TILE_GEMM = 0x1000, 0x2000, 0x4000, 0x8000
PLAN_MBCONV_ALWAYS = 0x20000
PLAN_NO_SMALL_CONV = 0x40000
PLAN_CLUSTER_SPLIT_K = 0x10000
STATIC_WS_BYTES = 32 << 20


class Attr(C.Structure):
    _fields_ = [("key", C.c_int32), ("n", C.c_int32), ("i", C.c_int64 * 8), ("f", C.c_double)]


class RewriteStats(C.Structure):
    _fields_ = [("ops_before", C.c_int32), ("ops_after", C.c_int32), ("flops_before", C.c_int64),
                ("flops_after", C.c_int64), ("rules_applied", C.c_int32), ("applied_by_rule", C.c_int32 * 16),
                ("folded_constants", C.c_int32), ("layout_transposes_removed", C.c_int32)]


class PlanStats(C.Structure):
    _fields_ = [("n_ops", C.c_int32), ("n_blocks", C.c_int32), ("n_kernels", C.c_int32), ("fusion_rate", C.c_double),
                ("irs_bytes_unfused", C.c_int64), ("irs_bytes_fused", C.c_int64), ("workspace_bytes", C.c_int64),
                ("n_yellow_decisions", C.c_int32), ("n_yellow_fused", C.c_int32),
                ("n_profile_hits", C.c_int32), ("n_profile_misses", C.c_int32)]


class BlockDesc(C.Structure):
    _fields_ = [("family", C.c_int32), ("mapping", C.c_int32), ("n_ops", C.c_int32), ("op_kinds", C.c_int32 * 48),
                ("n_inputs", C.c_int32), ("n_outputs", C.c_int32), ("bytes_in", C.c_int64), ("bytes_out", C.c_int64),
                ("flops", C.c_int64), ("n_microops", C.c_int32), ("grid", C.c_int32), ("threads", C.c_int32),
                ("variant", C.c_int32)]


EXPORTS = ["dnnf_graph_create", "dnnf_graph_destroy", "dnnf_add_tensor", "dnnf_add_op", "dnnf_mark_output",
           "dnnf_tensor_info", "dnnf_op_mapping", "dnnf_mapping_check", "dnnf_rewrite", "dnnf_rule_name", "dnnf_plan",
           "dnnf_block_count", "dnnf_block_info", "dnnf_block_tensors", "dnnf_tensor_location", "dnnf_block_program", "dnnf_op_block", "dnnf_op_count", "dnnf_op_kind",
           "dnnf_workspace_size", "dnnf_workspace_zero_bytes", "dnnf_bind", "dnnf_bind_workspace", "dnnf_run", "dnnf_run_static_ws", "dnnf_run_block", "dnnf_status", "dnnf_selftest_wait_expiry",
           "dnnf_launch_count", "dnnf_last_error", "dnnf_version",
           "dnnf_profile_db_set", "dnnf_profile_db_get", "dnnf_profile_db_size", "dnnf_profile_db_clear", "dnnf_profile_db_save",
           "dnnf_profile_db_load", "dnnf_block_signature", "dnnf_profile_miss_count", "dnnf_profile_miss", "dnnf_profile_measure"]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2108_13342_b200.build` "
                          "(there is no non-CUDA fallback)")
    lib = C.CDLL(LIB_PATH)
    lib.dnnf_last_error.restype = C.c_char_p
    lib.dnnf_version.restype = C.c_char_p
    lib.dnnf_rule_name.restype = C.c_char_p
    lib.dnnf_last_error.argtypes = [C.c_void_p]
    lib.dnnf_graph_create.argtypes = [C.POINTER(C.c_void_p)]
    lib.dnnf_graph_destroy.argtypes = [C.c_void_p]
    lib.dnnf_add_tensor.argtypes = [C.c_void_p, C.c_char_p, C.c_int, C.c_int, C.POINTER(C.c_int64), C.c_int, C.POINTER(C.c_int)]
    lib.dnnf_add_op.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(Attr), C.c_int, C.c_int,
                                C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.dnnf_mark_output.argtypes = [C.c_void_p, C.c_int]
    lib.dnnf_tensor_info.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int64)]
    lib.dnnf_op_mapping.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int)]
    lib.dnnf_mapping_check.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.dnnf_rewrite.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(RewriteStats)]
    lib.dnnf_rule_name.argtypes = [C.c_int]
    lib.dnnf_plan.argtypes = [C.c_void_p, C.c_uint32, C.POINTER(PlanStats)]
    lib.dnnf_block_count.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    lib.dnnf_block_info.argtypes = [C.c_void_p, C.c_int, C.POINTER(BlockDesc)]
    lib.dnnf_block_program.argtypes = [C.c_void_p, C.c_int, C.c_char_p, C.c_size_t]
    lib.dnnf_block_tensors.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int)]
    lib.dnnf_tensor_location.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int64)]
    lib.dnnf_op_block.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int)]
    lib.dnnf_op_count.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    lib.dnnf_op_kind.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.dnnf_workspace_size.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
    lib.dnnf_workspace_zero_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
    lib.dnnf_profile_db_set.argtypes = [C.c_char_p, C.c_double]
    lib.dnnf_profile_db_get.argtypes = [C.c_char_p, C.POINTER(C.c_double)]
    lib.dnnf_profile_db_size.argtypes = [C.POINTER(C.c_size_t)]
    lib.dnnf_profile_db_save.argtypes = [C.c_char_p]
    lib.dnnf_profile_db_load.argtypes = [C.c_char_p, C.POINTER(C.c_int)]
    lib.dnnf_block_signature.argtypes = [C.c_void_p, C.c_int, C.c_char_p, C.c_size_t]
    lib.dnnf_profile_miss_count.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    lib.dnnf_profile_miss.argtypes = [C.c_void_p, C.c_int, C.c_char_p, C.c_size_t]
    lib.dnnf_profile_measure.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_int, C.POINTER(C.c_int)]
    lib.dnnf_bind.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
    lib.dnnf_bind_workspace.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
    lib.dnnf_run.argtypes = [C.c_void_p, C.c_void_p]
    lib.dnnf_run_static_ws.argtypes = [C.c_void_p, C.c_void_p]
    lib.dnnf_run_block.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
    lib.dnnf_status.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
    lib.dnnf_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
    lib.dnnf_launch_count.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    return lib


lib = _load()


def mapping_check(first, second):
    f, c = C.c_int(), C.c_int()
    rc = lib.dnnf_mapping_check(first, second, C.byref(f), C.byref(c))
    if rc:
        raise DnnfError(rc, "mapping_check")
    return f.value, c.value


class Graph:
    """Thin object wrapper over a dnnf_graph handle (same call names as the C ABI)."""

    def __init__(self):
        self.h = C.c_void_p()
        self._check(lib.dnnf_graph_create(C.byref(self.h)))
        self.names = {}          # tensor name -> id

    def __del__(self):
        if getattr(self, "h", None) and lib is not None:      # `lib` is gone during interpreter shutdown
            lib.dnnf_graph_destroy(self.h)
            self.h = None

    def _check(self, rc):
        if rc != OK:
            msg = lib.dnnf_last_error(self.h).decode() if self.h else ""
            raise DnnfError(rc, msg)

    def add_tensor(self, name, dtype, dims, kind=INPUT):
        arr = (C.c_int64 * len(dims))(*dims)
        tid = C.c_int()
        self._check(lib.dnnf_add_tensor(self.h, name.encode(), dtype, len(dims), arr, kind, C.byref(tid)))
        self.names[name] = tid.value
        return tid.value

    def add_op(self, kind, inputs, **attrs):
        if isinstance(kind, str):
            kind = OP[kind]
        ins = (C.c_int * len(inputs))(*inputs)
        if "equation" in attrs:                      # "bhqd,bhkd->bhqk": one integer per axis label
            attrs = dict(attrs)
            lhs, out = attrs.pop("equation").replace(" ", "").split("->")
            a, b = lhs.split(",")
            attrs.update(labels_a=[ord(c) for c in a], labels_b=[ord(c) for c in b], labels_out=[ord(c) for c in out])
        alist = []
        for k, v in attrs.items():
            if k == "approx" and isinstance(v, str):
                v = {"erf": 0, "tanh": 1}[v]
            if k == "direction":
                continue
            if k == "to" and isinstance(v, str):
                v = CAST_TO[v]
            a = Attr()
            a.key = ATTR[k]
            if k in _FLOAT_ATTRS:
                a.f = float(v); a.n = 0
            elif isinstance(v, (list, tuple)):
                a.n = len(v)
                for j, x in enumerate(v):
                    a.i[j] = int(x)
            else:
                a.n = 1; a.i[0] = int(v)
            alist.append(a)
        aarr = (Attr * max(1, len(alist)))(*alist)
        outs = (C.c_int * 8)()
        n = C.c_int()
        self._check(lib.dnnf_add_op(self.h, kind, len(inputs), ins, aarr, len(alist), 8, outs, C.byref(n)))
        return [outs[i] for i in range(n.value)]

    def mark_output(self, tid):
        self._check(lib.dnnf_mark_output(self.h, tid))

    def tensor_info(self, tid):
        dt, rk = C.c_int(), C.c_int()
        dims = (C.c_int64 * 6)()
        self._check(lib.dnnf_tensor_info(self.h, tid, C.byref(dt), C.byref(rk), dims))
        return dt.value, tuple(dims[i] for i in range(rk.value))

    def op_mapping(self, op_index):
        m = C.c_int()
        self._check(lib.dnnf_op_mapping(self.h, op_index, C.byref(m)))
        return m.value

    def rewrite(self, flags=REWRITE_DEFAULT):
        st = RewriteStats()
        self._check(lib.dnnf_rewrite(self.h, flags, C.byref(st)))
        return st

    def plan(self, flags=PLAN_FUSED):
        st = PlanStats()
        self._check(lib.dnnf_plan(self.h, flags, C.byref(st)))
        return st

    def block_count(self):
        n = C.c_int()
        self._check(lib.dnnf_block_count(self.h, C.byref(n)))
        return n.value

    def block_info(self, b):
        d = BlockDesc()
        self._check(lib.dnnf_block_info(self.h, b, C.byref(d)))
        return d

    def block_tensors(self, b):
        """(input tensor ids, output tensor ids) of a planned block."""
        ins, outs = (C.c_int * 16)(), (C.c_int * 16)()
        ni, no = C.c_int(), C.c_int()
        self._check(lib.dnnf_block_tensors(self.h, b, ins, 16, C.byref(ni), outs, 16, C.byref(no)))
        return [ins[i] for i in range(min(ni.value, 16))], [outs[i] for i in range(min(no.value, 16))]

    def tensor_location(self, tid):
        """(where, offset): 0 caller-bound, 1 workspace at `offset` bytes, 2 inside its block, 3 alias of bound tensor `offset`."""
        w, off = C.c_int(), C.c_int64()
        self._check(lib.dnnf_tensor_location(self.h, tid, C.byref(w), C.byref(off)))
        return w.value, off.value

    def block_program(self, b):
        buf = C.create_string_buffer(4096)
        self._check(lib.dnnf_block_program(self.h, b, buf, 4096))
        return buf.value.decode()

    def op_block(self, op_index):
        b = C.c_int()
        self._check(lib.dnnf_op_block(self.h, op_index, C.byref(b)))
        return b.value

    def op_count(self):
        n = C.c_int()
        self._check(lib.dnnf_op_count(self.h, C.byref(n)))
        return n.value

    def op_kind(self, i):
        k, a = C.c_int(), C.c_int()
        self._check(lib.dnnf_op_kind(self.h, i, C.byref(k), C.byref(a)))
        return k.value, bool(a.value)

    def workspace_size(self):
        n = C.c_size_t()
        self._check(lib.dnnf_workspace_size(self.h, C.byref(n)))
        return n.value

    def workspace_zero_bytes(self):
        n = C.c_size_t(0)
        self._check(lib.dnnf_workspace_zero_bytes(self.h, C.byref(n)))
        return n.value

    def block_signature(self, block):
        buf = C.create_string_buffer(4096)
        self._check(lib.dnnf_block_signature(self.h, block, buf, 4096))
        return buf.value.decode()

    def profile_misses(self):
        n = C.c_int(0)
        self._check(lib.dnnf_profile_miss_count(self.h, C.byref(n)))
        out = []
        for i in range(n.value):
            buf = C.create_string_buffer(4096)
            self._check(lib.dnnf_profile_miss(self.h, i, buf, 4096))
            out.append(buf.value.decode())
        return out

    def profile_measure(self, scratch_ptr, scratch_bytes, stream=0, iters=20):
        n = C.c_int(0)
        self._check(lib.dnnf_profile_measure(self.h, C.c_void_p(scratch_ptr), scratch_bytes, C.c_void_p(stream), iters, C.byref(n)))
        return n.value

    def bind(self, tid, dev_ptr):
        self._check(lib.dnnf_bind(self.h, tid, C.c_void_p(dev_ptr)))

    def bind_workspace(self, dev_ptr, nbytes):
        self._check(lib.dnnf_bind_workspace(self.h, C.c_void_p(dev_ptr), nbytes))

    def run(self, stream=0):
        self._check(lib.dnnf_run(self.h, C.c_void_p(stream)))

    def run_static_ws(self, stream=0):
        """dnnf_run with the between-block intermediates in the library's built-in array (no workspace needed)."""
        self._check(lib.dnnf_run_static_ws(self.h, C.c_void_p(stream)))

    def run_block(self, b, stream=0):
        self._check(lib.dnnf_run_block(self.h, b, C.c_void_p(stream)))

    def selftest_wait_expiry(self, limit_ns, stream=0):
        self._check(lib.dnnf_selftest_wait_expiry(self.h, int(limit_ns), C.c_void_p(stream)))

    def status(self):
        s, b = C.c_int(), C.c_int()
        self._check(lib.dnnf_status(self.h, C.byref(s), C.byref(b)))
        return s.value, b.value

    def launch_count(self):
        n = C.c_int()
        self._check(lib.dnnf_launch_count(self.h, C.byref(n)))
        return n.value

    def blocks(self):
        out = []
        for b in range(self.block_count()):
            d = self.block_info(b)
            out.append({"family": FAMILY_NAMES[d.family], "mapping": MAPPING_NAMES[d.mapping],
                        "ops": [OP_NAMES[d.op_kinds[i]] for i in range(min(d.n_ops, 48))],
                        "bytes": d.bytes_in + d.bytes_out, "flops": d.flops, "grid": d.grid,
                        "threads": d.threads, "variant": d.variant, "n_microops": d.n_microops,
                        "n_inputs": d.n_inputs, "n_outputs": d.n_outputs})
        return out


# ---- profiling database (process-wide) -------------------------------------------------------------
def profile_db_set(signature, us):
    if lib.dnnf_profile_db_set(signature.encode(), float(us)) != 0:
        raise ValueError("bad profiling-database entry")


def profile_db_get(signature):
    v = C.c_double(0)
    return v.value if lib.dnnf_profile_db_get(signature.encode(), C.byref(v)) == 0 else None


def profile_db_size():
    n = C.c_size_t(0)
    lib.dnnf_profile_db_size(C.byref(n))
    return n.value


def profile_db_clear():
    lib.dnnf_profile_db_clear()


def profile_db_save(path):
    if lib.dnnf_profile_db_save(path.encode()) != 0:
        raise OSError(f"cannot write {path}")


def profile_db_load(path):
    n = C.c_int(0)
    if lib.dnnf_profile_db_load(path.encode(), C.byref(n)) != 0:
        raise OSError(f"cannot read {path}")
    return n.value

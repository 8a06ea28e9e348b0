"""Pins for the oracle: closed forms, invariants, brute-force index loops.

Every check here compares an oracle operator with something other than
itself: a value fixed by mathematics, a pure-Python loop over indices written
from the operator's definition, or an identity between two different oracle
code paths.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import interp as O
from paper_2108_13342_b200 import workloads as W


def rnd(shape, seed=0, lo=-2.0, hi=2.0):
    return np.random.default_rng(seed).uniform(lo, hi, size=shape)


# ---- elementwise closed forms ------------------------------------------------

def test_sigmoid_points():
    x = np.array([0.0, math.log(3.0), -math.log(3.0), 40.0, -40.0])
    y = O.op_sigmoid(x)
    assert y[0] == 0.5
    assert abs(y[1] - 0.75) < 1e-15 and abs(y[2] - 0.25) < 1e-15
    assert abs(y[3] - 1.0) < 1e-15 and 0.0 < y[4] < 1e-17


def test_swish_and_gelu_reflection():
    # x*sigma(x) - (-x)*sigma(-x) = x ; GELU(x) - GELU(-x) = x for both variants
    x = rnd((257,), 1, -6, 6)
    sw = lambda v: v * O.op_sigmoid(v)
    assert np.max(np.abs(sw(x) - sw(-x) - x)) < 1e-14
    for ap in ("erf", "tanh"):
        f = lambda v: O.op_gelu(v, ap)
        assert np.max(np.abs(f(x) - f(-x) - x)) < 1e-14
        assert f(np.zeros(1))[0] == 0.0


def test_gelu_tabulated():
    # Phi(1) = 0.8413447460685429, Phi(2) = 0.9772498680518208 (standard normal CDF)
    y = O.op_gelu(np.array([1.0, 2.0, -1.0]), "erf")
    assert abs(y[0] - 0.8413447460685429) < 1e-15
    assert abs(y[1] - 2 * 0.9772498680518208) < 1e-15
    assert abs(y[2] + (1 - 0.8413447460685429)) < 1e-15
    # tanh form, tabulated to 30 digits with an arbitrary-precision package (not recomputed here):
    # x = 1, 2, -1, 0.5.  A wrong 0.044715, a wrong sqrt(2/pi) or a misplaced cube moves these by > 1e-6.
    tab = {1.0: 0.841191990608276704781995777045, 2.0: 1.95459769408777501878104138615,
           -1.0: -0.158808009391723295218004222955, 0.5: 0.345714009825143922037757257365}
    for x, want in tab.items():
        assert abs(O.op_gelu(np.array([x]), "tanh")[0] - want) < 1e-15
    # the two variants agree to about 1e-3 on [-4, 4] (sanity, catches a wrong constant)
    x = np.linspace(-4, 4, 101)
    assert np.max(np.abs(O.op_gelu(x, "erf") - O.op_gelu(x, "tanh"))) < 1.1e-3


def test_erf_points():
    assert O.op_erf(np.array([0.0]))[0] == 0.0
    assert abs(O.op_erf(np.array([0.5]))[0] - 0.5204998778130465) < 1e-15
    assert abs(O.op_erf(np.array([-1.0]))[0] + 0.8427007929497149) < 1e-15


def test_clip_scaleshift_points():
    x = np.array([-1.0, 0.0, 3.0, 6.0, 7.5])
    assert list(O.op_clip(x, 0.0, 6.0)) == [0.0, 0.0, 3.0, 6.0, 6.0]
    assert list(O.op_relu(x)) == [0.0, 0.0, 3.0, 6.0, 7.5]
    a = np.arange(24, dtype=float).reshape(1, 2, 3, 4)
    s = np.array([1.0, 2.0, 3.0, 4.0]); t = np.array([0.5, 0.0, -1.0, 2.0])
    y = O.op_scaleshift(a, s, t, axis=-1)
    for n, h, w, c in itertools.product(range(1), range(2), range(3), range(4)):
        assert y[n, h, w, c] == a[n, h, w, c] * s[c] + t[c]
    s2 = np.array([2.0, -1.0]); t2 = np.array([1.0, 3.0])
    y = O.op_scaleshift(a, s2, t2, axis=1)          # NCHW flavour
    assert y[0, 1, 2, 3] == a[0, 1, 2, 3] * -1.0 + 3.0


def test_unary_inverse_pairs():
    x = rnd((64,), 2, 0.1, 3.0)
    assert np.max(np.abs(O.op_log(O.op_exp(x)) - x)) < 1e-14
    assert np.max(np.abs(O.op_square(O.op_sqrt(x)) - x)) < 1e-14
    assert np.max(np.abs(O.op_recip(x) * x - 1)) < 1e-15
    assert np.all(O.op_abs(-x) == x) and np.all(O.op_neg(x) == -x)
    assert np.max(np.abs(O.op_pow(x, 2.0) - x * x)) < 1e-14
    assert np.max(np.abs(O.op_pow(x, 0.5) - np.sqrt(x))) < 1e-15
    assert np.all(O.op_sub(x, x) == 0) and np.all(O.op_div(x, x) == 1)
    assert np.all(O.op_mulc(x, 0.5) == x / 2) and np.all(O.op_addc(x, 1.0) == x + 1)
    assert abs(O.op_tanh(np.array([0.5]))[0] - 0.46211715726000974) < 1e-15


def test_bitshift():
    a = np.array([1.0, 3.0, -4.0, 10.0])
    assert list(O.op_bitshift(a, 2)) == [4.0, 12.0, -16.0, 40.0]
    assert list(O.op_bitshift(np.array([9.0, 8.0]), 2, "right")) == [2.0, 2.0]


# ---- broadcasting against explicit expansion ---------------------------------

def test_broadcast_vs_explicit_loops():
    a = rnd((2, 3, 4, 5), 3)
    for bshape in [(5,), (4, 1), (3, 1, 1), (1, 3, 1, 1), (2, 1, 4, 1), (1,)]:
        b = rnd(bshape, 4)
        bb = np.zeros(a.shape)
        pad = (1,) * (4 - len(bshape)) + tuple(bshape)
        for idx in itertools.product(*[range(s) for s in a.shape]):
            j = tuple(i if p > 1 else 0 for i, p in zip(idx, pad))
            bb[idx] = b.reshape(pad)[j]
        assert np.array_equal(O.op_add(a, b), a + bb)
        assert np.array_equal(O.op_mul(a, b), a * bb)
        assert np.array_equal(O.op_sub(a, b), a - bb)
        assert np.array_equal(O.op_expand(b, a.shape), bb)


# ---- Reorganize / Shuffle ------------------------------------------------------

@pytest.mark.parametrize("shape", [(2, 3, 5, 7), (3, 5, 2), (7, 3)])
def test_transpose_bruteforce_all_perms(shape):
    x = np.arange(int(np.prod(shape)), dtype=float).reshape(shape)
    for perm in itertools.permutations(range(len(shape))):
        y = O.op_transpose(x, perm)
        assert y.shape == tuple(shape[p] for p in perm)
        for idx in itertools.product(*[range(s) for s in y.shape]):
            src = [0] * len(shape)
            for k, p in enumerate(perm):
                src[p] = idx[k]
            assert y[idx] == x[tuple(src)]
        inv = np.argsort(perm)
        assert np.array_equal(O.op_transpose(y, inv), x)


def test_nchw_nhwc_roundtrip_bits():
    x = rnd((2, 5, 3, 7), 5)
    x[0, 0, 0, 0] = -0.0
    x[1, 2, 1, 3] = np.inf
    y = O.op_transpose(x, (0, 2, 3, 1))
    assert y[1, 2, 6, 4] == x[1, 4, 2, 6]
    z = O.op_transpose(y, (0, 3, 1, 2))
    assert np.array_equal(z.view(np.uint64), x.view(np.uint64))


def test_reorganize_keeps_flat_order():
    x = rnd((2, 3, 4), 6)
    flat = x.ravel()
    assert np.array_equal(O.op_reshape(x, (4, 6)).ravel(), flat)
    assert O.op_reshape(x, (4, 6))[2, 3] == flat[2 * 6 + 3]
    assert np.array_equal(O.op_flatten(x, 1).shape, (2, 12))
    assert np.array_equal(O.op_flatten(x, 2).ravel(), flat)
    u = O.op_unsqueeze(x, [0, 3])
    assert u.shape == (1, 2, 3, 1, 4) and np.array_equal(u.ravel(), flat)
    assert O.op_squeeze(u, [0, 3]).shape == (2, 3, 4)


def test_split_concat_slice():
    x = rnd((3, 10, 2), 7)
    parts = O.op_split(x, 1, (2, 5, 3))
    assert [p.shape[1] for p in parts] == [2, 5, 3]
    assert parts[1][2, 4, 1] == x[2, 2 + 4, 1]
    assert np.array_equal(O.op_concat(parts, 1), x)
    assert np.array_equal(O.op_slice(x, 1, 2, 7), parts[1])
    assert np.array_equal(O.op_split(x, -1, (1, 1))[1][..., 0], x[..., 1])


def test_gather():
    x = rnd((5, 3), 8)
    y = O.op_gather(x, np.array([4.0, 0.0, 4.0]), 0)
    assert np.array_equal(y, np.stack([x[4], x[0], x[4]]))
    # any axis, index tensors of any rank: the index axes take the place of the gathered axis
    t = rnd((3, 4, 5), 9)
    idx = np.array([[3.0, 0.0], [1.0, 1.0], [2.0, 3.0]])
    y = O.op_gather(t, idx, 1)
    assert y.shape == (3, 3, 2, 5)
    for a, i, j, c in itertools.product(range(3), range(3), range(2), range(5)):
        assert y[a, i, j, c] == t[a, int(idx[i, j]), c]
    y = O.op_gather(t, np.array([4.0, 4.0, 0.0]), -1)
    for a, b, i in itertools.product(range(3), range(4), range(3)):
        assert y[a, b, i] == t[a, b, [4, 4, 0][i]]


def test_further_one_to_one_operators_at_known_points():
    assert np.allclose(O.op_sin(np.array([0.0, math.pi / 6, math.pi / 2, -math.pi / 2])), [0.0, 0.5, 1.0, -1.0], atol=1e-15)
    assert np.allclose(O.op_cos(np.array([0.0, math.pi / 3, math.pi])), [1.0, 0.5, -1.0], atol=1e-15)
    assert np.allclose(O.op_asin(np.array([0.0, 0.5, 1.0, -1.0])), [0.0, math.pi / 6, math.pi / 2, -math.pi / 2], atol=1e-15)
    x = rnd((50,), 40, -1.0, 1.0)
    assert np.allclose(O.op_sin(x) ** 2 + O.op_cos(x) ** 2, 1.0, atol=1e-15)
    assert np.allclose(O.op_sin(O.op_asin(x)), x, atol=1e-15)
    v = np.array([-2.5, -1.5, -0.5, -0.2, 0.0, 0.2, 0.5, 1.5, 2.5, 3.0])
    assert np.array_equal(O.op_ceil(v), [-2, -1, -0, -0, 0, 1, 1, 2, 3, 3])
    assert np.array_equal(O.op_floor(v), [-3, -2, -1, -1, 0, 0, 0, 1, 2, 3])
    assert np.array_equal(O.op_round(v), [-2, -2, -0, -0, 0, 0, 0, 2, 2, 3])          # ties go to the even neighbour
    assert np.array_equal(O.op_leakyrelu(np.array([-4.0, 0.0, 3.0]), 0.25), [-1.0, 0.0, 3.0])
    assert np.array_equal(O.op_not(np.array([0.0, 1.0, 0.0])), [1.0, 0.0, 1.0])
    a = np.array([[1.0, 5.0, 3.0], [4.0, 2.0, 6.0]])
    assert np.array_equal(O.op_greater(a, np.array([2.0, 2.0, 6.0])), [[0, 1, 0], [1, 0, 0]])      # broadcast over rows
    assert np.array_equal(O.op_greater(a, a), np.zeros((2, 3)))
    assert np.array_equal(O.op_prelu(np.array([[-2.0, 4.0], [-1.0, -8.0]]), np.array([0.5, 0.25])), [[-1.0, 4.0], [-0.5, -2.0]])
    assert np.array_equal(O.op_prelu(x, np.ones(50)), x)
    assert np.array_equal(O.op_prelu(x, np.zeros(50)), O.op_relu(x))


def test_depthtospace_spacetodepth_resize_index_loops():
    """Each element against the index formula of the operator's definition, in pure-Python loops; the two Shuffle
    operators undo each other; nearest-neighbour enlargement equals numpy's repeat along both image axes."""
    b = 2
    x = rnd((2, 3, 2, 12), 21)
    y = O.op_depthtospace(x, b)
    assert y.shape == (2, 6, 4, 3)
    for n, h, w, i, j, c in itertools.product(range(2), range(3), range(2), range(b), range(b), range(3)):
        assert y[n, h * b + i, w * b + j, c] == x[n, h, w, (i * b + j) * 3 + c]
    assert np.array_equal(O.op_spacetodepth(y, b), x)
    z = rnd((1, 6, 9, 2), 22)
    s2d = O.op_spacetodepth(z, 3)
    assert s2d.shape == (1, 2, 3, 18)
    for h, w, i, j, c in itertools.product(range(2), range(3), range(3), range(3), range(2)):
        assert s2d[0, h, w, (i * 3 + j) * 2 + c] == z[0, h * 3 + i, w * 3 + j, c]
    assert np.array_equal(O.op_depthtospace(s2d, 3), z)
    r = O.op_resize_nearest(z, 2)
    assert r.shape == (1, 12, 18, 2)
    for h, w, c in itertools.product(range(12), range(18), range(2)):
        assert r[0, h, w, c] == z[0, h // 2, w // 2, c]
    assert np.array_equal(r, np.repeat(np.repeat(z, 2, axis=1), 2, axis=2))
    assert np.array_equal(O.op_resize_nearest(z, 1), z)


# ---- Many-to-Many --------------------------------------------------------------

def test_convtranspose_bruteforce_and_pointwise_case():
    """Scalar loops from the scatter definition, with overlapping patches too (stride < kernel); a 1x1 kernel at
    stride 1 is the pointwise convolution."""
    x = rnd((2, 3, 4, 3), 41); w = rnd((3, 2, 2, 5), 42)
    for s in (2, 1):
        y = O.op_convtranspose(x, w, s)
        ref = np.zeros_like(y)
        for n, h, ww, c, i, j, o in itertools.product(range(2), range(3), range(4), range(3), range(2), range(2), range(5)):
            ref[n, h * s + i, ww * s + j, o] += x[n, h, ww, c] * w[c, i, j, o]
        assert y.shape == (2, (3 - 1) * s + 2, (4 - 1) * s + 2, 5)
        assert np.max(np.abs(y - ref)) < 1e-14
    w1 = rnd((3, 1, 1, 5), 43)
    assert np.allclose(O.op_convtranspose(x, w1, 1), O.op_conv1x1(x, w1[:, 0, 0, :]), atol=1e-14)
    # padding cuts the border: the gather form, written as index loops over the OUTPUT (kernel 4, stride 2, pad 1: the
    # result is exactly twice the input's size), and kernel 3, stride 2, pad 1
    for k, s, p in ((4, 2, 1), (3, 2, 1), (3, 1, 1)):
        w = rnd((3, k, k, 2), 44 + k)
        y = O.op_convtranspose(x, w, s, p)
        ho, wo = (3 - 1) * s + k - 2 * p, (4 - 1) * s + k - 2 * p
        assert y.shape == (2, ho, wo, 2)
        ref = np.zeros_like(y)
        for n, oh, ow, o in itertools.product(range(2), range(ho), range(wo), range(2)):
            acc = 0.0
            for i, j in itertools.product(range(k), range(k)):
                if (oh + p - i) % s or (ow + p - j) % s:
                    continue
                h, ww = (oh + p - i) // s, (ow + p - j) // s
                if 0 <= h < 3 and 0 <= ww < 4:
                    acc += sum(x[n, h, ww, c] * w[c, i, j, o] for c in range(3))
            ref[n, oh, ow, o] = acc
        assert np.max(np.abs(y - ref)) < 1e-13
    assert O.op_convtranspose(x, rnd((3, 4, 4, 2), 50), 2, 1).shape == (2, 6, 8, 2)
    # stride 1, kernel 3, pad 1 is a same-size correlation with the flipped kernel: a delta input returns the flipped taps
    d = np.zeros((1, 5, 5, 1)); d[0, 2, 2, 0] = 1.0
    wk = rnd((1, 3, 3, 1), 51)
    assert np.allclose(O.op_convtranspose(d, wk, 1, 1)[0, 1:4, 1:4, 0], wk[0, :, :, 0], atol=1e-15)


def test_pooling_bruteforce_and_special_cases():
    """Scalar loops from the definition (window clipped to the image; the mean counts only elements inside it);
    a global average pool is the mean over the image; a 1x1 window is the identity; a constant image stays
    constant under AveragePool whatever the padding; non-overlapping 2x2 MaxPool equals a reshape + max."""
    x = rnd((2, 5, 7, 3), 31)
    for k, s, p in [(3, 2, 1), (2, 2, 0), (3, 1, 1), (2, 1, 0), (3, 2, 0)]:
        ho, wo = (5 + 2 * p - k) // s + 1, (7 + 2 * p - k) // s + 1
        mx, av = O.op_maxpool(x, k, s, p), O.op_avgpool(x, k, s, p)
        assert mx.shape == av.shape == (2, ho, wo, 3)
        for n, i, j, c in itertools.product(range(2), range(ho), range(wo), range(3)):
            vals = [x[n, a, b, c] for a in range(i * s - p, i * s - p + k) for b in range(j * s - p, j * s - p + k)
                    if 0 <= a < 5 and 0 <= b < 7]
            assert mx[n, i, j, c] == max(vals)
            assert abs(av[n, i, j, c] - sum(vals) / len(vals)) < 1e-14
    sq = rnd((2, 6, 6, 4), 32)
    assert np.allclose(O.op_avgpool(sq, 6, 1, 0)[:, 0, 0, :], sq.mean(axis=(1, 2)), atol=1e-14)
    assert np.array_equal(O.op_maxpool(sq, 1, 1, 0), sq)
    assert np.allclose(O.op_avgpool(np.full((1, 5, 5, 2), 3.25), 3, 2, 1), 3.25)
    assert np.array_equal(O.op_maxpool(sq, 2, 2, 0), sq.reshape(2, 3, 2, 3, 2, 4).max(axis=(2, 4)))


def test_matmul_bruteforce_and_identities():
    a = rnd((2, 3, 4, 5), 9)
    b = rnd((3, 5, 6), 10)             # broadcast over the leading batch dim
    c = O.op_matmul(a, b)
    ref = np.zeros((2, 3, 4, 6))
    for n, h, i, j in itertools.product(range(2), range(3), range(4), range(6)):
        s = 0.0
        for k in range(5):
            s += a[n, h, i, k] * b[h, k, j]
        ref[n, h, i, j] = s
    assert np.max(np.abs(c - ref)) < 1e-14
    # not symmetric in its operands: A(4x5) x ones(5x6) gives row sums of A
    assert np.max(np.abs(O.op_matmul(a[0, 0], np.ones((5, 6)))[:, 0] - a[0, 0].sum(1))) < 1e-14
    assert np.array_equal(O.op_matmul(a[0, 0], np.eye(5)), a[0, 0])
    # exact associativity on small integers
    ri = np.random.default_rng(11)
    A, B, C = (ri.integers(-4, 5, size=s).astype(float) for s in [(6, 7), (7, 5), (5, 3)])
    assert np.array_equal(O.op_matmul(O.op_matmul(A, B), C), O.op_matmul(A, O.op_matmul(B, C)))


def test_conv1x1_equals_matmul_over_pixels():
    x = rnd((2, 3, 4, 5), 12); w = rnd((5, 7), 13)
    y = O.op_conv1x1(x, w)
    assert y.shape == (2, 3, 4, 7)
    ref = O.op_matmul(x.reshape(-1, 5), w).reshape(2, 3, 4, 7)
    assert np.max(np.abs(y - ref)) < 1e-14
    assert abs(y[1, 2, 3, 6] - sum(x[1, 2, 3, c] * w[c, 6] for c in range(5))) < 1e-14


def test_dwconv_delta_ones_and_bruteforce():
    x = rnd((2, 5, 6, 3), 14)
    k = np.zeros((3, 3, 3)); k[1, 1, :] = 1.0
    assert np.array_equal(O.op_dwconv3x3(x, k), x)
    ones = np.ones((1, 4, 5, 2))
    y = O.op_dwconv3x3(ones, np.ones((3, 3, 2)))
    assert y[0, 0, 0, 0] == 4 and y[0, 0, 2, 1] == 6 and y[0, 2, 2, 0] == 9 and y[0, 3, 4, 1] == 4
    k = rnd((3, 3, 3), 15)
    y = O.op_dwconv3x3(x, k)
    for n, h, w, c in itertools.product(range(2), range(5), range(6), range(3)):
        s = 0.0
        for dh in (-1, 0, 1):
            for dw in (-1, 0, 1):
                hh, ww = h + dh, w + dw
                if 0 <= hh < 5 and 0 <= ww < 6:
                    s += x[n, hh, ww, c] * k[dh + 1, dw + 1, c]
        assert abs(y[n, h, w, c] - s) < 1e-14
    # asymmetric kernel: a single tap at (0, 2) shifts the image down-left
    k = np.zeros((3, 3, 3)); k[0, 2, :] = 1.0
    y = O.op_dwconv3x3(x, k)
    assert y[0, 2, 2, 1] == x[0, 1, 3, 1] and y[0, 0, 0, 0] == 0.0


def test_softmax_invariants():
    x = rnd((3, 4, 17), 16, -5, 5)
    p = O.op_softmax(x)
    assert np.max(np.abs(p.sum(-1) - 1)) < 1e-14
    assert p.min() >= 0 and p.max() <= 1
    assert np.max(np.abs(O.op_softmax(x + 123.0) - p)) < 1e-13
    assert abs(p[1, 2, 3] - math.exp(x[1, 2, 3]) / sum(math.exp(v) for v in x[1, 2])) < 1e-15
    # two-element row is the logistic function of the difference
    q = O.op_softmax(np.array([[1.0, 3.0]]))
    assert abs(q[0, 1] - 1 / (1 + math.exp(-2.0))) < 1e-15
    # causal mask: row i is uniform 1/(i+1) on a constant row and exactly 0 above the diagonal
    m = W.causal_mask(6).astype(float)
    pc = O.op_softmax(np.zeros((6, 6)) + m)
    for i in range(6):
        assert np.max(np.abs(pc[i, :i + 1] - 1.0 / (i + 1))) < 1e-15
        assert np.all(pc[i, i + 1:] == 0.0)
    assert pc[0, 0] == 1.0
    # other axis
    p0 = O.op_softmax(x, axis=0)
    assert np.max(np.abs(p0.sum(0) - 1)) < 1e-14


def test_layernorm_closed_forms():
    x = rnd((5, 48), 17, -3, 3)
    g1, b0 = np.ones(48), np.zeros(48)
    eps = 1e-5
    y = O.op_layernorm(x, g1, b0, eps=eps)
    assert np.max(np.abs(y.mean(-1))) < 1e-14
    v = x.var(-1)                                   # biased
    assert np.max(np.abs(y.var(-1) - v / (v + eps))) < 1e-13
    # an unbiased variance would give (n-1)/n of that
    g = rnd((48,), 18); b = rnd((48,), 19)
    y2 = O.op_layernorm(x, g, b, eps=eps)
    assert np.max(np.abs(y2 - (y * g + b))) < 1e-14
    c = O.op_layernorm(np.full((2, 48), 3.25), g, b, eps=eps)
    assert np.array_equal(c, np.stack([b, b]))
    # scale invariance as eps -> 0
    ya = O.op_layernorm(x, g1, b0, eps=0.0); yb = O.op_layernorm(7.0 * x, g1, b0, eps=0.0)
    assert np.max(np.abs(ya - yb)) < 1e-13
    # eps sits inside the square root: a row with variance v scales by 1/sqrt(v+eps)
    r = np.array([[1.0, -1.0]])
    assert abs(O.op_layernorm(r, np.ones(2), np.zeros(2), eps=3.0)[0, 0] - 0.5) < 1e-15


def test_reductions():
    x = rnd((3, 4, 5), 20, 0.5, 1.5)
    assert np.max(np.abs(O.op_reducesum(x, -1, 1)[1, 2, 0] - sum(x[1, 2]))) < 1e-14
    assert O.op_reducesum(x, -1, 0).shape == (3, 4)
    assert abs(O.op_reducemean(x, 1, 1)[2, 0, 3] - sum(x[2, :, 3]) / 4) < 1e-15
    assert abs(O.op_reduceprod(x, -1, 1)[0, 1, 0] - math.prod(x[0, 1])) < 1e-14
    assert O.op_reducemax(x, 0, 0)[3, 4] == max(x[:, 3, 4])


# ---- Table 4: both sides of each printed rewrite identity ----------------------

def _t4_cases():
    m, n = 4, 6
    A = rnd((m, n), 21, 0.5, 2.0); B = rnd((m, n), 22, 0.5, 2.0); C = rnd((m, n), 23, -2.0, 2.0)
    rs = lambda v: O.op_reducesum(v, -1, 1)
    Ai = np.random.default_rng(24).integers(0, 9, size=(m, n)).astype(float)
    As = rnd((m, n), 25, -0.5, 0.5)
    return [
        ("assoc1", O.op_recip(A) * O.op_recip(A * B), O.op_square(O.op_recip(A)) * O.op_recip(B)),
        ("assoc2", (A * O.op_sqrt(B)) * (O.op_sqrt(B) * C), A * B * C),
        ("assoc3", O.op_abs(C) * B * O.op_abs(-A), O.op_abs(C * -A) * B),
        ("assoc4", (A * rs(B)) * (rs(B) * C), A * O.op_square(rs(B)) * C),
        # The row as printed (A.C + A.B -> (A+B).C) is not an identity; the shared factor must be
        # the one kept outside the sum (Fig. 2(b): two Mul by the same weight C, then Add).
        ("dist1", A * C + B * C, (A + B) * C),
        ("dist1-left-factor", A * C + A * B, A * (B + C)),
        ("dist2", A + A * B, A * (B + 1.0)),
        ("dist3", O.op_square(A + B) - (A + B) * C, (A + B) * (A + B - C)),
        ("comm1", A * B, B * A),
        ("comm2", rs(O.op_bitshift(Ai, 3)), O.op_bitshift(rs(Ai), 3)),
        ("comm3", O.op_reduceprod(O.op_exp(As), -1, 1), O.op_exp(rs(As))),
    ]


@pytest.mark.parametrize("case", _t4_cases(), ids=lambda c: c[0])
def test_table4_identities(case):
    _, lhs, rhs = case
    assert lhs.shape == rhs.shape
    assert np.max(np.abs(lhs - rhs) / (np.abs(rhs) + 1e-300)) < 1e-12


# ---- interpreter plumbing --------------------------------------------------------

def test_run_graph_composes_and_materialises():
    wl = W.swish_transpose(n=1, c=3, h=2, w=5)
    env = O.run_graph(wl.graph, wl.inputs, keep_all=True)
    X = wl.inputs["X"].astype(float); b = wl.inputs["b"].astype(float)
    Y = env["Y"]
    assert Y.shape == (1, 2, 5, 3)
    for c, h, w in itertools.product(range(3), range(2), range(5)):
        t = (X[0, c, h, w] + b[0, c, 0, 0]) * 0.5
        assert abs(Y[0, h, w, c] - t / (1 + math.exp(-t))) < 1e-15
    assert len(env) == 2 + 5          # every intermediate is kept


def test_encoder_primitives_match_macro_ops():
    # the 9-operator LayerNorm and 5-operator GELU expansions equal the single-operator forms
    g = W.GraphDesc()
    g.ext("x", (4, 16)); g.ext("g", (16,)); g.ext("b", (16,))
    y = W._layernorm_primitives(g, "x", "g", "b", 1e-5)
    z = W._gelu_erf_primitives(g, y)
    g.mark_output(y); g.mark_output(z)
    ins = {"x": rnd((4, 16), 30), "g": rnd((16,), 31), "b": rnd((16,), 32)}
    out = O.run_graph(g, ins)
    ln = O.op_layernorm(ins["x"], ins["g"], ins["b"], eps=1e-5)
    assert np.max(np.abs(out[y] - ln)) < 1e-13
    assert np.max(np.abs(out[z] - O.op_gelu(ln, "erf"))) < 1e-13


def test_encoder_graph_shape_and_op_count():
    wl = W.encoder(layers=2, batch=2, seq=8, hidden=16, heads=2, ffn=32)
    assert len(wl.graph.ops) == 2 * 48
    out = O.run_graph(wl.graph, wl.inputs)
    (y,) = out.values()
    assert y.shape == (2, 8, 16) and np.all(np.isfinite(y))
    # causality: changing the last token leaves earlier positions of the output unchanged
    ins2 = dict(wl.inputs); x2 = wl.inputs["x"].copy(); x2[:, -1, :] += 1.0; ins2["x"] = x2
    (y2,) = O.run_graph(wl.graph, ins2).values()
    assert np.max(np.abs(y2[:, :-1] - y[:, :-1])) < 1e-12
    assert np.max(np.abs(y2[:, -1] - y[:, -1])) > 1e-3


# ---- generators --------------------------------------------------------------------

def test_generators_are_counter_based_and_distributed():
    a = W.uniform(1, 3, (1000,), -1.0, 1.0); b = W.uniform(1, 3, (10,), -1.0, 1.0)
    assert np.array_equal(a[:10], b)                    # independent of length
    assert not np.array_equal(a, W.uniform(1, 4, (1000,), -1.0, 1.0))
    assert a.min() >= -1 and a.max() < 1 and abs(a.mean()) < 0.06
    z = W.normal(2, 1, (20000,), 1.0, 0.5)
    assert abs(z.mean() - 1.0) < 0.02 and abs(z.std() - 0.5) < 0.02
    r = W.round_to_bf16(np.array([1.0, 1.00390625, 1.01171875, 3.14159], dtype=np.float32))
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.015625    # ties to even, both directions
    assert np.array_equal(W.bf16_bits_to_f32(W.bf16_bits(r)), r)


# ---- Where, Cast, CumSum, InstanceNormalization (Table 2) -------------------------------------------------------------

def test_where_index_loops_and_selection_semantics():
    r = np.random.default_rng(5)
    cond = (r.random((3, 1, 5)) > 0.5).astype(np.float64)
    a = r.standard_normal((1, 4, 5)); b = r.standard_normal((3, 4, 1))
    y = O.op_where(cond, a, b)
    assert y.shape == (3, 4, 5)
    for i, j, k in itertools.product(range(3), range(4), range(5)):
        assert y[i, j, k] == (a[0, j, k] if cond[i, 0, k] != 0 else b[i, j, 0])
    np.testing.assert_array_equal(O.op_where(np.ones((2, 3)), a[0, :2, :3], 7.0), a[0, :2, :3])
    np.testing.assert_array_equal(O.op_where(np.zeros((2, 3)), a[0, :2, :3], 7.0), np.full((2, 3), 7.0))
    # the branch that is not taken leaves no trace: the usual masking with -inf, and a NaN on the other side
    y = O.op_where(np.array([1.0, 0.0, 1.0]), np.array([1.0, np.nan, 3.0]), np.array([-np.inf, 2.0, -np.inf]))
    np.testing.assert_array_equal(y, [1.0, 2.0, 3.0])
    # Where(Greater(x, 0), x, 0) is Relu; Where(Not(c), a, b) swaps the branches
    x = r.standard_normal(50)
    np.testing.assert_array_equal(O.op_where(O.op_greater(x, 0.0), x, 0.0), O.op_relu(x))
    c = (r.random(50) > 0.5).astype(float)
    np.testing.assert_array_equal(O.op_where(O.op_not(c), x, -x), O.op_where(c, -x, x))


def test_cast_points_and_properties():
    import torch
    # bfloat16 keeps 8 significand bits: spacing 2^-7 in [1, 2); ties go to the even neighbour
    e = 2.0 ** -7
    pts = {1.0: 1.0, 1.0 + e / 2: 1.0, 1.0 + 3 * e / 2: 1.0 + 2 * e, 1.0 + e / 2 + 2.0 ** -20: 1.0 + e, -1.0 - 3 * e / 2: -1.0 - 2 * e,
           3.140625: 3.140625, 0.0: 0.0, 2.0 ** -130: 2.0 ** -130, 65280.0: 65280.0, 1e-3: 131 / 128 * 2.0 ** -10}        # 0.001 = 1.024 * 2^-10 and 1.024 * 128 = 131.07
    for x, want in pts.items():
        assert O.op_cast(np.array([x]), "bf16")[0] == want, (x, want)
    r = np.random.default_rng(6)
    x = np.concatenate([r.standard_normal(4000) * 10.0 ** r.integers(-6, 6, 4000), [0.0, -0.0, 1e30, -1e-30]])
    y = O.op_cast(x, "bf16")
    x32 = x.astype(np.float32).astype(np.float64)
    assert np.all(np.abs(y - x32) <= 2.0 ** -8 * np.abs(x32))                         # half a unit in the last place: 2^-8 * 2^exponent
    assert np.all((y.astype(np.float32).view(np.uint32) & 0xFFFF) == 0)               # representable in 16 bits
    np.testing.assert_array_equal(O.op_cast(y, "bf16"), y)                            # idempotent
    lib = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(y, lib)                                             # the library's conversion
    # float -> integer conversion goes toward zero; bool is "non-zero"; f32 leaves values alone
    v = np.array([-2.7, -2.0, -0.5, 0.0, 0.5, 1.999, 2.0, 1e6 + 0.75])
    np.testing.assert_array_equal(O.op_cast(v, "i32"), [float(int(t)) for t in v])
    np.testing.assert_array_equal(O.op_cast(v, "bool"), [1, 1, 1, 0, 1, 1, 1, 1])
    np.testing.assert_array_equal(O.op_cast(v, "f32"), v)
    np.testing.assert_array_equal(O.op_cast(v, "bool"), O.op_not(O.op_not(v)))


def test_cumsum_running_loops_and_closed_forms():
    r = np.random.default_rng(7)
    x = r.standard_normal((3, 4, 6))
    for axis in (0, 1, 2, -1):
        for exclusive in (0, 1):
            for reverse in (0, 1):
                y = O.op_cumsum(x, axis, exclusive, reverse)
                ax = axis % 3
                xm = np.moveaxis(x, ax, -1); ym = np.moveaxis(y, ax, -1)
                L = xm.shape[-1]
                for i, j in itertools.product(range(xm.shape[0]), range(xm.shape[1])):
                    order = range(L - 1, -1, -1) if reverse else range(L)
                    run = 0.0
                    for k in order:
                        if exclusive:
                            assert abs(ym[i, j, k] - run) < 1e-12
                        run += xm[i, j, k]
                        if not exclusive:
                            assert abs(ym[i, j, k] - run) < 1e-12
    n = 37
    np.testing.assert_array_equal(O.op_cumsum(np.ones(n)), np.arange(1, n + 1))
    np.testing.assert_array_equal(O.op_cumsum(np.ones(n), exclusive=1), np.arange(n))
    np.testing.assert_array_equal(O.op_cumsum(np.ones(n), reverse=1), np.arange(n, 0, -1))
    np.testing.assert_array_equal(O.op_cumsum(np.arange(1, n + 1)), [k * (k + 1) // 2 for k in range(1, n + 1)])   # triangular numbers
    q = 0.5 ** np.arange(20)
    np.testing.assert_allclose(O.op_cumsum(q), 2.0 - q, rtol=1e-15)                                                # geometric series
    y = O.op_cumsum(x, -1)
    np.testing.assert_allclose(y[..., -1], O.op_reducesum(x, -1, 0), rtol=1e-14)                                    # last element is the sum
    np.testing.assert_allclose(np.diff(y, axis=-1), x[..., 1:], atol=1e-14)                                         # differences give x back
    np.testing.assert_allclose(O.op_cumsum(x, -1) - O.op_cumsum(x, -1, exclusive=1), x, atol=1e-14)
    np.testing.assert_allclose(O.op_cumsum(x, -1) + O.op_cumsum(x, -1, exclusive=1, reverse=1),
                               np.broadcast_to(x.sum(-1, keepdims=True), x.shape), atol=1e-13)


def test_instancenorm_index_loops_and_invariants():
    r = np.random.default_rng(8)
    N, H, Wd, Cc = 2, 3, 5, 4
    x = r.standard_normal((N, H, Wd, Cc)) * 3 + 1
    s = r.uniform(0.5, 1.5, Cc); b = r.uniform(-1, 1, Cc)
    eps = 1e-5
    y = O.op_instancenorm(x, s, b, eps)
    for n, c in itertools.product(range(N), range(Cc)):
        vals = [x[n, h, w, c] for h in range(H) for w in range(Wd)]
        m = sum(vals) / len(vals)
        v = sum((t - m) ** 2 for t in vals) / len(vals)
        for h, w in itertools.product(range(H), range(Wd)):
            assert abs(y[n, h, w, c] - ((x[n, h, w, c] - m) / math.sqrt(v + eps) * s[c] + b[c])) < 1e-12
    # unit scale, zero shift: every (image, channel) plane has mean 0 and variance var / (var + eps)
    z = O.op_instancenorm(x, np.ones(Cc), np.zeros(Cc), eps)
    var = x.var(axis=(1, 2))
    np.testing.assert_allclose(z.mean(axis=(1, 2)), 0.0, atol=1e-14)
    np.testing.assert_allclose(z.var(axis=(1, 2)), var / (var + eps), rtol=1e-12)
    # a per-plane affine change of the input is removed (exactly so as eps -> 0); planes do not see each other
    a = r.uniform(0.5, 2.0, (N, 1, 1, Cc)); t = r.standard_normal((N, 1, 1, Cc))
    np.testing.assert_allclose(O.op_instancenorm(a * x + t, s, b, 0.0), O.op_instancenorm(x, s, b, 0.0), atol=1e-12)
    x2 = x.copy(); x2[1, :, :, 2] = r.standard_normal((H, Wd))
    y2 = O.op_instancenorm(x2, s, b, eps)
    mask = np.ones_like(x, dtype=bool); mask[1, :, :, 2] = False
    np.testing.assert_array_equal(y2[mask], y[mask])
    # a constant plane maps to the shift; it is LayerNorm over the H*W positions of the channels-first view
    np.testing.assert_allclose(O.op_instancenorm(np.full((1, 2, 2, Cc), 5.0), s, b, eps), np.broadcast_to(b, (1, 2, 2, Cc)), atol=1e-12)
    xt = x.transpose(0, 3, 1, 2).reshape(N, Cc, H * Wd)
    ln = O.op_layernorm(xt, np.ones(H * Wd), np.zeros(H * Wd), -1, eps).reshape(N, Cc, H, Wd).transpose(0, 2, 3, 1)
    np.testing.assert_allclose(y, ln * s + b, atol=1e-12)


def test_einsum_index_loops_and_matrix_product_cases():
    r = np.random.default_rng(9)
    a = r.standard_normal((2, 3, 4, 5)); b = r.standard_normal((2, 3, 6, 5))
    y = O.op_einsum(a, b, "bhqd,bhkd->bhqk")
    assert y.shape == (2, 3, 4, 6)
    for i, j, q, k in itertools.product(range(2), range(3), range(4), range(6)):
        assert abs(y[i, j, q, k] - sum(a[i, j, q, d] * b[i, j, k, d] for d in range(5))) < 1e-12
    np.testing.assert_allclose(y, O.op_matmul(a, np.swapaxes(b, -1, -2)), atol=1e-12)         # Q K^T
    # a permuted result, two summed labels, free labels on both sides that are not adjacent
    a = r.standard_normal((3, 2, 4)); b = r.standard_normal((4, 5, 2))
    y = O.op_einsum(a, b, "mck,knc->nm")
    for n, m in itertools.product(range(5), range(3)):
        assert abs(y[n, m] - sum(a[m, c, k] * b[k, n, c] for c in range(2) for k in range(4))) < 1e-12
    # plain cases: matrix product, matrix-vector, a 1x1 convolution over NHWC pixels
    A = r.standard_normal((4, 7)); Bm = r.standard_normal((7, 3)); v = r.standard_normal(7)
    np.testing.assert_allclose(O.op_einsum(A, Bm, "ik,kj->ij"), O.op_matmul(A, Bm), atol=1e-12)
    np.testing.assert_allclose(O.op_einsum(A, v, "ik,k->i"), A @ v, atol=1e-12)
    x = r.standard_normal((2, 3, 3, 7))
    np.testing.assert_allclose(O.op_einsum(x, Bm, "nhwc,co->nhwo"), O.op_conv1x1(x, Bm), atol=1e-12)
    # linear in each operand; ones as the second operand sum the label away
    np.testing.assert_allclose(O.op_einsum(2.0 * A, Bm, "ik,kj->ij"), 2.0 * O.op_einsum(A, Bm, "ik,kj->ij"), atol=1e-12)
    np.testing.assert_allclose(O.op_einsum(A, np.ones((7, 1)), "ik,kj->ij")[:, 0], O.op_reducesum(A, -1, 0), atol=1e-12)

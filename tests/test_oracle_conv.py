"""Pins for the convolution oracle: a brute-force dense conv written here in numpy loops, a
library fp64 convolution, a plain matrix product for 1x1, and hand-worked fixtures."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def brute_dense_conv(w_ohwi, x, stride, pad, dil, bias=None, relu=False):
    """Seven nested loops over (n, oh, ow, o, kh, kw, c), fp64, written apart from the oracle."""
    co, kh, kw, ci = w_ohwi.shape
    b, h, wd, _ = x.shape
    ho = (h + 2 * pad[0] - dil[0] * (kh - 1) - 1) // stride[0] + 1
    wo = (wd + 2 * pad[1] - dil[1] * (kw - 1) - 1) // stride[1] + 1
    y = np.zeros((b, ho, wo, co), dtype=np.float64)
    for n in range(b):
        for oh in range(ho):
            for ow in range(wo):
                for o in range(co):
                    acc = 0.0 if bias is None else float(bias[o])
                    for a in range(kh):
                        ih = oh * stride[0] - pad[0] + a * dil[0]
                        if not 0 <= ih < h:
                            continue
                        for c_ in range(kw):
                            iw = ow * stride[1] - pad[1] + c_ * dil[1]
                            if not 0 <= iw < wd:
                                continue
                            for c in range(ci):
                                acc += float(w_ohwi[o, a, c_, c]) * float(x[n, ih, iw, c])
                    y[n, oh, ow, o] = max(acc, 0.0) if relu else acc
    return y


def _pruned_dense(w, n, m, t):
    values, indices = oracle.prune(w, n, m, t)
    dense = oracle.expand(values, indices, int(np.prod(w.shape[1:])), t).reshape(w.shape)
    return values, indices, dense


def _load_golden(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            rows[key] = np.array([float(v) for v in vals], dtype=np.float32)
    return rows


# ---- hand-worked fixtures ----------------------------------------------------------------------

@pytest.mark.parametrize("key,stride,pad,dil,shape", [("s1p1", 1, 1, 1, (4, 4)), ("s2p1", 2, 1, 1, (2, 2)),
                                                      ("d2p2", 1, 2, 2, (4, 4))])
def test_hand_worked_3x3(key, stride, pad, dil, shape):
    g = _load_golden("hand_conv3x3.txt")
    x = g["image"].reshape(1, 4, 4, 1)
    w = g["kernel"].reshape(1, 3, 3, 1)
    values, indices = oracle.prune(w, 1, 1, 1)  # keep everything
    y = oracle.conv2d(values, indices, 3, 3, 1, 1, x, (stride, stride), (pad, pad), (dil, dil))
    assert y.shape == (1,) + shape + (1,)
    assert y.reshape(-1).tolist() == g[key].tolist()


def test_hand_worked_pruned_two_channels():
    # 1x1 conv, 4 input channels, two output tiles of one row each, 2:4.
    # row 0 = (3, -1, 0.5, 2) keeps cols {0, 3}; row 1 = (0, 4, -4, 1) keeps cols {1, 2}
    w = np.array([[3, -1, 0.5, 2], [0, 4, -4, 1]], dtype=np.float32).reshape(2, 1, 1, 4)
    x = np.array([[1, 10, 100, 1000], [2, 3, 5, 7]], dtype=np.float32).reshape(1, 1, 2, 4)
    values, indices = oracle.prune(w, 2, 4, 1)
    y = oracle.conv2d(values, indices, 1, 1, 4, 1, x, bias=np.array([1, -1], dtype=np.float32))
    # pixel 0: 3*1 + 2*1000 + 1 = 2004 ; 4*10 - 4*100 - 1 = -361.  pixel 1: 6+14+1 = 21 ; 12-20-1 = -9
    assert y.reshape(2, 2).tolist() == [[2004, -361], [21, -9]]
    y = oracle.conv2d(values, indices, 1, 1, 4, 1, x, bias=np.array([1, -1], dtype=np.float32), relu=True)
    assert y.reshape(2, 2).tolist() == [[2004, 0], [21, 0]]


# ---- brute force on the zero-expanded weights ---------------------------------------------------

CASES = [
    # b, h, w, ci, co, kh, kw, stride, pad, dil, n, m, t
    (2, 6, 7, 4, 6, 3, 3, (1, 1), (1, 1), (1, 1), 2, 4, 2),
    (1, 9, 8, 8, 5, 3, 2, (2, 1), (1, 0), (1, 2), 1, 4, 4),   # asymmetric everything, tail tile
    (2, 7, 7, 3, 4, 5, 3, (1, 2), (2, 1), (1, 1), 3, 4, 3),   # K = 45: tail group
    (1, 10, 9, 8, 8, 2, 3, (2, 2), (0, 2), (3, 2), 2, 8, 8),  # dilation, 2:8
    (3, 5, 5, 16, 7, 1, 1, (1, 1), (0, 0), (1, 1), 1, 8, 1),  # 1x1, T = 1
    (1, 8, 8, 4, 4, 3, 3, (2, 2), (1, 1), (1, 1), 2, 4, 8),   # T larger than c_out
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("relu", [False, True])
def test_equals_bruteforce_dense_conv_on_expanded_weights(case, relu):
    b, h, wd, ci, co, kh, kw, stride, pad, dil, n, m, t = case
    r = _rng(hash(case) % 1000)
    w = r.standard_normal((co, kh, kw, ci)).astype(np.float32)
    x = r.standard_normal((b, h, wd, ci)).astype(np.float32)
    bias = r.standard_normal(co).astype(np.float32)
    values, indices, dense = _pruned_dense(w, n, m, t)
    got = oracle.conv2d(values, indices, kh, kw, ci, t, x, stride, pad, dil, bias, relu)
    ref = brute_dense_conv(dense, x, stride, pad, dil, bias, relu)
    assert got.shape == ref.shape
    # both sides accumulate in fp64 (different order) and round once: within one fp32 ulp
    np.testing.assert_allclose(got, ref.astype(np.float32), rtol=2.5e-7, atol=1e-6)


def test_integer_inputs_agree_exactly_with_bruteforce():
    r = _rng(11)
    w = r.integers(-4, 5, size=(8, 3, 3, 8)).astype(np.float32)
    x = r.integers(-4, 5, size=(2, 6, 6, 8)).astype(np.float32)
    bias = r.integers(-4, 5, size=8).astype(np.float32)
    values, indices, dense = _pruned_dense(w, 2, 4, 4)
    got = oracle.conv2d(values, indices, 3, 3, 8, 4, x, (1, 1), (1, 1), (1, 1), bias, True)
    ref = brute_dense_conv(dense, x, (1, 1), (1, 1), (1, 1), bias, True)
    assert np.array_equal(got.astype(np.float64), ref)


# ---- library cross-checks ------------------------------------------------------------------------

@pytest.mark.parametrize("n,m,t", [(2, 4, 8), (1, 4, 32), (2, 8, 16), (4, 4, 8)])
def test_equals_library_fp64_conv(n, m, t):
    r = _rng(20 + n + m)
    co, kh, kw, ci = 32, 3, 3, 16
    w = r.standard_normal((co, kh, kw, ci)).astype(np.float32)
    x = r.standard_normal((2, 14, 14, ci)).astype(np.float32)
    bias = r.standard_normal(co).astype(np.float32)
    values, indices, dense = _pruned_dense(w, n, m, t)
    got = oracle.conv2d(values, indices, kh, kw, ci, t, x, (2, 1), (1, 1), (1, 1), bias, False)
    ref = torch.nn.functional.conv2d(
        torch.from_numpy(x).double().permute(0, 3, 1, 2), torch.from_numpy(dense).double().permute(0, 3, 1, 2),
        torch.from_numpy(bias).double(), stride=(2, 1), padding=(1, 1)).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(got, ref.astype(np.float32), rtol=2.5e-7, atol=1e-6)
    if n == m:  # N = M: nothing pruned, the result is the unpruned dense convolution
        assert np.array_equal(dense, w)


def test_1x1_equals_plain_matrix_product():
    r = _rng(31)
    ci, co = 64, 24
    w = r.standard_normal((co, 1, 1, ci)).astype(np.float32)
    x = r.standard_normal((2, 5, 6, ci)).astype(np.float32)
    values, indices, dense = _pruned_dense(w, 1, 4, 8)
    got = oracle.conv2d(values, indices, 1, 1, ci, 8, x)
    # triple loop written here
    xm = x.reshape(-1, ci).astype(np.float64)
    wm = dense.reshape(co, ci).astype(np.float64)
    ref = np.zeros((xm.shape[0], co))
    for p in range(xm.shape[0]):
        for o in range(co):
            s = 0.0
            for c in range(ci):
                s += xm[p, c] * wm[o, c]
            ref[p, o] = s
    np.testing.assert_allclose(got.reshape(-1, co), ref.astype(np.float32), rtol=2.5e-7, atol=1e-6)
    np.testing.assert_allclose(got.reshape(-1, co), (xm @ wm.T).astype(np.float32), rtol=2.5e-7, atol=1e-6)


def test_rejects_bad_arguments():
    values = np.zeros((2, 2), np.float32)
    indices = np.zeros((1, 2), np.uint16)
    x = np.zeros((1, 2, 2, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.conv2d(values, indices, 3, 3, 4, 2, x)  # 3x3 on 2x2 without padding: no output
    with pytest.raises(ValueError):
        oracle.conv2d(values, indices, 1, 1, 5, 2, x)  # channel mismatch


# ---- shortcut-adding form (residual blocks of the ResNets of Sec. 4.5) -------------------------------

def _res_case(seed=5, integer=False):
    rng = np.random.default_rng(seed)
    c_out, kh, kw, c_in = 12, 3, 3, 8
    if integer:
        w = rng.integers(-3, 4, (c_out, kh, kw, c_in)).astype(np.float32)
        x = rng.integers(-3, 4, (2, 7, 6, c_in)).astype(np.float32)
        b = rng.integers(-3, 4, (c_out,)).astype(np.float32)
    else:
        w = rng.standard_normal((c_out, kh, kw, c_in)).astype(np.float32)
        x = rng.standard_normal((2, 7, 6, c_in)).astype(np.float32)
        b = rng.standard_normal((c_out,)).astype(np.float32)
    v, i = oracle.prune(w, 2, 4, 4)
    return v, i, x, b, (kh, kw, c_in, 4)


def test_residual_form_with_zero_or_no_residual_is_the_plain_form():
    v, i, x, b, (kh, kw, c_in, t) = _res_case()
    plain = oracle.conv2d(v, i, kh, kw, c_in, t, x, (1, 1), (1, 1), (1, 1), b, True)
    none = oracle.conv2d_res(v, i, kh, kw, c_in, t, x, (1, 1), (1, 1), (1, 1), b, None, True)
    zero = oracle.conv2d_res(v, i, kh, kw, c_in, t, x, (1, 1), (1, 1), (1, 1), b, np.zeros_like(plain), True)
    assert np.array_equal(plain, none) and np.array_equal(plain, zero)


def test_residual_is_added_before_the_activation_exactly_on_integers():
    v, i, x, b, (kh, kw, c_in, t) = _res_case(integer=True)
    lin = oracle.conv2d(v, i, kh, kw, c_in, t, x, (2, 1), (1, 0), (1, 1), b, False)       # no activation
    res = np.random.default_rng(9).integers(-20, 21, lin.shape).astype(np.float32)
    got = oracle.conv2d_res(v, i, kh, kw, c_in, t, x, (2, 1), (1, 0), (1, 1), b, res, True)
    assert np.array_equal(got, np.maximum(lin + res, 0.0))      # everything is an exact small integer
    # a ReLU applied before the addition would give something else on this data
    assert not np.array_equal(got, np.maximum(lin, 0.0) + res)


def test_residual_form_equals_library_fp64_conv_plus_residual():
    torch = pytest.importorskip("torch")
    v, i, x, b, (kh, kw, c_in, t) = _res_case(seed=11)
    dense = oracle.expand(v, i, kh * kw * c_in, t).reshape(v.shape[0], kh, kw, c_in)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2),
                                     torch.from_numpy(dense).double().permute(0, 3, 1, 2),
                                     torch.from_numpy(b).double(), stride=1, padding=1).permute(0, 2, 3, 1).numpy()
    res = np.random.default_rng(3).standard_normal(ref.shape).astype(np.float32)
    want = np.maximum(ref + res.astype(np.float64), 0.0)
    got = oracle.conv2d_res(v, i, kh, kw, c_in, t, x, (1, 1), (1, 1), (1, 1), b, res, True)
    assert np.allclose(got, want, rtol=0, atol=1e-5 * np.abs(want).max())

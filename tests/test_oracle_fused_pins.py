"""Pins for the oracle of the operators fused behind the convolution (residual addition, ReLU,
2x2 max-pool, re-quantisation): hand-computed values, an array-library restatement with a
different structure, algebraic identities, and exact integer arithmetic for the re-quantised
codes.  The convolution in front of them is pinned in test_oracle_pins.py."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_fused_4x4.txt")
PRE = np.array([[1, -2, 3, 4], [-5, 6, -7, 8], [9, -10, 11, -12], [-13, 14, -15, 16]], dtype=np.float64)
RES = np.array([[0, 5, -10, 0], [1, 1, 1, 1], [-9, 20, -11, 2], [0, 0, 30, -40]], dtype=np.float64)


def _gold():
    out = {}
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("|")
        out[k.strip()] = [float(t) for t in v.split()]
    return out


def _identity_layer(pre, dtype):
    """A layer whose convolution output is `pre`: one channel, the centre tap with weight 1."""
    x = pre.reshape(1, 4, 4, 1)
    w = np.zeros((1, 1, 3, 3))
    w[0, 0, 1, 1] = 1
    masks = np.array([0x01B], dtype=np.uint16)          # taps 0, 1, 3, 4: contains the centre
    pid = np.zeros((1, 1), np.int16)
    if dtype == "i8":
        return x.astype(np.uint8), w.astype(np.int8), pid, masks
    return x, w, pid, masks


def test_hand_computed_fp():
    g = _gold()
    x, w, pid, masks = _identity_layer(PRE, "f64")
    res = RES.reshape(1, 4, 4, 1)
    assert oracle.conv_fused(x, w, pid, masks, relu=True, residual=res, pool=2).ravel().tolist() == g["pool_relu_res"]
    assert oracle.conv_fused(x, w, pid, masks, relu=False, residual=res, pool=2).ravel().tolist() == g["pool_res"]
    assert oracle.conv_fused(x, w, pid, masks, relu=False, pool=2).ravel().tolist() == g["pool_plain"]
    assert oracle.conv_fused(-x, w, pid, masks, relu=False, pool=2).ravel().tolist() == g["pool_neg"]
    # no pool: the element-wise part alone
    v = oracle.conv_fused(x, w, pid, masks, relu=True, residual=res)
    assert v.reshape(4, 4).tolist() == np.maximum(PRE + RES, 0).tolist()


def test_hand_computed_requantisation():
    g = _gold()
    # integer layer: x >= 0 is required of uint8 activations, so pre is built from a bias
    x = np.zeros((1, 4, 4, 1), np.uint8)
    w = np.zeros((1, 1, 3, 3), np.int8)
    pid = np.zeros((1, 1), np.int16)
    masks = np.array([0x01B], dtype=np.uint16)
    x[0, :, :, 0] = (PRE + 20).astype(np.uint8)          # 20 + pre is in 5..36
    w[0, 0, 1, 1] = 1
    bias = np.array([-20], np.int32)
    res = RES.reshape(1, 4, 4, 1).astype(np.int32)
    v = oracle.conv_fused(x, w, pid, masks, bias=bias, residual=res)
    assert v.dtype == np.int64 and v.reshape(4, 4).tolist() == (PRE + RES).astype(int).tolist()
    half = np.array([0.5], np.float32)
    q = oracle.conv_fused(x, w, pid, masks, bias=bias, relu=True, residual=res, pool=2, requant_scale=half)
    assert q.dtype == np.uint8 and q.ravel().tolist() == g["requant_half"]
    q = oracle.conv_fused(x, w, pid, masks, bias=bias, relu=True, residual=res, pool=2,
                          requant_scale=np.array([20.0], np.float32), zero_point=3)
    assert q.ravel().tolist() == g["requant_clamp"]
    q = oracle.conv_fused(x, w, pid, masks, bias=bias, relu=False, residual=res, requant_scale=half, zero_point=10)
    assert q.reshape(4, 4)[3].tolist() == g["requant_row3"]


def _case(dtype, stride=1, seed=7, n=2, ci=5, co=6, h=8, w=12):
    spec = wl.LayerSpec("t", n, ci, co, h, w, stride, dtype, 0.3, 12, 0.5,
                        "u01" if dtype == "i8" else "upm1", 0.3, False, seed % 89)
    return wl.make_layer(spec, seed=seed)


@pytest.mark.parametrize("stride", [1, 2])
def test_pool_against_array_reshape(stride):
    d = _case("f32", stride)
    pre = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, stride=stride)
    n, ho, wo, c = pre.shape
    res = wl.normal(3, "AUX", 1, pre.size).reshape(pre.shape)
    got = oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=stride, residual=res, pool=2)
    want = np.maximum(pre + res, 0).reshape(n, ho // 2, 2, wo // 2, 2, c).max(axis=(2, 4))
    assert np.array_equal(got, want)
    # ReLU and max commute
    lin = oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=False, stride=stride, residual=res, pool=2)
    assert np.array_equal(np.maximum(lin, 0), got)
    # nothing fused = the plain layer
    assert np.array_equal(oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=stride),
                          oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=stride))
    # a zero residual changes nothing, and the residual enters linearly before the activation
    assert np.array_equal(oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, stride=stride, residual=np.zeros_like(pre)), pre)
    assert np.allclose(oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, stride=stride, residual=res) - pre, res, rtol=0, atol=1e-12)


def test_odd_extents_cannot_be_pooled():
    d = _case("f32", 1, h=7, w=8)
    with pytest.raises(ValueError):
        oracle.conv_fused(d.x, d.w, d.pid, d.masks, pool=2)


def _rne_div_pow2(v, k):
    """round-half-even of v / 2^k in exact integer arithmetic."""
    q, r = divmod(v, 1 << k)
    half = 1 << (k - 1)
    if r > half or (r == half and (q & 1)):
        q += 1
    return q


def test_requantisation_exact_integer_arithmetic():
    d = _case("i8", 1, ci=6, co=5)
    pre = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias)
    assert np.abs(pre).max() < 2 ** 24                   # int32 -> fp32 is exact here
    res = wl.integers(5, "AUX", 2, pre.size, -3000, 3000).reshape(pre.shape).astype(np.int32)
    # power-of-two scales: the fp32 product is exact, so the code is the exactly rounded quotient
    ks = np.array([6, 7, 8, 9, 10], dtype=np.int64)
    scale = (2.0 ** -ks).astype(np.float32)
    for relu, zp in ((True, 0), (False, 128)):
        got = oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=relu, residual=res,
                                requant_scale=scale, zero_point=zp)
        v = pre + res
        if relu:
            v = np.maximum(v, 0)
        want = np.empty_like(v)
        for idx in np.ndindex(*v.shape):
            want[idx] = min(255, max(0, _rne_div_pow2(int(v[idx]), int(ks[idx[3]])) + zp))
        assert np.array_equal(got.astype(np.int64), want)
    # general scales: every code is within half a step of the exact rational value, allowing
    # for the one fp32 rounding of the product (relative 2^-24)
    scale = (wl.uniform01(9, "AUX", 3, 5) * 0.01 + 1e-4).astype(np.float32)
    got = oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, requant_scale=scale).astype(np.int64)
    v = np.maximum(pre, 0)
    for idx in list(np.ndindex(*v.shape))[::7]:
        exact = Fraction(int(v[idx])) * Fraction(float(scale[idx[3]]))
        if exact > 255:
            assert got[idx] == 255
        else:
            assert abs(Fraction(int(got[idx])) - exact) <= Fraction(1, 2) + abs(exact) * Fraction(1, 2 ** 23)
    # and the same decision restated with an array library in fp32
    want = np.clip(np.rint(v.astype(np.float32) * scale[None, None, None, :]), 0, 255).astype(np.int64)
    assert np.array_equal(got, want)


def test_integer_pool_and_residual():
    d = _case("i8", 2, ci=4, co=3, h=8, w=8)
    pre = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, stride=2)
    n, ho, wo, c = pre.shape
    res = wl.integers(6, "AUX", 4, pre.size, -(1 << 15), 1 << 15).reshape(pre.shape).astype(np.int32)
    got = oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=2, residual=res, pool=2)
    want = np.maximum(pre + res, 0).reshape(n, ho // 2, 2, wo // 2, 2, c).max(axis=(2, 4))
    assert got.dtype == np.int64 and np.array_equal(got, want)

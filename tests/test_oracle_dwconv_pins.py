"""Pins of the depthwise pattern-pruned oracle: a case worked by hand, the full layer's
oracle with a diagonal connectivity (a different routine), closed forms and invariants."""
import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import workloads as wl


def test_hand_computed_case():
    """One channel, 3x3 input 1..9, pattern keeps taps (0,1), (1,0), (1,1), (1,2) with weights
    2, -1, 3, 0.5: worked by hand for stride 1 and for the single stride-2 corner outputs."""
    x = np.arange(1.0, 10.0).reshape(1, 3, 3, 1)
    w = np.zeros((1, 3, 3))
    w[0, 0, 1], w[0, 1, 0], w[0, 1, 1], w[0, 1, 2] = 2.0, -1.0, 3.0, 0.5
    w[0, 2, 2] = 100.0                                       # not in the pattern: ignored
    masks = np.array([(1 << 1) | (1 << 3) | (1 << 4) | (1 << 5)], np.uint16)
    pid = np.array([0], np.int16)
    y, s = oracle.depthwise(x, w, pid, masks, bias=np.array([0.25]), with_scale=True)
    # y[oy,ox] = 0.25 + 2*x[oy-1,ox] - x[oy,ox-1] + 3*x[oy,ox] + 0.5*x[oy,ox+1]
    want = np.array([[0.25 + 3 * 1 + 0.5 * 2, 0.25 - 1 + 3 * 2 + 0.5 * 3, 0.25 - 2 + 3 * 3],
                     [0.25 + 2 * 1 + 3 * 4 + 0.5 * 5, 0.25 + 2 * 2 - 4 + 3 * 5 + 0.5 * 6, 0.25 + 2 * 3 - 5 + 3 * 6],
                     [0.25 + 2 * 4 + 3 * 7 + 0.5 * 8, 0.25 + 2 * 5 - 7 + 3 * 8 + 0.5 * 9, 0.25 + 2 * 6 - 8 + 3 * 9]])
    assert np.array_equal(y[0, :, :, 0], want)
    want_s = np.array([[0.25 + 3 + 1, 0.25 + 1 + 6 + 1.5, 0.25 + 2 + 9],
                       [0.25 + 2 + 12 + 2.5, 0.25 + 4 + 4 + 15 + 3, 0.25 + 6 + 5 + 18],
                       [0.25 + 8 + 21 + 4, 0.25 + 10 + 7 + 24 + 4.5, 0.25 + 12 + 8 + 27]])
    assert np.array_equal(s[0, :, :, 0], want_s)
    y2 = oracle.depthwise(x, w, pid, masks, bias=np.array([0.25]), stride=2)
    assert np.array_equal(y2[0, :, :, 0], want[::2, ::2])


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_equals_the_full_layer_with_diagonal_connectivity(stride, dtype):
    """The depthwise layer is the full pattern-pruned layer whose kernel (oc, ic) exists only for oc == ic."""
    d = wl.make_depthwise(wl.DepthwiseSpec("t", 2, 6, 7, 9, stride, dtype, 0.34, 8, "upm1", 0.3, True, 1))
    c = 6
    wfull = np.zeros((c, c, 3, 3), d.w.dtype)
    pidfull = np.full((c, c), -1, np.int16)
    for ch in range(c):
        wfull[ch, ch] = d.w[ch]
        pidfull[ch, ch] = d.pid[ch]
    for relu in (False, True):
        y, s = oracle.depthwise(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=relu, stride=stride, with_scale=True)
        yf, sf = oracle.conv(d.x, wfull, pidfull, d.masks, bias=d.bias, relu=relu, stride=stride, with_scale=True)
        assert np.array_equal(y, yf) and np.array_equal(s, sf)
    assert (d.pid == -1).sum() == 2


def test_closed_forms_and_what_contributes_nothing():
    d = wl.make_depthwise(wl.DepthwiseSpec("t", 1, 8, 6, 6, 1, "f32", 0.25, 8, "upm1", 0.2, False, 2))
    ones = np.ones_like(d.x)
    y = oracle.depthwise(ones, d.w, d.pid, d.masks)
    for ch in range(8):
        kept = [t for t in range(9) if d.pid[ch] >= 0 and (d.masks[d.pid[ch]] >> t) & 1]
        want = sum(float(d.w[ch].reshape(9)[t]) for t in kept)      # interior: all four taps inside
        assert np.allclose(y[0, 1:-1, 1:-1, ch], want, rtol=0, atol=1e-15)
        if d.pid[ch] < 0:
            assert (y[..., ch] == 0).all()                            # a removed kernel gives nothing
    # values at pruned taps never matter
    wp = d.w.astype(np.float64).copy()
    for ch in range(8):
        for t in range(9):
            if d.pid[ch] < 0 or not (d.masks[d.pid[ch]] >> t) & 1:
                wp[ch].reshape(9)[t] = 1e30
    assert np.array_equal(oracle.depthwise(d.x, wp, d.pid, d.masks, bias=d.bias),
                          oracle.depthwise(d.x, d.w, d.pid, d.masks, bias=d.bias))
    # zero input gives the bias; channels do not mix
    assert np.array_equal(oracle.depthwise(np.zeros_like(d.x), d.w, d.pid, d.masks, bias=d.bias),
                          np.broadcast_to(d.bias.astype(np.float64), y.shape))
    x2 = d.x.copy()
    x2[..., 3] = 7.0
    ya, yb = oracle.depthwise(d.x, d.w, d.pid, d.masks), oracle.depthwise(x2, d.w, d.pid, d.masks)
    assert np.array_equal(np.delete(ya, 3, axis=3), np.delete(yb, 3, axis=3))


def test_linearity_and_error_scale():
    d = wl.make_depthwise(wl.DepthwiseSpec("t", 2, 5, 5, 8, 2, "f32", 0.0, 12, "upm1", 0.2, False, 3))
    xa = d.x.astype(np.float64)
    xb = xa[::-1] * 0.5
    f = lambda x, **kw: oracle.depthwise(x, d.w, d.pid, d.masks, stride=2, **kw)
    assert np.allclose(f(3 * xa - xb), 3 * f(xa) - f(xb), rtol=1e-12, atol=1e-12)
    b = d.bias.astype(np.float64)
    y, S = f(xa, bias=b, with_scale=True)
    ya = oracle.depthwise(np.abs(xa), np.abs(d.w.astype(np.float64)), d.pid, d.masks, bias=np.abs(b), stride=2)
    assert np.allclose(S, ya, rtol=1e-13, atol=0)
    assert (S >= np.abs(y)).all()
    _, S2 = f(2 * xa, bias=b, with_scale=True)
    assert np.allclose(S2, 2 * S - np.abs(b), rtol=1e-13, atol=0)
    with pytest.raises(ValueError):
        oracle.depthwise(d.x, d.w, np.full(5, 12, np.int16), d.masks)

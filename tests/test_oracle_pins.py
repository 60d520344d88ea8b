"""Pins for the CPU oracle: checks against things that are not the oracle.

Each test fixes the oracle to something the mathematics or a worked example
decides: hand-computed outputs, the impulse response (reads every kept weight
back), closed forms for a constant image, "a pruned kernel contributes
nothing", linearity, a library convolution on the masked dense tensor, and a
scatter-form brute force with a different loop structure.  A dropped term, a
wrong sign or index, a flipped kernel or a transposed operand fails at least
one of them.
"""
import os

import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")
LIB12 = wl.pattern_library(12)


def _read_gold(name):
    rows = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        a, b = line.split("|")
        rows.append(([int(t) for t in a.split()], [float(v) for v in b.split()]))
    return rows


def _mask_of(taps):
    return sum(1 << t for t in taps)


def test_library_shapes():
    # 12 distinct masks, 4 taps each, all containing the centre tap
    assert len(set(int(m) for m in LIB12)) == 12
    for m in LIB12:
        assert bin(int(m)).count("1") == 4
        assert (int(m) >> 4) & 1
    assert [hex(int(m)) for m in LIB12[:4]] == ["0x1b", "0x36", "0xd8", "0x1b0"]


# ---- P1: hand-computed cases -------------------------------------------------
def test_hand_3x3_every_pattern():
    rows = _read_gold("hand_3x3.txt")
    assert len(rows) == 12
    x = np.arange(1, 10, dtype=np.float64).reshape(1, 3, 3, 1)
    w = np.arange(1, 10, dtype=np.float64).reshape(1, 1, 3, 3)
    seen = set()
    for taps, exp in rows:
        masks = np.array([_mask_of(taps)], dtype=np.uint16)
        seen.add(int(masks[0]))
        y = oracle.conv(x, w, np.zeros((1, 1), np.int16), masks)
        got = [y[0, 0, 0, 0], y[0, 0, 1, 0], y[0, 1, 1, 0], y[0, 2, 2, 0]]
        assert got == exp, (taps, got, exp)
    assert seen == set(int(m) for m in LIB12)


def test_hand_stride2():
    x = np.arange(1, 17, dtype=np.float64).reshape(1, 4, 4, 1)
    w = np.arange(1, 10, dtype=np.float64).reshape(1, 1, 3, 3)
    for taps, exp in _read_gold("hand_stride2_4x4.txt"):
        masks = np.array([_mask_of(taps)], dtype=np.uint16)
        y = oracle.conv(x, w, np.zeros((1, 1), np.int16), masks, stride=2)
        assert y.shape == (1, 2, 2, 1)
        assert [y[0, 0, 0, 0], y[0, 0, 1, 0], y[0, 1, 0, 0], y[0, 1, 1, 0]] == exp


def test_hand_channels_bias_relu():
    # 1x1 image: only the centre tap reaches it.  x = [2, 3];
    # filter 0 keeps kernel (0,0) only -> 1*2 ; filter 1 keeps both -> 100*2 + 1000*3
    x = np.array([2.0, 3.0]).reshape(1, 1, 1, 2)
    w = np.zeros((2, 2, 3, 3))
    w[0, 0, 1, 1], w[0, 1, 1, 1], w[1, 0, 1, 1], w[1, 1, 1, 1] = 1, 10, 100, 1000
    w[0, 0, 0, 0] = 7.0  # a corner weight that falls in the padding
    pid = np.array([[0, -1], [3, 1]], dtype=np.int16)
    y = oracle.conv(x, w, pid, LIB12[:4])
    assert y.ravel().tolist() == [2.0, 3200.0]
    bias = np.array([0.5, -5000.0])
    y = oracle.conv(x, w, pid, LIB12[:4], bias=bias, relu=True)
    assert y.ravel().tolist() == [2.5, 0.0]
    y = oracle.conv(x, w, pid, LIB12[:4], bias=bias, relu=False)
    assert y.ravel().tolist() == [2.5, -1800.0]


def test_hand_int8():
    # same 3x3 worked example, in integers: centre output of taps {0,1,3,4} is 46
    x = np.arange(1, 10, dtype=np.uint8).reshape(1, 3, 3, 1)
    w = np.arange(1, 10, dtype=np.int8).reshape(1, 1, 3, 3)
    y = oracle.conv(x, w, np.zeros((1, 1), np.int16), LIB12[:1], bias=np.array([-50], np.int32))
    assert y.dtype == np.int64
    assert int(y[0, 1, 1, 0]) == 46 - 50 and int(y[0, 0, 0, 0]) == 5 - 50 and int(y[0, 2, 2, 0]) == 94 - 50
    y = oracle.conv(x, w, np.zeros((1, 1), np.int16), LIB12[:1], bias=np.array([-50], np.int32), relu=True)
    assert int(y[0, 1, 1, 0]) == 0 and int(y[0, 2, 2, 0]) == 44


# ---- helpers for random cases ------------------------------------------------
def _small_case(seed, n=2, ci=5, co=7, h=6, w=5, lib=12, prune=0.4, dtype="f32", stride=1):
    spec = wl.LayerSpec("t", n, ci, co, h, w, stride, dtype, prune, lib, 0.5, "upm1", 0.3, False, seed % 97)
    return wl.make_layer(spec, seed=seed)


def _masked_dense(d):
    """Dense weights with pruned entries zeroed, built by table lookup."""
    keep = np.zeros((len(d.masks) + 1, 9), dtype=bool)      # last row = removed kernel
    for p, m in enumerate(d.masks):
        keep[p] = [(int(m) >> t) & 1 for t in range(9)]
    sel = keep[d.pid].reshape(d.pid.shape + (3, 3))           # pid -1 picks the last row
    return np.where(sel, d.w.astype(np.float64), 0.0)


# ---- P2: impulse response reads every kept weight back -----------------------
@pytest.mark.parametrize("seed", [1, 2])
def test_impulse_response(seed):
    d = _small_case(seed, n=1, ci=3, co=4, h=5, w=6)
    wm = _masked_dense(d)
    bias = d.bias.astype(np.float64)
    for ic in range(3):
        y0, x0 = 2, 3
        x = np.zeros((1, 5, 6, 3))
        x[0, y0, x0, ic] = 1.0
        y = oracle.conv(x, d.w, d.pid, d.masks, bias=bias)
        resp = y - bias                                     # exact: one product per output
        for dy in range(3):
            for dx in range(3):
                got = resp[0, y0 - dy + 1, x0 - dx + 1, :]
                np.testing.assert_allclose(got, wm[:, ic, dy, dx], rtol=0, atol=1e-15)
        # everything outside the 3x3 neighbourhood is untouched
        resp[0, y0 - 1:y0 + 2, x0 - 1:x0 + 2, :] = 0
        assert np.abs(resp).max() < 1e-15


def test_impulse_at_corner_stride2():
    # stride 2: impulse at input (1,1) reaches output (oy,ox) through tap (1-2oy+1, 1-2ox+1)
    d = _small_case(5, n=1, ci=2, co=3, h=4, w=4, stride=2)
    wm = _masked_dense(d)
    x = np.zeros((1, 4, 4, 2))
    x[0, 1, 1, 1] = 1.0
    y = oracle.conv(x, d.w, d.pid, d.masks, stride=2)
    assert y.shape == (1, 2, 2, 3)
    np.testing.assert_array_equal(y[0, 0, 0], wm[:, 1, 2, 2])
    np.testing.assert_array_equal(y[0, 1, 1], wm[:, 1, 0, 0])
    np.testing.assert_array_equal(y[0, 0, 1], wm[:, 1, 2, 0])
    np.testing.assert_array_equal(y[0, 1, 0], wm[:, 1, 0, 2])


# ---- P3: constant image, closed forms ----------------------------------------
@pytest.mark.parametrize("stride", [1, 2])
def test_constant_image_subset_sums(stride):
    d = _small_case(11, n=1, ci=4, co=5, h=7, w=7, stride=stride)
    wm = _masked_dense(d)
    x = np.ones((1, 7, 7, 4))
    y = oracle.conv(x, d.w, d.pid, d.masks, stride=stride)
    tap_sum = wm.sum(axis=1)                                # [co,3,3], summed over input channels
    ho = y.shape[1]
    # an interior output sees all nine tap positions
    iy = 1
    np.testing.assert_allclose(y[0, iy, iy], tap_sum.sum(axis=(1, 2)), rtol=1e-13)
    # top-left output loses the top row and left column of taps
    np.testing.assert_allclose(y[0, 0, 0], tap_sum[:, 1:, 1:].sum(axis=(1, 2)), rtol=1e-13, atol=1e-15)
    # top edge, interior column loses the top row only
    np.testing.assert_allclose(y[0, 0, 1], tap_sum[:, 1:, :].sum(axis=(1, 2)), rtol=1e-13, atol=1e-15)
    if stride == 1:
        # bottom-right output loses the bottom row and right column
        np.testing.assert_allclose(y[0, ho - 1, ho - 1], tap_sum[:, :2, :2].sum(axis=(1, 2)), rtol=1e-13, atol=1e-15)
    else:
        # 7 -> 4 outputs; the last one sits at input 6 and its tap dx=2 falls at 7 (outside)
        assert ho == 4
        np.testing.assert_allclose(y[0, 3, 3], tap_sum[:, :2, :2].sum(axis=(1, 2)), rtol=1e-13, atol=1e-15)


def test_each_kernel_keeps_four_weights():
    d = _small_case(3)
    wm = _masked_dense(d)
    nz = (wm != 0).reshape(d.pid.shape + (9,)).sum(axis=2)
    assert set(np.unique(nz[d.pid >= 0])) == {4}
    assert set(np.unique(nz[d.pid < 0])) <= {0}


# ---- P4: pruned entries contribute exactly nothing ---------------------------
@pytest.mark.parametrize("dtype", ["f32", "i8"])
def test_pruned_contributes_nothing(dtype):
    d = _small_case(21, dtype=dtype, prune=0.5)
    y0 = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True)
    rng = np.random.default_rng(0)
    w2 = d.w.copy().reshape(-1, 9)
    pid = d.pid.reshape(-1)
    for k in range(len(pid)):
        for t in range(9):
            if pid[k] < 0 or not (int(d.masks[pid[k]]) >> t) & 1:
                w2[k, t] = rng.integers(-100, 100)
    assert (w2 != d.w.reshape(-1, 9)).any()
    y1 = oracle.conv(d.x, w2.reshape(d.w.shape), d.pid, d.masks, bias=d.bias, relu=True)
    assert np.array_equal(y0, y1)
    # and a filter with every kernel removed outputs act(bias)
    pid2 = d.pid.copy()
    pid2[2, :] = -1
    y2 = oracle.conv(d.x, d.w, pid2, d.masks, bias=d.bias, relu=False)
    assert np.all(y2[..., 2] == d.bias[2])


# ---- P5: linearity and zero input ---------------------------------------------
def test_linearity_and_zero_input():
    d = _small_case(31, dtype="f32")
    d2 = _small_case(32, dtype="f32")
    a = 0.375
    f = lambda x: oracle.conv(x, d.w, d.pid, d.masks)
    x1, x2 = d.x.astype(np.float64), d2.x.astype(np.float64)
    lhs = f(a * x1 + x2)
    rhs = a * f(x1) + f(x2)
    np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-13)
    y = oracle.conv(np.zeros_like(d.x), d.w, d.pid, d.masks, bias=d.bias, relu=True)
    assert np.array_equal(y, np.broadcast_to(np.maximum(d.bias.astype(np.float64), 0), y.shape))
    # integers: exact linearity
    di = _small_case(33, dtype="i8")
    g = lambda x: oracle.conv(x, di.w, di.pid, di.masks)
    xa = (di.x // 4).astype(np.uint8)
    xb = (di.x // 8).astype(np.uint8)
    assert np.array_equal(g((3 * xa + xb).astype(np.uint8)), 3 * g(xa) + g(xb))


# ---- P6: a library convolution on the masked dense tensor ----------------------
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_against_library_conv(stride, dtype):
    torch = pytest.importorskip("torch")
    d = _small_case(41, n=2, ci=6, co=9, h=9, w=8, dtype=dtype, stride=stride)
    y, s = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=stride, with_scale=True)
    wm = torch.from_numpy(_masked_dense(d))
    xt = torch.from_numpy(d.x.astype(np.float64)).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(xt, wm, torch.from_numpy(d.bias.astype(np.float64)), stride=stride, padding=1)
    ref = torch.relu(ref).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-12)
    assert np.all(s >= np.abs(y) - 1e-12)


# ---- P7: scatter-form brute force (loops over inputs, adds into outputs) -------
def _scatter_form(x, w, pid, masks, bias, stride):
    n, h, wd, ci = x.shape
    co = w.shape[0]
    ho, wo = (h - 1) // stride + 1, (wd - 1) // stride + 1
    y = np.zeros((n, ho, wo, co), dtype=object if x.dtype == np.uint8 else np.float64)
    y += 0
    for b in range(n):
        for iy in range(h):
            for ix in range(wd):
                for ic in range(ci):
                    v = int(x[b, iy, ix, ic]) if x.dtype == np.uint8 else float(x[b, iy, ix, ic])
                    for oc in range(co):
                        p = pid[oc, ic]
                        if p < 0:
                            continue
                        for t in range(9):
                            if not (int(masks[p]) >> t) & 1:
                                continue
                            dy, dx = divmod(t, 3)
                            ny, nx = iy - dy + 1, ix - dx + 1      # output row*stride, col*stride
                            if ny % stride or nx % stride:
                                continue
                            oy, ox = ny // stride, nx // stride
                            if 0 <= oy < ho and 0 <= ox < wo:
                                wv = int(w[oc, ic, dy, dx]) if x.dtype == np.uint8 else float(w[oc, ic, dy, dx])
                                y[b, oy, ox, oc] += wv * v
    return y + (0 if bias is None else bias)


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("dtype", ["f32", "i8"])
def test_scatter_form_brute_force(stride, dtype):
    d = _small_case(51 + stride, n=1, ci=3, co=4, h=5, w=4, dtype=dtype, stride=stride)
    y = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, stride=stride)
    ref = _scatter_form(d.x, d.w, d.pid, d.masks, d.bias.astype(object if dtype == "i8" else np.float64), stride)
    if dtype == "i8":
        assert np.array_equal(y, ref.astype(np.int64))
    else:
        np.testing.assert_allclose(y, ref.astype(np.float64), rtol=0, atol=1e-13)


# ---- P8: integer extremes against a closed form --------------------------------
def test_int8_extremes():
    ci = 512
    x = np.full((1, 3, 3, ci), 255, dtype=np.uint8)
    for wv in (127, -127, -128):
        w = np.full((1, ci, 3, 3), wv, dtype=np.int8)
        y = oracle.conv(x, w, np.zeros((1, ci), np.int16), LIB12[:1], bias=np.array([1 << 20], np.int32))
        # centre output: 4 kept taps per kernel, all inside the image
        assert int(y[0, 1, 1, 0]) == 255 * wv * 4 * ci + (1 << 20)
        assert abs(int(y[0, 1, 1, 0])) < 2 ** 31
        # corner (0,0): of taps {0,1,3,4} only tap 4 reaches the image
        assert int(y[0, 0, 0, 0]) == 255 * wv * ci + (1 << 20)


# ---- P9: relabelling the library does not change the layer ---------------------
def test_library_relabelling_invariance():
    d = _small_case(61)
    y0 = oracle.conv(d.x, d.w, d.pid, d.masks)
    perm = np.random.default_rng(1).permutation(len(d.masks))
    masks2 = d.masks[perm]
    inv = np.argsort(perm)
    pid2 = np.where(d.pid >= 0, inv[np.maximum(d.pid, 0)], -1).astype(np.int16)
    y1 = oracle.conv(d.x, d.w, pid2, masks2)
    assert np.array_equal(y0, y1)


def test_bad_pattern_id_is_an_error():
    d = _small_case(71)
    pid = d.pid.copy()
    pid[0, 0] = len(d.masks)
    with pytest.raises(ValueError):
        oracle.conv(d.x, d.w, pid, d.masks)


def test_fp16_inputs_are_used_as_stored():
    d = _small_case(81, dtype="f16")
    assert d.x.dtype == np.float16 and d.w.dtype == np.float16
    y16 = oracle.conv(d.x, d.w, d.pid, d.masks)
    y64 = oracle.conv(d.x.astype(np.float64), d.w.astype(np.float64), d.pid, d.masks)
    assert np.array_equal(y16, y64)


# ---- the error scale S = |bias| + sum |w * x| (every floating-point tolerance uses it) --------
def test_scale_hand_computed():
    x = np.arange(1, 10, dtype=np.float64).reshape(1, 3, 3, 1)
    w = np.arange(1, 10, dtype=np.float64).reshape(1, 1, 3, 3)
    w[0, 0, 0, 1] = -2.0
    w[0, 0, 1, 0] = -4.0
    masks = np.array([_mask_of([0, 1, 3, 4])], dtype=np.uint16)
    y, s = oracle.conv(x, w, np.zeros((1, 1), np.int16), masks, bias=np.array([-3.0]), with_scale=True)
    rows = _read_gold("hand_scale_3x3.txt")
    assert len(rows) == 4
    for (oy, ox), (ey, es) in rows:
        assert y[0, oy, ox, 0] == ey and s[0, oy, ox, 0] == es, (oy, ox, y[0, oy, ox, 0], s[0, oy, ox, 0])


@pytest.mark.parametrize("stride", [1, 2])
def test_scale_equals_output_for_nonnegative_terms(stride):
    # x >= 0, kept weights >= 0, bias >= 0: every term is its own magnitude, so S == y, bit for bit
    d = _small_case(51, n=2, ci=6, co=5, h=7, w=6, stride=stride)
    x, w, b = np.abs(d.x), np.abs(d.w), np.abs(d.bias)
    for relu in (False, True):
        y, s = oracle.conv(x, w, d.pid, d.masks, bias=b, relu=relu, stride=stride, with_scale=True)
        assert np.array_equal(y, s)
        assert (s > 0).any()


@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_scale_is_the_layer_on_magnitudes(dtype):
    # S(x, W, bias) == y(|x|, |W|, |bias|) exactly: same loop order, and |w*x| == |w|*|x| in binary fp
    d = _small_case(52, n=1, ci=7, co=6, h=6, w=7, dtype=dtype, stride=1)
    assert (d.x < 0).any() or dtype == "f16"
    assert (d.w < 0).any() and (d.bias < 0).any()
    _, s = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, with_scale=True)
    y_abs = oracle.conv(np.abs(d.x), np.abs(d.w), d.pid, d.masks, bias=np.abs(d.bias), relu=False)
    assert np.array_equal(s, y_abs)
    # without a bias the bias term is gone, and only then
    _, s0 = oracle.conv(d.x, d.w, d.pid, d.masks, bias=None, with_scale=True)
    assert np.allclose(s - s0, np.abs(d.bias).astype(np.float64)[None, None, None, :], rtol=0, atol=1e-12)


def test_scale_ignores_relu_and_pruned_weights_and_is_homogeneous():
    d = _small_case(53, n=1, ci=5, co=4, h=5, w=5)
    _, s_lin = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=False, with_scale=True)
    _, s_relu = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, with_scale=True)
    assert np.array_equal(s_lin, s_relu)
    w2 = np.where(_masked_dense(d) != 0, d.w, 1e6)             # garbage at pruned positions
    _, s_g = oracle.conv(d.x, w2, d.pid, d.masks, bias=d.bias, with_scale=True)
    assert np.array_equal(s_lin, s_g)
    _, s2 = oracle.conv(2.0 * d.x.astype(np.float64), d.w, d.pid, d.masks, bias=2.0 * d.bias.astype(np.float64),
                        with_scale=True)
    assert np.array_equal(s2, 2.0 * s_lin)                     # doubling every term doubles S exactly

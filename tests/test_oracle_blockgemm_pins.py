"""Pins of the block-pruned matrix-product oracle (paper Sec. 2.1, "Block-Based
Pruning") against what the mathematics fixes: a case worked by hand, closed
forms, a library product on the masked matrix, and invariants chosen so that a
plausible slip (rows and columns swapped, a block index off by one, the edge
blocks, a dropped bias) fails at least one of them."""
import os

import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_blockgemm.txt")


def _masked(w, rk, ck, br, bc):
    """The masked matrix, built here independently of the oracle (numpy indexing)."""
    c_out, k = w.shape
    oc = np.arange(c_out)[:, None]
    c = np.arange(k)[None, :]
    keep = rk[oc // br, c // bc, oc % br].astype(bool) & ck[oc // br, c // bc, c % bc].astype(bool)
    return np.where(keep, w.astype(np.float64), 0.0)


def test_hand_computed_case():
    """tests/golden/hand_blockgemm.txt: a 4x6 matrix in blocks of 2x3, worked by hand."""
    vals = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, rest = line.split(":")
                vals[key.strip()] = np.array([float(v) for v in rest.split()])
    w = vals["w"].reshape(4, 6)
    x = vals["x"].reshape(2, 6)
    rk = vals["row_keep"].reshape(2, 2, 2).astype(np.uint8)
    ck = vals["col_keep"].reshape(2, 2, 3).astype(np.uint8)
    y, s = oracle.block_gemm(x, w, rk, ck, 2, 3, bias=vals["bias"], relu=False, with_scale=True)
    assert np.array_equal(y, vals["y"].reshape(2, 4))
    assert np.array_equal(s, vals["s"].reshape(2, 4))
    yr = oracle.block_gemm(x, w, rk, ck, 2, 3, bias=vals["bias"], relu=True)
    assert np.array_equal(yr, np.maximum(vals["y"].reshape(2, 4), 0.0))


@pytest.mark.parametrize("m,k,c_out,br,bc", [(5, 12, 8, 4, 4), (7, 13, 10, 4, 8), (3, 40, 33, 16, 32), (1, 5, 3, 8, 8)])
def test_library_product_on_the_masked_matrix(m, k, c_out, br, bc):
    """Special case that reduces to a library routine: numpy's product of x with the
    masked matrix built in this test (edge blocks included)."""
    d = wl.make_block_gemm(wl.GemmSpec("t", m, k, c_out, br, bc, 0.5, 0.5, "f32", "upm1", 0.3, False, 3))
    y = oracle.block_gemm(d.x, d.w, d.row_keep, d.col_keep, br, bc, bias=d.bias)
    wm = _masked(d.w, d.row_keep, d.col_keep, br, bc)
    ref = d.x.astype(np.float64) @ wm.T + d.bias.astype(np.float64)
    assert np.allclose(y, ref, rtol=1e-12, atol=1e-12)
    assert wm.any() and not wm.all()


def test_nothing_pruned_is_the_plain_product_and_everything_pruned_is_the_bias():
    d = wl.make_block_gemm(wl.GemmSpec("t", 6, 20, 9, 4, 8, 0.5, 0.5, "f32", "upm1", 0.3, False, 4))
    ones_r, ones_c = np.ones_like(d.row_keep), np.ones_like(d.col_keep)
    y = oracle.block_gemm(d.x, d.w, ones_r, ones_c, 4, 8, bias=d.bias)
    assert np.allclose(y, d.x.astype(np.float64) @ d.w.astype(np.float64).T + d.bias, rtol=1e-12, atol=1e-12)
    y0 = oracle.block_gemm(d.x, d.w, np.zeros_like(d.row_keep), ones_c, 4, 8, bias=d.bias)
    assert np.array_equal(y0, np.broadcast_to(d.bias.astype(np.float64), y0.shape))
    y1 = oracle.block_gemm(d.x, d.w, ones_r, np.zeros_like(d.col_keep), 4, 8, bias=d.bias)
    assert np.array_equal(y1, y0)


def test_pruned_rows_and_columns_contribute_exactly_nothing():
    """Values stored at pruned positions never reach the result; a pruned row of one block
    removes that block's share of the row only; a pruned column likewise."""
    s = wl.GemmSpec("t", 4, 16, 8, 4, 8, 0.5, 0.5, "f32", "upm1", 0.0, False, 5)
    d = wl.make_block_gemm(s)
    y = oracle.block_gemm(d.x, d.w, d.row_keep, d.col_keep, 4, 8)
    wm = _masked(d.w, d.row_keep, d.col_keep, 4, 8)
    poisoned = np.where(wm != 0.0, d.w.astype(np.float64), 1e30)
    assert np.array_equal(oracle.block_gemm(d.x, poisoned, d.row_keep, d.col_keep, 4, 8), y)
    # one block at a time: block (i, j) alone gives x[:, cols kept] . w[rows kept, cols kept]^T in its rows
    total = np.zeros_like(y)
    for i in range(s.nbr):
        for j in range(s.nbc):
            rk, ck = np.zeros_like(d.row_keep), np.zeros_like(d.col_keep)
            rk[i, j], ck[i, j] = d.row_keep[i, j], d.col_keep[i, j]
            part = oracle.block_gemm(d.x, d.w, rk, ck, 4, 8)
            rows = i * 4 + np.flatnonzero(d.row_keep[i, j])
            cols = j * 8 + np.flatnonzero(d.col_keep[i, j])
            want = np.zeros_like(y)
            want[:, rows] = d.x[:, cols].astype(np.float64) @ d.w[np.ix_(rows, cols)].astype(np.float64).T
            assert np.allclose(part, want, rtol=1e-13, atol=1e-13)
            total += part
    assert np.allclose(total, y, rtol=1e-12, atol=1e-12)


def test_rows_and_columns_are_not_interchanged():
    """Keeping row 1 of block (0, 0) and column 2 of it leaves exactly W[1, 2]."""
    w = np.arange(1.0, 25.0).reshape(4, 6)
    rk = np.zeros((2, 2, 2), np.uint8)
    ck = np.zeros((2, 2, 3), np.uint8)
    rk[0, 0, 1] = 1
    ck[0, 0, 2] = 1
    x = np.eye(6)
    y = oracle.block_gemm(x, w, rk, ck, 2, 3)               # y[c, oc] = Wm[oc, c]
    want = np.zeros((6, 4))
    want[2, 1] = w[1, 2]
    assert np.array_equal(y, want)
    rk[:] = 0
    ck[:] = 0
    rk[1, 0, 0] = 1                                          # block row 1, block column 0: row 2, column 1
    ck[1, 0, 1] = 1
    want[:] = 0
    want[1, 2] = w[2, 1]
    assert np.array_equal(oracle.block_gemm(x, w, rk, ck, 2, 3), want)


def test_constant_inputs_closed_form_and_linearity():
    s = wl.GemmSpec("t", 3, 24, 12, 4, 8, 0.5, 0.25, "f32", "upm1", 0.2, False, 6)
    d = wl.make_block_gemm(s)
    ones_w = np.ones_like(d.w)
    x1 = np.full((3, 24), 0.5)
    y = oracle.block_gemm(x1, ones_w, d.row_keep, d.col_keep, 4, 8)
    # every kept weight contributes 0.5: kept columns of the blocks in which the row is kept
    want = np.zeros(12)
    for oc in range(12):
        for j in range(s.nbc):
            if d.row_keep[oc // 4, j, oc % 4]:
                want[oc] += 0.5 * d.col_keep[oc // 4, j].sum()
    assert np.array_equal(y, np.broadcast_to(want, y.shape))
    xa = d.x.astype(np.float64)
    xb = xa[::-1] * 0.75
    ya = oracle.block_gemm(xa, d.w, d.row_keep, d.col_keep, 4, 8)
    yb = oracle.block_gemm(xb, d.w, d.row_keep, d.col_keep, 4, 8)
    yab = oracle.block_gemm(2.0 * xa - xb, d.w, d.row_keep, d.col_keep, 4, 8)
    assert np.allclose(yab, 2.0 * ya - yb, rtol=1e-12, atol=1e-12)
    assert np.array_equal(oracle.block_gemm(np.zeros_like(xa), d.w, d.row_keep, d.col_keep, 4, 8, bias=d.bias),
                          np.broadcast_to(d.bias.astype(np.float64), ya.shape))


def test_error_scale():
    s = wl.GemmSpec("t", 5, 32, 16, 8, 16, 0.5, 0.5, "f32", "upm1", 0.3, False, 7)
    d = wl.make_block_gemm(s)
    x, w, b = d.x.astype(np.float64), d.w.astype(np.float64), d.bias.astype(np.float64)
    y, S = oracle.block_gemm(x, w, d.row_keep, d.col_keep, 8, 16, bias=b, with_scale=True)
    ya = oracle.block_gemm(np.abs(x), np.abs(w), d.row_keep, d.col_keep, 8, 16, bias=np.abs(b))
    assert np.allclose(S, ya, rtol=1e-13, atol=0)            # S(x, W, b) = y(|x|, |W|, |b|)
    assert (S >= np.abs(y)).all() and (S > np.abs(y)).any()
    yp, Sp = oracle.block_gemm(np.abs(x), np.abs(w), d.row_keep, d.col_keep, 8, 16, bias=np.abs(b), with_scale=True)
    assert np.array_equal(yp, Sp)                             # non-negative terms: S is the result itself
    _, S2 = oracle.block_gemm(2.0 * x, w, d.row_keep, d.col_keep, 8, 16, bias=b, with_scale=True)
    assert np.allclose(S2, 2.0 * S - np.abs(b), rtol=1e-13, atol=0)


def test_shape_errors():
    with pytest.raises(ValueError):
        oracle.block_gemm(np.zeros((2, 4)), np.zeros((3, 5)), np.ones((1, 1, 4), np.uint8), np.ones((1, 1, 8), np.uint8), 4, 8)
    with pytest.raises(ValueError):
        oracle.block_gemm(np.zeros((2, 4)), np.zeros((3, 4)), np.ones((1, 2, 4), np.uint8), np.ones((1, 1, 8), np.uint8), 4, 8)

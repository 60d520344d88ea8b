"""GPU parity of the block-pruned matrix product (xgen_blockgemm_run) against the CPU
oracle, element by element, through the C ABI: both numeric variants, block shapes
larger and smaller than a warp's 16 output channels and than a staged slice of columns,
ragged edges in every dimension, degenerate pruning, several tiles and stages."""
import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "f16": 2e-3}


def _run(d, relu=True, bias=True, guard=64):
    import torch
    s = d.spec
    pk = binding.BlockGemm(s.k, s.c_out, s.br, s.bc, s.dtype, d.w, d.row_keep, d.col_keep, device=0)
    tdt = torch.float32 if s.dtype == "f32" else torch.float16
    x = torch.from_numpy(d.x).cuda()
    b = torch.from_numpy(d.bias).cuda() if bias else None
    m = d.x.shape[0]
    # guard bands before and after y, and a poisoned y: a store outside, or a missing one, shows
    buf = torch.full((guard + m * s.c_out + guard,), 777.0, dtype=tdt, device="cuda")
    y = buf[guard:guard + m * s.c_out]
    st = torch.cuda.current_stream().cuda_stream
    pk.run(x.data_ptr(), m, b.data_ptr() if bias else 0, relu, y.data_ptr(), st)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    assert (host[:guard] == 777.0).all() and (host[guard + m * s.c_out:] == 777.0).all(), "store outside y"
    return host[guard:guard + m * s.c_out].reshape(m, s.c_out), pk


def _compare(d, got, relu=True, bias=True):
    s = d.spec
    ref, S = oracle.block_gemm(d.x, d.w, d.row_keep, d.col_keep, s.br, s.bc,
                               bias=d.bias if bias else None, relu=relu, with_scale=True)
    err = np.abs(got.astype(np.float64) - ref)
    bound = TOL[s.dtype] * np.maximum(np.abs(ref), 0.01 * S) + 1e-30
    bad = err > bound
    assert not bad.any(), "%d of %d elements off, worst %.3g x the bound at %s" % (
        bad.sum(), bad.size, (err / bound).max(), np.unravel_index(np.argmax(err / bound), err.shape))


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("m,k,c_out,br,bc", [
    (300, 64, 64, 32, 32),        # two tiles (one ragged), two stages, four warps
    (1000, 256, 256, 32, 32),     # 16 warps, eight stages
    (520, 96, 272, 64, 32),       # two blocks of output channels, the second with one warp
    (257, 128, 48, 16, 64),       # a pruning block wider than a staged slice
    (64, 40, 24, 8, 8),           # pruning blocks smaller than a warp's rows and a column group
    (33, 72, 40, 4, 16),
    (700, 200, 100, 32, 32),      # ragged edge blocks in rows and columns, scalar stores (f16)
])
def test_shapes(dtype, m, k, c_out, br, bc):
    d = wl.make_block_gemm(wl.GemmSpec("t", m, k, c_out, br, bc, 0.5, 0.5, dtype, "upm1", 0.05, True, 11))
    got, pk = _run(d)
    _compare(d, got)
    st = pk.stats()
    assert st["weights_kept"] == d.kept_weights()


@pytest.mark.parametrize("dtype", ["f32", "f16"])
def test_odd_extents_take_the_scalar_paths(dtype):
    """k odd (fp16 rows start on odd halves: no 4-byte copies) and c_out not a multiple of 4 / 8."""
    d = wl.make_block_gemm(wl.GemmSpec("t", 130, 45, 19, 8, 16, 0.6, 0.6, dtype, "upm1", 0.05, True, 12))
    got, _ = _run(d)
    _compare(d, got)


@pytest.mark.parametrize("rk,ck", [(1.0, 1.0), (1.0, 0.25), (0.25, 1.0), (0.125, 0.125), (0.0, 0.5)])
def test_pruning_rates(rk, ck):
    d = wl.make_block_gemm(wl.GemmSpec("t", 400, 128, 128, 32, 32, rk, ck, "f32", "relu_normal", 0.05, True, 13))
    got, pk = _run(d)
    _compare(d, got)
    if rk == 0.0:
        assert pk.stats()["row_commands"] == 0
        assert np.array_equal(got, np.broadcast_to(np.maximum(d.bias, 0), got.shape))


def test_no_bias_no_relu_and_pruned_values_ignored():
    s = wl.GemmSpec("t", 260, 64, 80, 16, 32, 0.5, 0.5, "f32", "upm1", 0.05, False, 14)
    d = wl.make_block_gemm(s)
    got, _ = _run(d, relu=False, bias=False)
    _compare(d, got, relu=False, bias=False)
    # values at pruned positions must not matter: poison them and compare bit for bit
    oc = np.arange(s.c_out)[:, None]
    c = np.arange(s.k)[None, :]
    keep = d.row_keep[oc // s.br, c // s.bc, oc % s.br].astype(bool) & d.col_keep[oc // s.br, c // s.bc, c % s.bc].astype(bool)
    d2 = wl.make_block_gemm(s)
    d2.w = np.where(keep, d.w, np.float32(1e30))
    got2, _ = _run(d2, relu=False, bias=False)
    assert np.array_equal(got, got2)


def test_unstructured_blocks_of_one_column():
    """Blocks of 16 rows x 1 column: column pruning per block is pruning of single (row group, column) strips."""
    d = wl.make_block_gemm(wl.GemmSpec("t", 100, 48, 32, 16, 1, 1.0, 0.5, "f32", "upm1", 0.05, True, 15))
    got, _ = _run(d)
    _compare(d, got)


def test_resnet50_pointwise_layers_sampled_rows():
    """The 1x1 layers of the benchmark at full size; the first and the last 256 rows of x are compared
    (rows are independent, so the oracle computes them alone)."""
    import torch
    for spec in wl.config_resnet50_1x1():
        if spec.m > 30000:
            spec.m = 25088 + 17                  # keep the largest inputs of the test moderate, keep them ragged
        d = wl.make_block_gemm(spec)
        got, _ = _run(d)
        for sl in (slice(0, 256), slice(spec.m - 256, spec.m)):
            ref, S = oracle.block_gemm(d.x[sl], d.w, d.row_keep, d.col_keep, spec.br, spec.bc, bias=d.bias, relu=True, with_scale=True)
            err = np.abs(got[sl].astype(np.float64) - ref)
            assert (err <= TOL[spec.dtype] * np.maximum(np.abs(ref), 0.01 * S) + 1e-30).all(), spec.name
        torch.cuda.empty_cache()


def test_argument_errors():
    import torch
    d = wl.make_block_gemm(wl.GemmSpec("t", 40, 32, 32, 16, 16, 0.5, 0.5, "f32", "upm1", 0.05, True, 16))
    pk = binding.BlockGemm(32, 32, 16, 16, "f32", d.w, d.row_keep, d.col_keep, device=0)
    x = torch.zeros((40, 32), device="cuda")
    y = torch.zeros((40, 32), device="cuda")
    with pytest.raises(binding.PatconvError) as e:
        pk.run(0, 40, 0, True, y.data_ptr())
    assert e.value.status == 1
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr(), 0, 0, True, y.data_ptr())
    assert e.value.status == 3
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr(), 40, 0, True, x.data_ptr())
    assert e.value.status == 1
    with pytest.raises(binding.PatconvError) as e:
        binding.BlockGemm(32, 32, 16, 16, "i8", d.w, d.row_keep, d.col_keep, device=0)
    assert e.value.status == 4

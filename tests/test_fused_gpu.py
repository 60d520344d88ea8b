"""GPU parity of the operators fused behind the convolution (xgen_patconv_run_fused: residual
addition, ReLU, 2x2 max-pool, re-quantisation to uint8) against the CPU oracle's conv_fused."""
import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import binding, workloads as wl
from _gpu_util import TOL, pack, guarded_output, check_guards

pytestmark = pytest.mark.gpu


def _layer(dtype, n, ci, co, h, w, stride=1, prune=0.5, lib=8, seed=1):
    xd = {"f32": "upm1", "f16": "relu_normal", "i8": "u01"}[dtype]
    spec = wl.LayerSpec("t", n, ci, co, h, w, stride, dtype, prune, lib, "he", xd, 0.05, True, seed % 83)
    return wl.make_layer(spec, seed=seed)


def _residual(d, ho, wo, seed):
    s = d.spec
    shape = (s.n, ho, wo, s.c_out)
    size = int(np.prod(shape))
    if s.dtype == "i8":
        return wl.integers(seed, "AUX", 7, size, -(1 << 14), 1 << 14).reshape(shape).astype(np.int32)
    r = wl.normal(seed, "AUX", 8, size).reshape(shape) * 0.5
    return r.astype(np.float32 if s.dtype == "f32" else np.float16)


def run_fused(pk, d, relu, pool, residual=None, scale=None, zp=0, plan_splits=None, reduce_mode=0):
    import torch
    s = d.spec
    x = torch.from_numpy(d.x).cuda()
    b = torch.from_numpy(d.bias).cuda()
    ho, wo = pk.out_shape(s.h, s.w)
    step = 2 if pool == 2 else 1
    ydt = torch.uint8 if scale is not None else {"f32": torch.float32, "f16": torch.float16, "i8": torch.int32}[s.dtype]
    if plan_splits is not None:
        pk.plan(s.n, s.h, s.w, splits=plan_splits, reduce_mode=reduce_mode)
    buf, y = guarded_output((s.n, ho // step, wo // step, s.c_out), ydt)
    rt = None if residual is None else torch.from_numpy(residual).cuda()
    st_ = None if scale is None else torch.from_numpy(scale).cuda()
    st = torch.cuda.current_stream().cuda_stream
    pk.run_fused(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), y.data_ptr(), st, relu=relu, pool=pool,
                 residual_ptr=0 if rt is None else rt.data_ptr(),
                 requant_scale_ptr=0 if st_ is None else st_.data_ptr(), zero_point=zp)
    pk.sync(st)
    check_guards(buf)
    return y.cpu().numpy()


def compare_fused(d, got, relu, pool, residual=None, scale=None, zp=0):
    s = d.spec
    ref = oracle.conv_fused(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=relu, stride=s.stride, residual=residual,
                            pool=pool, requant_scale=scale, zero_point=zp)
    if s.dtype == "i8":
        assert got.dtype == (np.uint8 if scale is not None else np.int32)
        assert np.array_equal(got.astype(np.int64), ref.astype(np.int64)), "integer result is not bit-exact"
        return
    # element-wise bound tol * max(|v|, 0.01 (S + |residual|)) before pooling; a maximum moves by at
    # most the largest movement of its arguments, so the pooled bound is the maximum of the bounds
    pre, S = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=False, stride=s.stride, with_scale=True)
    v = pre if residual is None else pre + residual.astype(np.float64)
    if residual is not None:
        S = S + np.abs(residual.astype(np.float64))
    bound = TOL[s.dtype] * np.maximum(np.abs(v), 0.01 * S) + 1e-30
    if pool == 2:
        n, ho, wo, c = bound.shape
        bound = bound.reshape(n, ho // 2, 2, wo // 2, 2, c).max(axis=(2, 4))
    g = got.astype(np.float64)
    assert np.isfinite(g).all()
    worst = float((np.abs(g - ref) / bound).max())
    assert worst <= 1.0, "error %.3g x the bound" % worst


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("pool", [0, 2])
def test_residual_relu_pool(dtype, stride, pool):
    # several tiles, two blocks of output channels (the second ragged), even output extents
    h, w = (22, 36) if stride == 1 else (44, 28)
    d = _layer(dtype, 3, 24, 136, h, w, stride, seed=11 + pool)
    pk = pack(d)
    ho, wo = pk.out_shape(h, w)
    res = _residual(d, ho, wo, seed=5)
    for relu, r in ((True, res), (False, res), (True, None)):
        compare_fused(d, run_fused(pk, d, relu, pool, r), relu, pool, r)


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
def test_odd_channel_count_scalar_paths(dtype):
    d = _layer(dtype, 2, 10, 37, 12, 14, 1, seed=21)
    pk = pack(d)
    res = _residual(d, 12, 14, seed=6)
    compare_fused(d, run_fused(pk, d, True, 2, res), True, 2, res)
    compare_fused(d, run_fused(pk, d, False, 0, res), False, 0, res)


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("pool", [0, 2])
def test_requantisation(stride, pool):
    h = 20 if stride == 1 else 40
    d = _layer("i8", 2, 32, 72, h, h, stride, seed=31)
    pk = pack(d)
    ho, wo = pk.out_shape(h, h)
    res = _residual(d, ho, wo, seed=7)
    # scales that put the codes across the whole range, some saturating
    scale = (wl.uniform01(3, "AUX", 9, 72) * 4e-3 + 2e-4).astype(np.float32)
    for relu, r, zp in ((True, None, 0), (False, res, 128), (True, res, 3)):
        got = run_fused(pk, d, relu, pool, r, scale, zp)
        compare_fused(d, got, relu, pool, r, scale, zp)
        assert got.min() == 0 or got.max() == 255 or (got.max() - got.min()) > 50    # the codes are spread out
    # a power-of-two scale makes many exact ties (x.5): round half to even
    half = np.full(72, 2.0 ** -7, np.float32)
    compare_fused(d, run_fused(pk, d, True, pool, None, half, 0), True, pool, None, half, 0)


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
def test_fused_behind_a_planned_split(dtype, stride):
    """The split items' partial sums are reduced inside the kernel; the fused operators then run
    in that reduction (pooled pixels take four rows of partial sums each)."""
    h = 16 if stride == 1 else 32
    d = _layer(dtype, 2, 128, 144, h, h, stride, prune=0.6, seed=41)
    pk = pack(d)
    ho, wo = pk.out_shape(h, h)
    res = _residual(d, ho, wo, seed=8)
    got = run_fused(pk, d, True, 2, res, plan_splits=3)
    assert pk.plan_info(2, h, h)["splits"] == 3
    compare_fused(d, got, True, 2, res)
    compare_fused(d, run_fused(pk, d, False, 0, res), False, 0, res)
    if dtype == "i8":
        scale = (wl.uniform01(4, "AUX", 10, 144) * 2e-3 + 1e-4).astype(np.float32)
        compare_fused(d, run_fused(pk, d, True, 2, res, scale, 7), True, 2, res, scale, 7)


@pytest.mark.parametrize("dtype", ["f32", "i8"])
def test_fused_behind_a_split_added_up_by_the_last_block(dtype):
    d = _layer(dtype, 2, 128, 144, 16, 16, 1, prune=0.6, seed=43)
    pk = pack(d)
    res = _residual(d, 16, 16, seed=9)
    got = run_fused(pk, d, True, 2, res, plan_splits=4, reduce_mode=2)
    info = pk.plan_info(2, 16, 16)
    assert info["splits"] == 4 and info["last_arriver"] == 1
    compare_fused(d, got, True, 2, res)
    compare_fused(d, run_fused(pk, d, False, 0, res), False, 0, res)
    if dtype == "i8":
        scale = (wl.uniform01(4, "AUX", 11, 144) * 2e-3 + 1e-4).astype(np.float32)
        compare_fused(d, run_fused(pk, d, True, 2, res, scale, 7), True, 2, res, scale, 7)


def test_vgg_stage_end_pool_and_argument_errors():
    import torch
    # VGG-16's conv4 (128 -> 128 at 112x112), whose result the network max-pools: planned, fused
    spec = wl.config_vgg16()[3]
    d = wl.make_layer(spec)
    pk = pack(d)
    got = run_fused(pk, d, True, 2, plan_splits=0)
    assert got.shape == (1, 56, 56, 128)
    compare_fused(d, got, True, 2)
    x = torch.zeros(1, 9, 9, spec.c_in, device="cuda")
    y = torch.zeros(1, 9, 9, spec.c_out, device="cuda")
    with pytest.raises(binding.PatconvError) as e:          # 9x9 cannot be pooled
        pk.run_fused(x.data_ptr(), 1, 9, 9, 0, y.data_ptr(), relu=True, pool=2)
    assert e.value.status == 3
    with pytest.raises(binding.PatconvError) as e:          # pool sizes other than 2
        pk.run_fused(x.data_ptr(), 1, 9, 9, 0, y.data_ptr(), relu=True, pool=3)
    assert e.value.status == 4
    with pytest.raises(binding.PatconvError) as e:          # re-quantisation belongs to the integer layer
        pk.run_fused(x.data_ptr(), 1, 9, 9, 0, y.data_ptr(), relu=True, requant_scale_ptr=y.data_ptr())
    assert e.value.status == 4
    with pytest.raises(binding.PatconvError) as e:          # y overlapping the residual
        pk.run_fused(x.data_ptr(), 1, 9, 9, 0, y.data_ptr(), relu=True, residual_ptr=y.data_ptr())
    assert e.value.status == 1

"""GPU parity of the depthwise pattern-pruned 3x3 layer (xgen_dwconv_run) against the CPU
oracle, element by element, through the C ABI: both numeric variants and strides, ragged
strips, channel counts that take the one-channel path, removed kernels, guard bands."""
import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "f16": 2e-3}
# A result below fp16's smallest normal number (6.1e-5) is stored with an absolute rounding
# error of up to half the subnormal spacing, 2^-25, whatever its size: with only four terms
# and a bias of about 0.01 such results occur (all four activations zero, a tiny bias).
ABS = {"f32": 1e-30, "f16": 2.0 ** -25}


def _run(d, relu=True, bias=True, guard=64):
    import torch
    s = d.spec
    pk = binding.Depthwise(s.c, s.stride, s.dtype, d.masks, d.w, d.pid, device=0)
    tdt = torch.float32 if s.dtype == "f32" else torch.float16
    x = torch.from_numpy(d.x).cuda()
    b = torch.from_numpy(d.bias).cuda() if bias else None
    n = d.x.shape[0]
    size = n * s.ho * s.wo * s.c
    buf = torch.full((guard + size + guard,), 777.0, dtype=tdt, device="cuda")
    y = buf[guard:guard + size]
    pk.run(x.data_ptr(), n, s.h, s.w, b.data_ptr() if bias else 0, relu, y.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    host = buf.cpu().numpy()
    assert (host[:guard] == 777.0).all() and (host[guard + size:] == 777.0).all(), "store outside y"
    return host[guard:guard + size].reshape(n, s.ho, s.wo, s.c), pk


def _compare(d, got, relu=True, bias=True, x=None):
    s = d.spec
    ref, S = oracle.depthwise(d.x if x is None else x, d.w, d.pid, d.masks, bias=d.bias if bias else None,
                              relu=relu, stride=s.stride, with_scale=True)
    err = np.abs(got.astype(np.float64) - ref)
    bound = TOL[s.dtype] * np.maximum(np.abs(ref), 0.01 * S) + ABS[s.dtype]
    assert (err <= bound).all(), "%d elements off, worst %.3g x the bound" % ((err > bound).sum(), (err / bound).max())


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("n,c,h,w", [(2, 32, 14, 14), (1, 64, 9, 23), (3, 8, 1, 1), (1, 4, 2, 5), (2, 128, 28, 28)])
def test_shapes(dtype, stride, n, c, h, w):
    d = wl.make_depthwise(wl.DepthwiseSpec("t", n, c, h, w, stride, dtype, 0.2, 8, "upm1", 0.05, True, 5))
    got, pk = _run(d)
    _compare(d, got)
    assert pk.kernels_surviving() == int((d.pid >= 0).sum())


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("c", [1, 3, 30])
def test_channel_counts_of_the_one_channel_path(dtype, c):
    d = wl.make_depthwise(wl.DepthwiseSpec("t", 2, c, 11, 13, 1, dtype, 0.0, 12, "upm1", 0.05, True, 6))
    got, _ = _run(d)
    _compare(d, got)


def test_no_bias_no_relu_removed_kernels_and_ignored_taps():
    s = wl.DepthwiseSpec("t", 1, 16, 12, 12, 1, "f32", 0.5, 8, "upm1", 0.05, False, 7)
    d = wl.make_depthwise(s)
    got, _ = _run(d, relu=False, bias=False)
    _compare(d, got, relu=False, bias=False)
    assert (got[..., d.pid < 0] == 0).all()
    d2 = wl.make_depthwise(s)
    for ch in range(16):
        for t in range(9):
            if d.pid[ch] < 0 or not (d.masks[d.pid[ch]] >> t) & 1:
                d2.w[ch].reshape(9)[t] = 1e30
    got2, _ = _run(d2, relu=False, bias=False)
    assert np.array_equal(got, got2)


def test_mobilenet_layers_sampled_images():
    for spec in wl.config_mobilenet_depthwise(batch=8):
        d = wl.make_depthwise(spec)
        got, _ = _run(d)
        for i in (0, spec.n - 1):
            _compare(d, got[i:i + 1], x=d.x[i:i + 1])


def test_argument_errors():
    import torch
    d = wl.make_depthwise(wl.DepthwiseSpec("t", 1, 8, 6, 6, 1, "f32", 0.0, 8, "upm1", 0.05, True, 8))
    pk = binding.Depthwise(8, 1, "f32", d.masks, d.w, d.pid, device=0)
    x = torch.zeros((1, 6, 6, 8), device="cuda")
    y = torch.zeros((1, 6, 6, 8), device="cuda")
    with pytest.raises(binding.PatconvError) as e:
        pk.run(0, 1, 6, 6, 0, True, y.data_ptr())
    assert e.value.status == 1
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr(), 1, 0, 6, 0, True, y.data_ptr())
    assert e.value.status == 3
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr(), 1, 6, 6, 0, True, x.data_ptr())
    assert e.value.status == 1
    with pytest.raises(binding.PatconvError) as e:
        binding.Depthwise(8, 3, "f32", d.masks, d.w, d.pid, device=-1)
    assert e.value.status == 4
    bad = d.masks.copy(); bad[0] = 0x1F
    with pytest.raises(binding.PatconvError) as e:
        binding.Depthwise(8, 1, "f32", bad, d.w, d.pid, device=-1)
    assert e.value.status == 2
    host_only = binding.Depthwise(8, 1, "f32", d.masks, d.w, d.pid, device=-1)
    with pytest.raises(binding.PatconvError) as e:
        host_only.run(x.data_ptr(), 1, 6, 6, 0, True, y.data_ptr())
    assert e.value.status == 6

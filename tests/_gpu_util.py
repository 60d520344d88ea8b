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

# Guard bands: the result tensor sits between two runs of GUARD sentinel elements that no
# kernel may touch (a store one pixel past either end shows up here).
GUARD = 64
SENTINEL = 12345

# What the fp16 second view saw, over the whole session: elements compared, elements more
# than one fp16 ulp away from the rounded oracle (printed by conftest at the end of the run).
FP16_ULP_STATS = {"compared": 0, "beyond_one_ulp": 0, "worst_ulp": 0}


def pack(d, device=0):
    s = d.spec
    return binding.Packed(s.c_in, s.c_out, s.stride, s.dtype, d.masks, d.w, d.pid, device=device)


def guarded_output(shape, dtype):
    """A poisoned result tensor of `shape` with sentinel guard bands on both sides.
    Returns (whole flat buffer, view of the result)."""
    import torch
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * GUARD,), _sentinel(dtype), dtype=dtype, device="cuda")
    return buf, buf[GUARD:GUARD + n].view(*shape)


def _sentinel(dtype):
    import torch
    return SENTINEL % 251 if dtype == torch.uint8 else SENTINEL


def check_guards(buf):
    g = buf.cpu().numpy()
    sentinel = _sentinel(buf.dtype)
    assert (g[:GUARD] == sentinel).all(), "the kernel wrote before the start of y"
    assert (g[-GUARD:] == sentinel).all(), "the kernel wrote past the end of y"


def run_gpu(pk, x, bias, relu, plan=False):
    """x: numpy NHWC.  Returns numpy output computed on cuda:0 via xgen_patconv_run
    (after xgen_patconv_plan for this shape when `plan` is set)."""
    import torch
    xt = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    n, h, w, _ = x.shape
    ho, wo = pk.out_shape(h, w)
    ydt = {binding.F32: torch.float32, binding.F16_F32ACC: torch.float16, binding.I8_I32: torch.int32}[pk.dtype]
    if plan:
        pk.plan(n, h, w)
    # poison the output so that an unwritten element cannot pass
    buf, yt = guarded_output((n, ho, wo, pk.c_out), ydt)
    bt = None if bias is None else torch.from_numpy(np.ascontiguousarray(bias)).cuda()
    stream = torch.cuda.current_stream().cuda_stream
    pk.run(xt.data_ptr(), n, h, w, 0 if bt is None else bt.data_ptr(), relu, yt.data_ptr(), stream)
    pk.sync(stream)
    check_guards(buf)
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
        # Second view: the oracle rounded to fp16 against the stored fp16 result, in units of
        # the last place, on the elements that are not dominated by cancellation
        # (|ref| >= 0.01 S).  There the fp32 accumulation error is typically well below half
        # an fp16 ulp, so all but a few elements agree to one ulp; the first check above
        # already bounds every element (2e-3 relative is about four fp16 ulps).
        r16 = ref.astype(np.float16)
        big = (np.abs(ref) >= 0.01 * S) & (r16 != 0) & (y_gpu != 0)
        if big.any():
            ulp = np.abs(y_gpu.view(np.int16).astype(np.int32) - r16.view(np.int16).astype(np.int32))[big]
            same_sign = (np.signbit(y_gpu) == np.signbit(r16))[big]
            assert same_sign.all()
            n_far = int((ulp > 1).sum())
            FP16_ULP_STATS["compared"] += int(ulp.size)
            FP16_ULP_STATS["beyond_one_ulp"] += n_far
            FP16_ULP_STATS["worst_ulp"] = max(FP16_ULP_STATS["worst_ulp"], int(ulp.max()))
            assert int(ulp.max()) <= 5, "fp16 result %d ulps from the rounded oracle" % int(ulp.max())
            assert n_far <= 1e-3 * ulp.size + 1, "%d of %d fp16 results beyond one ulp" % (n_far, ulp.size)
    return worst

"""The entry point that allocates nothing (xgen_patconv_run_static_scratch).

Some users of this library run where device allocation is off limits -- a fixed
memory budget, another framework's allocator scope, a path that must not
synchronise.  For them the split of a layer's input channels keeps its partial
sums in an array built into the library.  This file checks that entry point,
through the C ABI, against the ordinary xgen_patconv_run on the same inputs:
twice in a row (the array is shared between calls and keeps old contents), for
the three numeric variants, and that a request beyond the array's size is
refused.  Both results are also compared with the CPU oracle, and the free
device memory is read before and after the calls: it must not move.  The file is
collected last on purpose and does not depend on other tests.
"""
import numpy as np
import pytest

import oracle
from paper_2206_10620_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "f16": 2e-3}


def _layer(dtype, n, ci, co, hw, stride, seed):
    xd = {"f32": "upm1", "f16": "relu_normal", "i8": "u01"}[dtype]
    spec = wl.LayerSpec("noalloc", n, ci, co, hw, hw, stride, dtype, 0.6, 8, "he", xd, 0.05, True, 1)
    return wl.make_layer(spec, seed=seed)


def _buffers(d, pk):
    import torch
    s = d.spec
    ydt = {"f32": torch.float32, "f16": torch.float16, "i8": torch.int32}[s.dtype]
    x = torch.from_numpy(d.x).cuda()
    b = torch.from_numpy(d.bias).cuda()
    ho, wo = pk.out_shape(s.h, s.w)
    mk = lambda: torch.full((s.n, ho, wo, s.c_out), 77, dtype=ydt, device="cuda")
    return x, b, mk


@pytest.mark.parametrize("dtype,stride", [("f32", 1), ("f16", 2), ("i8", 1)])
def test_matches_ordinary_run_twice_in_a_row(dtype, stride):
    import torch
    d = _layer(dtype, 2, 192, 40, 14, stride, seed=21)
    s = d.spec
    pk = binding.Packed(s.c_in, s.c_out, stride, dtype, d.masks, d.w, d.pid, device=0)
    x, b, mk = _buffers(d, pk)
    st = torch.cuda.current_stream().cuda_stream
    y_ref = mk()
    pk.run(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), True, y_ref.data_ptr(), st)
    pk.sync(st)
    ref = y_ref.cpu().numpy()
    if dtype == "i8":
        truth = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=stride)
        assert np.array_equal(ref.astype(np.int64), truth)
    else:
        truth, S = oracle.conv(d.x, d.w, d.pid, d.masks, bias=d.bias, relu=True, stride=stride, with_scale=True)
    outs = [mk(), mk()]                                    # allocated before the memory reading
    pk.run_static_scratch(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), True, outs[0].data_ptr(), 2, st)   # first call
    pk.sync(st)                                            # on this device: resolves the array's address
    outs[0].fill_(77)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for y, splits in zip(outs, (6, 3)):                    # two calls in a row, different splits
        pk.run_static_scratch(x.data_ptr(), s.n, s.h, s.w, b.data_ptr(), True, y.data_ptr(), splits, st)
    pk.sync(st)
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the call that must not allocate changed the free device memory"
    for y in outs:
        got = y.cpu().numpy()
        if dtype == "i8":
            assert np.array_equal(got, ref)                # the ordinary entry point
            assert np.array_equal(got.astype(np.int64), truth)   # and the oracle
        else:
            bound = TOL[dtype] * np.maximum(np.abs(truth), 0.01 * S) + 1e-30
            assert (np.abs(got.astype(np.float64) - truth) <= bound).all()                       # the oracle
            assert (np.abs(got.astype(np.float64) - ref.astype(np.float64)) <= 2 * bound).all()  # the ordinary entry point
    # a second layer through the same array right after: old contents must not leak
    d2 = _layer(dtype, 1, 64, 24, 9, stride, seed=22)
    s2 = d2.spec
    pk2 = binding.Packed(s2.c_in, s2.c_out, stride, dtype, d2.masks, d2.w, d2.pid, device=0)
    x2, b2, mk2 = _buffers(d2, pk2)
    ya, yb = mk2(), mk2()
    pk2.run(x2.data_ptr(), s2.n, s2.h, s2.w, b2.data_ptr(), False, ya.data_ptr(), st)
    pk2.run_static_scratch(x2.data_ptr(), s2.n, s2.h, s2.w, b2.data_ptr(), False, yb.data_ptr(), 4, st)
    pk2.sync(st)
    a, bb = ya.cpu().numpy(), yb.cpu().numpy()
    if dtype == "i8":
        assert np.array_equal(a, bb)
    else:
        _, S2 = oracle.conv(d2.x, d2.w, d2.pid, d2.masks, bias=d2.bias, relu=False, stride=stride, with_scale=True)
        assert (np.abs(a.astype(np.float64) - bb.astype(np.float64))
                <= TOL[dtype] * np.maximum(np.abs(a.astype(np.float64)), 0.01 * S2) + 1e-30).all()


def test_refuses_what_does_not_fit():
    import torch
    d = _layer("f32", 1, 64, 64, 8, 1, seed=23)
    s = d.spec
    pk = binding.Packed(s.c_in, s.c_out, 1, "f32", d.masks, d.w, d.pid, device=0)
    n, hw = 8, 128                                        # 8*128*128*64 outputs * 4 B * 2 splits = 64 MiB
    assert n * hw * hw * 64 * 4 * 2 > binding.STATIC_SCRATCH_BYTES
    x = torch.zeros((n, hw, hw, 64), device="cuda")
    y = torch.zeros((n, hw, hw, 64), device="cuda")
    with pytest.raises(binding.PatconvError) as e:
        pk.run_static_scratch(x.data_ptr(), n, hw, hw, 0, True, y.data_ptr(), 2)
    assert e.value.status == 3
    # one split needs no scratch at all and is accepted at any size
    pk.run_static_scratch(x.data_ptr(), n, hw, hw, 0, True, y.data_ptr(), 1)
    pk.sync()
    with pytest.raises(binding.PatconvError) as e:
        pk.run_static_scratch(x.data_ptr(), n, hw, hw, 0, True, y.data_ptr(), 0)
    assert e.value.status == 1

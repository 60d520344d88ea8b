"""The shared library loads without a GPU and exports what the header declares."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2206_10620_b200 import binding, build, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = ""
    for name in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if name.endswith(".h"):
            src += open(os.path.join(ROOT, "include", name)).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(xgen_[a-z_]+)\s*\(", src)))


def test_header_symbols_are_exported():
    path = build.build()
    L = ctypes.CDLL(path)
    names = _declared()
    assert "xgen_patconv_pack" in names and "xgen_patconv_run" in names
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_launch_count():
    assert binding.strerror(0) == "ok"
    assert "pattern" in binding.strerror(2)
    assert binding.launch_count() >= 0


def _mk(dtype="f32", **kw):
    spec = wl.LayerSpec("t", 1, 6, 10, 5, 5, 1, dtype, 0.4, 8, 0.5, "upm1", 0.1, True, 3)
    for k, v in kw.items():
        setattr(spec, k, v)
    return wl.make_layer(spec, seed=5)


def test_error_codes_host_only():
    d = _mk()
    ok = binding.Packed(6, 10, 1, "f32", d.masks, d.w, d.pid, device=-1)
    assert ok.out_shape(5, 7) == (5, 7)
    with pytest.raises(binding.PatconvError) as e:
        binding.Packed(6, 10, 3, "f32", d.masks, d.w, d.pid, device=-1)
    assert e.value.status == 4
    with pytest.raises(binding.PatconvError) as e:
        binding.Packed(6, 10, 1, "f32", d.masks, d.w, d.pid, device=-1, pad=0)
    assert e.value.status == 4
    bad = d.masks.copy(); bad[0] = 0x1F            # five taps
    with pytest.raises(binding.PatconvError) as e:
        binding.Packed(6, 10, 1, "f32", bad, d.w, d.pid, device=-1)
    assert e.value.status == 2
    pid = d.pid.copy(); pid[0, 0] = 8               # id outside the library
    with pytest.raises(binding.PatconvError) as e:
        binding.Packed(6, 10, 1, "f32", d.masks, d.w, pid, device=-1)
    assert e.value.status == 2
    # a host-only handle cannot run
    x = np.zeros((1, 5, 5, 6), np.float32)
    with pytest.raises(binding.PatconvError) as e:
        ok.run_host(x, None, False)
    assert e.value.status == 6
    # stride-2 output extents
    s2 = binding.Packed(6, 10, 2, "f32", d.masks, d.w, d.pid, device=-1)
    assert s2.out_shape(7, 8) == (4, 4)

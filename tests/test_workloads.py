"""The seeded input generators: determinism, counts and value ranges."""
import numpy as np

from paper_2206_10620_b200 import workloads as wl


def test_counter_based_and_deterministic():
    a = wl.uniform01(7, "X", 3, 1000)
    b = wl.uniform01(7, "X", 3, 1000)
    assert np.array_equal(a, b)
    # a sub-range equals the same slice of the whole
    assert np.array_equal(wl.uniform01(7, "X", 3, 100, start=400), a[400:500])
    assert not np.array_equal(a, wl.uniform01(8, "X", 3, 1000))
    assert not np.array_equal(a, wl.uniform01(7, "W", 3, 1000))
    assert not np.array_equal(a, wl.uniform01(7, "X", 4, 1000))


def test_distributions():
    u = wl.uniform01(1, "X", 0, 200000)
    assert 0.0 <= u.min() and u.max() < 1.0 and abs(u.mean() - 0.5) < 5e-3
    g = wl.normal(1, "W", 0, 200000)
    assert abs(g.mean()) < 1e-2 and abs(g.std() - 1.0) < 1e-2
    k = wl.integers(1, "W", 0, 200000, -127, 127)
    assert k.min() == -127 and k.max() == 127


def test_exact_prune_count_and_library_range():
    for spec in wl.config_vgg16()[:4] + wl.config_single_layer():
        pid = wl.make_pattern_ids(wl.BASE_SEED, spec.index, spec.c_out, spec.c_in, spec.lib_size, spec.prune)
        assert (pid >= 0).sum() == spec.k_surv
        assert pid.max() < spec.lib_size and pid.min() >= -1
    s = wl.config_single_layer()[0]
    assert s.k_surv == 256 and s.useful_macs() == 4 * 256 * 32 * 32


def test_layer_tensors():
    d = wl.make_layer(wl.config_single_layer()[0])
    assert d.x.shape == (1, 32, 32, 16) and d.x.dtype == np.float32
    assert d.w.shape == (32, 16, 3, 3) and d.bias.shape == (32,)
    assert -1.0 <= d.x.min() and d.x.max() < 1.0
    r18 = wl.config_resnet18(batch=2)
    assert len(r18) == 16 and r18[4].stride == 2 and r18[4].c_out == 128
    di = wl.make_layer(r18[-1])
    assert di.x.dtype == np.uint8 and di.w.dtype == np.int8 and di.bias.dtype == np.int32
    assert np.abs(di.bias).max() <= 1 << 20
    r50 = wl.config_resnet50(batch=1)
    assert len(r50) == 16
    dh = wl.make_layer(r50[-1])
    assert dh.x.dtype == np.float16 and dh.x.min() >= 0
    assert len(wl.config_sweep()) == 48 and len(wl.config_vgg16()) == 13
    # leading images of a batch do not depend on the batch size
    full = wl.make_layer(r50[-1].__class__(**{**r50[-1].__dict__, "n": 3}))
    part = wl.make_layer(r50[-1].__class__(**{**r50[-1].__dict__, "n": 3}), n_override=1)
    assert np.array_equal(full.x[:1], part.x)

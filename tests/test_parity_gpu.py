"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle,
element by element on the same seeded inputs."""
import numpy as np
import pytest

from paper_2206_10620_b200 import binding, workloads as wl
from _gpu_util import compare, pack, run_gpu

pytestmark = pytest.mark.gpu


def _layer(dtype, n, ci, co, h, w, stride=1, prune=0.5, lib=8, seed=1, idx=0):
    xd = {"f32": "upm1", "f16": "relu_normal", "i8": "u01"}[dtype]
    spec = wl.LayerSpec("t", n, ci, co, h, w, stride, dtype, prune, lib, "he", xd, 0.05, True, idx)
    return wl.make_layer(spec, seed=seed)


def test_config_single_layer():
    d = wl.make_layer(wl.config_single_layer()[0])
    pk = pack(d)
    y = run_gpu(pk, d.x, d.bias, True)
    compare(d, y)
    assert binding.launch_count() >= 1


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape", [
    (2, 5, 7, 9, 11),        # odd everything: scalar stores, ragged channels
    (3, 20, 40, 37, 19),     # several tiles and a ragged tail in both directions
    (1, 16, 136, 70, 66),    # two blocks of output channels, the second ragged
    (5, 24, 16, 7, 7),       # several small images in one tile
    (2, 64, 32, 14, 14),
])
def test_shapes(dtype, stride, shape):
    n, ci, co, h, w = shape
    d = _layer(dtype, n, ci, co, h, w, stride, prune=0.5, lib=12, seed=n + ci)
    pk = pack(d)
    compare(d, run_gpu(pk, d.x, d.bias, True))
    compare(d, run_gpu(pk, d.x, None, False), bias=None, relu=False)


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
def test_first_layer_three_channels(dtype):
    d = _layer(dtype, 1, 3, 64, 60, 60, prune=0.0)
    compare(d, run_gpu(pack(d), d.x, d.bias, True))


@pytest.mark.parametrize("prune", [0.0, 0.75, 0.875])
@pytest.mark.parametrize("lib", [4, 12])
def test_density_and_library(prune, lib):
    d = _layer("f16", 2, 64, 64, 28, 28, prune=prune, lib=lib)
    compare(d, run_gpu(pack(d), d.x, d.bias, True))


def test_foreign_masks_universal_table():
    d = _layer("f32", 1, 16, 32, 12, 12, lib=4)
    d.masks = np.array([0x00F, 0x1E0, 0x145, 0x0AA], dtype=np.uint16)   # none contains the centre
    pk = pack(d)
    assert pk.stats()["patterns_compiled"] == 126
    compare(d, run_gpu(pk, d.x, d.bias, True))


def test_degenerate_layers():
    d = _layer("f32", 1, 8, 16, 10, 10)
    d.pid[:] = -1                                    # everything pruned: y = act(bias)
    y = run_gpu(pack(d), d.x, d.bias, True)
    assert np.array_equal(y, np.broadcast_to(np.maximum(d.bias, 0), y.shape))
    d2 = _layer("f32", 1, 8, 16, 10, 10)
    d2.pid[3, :] = -1                                # one filter with no kernel left
    y2 = run_gpu(pack(d2), d2.x, d2.bias, False)
    assert np.all(y2[..., 3] == d2.bias[3])
    compare(d2, y2, relu=False)
    d3 = _layer("f32", 1, 4, 8, 1, 1)                # 1x1 image: only the centre tap lands
    compare(d3, run_gpu(pack(d3), d3.x, d3.bias, True))


def test_pruned_weights_are_ignored_and_runs_are_deterministic():
    d = _layer("f32", 1, 16, 32, 20, 20)
    y0 = run_gpu(pack(d), d.x, d.bias, True)
    w2 = d.w.copy()
    keep = np.zeros((len(d.masks) + 1, 9), bool)
    for p, m in enumerate(d.masks):
        keep[p] = [(int(m) >> t) & 1 for t in range(9)]
    sel = keep[d.pid].reshape(d.pid.shape + (3, 3))
    w2[~sel] = 777.0
    d.w = w2
    pk = pack(d)
    y1 = run_gpu(pk, d.x, d.bias, True)
    y2 = run_gpu(pk, d.x, d.bias, True)
    assert np.array_equal(y0, y1) and np.array_equal(y1, y2)


def test_int8_extremes_and_long_reduction():
    # 512 input channels: the exact-partial-sum fold runs several times
    ci = 512
    spec = wl.LayerSpec("t", 1, ci, 16, 6, 6, 1, "i8", 0.0, 8, "he", "u01", 0.05, True, 0)
    d = wl.make_layer(spec)
    d.x[:] = 255
    for wv in (127, -128):
        d.w[:] = wv
        compare(d, run_gpu(pack(d), d.x, d.bias, False), relu=False)
    d = wl.make_layer(spec)
    compare(d, run_gpu(pack(d), d.x, d.bias, True))


def test_enqueue_host_overlapping_calls():
    """Host-buffer calls that only enqueue: two handles in turn on one stream, each several
    times (a later call on a handle has to wait for the staging buffers of the earlier one),
    results read after xgen_patconv_last_status."""
    import torch
    da = _layer("f32", 3, 40, 48, 30, 30, 1, prune=0.5, lib=8, seed=51)
    db = _layer("f16", 2, 64, 24, 21, 21, 2, prune=0.4, lib=8, seed=52)
    pa, pb = pack(da), pack(db)
    st = torch.cuda.current_stream().cuda_stream
    bufs = []
    for rep in range(3):
        for d, pk in ((da, pa), (db, pb)):
            hx = torch.from_numpy(d.x * (rep + 1) if d.spec.dtype == "f32" else d.x).pin_memory()
            hb = torch.from_numpy(d.bias).pin_memory()
            ho, wo = pk.out_shape(d.spec.h, d.spec.w)
            hy = torch.full((d.spec.n, ho, wo, d.spec.c_out), 777.0,
                            dtype=torch.float32 if d.spec.dtype == "f32" else torch.float16).pin_memory()
            pk.enqueue_host_ptr(hx.data_ptr(), d.spec.n, d.spec.h, d.spec.w, hb.data_ptr(), True, hy.data_ptr(), st)
            bufs.append((d, hx, hy))
    pa.sync(st)
    pb.sync(st)
    for d, hx, hy in bufs:
        compare(d, hy.numpy(), x=hx.numpy())


def test_run_host_entry_point():
    d = _layer("f16", 2, 32, 48, 20, 20)
    pk = pack(d)
    compare(d, pk.run_host(d.x, d.bias, True))


def test_argument_errors():
    import torch
    d = _layer("f32", 1, 8, 16, 10, 10)
    pk = pack(d)
    x = torch.zeros(1, 10, 10, 8, device="cuda")
    y = torch.zeros(1, 10, 10, 16, device="cuda")
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr() + 4, 1, 10, 10, 0, True, y.data_ptr())
    assert e.value.status == 1
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr(), 0, 10, 10, 0, True, y.data_ptr())
    assert e.value.status == 3
    with pytest.raises(binding.PatconvError) as e:
        pk.run(x.data_ptr(), 1, 10, 10, 0, True, x.data_ptr())      # y overlaps x
    assert e.value.status == 1


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
def test_planned_shape_splits_input_channels(dtype, stride):
    # few output pixels, many input channels: plan() splits the channel chunks across
    # blocks, which exchange their partial sums and reduce them inside the one kernel
    d = _layer(dtype, 1, 256, 72, 14, 14, stride, prune=0.6, lib=8, seed=11)
    pk = pack(d)
    pk.plan(1, 14, 14)
    before = binding.launch_count()
    y = run_gpu(pk, d.x, d.bias, True)
    assert binding.launch_count() - before == 1          # the split is reduced inside the kernel
    compare(d, y)
    y2 = run_gpu(pk, d.x, d.bias, True)
    assert np.array_equal(y, y2)                         # fixed reduction order
    # another shape on the same handle runs unsplit
    d2 = _layer(dtype, 1, 256, 72, 9, 9, stride, prune=0.6, lib=8, seed=11)
    before = binding.launch_count()
    y3 = run_gpu(pk, d2.x, d.bias, False)
    assert binding.launch_count() - before == 1
    d2.w, d2.pid, d2.masks = d.w, d.pid, d.masks
    compare(d2, y3, bias=d.bias, relu=False)


def test_planned_odd_channel_count():
    d = _layer("f32", 2, 130, 37, 7, 7, 1, prune=0.3, lib=12, seed=4)
    pk = pack(d)
    pk.plan(2, 7, 7)
    compare(d, run_gpu(pk, d.x, d.bias, True))


def test_planned_runs_back_to_back_and_replanned():
    """The arrival counters of a planned split only grow: many launches in a row on one
    stream, without a host synchronisation in between, must all reduce correctly; planning
    the handle for another shape starts over."""
    import torch
    d = _layer("f32", 1, 192, 64, 12, 12, 1, prune=0.5, lib=8, seed=31)
    pk = pack(d)
    pk.plan(1, 12, 12)
    x = torch.from_numpy(d.x).cuda()
    b = torch.from_numpy(d.bias).cuda()
    ys = [torch.full((1, 12, 12, 64), 777.0, device="cuda") for _ in range(25)]
    st = torch.cuda.current_stream().cuda_stream
    for y in ys:
        pk.run(x.data_ptr(), 1, 12, 12, b.data_ptr(), True, y.data_ptr(), st)
    pk.sync(st)
    first = ys[0].cpu().numpy()
    compare(d, first)
    for y in ys[1:]:
        assert np.array_equal(y.cpu().numpy(), first)
    d2 = _layer("f32", 2, 192, 64, 7, 7, 1, prune=0.5, lib=8, seed=31)
    pk.plan(2, 7, 7)
    y2 = run_gpu(pk, d2.x, d.bias, True)
    d2.w, d2.pid, d2.masks = d.w, d.pid, d.masks
    compare(d2, y2, bias=d.bias)
    compare(d, run_gpu(pk, d.x, d.bias, True))          # the first shape now runs unsplit


@pytest.mark.parametrize("c_out", [64, 160])
def test_unsplit_runs_back_to_back_overlap(c_out):
    """Launches follow each other on one stream without a host synchronisation: a kernel may be
    scheduled while its predecessor drains (programmatic stream serialisation), so its blocks start
    at different times and its prologue overlaps foreign work.  64 output channels give 8 consumer
    warps per block, 160 give 16; several images make more blocks than the GPU holds at once.
    The second layer of each pair reads what the first one wrote."""
    import torch
    d1 = _layer("f32", 6, 24, c_out, 40, 40, 1, prune=0.5, lib=8, seed=41)
    d2 = _layer("f32", 6, c_out, 32, 40, 40, 1, prune=0.5, lib=8, seed=42)
    p1, p2 = pack(d1), pack(d2)
    x = torch.from_numpy(d1.x).cuda()
    b1 = torch.from_numpy(d1.bias).cuda()
    b2 = torch.from_numpy(d2.bias).cuda()
    st = torch.cuda.current_stream().cuda_stream
    mids = [torch.full((6, 40, 40, c_out), 777.0, device="cuda") for _ in range(6)]
    outs = [torch.full((6, 40, 40, 32), 777.0, device="cuda") for _ in range(6)]
    for m, o in zip(mids, outs):
        p1.run(x.data_ptr(), 6, 40, 40, b1.data_ptr(), True, m.data_ptr(), st)
        p2.run(m.data_ptr(), 6, 40, 40, b2.data_ptr(), True, o.data_ptr(), st)
    p2.sync(st)
    mid = mids[0].cpu().numpy()
    compare(d1, mid)
    out = outs[0].cpu().numpy()
    compare(d2, out, x=mid)
    for m, o in zip(mids[1:], outs[1:]):
        assert np.array_equal(m.cpu().numpy(), mid)
        assert np.array_equal(o.cpu().numpy(), out)


def test_planned_long_integer_layer():
    # more than 128 input channels: the integer variant folds its exact fp32 partial sums into
    # int32 totals on the way, and the split exchanges those totals
    d = _layer("i8", 1, 320, 48, 10, 10, 1, prune=0.4, lib=8, seed=17)
    pk = pack(d)
    pk.plan(1, 10, 10)
    compare(d, run_gpu(pk, d.x, d.bias, True))

"""GPU parity of planned runs (xgen_patconv_plan before xgen_patconv_run), i.e. of the launch
configuration bench.py times: channel splits exchanged and reduced inside the kernel, over
several pixel tiles and several blocks of output channels.  Every comparison is against the CPU
oracle, through the C ABI."""
import numpy as np
import pytest

from paper_2206_10620_b200 import binding, workloads as wl
from _gpu_util import compare, pack, run_gpu, guarded_output, check_guards

pytestmark = pytest.mark.gpu


def _layer(dtype, n, ci, co, h, w, stride=1, prune=0.5, lib=8, seed=1, idx=0):
    xd = {"f32": "upm1", "f16": "relu_normal", "i8": "u01"}[dtype]
    spec = wl.LayerSpec("t", n, ci, co, h, w, stride, dtype, prune, lib, "he", xd, 0.05, True, idx)
    return wl.make_layer(spec, seed=seed)


def test_vgg16_planned_every_layer_every_element():
    """The benchmark's own stack, planned as the benchmark plans it: 11 of the 13 layers run as
    in-kernel splits over several (tile x filter block) items."""
    split_layers, most_items = 0, 0
    for spec in wl.config_vgg16():
        d = wl.make_layer(spec)
        pk = pack(d)
        y = run_gpu(pk, d.x, d.bias, True, plan=True)
        info = pk.plan_info(spec.n, spec.h, spec.w)
        assert info["blocks"] == info["whole_items"] + (info["items"] - info["whole_items"]) * info["splits"]
        if info["splits"] > 1:
            split_layers += 1
            most_items = max(most_items, info["items"])
            assert info["workspace_bytes"] > 0
        compare(d, y)
    assert split_layers >= 8 and most_items >= 4


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
def test_planned_split_over_several_tiles_and_filter_blocks(dtype, stride):
    d = _layer(dtype, 2, 128, 264, 40, 40, stride, prune=0.6, lib=8, seed=61)
    pk = pack(d)
    pk.plan(2, 40, 40, splits=3)
    info = pk.plan_info(2, 40, 40)
    assert info["splits"] == 3 and info["tiles"] > 1 and info["filter_blocks"] > 1
    assert info["items"] == info["tiles"] * info["filter_blocks"] and info["items"] > 4
    y = run_gpu(pk, d.x, d.bias, True)
    compare(d, y)
    y2 = run_gpu(pk, d.x, None, False)
    compare(d, y2, bias=None, relu=False)
    assert np.array_equal(run_gpu(pk, d.x, d.bias, True), y)        # fixed reduction order


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
def test_split_added_up_by_the_last_block_to_arrive(dtype, stride):
    """Splits that do not wait for each other: more blocks than any GPU holds at once, running in
    waves; the block of an item that counts itself in last adds up all of its partial sums."""
    n = 24 if stride == 1 else 40
    d = _layer(dtype, n, 64, 72, 40, 40, stride, prune=0.6, lib=8, seed=71)
    pk = pack(d)
    pk.plan(n, 40, 40, splits=4, reduce_mode=2)
    info = pk.plan_info(n, 40, 40)
    assert info["last_arriver"] == 1 and info["splits"] == 4 and info["whole_items"] == 0
    assert info["blocks"] == 4 * info["items"] and info["blocks"] > 160
    before = binding.launch_count()
    y = run_gpu(pk, d.x, d.bias, True)
    assert binding.launch_count() - before == 1
    compare(d, y)
    compare(d, run_gpu(pk, d.x, None, False), bias=None, relu=False)
    assert np.array_equal(run_gpu(pk, d.x, d.bias, True), y)        # fixed order of the additions
    # the same sums in the same order as splits that wait (2 x 4 blocks are resident anywhere)
    small = _layer(dtype, 1, 64, 72, 16, 16, stride, prune=0.6, lib=8, seed=72)
    pk2 = pack(small)
    pk2.plan(1, 16, 16, splits=4, reduce_mode=1)
    assert pk2.plan_info(1, 16, 16)["last_arriver"] == 0
    y_wait = run_gpu(pk2, small.x, small.bias, True)
    pk2.plan(1, 16, 16, splits=4, reduce_mode=2)
    assert pk2.plan_info(1, 16, 16)["last_arriver"] == 1
    assert np.array_equal(run_gpu(pk2, small.x, small.bias, True), y_wait)


def test_two_handles_at_once_with_splits_that_do_not_wait():
    """Planned layers of two handles on two streams at the same time: with reduce_mode=2 no block
    waits for another, so the launches may share the GPU in any interleaving."""
    import torch
    ds = [_layer("f32", 8, 64, 72, 24, 24, 1, prune=0.6, lib=8, seed=s) for s in (73, 74)]
    pks = [pack(d) for d in ds]
    streams = [torch.cuda.Stream() for _ in ds]
    xs, bs, ys = [], [], []
    for d, pk in zip(ds, pks):
        pk.plan(8, 24, 24, splits=4, reduce_mode=2)
        assert pk.plan_info(8, 24, 24)["last_arriver"] == 1
        xs.append(torch.from_numpy(d.x).cuda()); bs.append(torch.from_numpy(d.bias).cuda())
        ys.append(guarded_output((8, 24, 24, 72), torch.float32))
    torch.cuda.synchronize()
    for rep in range(3):
        for d, pk, st, x, b, (buf, y) in zip(ds, pks, streams, xs, bs, ys):
            pk.run(x.data_ptr(), 8, 24, 24, b.data_ptr(), True, y.data_ptr(), st.cuda_stream)
    for d, pk, st, (buf, y) in zip(ds, pks, streams, ys):
        pk.sync(st.cuda_stream)
        check_guards(buf)
        compare(d, y.cpu().numpy())


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
def test_last_wave_is_split(dtype):
    """More items than the GPU holds blocks: the items of the last, partly filled wave are split
    (and reduced inside the kernel), all earlier items run whole -- in one launch."""
    d = _layer(dtype, 60, 32, 16, 40, 40, 1, prune=0.5, lib=8, seed=111)
    pk = pack(d)
    pk.plan(60, 40, 40, splits=2, reduce_mode=1)
    info = pk.plan_info(60, 40, 40)
    assert 150 < info["items"] < 220             # 188 tiles of 32 blocks (row tiling) x 1 filter block
    if info["splits"] == 2:                      # a GPU with 148 block slots: 148 whole + 40 x 2
        assert 0 < info["whole_items"] < info["items"]
        assert info["blocks"] == info["whole_items"] + (info["items"] - info["whole_items"]) * 2
    before = binding.launch_count()
    y = run_gpu(pk, d.x, d.bias, True)
    assert binding.launch_count() - before == 1
    compare(d, y)
    assert np.array_equal(run_gpu(pk, d.x, d.bias, True), y)


def _sampled_batch_planned(spec, images):
    d = wl.make_layer(spec)
    pk = pack(d)
    y = run_gpu(pk, d.x, d.bias, True, plan=True)
    for i in images:
        compare(d, y[i:i + 1], x=d.x[i:i + 1])
    return pk.plan_info(spec.n, spec.h, spec.w)


def test_resnet50_planned_one_layer_per_shape():
    seen, splits = set(), []
    for spec in wl.config_resnet50():
        key = (spec.c_in, spec.h, spec.stride)
        if key in seen:
            continue
        seen.add(key)
        splits.append(_sampled_batch_planned(spec, [0, spec.n - 1])["splits"])
    assert max(splits) > 1


def test_resnet18_planned_one_layer_per_shape():
    seen, splits = set(), []
    for spec in wl.config_resnet18():
        key = (spec.c_in, spec.c_out, spec.h, spec.stride)
        if key in seen:
            continue
        seen.add(key)
        splits.append(_sampled_batch_planned(spec, [0, spec.n - 1])["splits"])
    assert max(splits) > 1


@pytest.mark.parametrize("lib", [4, 8, 12])
def test_sweep_every_point_planned(lib):
    """All 48 points of the single-layer sweep (16 per library size), planned as in the benchmark;
    the first and the last image of every batch against the oracle."""
    pts = [s for s in wl.config_sweep() if s.lib_size == lib]
    assert len(pts) == 16 and sorted({s.n for s in pts}) == [1, 8, 64, 256]
    for spec in pts:
        _sampled_batch_planned(spec, [0] if spec.n == 1 else [0, spec.n - 1])


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("case", [
    (3, 28, 28, 1, True),      # 7 x 7 blocks per image: 147 blocks, 4.6 tiles; tiles straddle images
    (5, 30, 27, 1, True),      # ragged: blocks hang over the right and the bottom edge
    (9, 20, 12, 1, True),      # 3 blocks per row: a tile touches up to 11 block rows
    (2, 56, 56, 1, False),     # 14 blocks per row: the staged slots may not fit; any tiling must be right
    (4, 56, 56, 2, False),     # stride 2: 14 x 7 blocks of 2 x 4 pixels
    (7, 26, 30, 2, False),
])
def test_row_tiling(dtype, case):
    """Shapes for which a tile is 32 consecutive pixel blocks of the row-by-row numbering over all
    images (every block row staged as a slot of its own).  Planning the shape may rebuild the
    command stream with smaller channel chunks so that the slots fit shared memory."""
    n, h, w, stride, expect_rows = case
    d = _layer(dtype, n, 48, 40, h, w, stride, prune=0.5, lib=8, seed=101 + n)
    pk = pack(d)
    compare(d, run_gpu(pk, d.x, d.bias, True))               # as packed, whatever tiling fits
    pk.plan(n, h, w, splits=1)
    info = pk.plan_info(n, h, w)
    if expect_rows:
        assert info["row_tiling"] == 1 and info["covered"] > 0.8 and info["tiles"] > 1
        assert info["uses_copy_engine"] == 1
    compare(d, run_gpu(pk, d.x, d.bias, True))
    pk.plan(n, h, w, splits=2)
    assert pk.plan_info(n, h, w)["splits"] == 2
    compare(d, run_gpu(pk, d.x, d.bias, True))
    pk.plan(n, h, w, splits=2, no_copy_engine=True)
    assert pk.plan_info(n, h, w)["uses_copy_engine"] == 0
    compare(d, run_gpu(pk, d.x, None, False), bias=None, relu=False)


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("shape", [(1, 14, 14), (1, 7, 7), (1, 13, 10), (2, 6, 5)])
def test_small_blocks_for_small_images(dtype, shape):
    """A single small image leaves most lanes of every 4x4-pixel tiling idle: planning such a shape
    switches the handle to 4x2 pixels per thread and 16 filters per warp (the command stream is
    rebuilt); planning a large shape switches it back."""
    import torch
    n, h, w = shape
    d = _layer(dtype, n, 96, 200, h, w, 1, prune=0.6, lib=12, seed=121)
    pk = pack(d)
    assert pk.plan_info(n, h, w)["pixels_per_lane"] == 16
    y0 = run_gpu(pk, d.x, d.bias, True)
    compare(d, y0)
    pk.plan(n, h, w)
    info = pk.plan_info(n, h, w)
    assert info["pixels_per_lane"] == 8 and pk.stats()["filters_per_group"] == 16
    compare(d, run_gpu(pk, d.x, d.bias, True))
    compare(d, run_gpu(pk, d.x, None, False), bias=None, relu=False)
    pk.plan(n, h, w, splits=3)
    assert pk.plan_info(n, h, w)["splits"] == 3
    y1 = run_gpu(pk, d.x, d.bias, True)
    compare(d, y1)
    # the fused operators need the large block
    x = torch.from_numpy(d.x).cuda()
    y = torch.empty((n, h, w, 200), dtype={"f32": torch.float32, "f16": torch.float16, "i8": torch.int32}[dtype], device="cuda")
    with pytest.raises(binding.PatconvError) as e:
        pk.run_fused(x.data_ptr(), n, h, w, 0, y.data_ptr(), relu=True)
    assert e.value.status == 4
    pk.plan(n, h, w, no_small_blocks=True)
    assert pk.plan_info(n, h, w)["pixels_per_lane"] == 16
    pk.run_fused(x.data_ptr(), n, h, w, 0, y.data_ptr(), relu=True)
    pk.sync()
    compare(d, y.cpu().numpy(), bias=None)
    # another, large shape on the same handle: back to 4x4 blocks
    pk.plan(n, h, w)
    assert pk.plan_info(n, h, w)["pixels_per_lane"] == 8
    d2 = _layer(dtype, 2, 96, 200, 40, 40, 1, prune=0.6, lib=12, seed=121)
    pk.plan(2, 40, 40)
    assert pk.plan_info(2, 40, 40)["pixels_per_lane"] == 16
    d2.w, d2.pid, d2.masks = d.w, d.pid, d.masks
    compare(d2, run_gpu(pk, d2.x, d.bias, True), bias=d.bias)


def test_small_blocks_universal_table():
    d = _layer("f32", 1, 32, 48, 12, 12, 1, prune=0.4, lib=4, seed=131)
    d.masks = np.array([0x00F, 0x1E0, 0x145, 0x0AA], dtype=np.uint16)
    pk = pack(d)
    pk.plan(1, 12, 12)
    assert pk.plan_info(1, 12, 12)["pixels_per_lane"] == 8 and pk.stats()["patterns_compiled"] == 126
    compare(d, run_gpu(pk, d.x, d.bias, True))


@pytest.mark.parametrize("dtype,stride", [("f32", 2), ("f16", 1), ("f16", 2), ("i8", 1), ("i8", 2)])
def test_universal_table_other_variants(dtype, stride):
    d = _layer(dtype, 2, 24, 40, 13, 15, stride, prune=0.4, lib=4, seed=71)
    d.masks = np.array([0x00F, 0x1E0, 0x145, 0x0AA], dtype=np.uint16)     # none of the built-in shapes
    pk = pack(d)
    assert pk.stats()["patterns_compiled"] == 126
    compare(d, run_gpu(pk, d.x, d.bias, True))


@pytest.mark.parametrize("knob", ["no_copy_engine", "no_launch_overlap"])
@pytest.mark.parametrize("dtype", ["f32", "i8"])
def test_tuning_switches_keep_the_result(knob, dtype):
    d = _layer(dtype, 2, 64, 48, 22, 22, 1, prune=0.5, lib=8, seed=81)
    pk = pack(d)
    pk.plan(2, 22, 22, splits=2)
    assert pk.plan_info(2, 22, 22)["uses_copy_engine"] == 1
    y0 = run_gpu(pk, d.x, d.bias, True)
    pk.plan(2, 22, 22, splits=2, **{knob: True})
    info = pk.plan_info(2, 22, 22)
    assert info["splits"] == 2
    if knob == "no_copy_engine":
        assert info["uses_copy_engine"] == 0
    y1 = run_gpu(pk, d.x, d.bias, True)
    compare(d, y1)
    assert np.array_equal(y0, y1)        # same sums in the same order, whatever stages the tiles


@pytest.mark.parametrize("dtype,stride", [("f32", 1), ("f16", 2), ("i8", 1)])
def test_tuned_grouping_keeps_the_result(dtype, stride):
    """The tuning-decided parameters of a layer (channels per chunk, filter groups per block) rebuild
    the command stream at plan time; every grouping computes the same layer."""
    d = _layer(dtype, 2, 64, 200, 24, 24, stride, prune=0.5, lib=8, seed=83)
    pk = pack(d)
    pk.plan(2, 24, 24)
    base = pk.plan_info(2, 24, 24)
    compare(d, run_gpu(pk, d.x, d.bias, True))
    seen = set()
    for cc, g in ((4, 0), (16, 0), (0, 4), (8, 8), (4, 1)):
        pk.plan(2, 24, 24, channels_per_chunk=cc, groups_per_block=g)
        info, st = pk.plan_info(2, 24, 24), pk.stats()
        if cc:
            assert st["channels_per_chunk"] in (cc, cc // 2, cc // 4)    # halved while a chunk's commands overflow their stage
        if g:
            assert st["groups_per_block"] == min(g, base["threads_per_block"] // 32 - 4)
            assert info["threads_per_block"] == 32 * (st["groups_per_block"] + 4)
        seen.add((st["channels_per_chunk"], st["groups_per_block"]))
        compare(d, run_gpu(pk, d.x, d.bias, True))
    assert len(seen) >= 4
    pk.plan(2, 24, 24)                               # back to the library's own grouping
    assert pk.plan_info(2, 24, 24)["filter_blocks"] == base["filter_blocks"]
    compare(d, run_gpu(pk, d.x, d.bias, True))
    with pytest.raises(binding.PatconvError) as e:
        pk.plan(2, 24, 24, channels_per_chunk=5)
    assert e.value.status == 1


def test_bounded_wait_runs_out_and_the_handle_recovers():
    """A planned split told to expect one arrival that never comes: every block's wait runs out
    after the (shortened) limit, the kernel ends by itself, xgen_patconv_last_status reports
    the timeout once, and the next ordinary run is correct again.  Nothing traps or spins on."""
    import torch
    d = _layer("f32", 1, 128, 32, 12, 12, 1, prune=0.5, lib=8, seed=91)
    pk = pack(d)
    pk.plan(1, 12, 12, splits=4, wait_limit_ms=20, reduce_mode=1)
    info = pk.plan_info(1, 12, 12)
    assert info["splits"] == 4 and info["last_arriver"] == 0
    compare(d, run_gpu(pk, d.x, d.bias, True))
    pk.test_expect_arrivals(1)
    x = torch.from_numpy(d.x).cuda()
    b = torch.from_numpy(d.bias).cuda()
    buf, y = guarded_output((1, 12, 12, 32), torch.float32)
    st = torch.cuda.current_stream().cuda_stream
    pk.run(x.data_ptr(), 1, 12, 12, b.data_ptr(), True, y.data_ptr(), st)      # only enqueues: OK
    with pytest.raises(binding.PatconvError) as e:
        pk.sync(st)
    assert e.value.status == 7
    check_guards(buf)
    pk.sync(st)                                                                # reported once
    pk.test_expect_arrivals(0)
    compare(d, run_gpu(pk, d.x, d.bias, True))
    compare(d, run_gpu(pk, d.x, d.bias, True))

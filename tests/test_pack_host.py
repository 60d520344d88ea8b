"""The packer, checked on the CPU: the packed command stream must describe
exactly the masked dense weight tensor.  A small interpreter written here walks
the stream (it shares no code with the library) and rebuilds that tensor."""
import numpy as np
import pytest

from paper_2206_10620_b200 import binding, workloads as wl


def _masked_dense(d):
    keep = np.zeros((len(d.masks) + 1, 9), dtype=bool)
    for p, m in enumerate(d.masks):
        keep[p] = [(int(m) >> t) & 1 for t in range(9)]
    sel = keep[d.pid].reshape(d.pid.shape + (3, 3))
    return np.where(sel, d.w.astype(np.float64), 0.0)


def _walk(pk, c_in, c_out, stride=1):
    """Rebuild [c_out,c_in,9] from the stream; also return counters."""
    st, v = pk.stats(), pk.view()
    J, G, cc = st["filters_per_group"], st["groups_per_block"], st["channels_per_chunk"]
    npc = st["patterns_compiled"]
    dense = np.zeros((c_out, c_in, 9))
    seen = np.zeros((c_out, c_in), dtype=int)
    loads = 0
    for b in range(st["n_blocks"]):
        for c in range(st["n_chunks"]):
            for g in range(G):
                lo, hi = v["seg_off"][b, c, g], v["seg_off"][b, c, g + 1]
                ic, last_key = None, None
                assert hi > lo and v["slots"][hi - 1, 0] == npc + 1      # run ends with END
                for s in v["slots"][lo:hi - 1]:
                    op, operand = int(s[0]), int(s[1])
                    if op == npc:
                        ic = c * cc + operand
                        assert ic < c_in
                        loads += 1
                        last_key = None
                    else:
                        T = 16 if stride == 1 else 8
                        assert op < npc and ic is not None and operand % T == 0
                        j = operand // T
                        oc = int(v["slot_oc"][b, g, j])
                        assert 0 <= oc < c_out
                        key = (op, j)
                        assert last_key is None or key > last_key      # sorted by (pattern, slot)
                        last_key = key
                        taps = [t for t in range(9) if (int(v["masks"][op]) >> t) & 1]
                        assert len(taps) == 4
                        dense[oc, ic, taps] = s[4:8].view(np.float32).astype(np.float64)
                        seen[oc, ic] += 1
    return dense, seen, loads


@pytest.mark.parametrize("dtype", ["f32", "f16", "i8"])
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("shape", [(5, 7), (16, 32), (40, 150), (3, 64), (300, 20)])
def test_stream_rebuilds_masked_tensor(dtype, stride, shape):
    ci, co = shape
    spec = wl.LayerSpec("t", 1, ci, co, 4, 4, stride, dtype, 0.45, 12, 0.5, "upm1", 0.1, True, 2)
    d = wl.make_layer(spec, seed=9)
    pk = binding.Packed(ci, co, stride, dtype, d.masks, d.w, d.pid, device=-1)
    dense, seen, loads = _walk(pk, ci, co, stride)
    np.testing.assert_array_equal(dense.reshape(co, ci, 3, 3), _masked_dense(d))
    np.testing.assert_array_equal(seen, (d.pid >= 0).astype(int))          # each survivor exactly once
    st = pk.stats()
    assert st["kernels_surviving"] == int((d.pid >= 0).sum())
    assert st["macs_per_pixel"] == 4 * st["kernels_surviving"]
    assert st["load_commands"] == loads
    v = pk.view()
    oc = v["slot_oc"].ravel()
    assert sorted(oc[oc >= 0].tolist()) == list(range(co))               # a bijection onto the filters
    # every group is an aligned run of J consecutive output channels
    J = st["filters_per_group"]
    for grp in v["slot_oc"].reshape(-1, J):
        if grp[0] < 0:
            assert (grp < 0).all()
            continue
        assert grp[0] % J == 0
        for j in range(J):
            assert grp[j] == (grp[0] + j if grp[0] + j < co else -1)


def test_index_overhead_below_csr_and_balance():
    spec = wl.config_vgg16()[5]
    pid = wl.make_pattern_ids(wl.BASE_SEED, spec.index, spec.c_out, spec.c_in, 8, 0.7)
    w = np.zeros((spec.c_out, spec.c_in, 3, 3), np.float32)
    pk = binding.Packed(spec.c_in, spec.c_out, 1, "f32", wl.pattern_library(8), w, pid, device=-1)
    st = pk.stats()
    assert st["kernels_surviving"] == spec.k_surv
    # information content of the layout (one opcode and one operand byte per command plus the
    # tables) against CSR's one 4-byte index per weight
    assert st["compact_index_bytes"] < st["csr_index_bytes"] / 4
    # what the device copy really stores beyond the kept weights: 48-byte slots and the tables
    v = pk.view()
    tables = 4 * (v["seg_off"].size + v["slot_oc"].size)
    assert st["stream_bytes"] == 48 * len(v["slots"])
    assert st["index_bytes"] == st["stream_bytes"] + tables - st["weight_bytes"]
    assert st["weight_bytes"] == 16 * st["kernels_surviving"]
    # per kernel that is 32 bytes (opcode, operand and the duplicate of the weights) plus the
    # LOAD and END slots: about twice CSR's 16 bytes -- the price of decoding a command with
    # two vector loads straight into the operand pairs of the packed FMAs
    assert 1.5 * st["csr_index_bytes"] < st["index_bytes"] < 4 * st["csr_index_bytes"]
    assert 1.0 <= st["group_imbalance"] < 1.05
    assert st["patterns_compiled"] == 8


def test_library_sizes_and_foreign_masks():
    d = wl.make_layer(wl.LayerSpec("t", 1, 8, 16, 4, 4, 1, "f32", 0.3, 4, 0.5, "upm1", 0.1, True, 1), seed=3)
    assert binding.Packed(8, 16, 1, "f32", d.masks, d.w, d.pid, device=-1).stats()["patterns_compiled"] == 4
    # masks in any order, and one outside the built-in library -> universal table
    masks = np.array([0x1B0, 0x00F, 0x134, 0x01B], dtype=np.uint16)
    d.masks = masks
    pk = binding.Packed(8, 16, 1, "f32", masks, d.w, d.pid, device=-1)
    assert pk.stats()["patterns_compiled"] == 126
    dense, seen, _ = _walk(pk, 8, 16)
    np.testing.assert_array_equal(dense.reshape(16, 8, 3, 3), _masked_dense(d))
    # reordered built-in masks still use the small table
    masks2 = np.array([0x1B0, 0x036, 0x01B, 0x0D8], dtype=np.uint16)
    d.masks = masks2
    pk2 = binding.Packed(8, 16, 1, "f32", masks2, d.w, d.pid, device=-1)
    assert pk2.stats()["patterns_compiled"] == 4
    dense, _, _ = _walk(pk2, 8, 16)
    np.testing.assert_array_equal(dense.reshape(16, 8, 3, 3), _masked_dense(d))


def test_all_pruned_and_empty_filter():
    d = wl.make_layer(wl.LayerSpec("t", 1, 8, 16, 4, 4, 1, "f32", 0.3, 8, 0.5, "upm1", 0.1, True, 1), seed=3)
    pid = np.full_like(d.pid, -1)
    pk = binding.Packed(8, 16, 1, "f32", d.masks, d.w, pid, device=-1)
    st = pk.stats()
    assert st["kernels_surviving"] == 0 and st["load_commands"] == 0
    dense, seen, _ = _walk(pk, 8, 16)
    assert not dense.any()

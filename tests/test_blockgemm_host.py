"""The block-pruned packer on the host (no GPU): an interpreter in this test walks the packed
stream the way the kernel's warps do and rebuilds the masked dense matrix from it."""
import numpy as np
import pytest

from paper_2206_10620_b200 import binding, workloads as wl


def _masked(d):
    s = d.spec
    oc = np.arange(s.c_out)[:, None]
    c = np.arange(s.k)[None, :]
    keep = d.row_keep[oc // s.br, c // s.bc, oc % s.br].astype(bool) & d.col_keep[oc // s.br, c // s.bc, c % s.bc].astype(bool)
    return np.where(keep, d.w.astype(np.float32), np.float32(0))


def _rebuild(pk, k, c_out):
    st = pk.stats()
    units, seg = pk.view()
    W, ks, ns = st["warps_per_block"], st["stage_cols"], st["n_stages"]
    out = np.zeros((c_out, k), np.float32)
    hits = np.zeros((c_out, k), np.int32)
    padded = groups = rows = 0
    for rb in range(st["row_blocks"]):
        for s in range(ns):
            base = (rb * ns + s) * (W + 1)
            assert seg[base + W] - seg[base] <= st["max_stage_bytes"] // 16
            for w in range(W):
                u, end = seg[base + w], seg[base + w + 1]
                r0 = rb * 16 * W + 16 * w
                while u < end:
                    n_rows = int(units[u, 0])
                    cols = [(int(units[u, 1 + i // 4]) >> (8 * (i % 4))) & 0xFF for i in range(8)]
                    assert units[u, 3] == 0 and n_rows >= 1
                    groups += 1
                    seen = set()
                    for r in range(n_rows):
                        hdr = units[u + 1 + 3 * r]
                        assert hdr[0] % 8 == 0 and 0 <= hdr[0] < 128 and hdr[0] not in seen
                        seen.add(int(hdr[0]))                      # a row at most once per group
                        oc = r0 + int(hdr[0]) // 8
                        wts = np.concatenate([units[u + 2 + 3 * r], units[u + 3 + 3 * r]]).view(np.float32)
                        for i, ci in enumerate(cols):
                            if ci == ks:
                                assert wts[i] == 0.0
                                padded += 1
                            else:
                                assert ci < ks and s * ks + ci < k and oc < c_out
                                out[oc, s * ks + ci] += wts[i]
                                hits[oc, s * ks + ci] += 1
                        rows += 1
                    u += 1 + 3 * n_rows
                assert u == end
    assert padded == st["padded_slots"] and groups == st["column_groups"] and rows == st["row_commands"]
    return out, hits


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("k,c_out,br,bc,rk,ck", [
    (64, 64, 32, 32, 0.5, 0.5), (200, 100, 32, 32, 0.4, 0.4), (96, 272, 64, 32, 0.5, 0.25),
    (40, 24, 8, 8, 0.5, 0.5), (72, 40, 4, 16, 0.75, 0.5), (45, 19, 8, 16, 0.6, 0.6),
    (128, 48, 16, 64, 1.0, 1.0), (5, 3, 2, 2, 0.5, 0.5), (48, 32, 16, 1, 1.0, 0.5)])
def test_stream_rebuilds_the_masked_matrix(dtype, k, c_out, br, bc, rk, ck):
    d = wl.make_block_gemm(wl.GemmSpec("t", 4, k, c_out, br, bc, rk, ck, dtype, "upm1", 0.05, True, 21))
    pk = binding.BlockGemm(k, c_out, br, bc, dtype, d.w, d.row_keep, d.col_keep, device=-1)
    out, hits = _rebuild(pk, k, c_out)
    wm = _masked(d)
    assert np.array_equal(out, wm)
    # every kept entry exactly once, no pruned entry at all
    oc = np.arange(c_out)[:, None]
    c = np.arange(k)[None, :]
    keep = d.row_keep[oc // br, c // bc, oc % br].astype(bool) & d.col_keep[oc // br, c // bc, c % bc].astype(bool)
    assert np.array_equal(hits, keep.astype(np.int32))
    st = pk.stats()
    assert st["weights_kept"] == d.kept_weights() == int(keep.sum())
    assert st["weights_total"] == k * c_out
    assert st["stream_bytes"] >= 16 * (st["column_groups"] + 3 * st["row_commands"])


def test_everything_pruned_gives_an_empty_stream_and_errors_are_reported():
    d = wl.make_block_gemm(wl.GemmSpec("t", 4, 32, 32, 16, 16, 0.0, 0.5, "f32", "upm1", 0.05, True, 22))
    pk = binding.BlockGemm(32, 32, 16, 16, "f32", d.w, d.row_keep, d.col_keep, device=-1)
    assert pk.stats()["row_commands"] == 0 and pk.stats()["weights_kept"] == 0
    with pytest.raises(binding.PatconvError) as e:
        binding.BlockGemm(32, 32, 16, 16, "i8", d.w, d.row_keep, d.col_keep, device=-1)
    assert e.value.status == 4
    with pytest.raises(binding.PatconvError) as e:
        pk.run(1 << 20, 4, 0, True, 2 << 20)                 # a host-only handle cannot run
    assert e.value.status == 6


def test_neighbouring_blocks_with_the_same_rows_share_column_groups():
    """No row pruning, blocks of 4 columns of which 2 are kept: four blocks fill one group of eight."""
    d = wl.make_block_gemm(wl.GemmSpec("t", 4, 64, 16, 16, 4, 1.0, 0.5, "f32", "upm1", 0.05, True, 23))
    pk = binding.BlockGemm(64, 16, 16, 4, "f32", d.w, d.row_keep, d.col_keep, device=-1)
    st = pk.stats()
    assert st["padded_slots"] == 0
    assert st["column_groups"] == (64 // 4 * 2) // 8

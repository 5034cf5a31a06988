"""CPU tests of the host-side work split: the share bounds handed to the CTAs of a launch must cover every work
item of every layer exactly once, in order, whatever the grid, the number of dynamic shares and the kernel variant
(the kernel walks from one bound to the next without any check of its own), and the static shares must be balanced
by cost."""
import numpy as np
import pytest

from paper_2608_15602_b200 import build, fluxbin, synth


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def header_of(M, N, Kb, Ks, g, n_sal, seed=1):
    """First 256 bytes of a packed layer of these dimensions (the bits do not matter for the split)."""
    idx = None
    if Ks and n_sal:
        idx = np.sort(np.random.default_rng(seed).choice(N, n_sal, replace=False)).astype(np.int32)
    L = synth.make_linear(seed, 9, M, N, Kb, Ks, g, idx)
    return np.ascontiguousarray(fluxbin.pack_host(L)[:256])


def walk(cuts, items):
    """Emulate the kernel's walk over its shares; returns per layer how often each work item was visited."""
    cover = [np.zeros(n, np.int32) for n in items]
    for s in range(len(cuts) - 1):
        (e0, i0), (e1, i1) = cuts[s], cuts[s + 1]
        for e in range(e0, e1 + 1):
            if e == e1 and i1 == 0:
                break
            assert e < len(items), "a share reaches past the last layer"
            cur = i0 if e == e0 else 0
            end = i1 if e == e1 else items[e]
            assert 0 <= cur <= end <= items[e]
            cover[e][cur:end] += 1
    return cover


LAYERS = [(70, 256, 2, 0, 128, 0), (1000, 512, 2, 1, 128, 26), (33, 1024, 4, 2, 128, 64), (4096, 256, 2, 1, 128, 13),
          (1, 256, 2, 0, 128, 0), (257, 2048, 2, 1, 128, 100)]


@pytest.mark.parametrize("np_", [1, 2])
@pytest.mark.parametrize("grid,nshares,static_pct", [(1, 1, 100), (7, 7, 100), (148, 148, 100), (444, 444, 100),
                                                     (444, 1776, 90), (37, 148, 50), (3, 12, 99)])
@pytest.mark.parametrize("mode", [1, 4, 16 + 8])
def test_shares_cover_every_work_item_exactly_once(np_, grid, nshares, static_pct, mode):
    headers = [header_of(*d) for d in LAYERS]
    cuts, items = fluxbin.debug_cut_shares(headers, mode, np_, grid, nshares, static_pct)
    assert tuple(cuts[0]) == (0, 0) and tuple(cuts[-1]) == (len(LAYERS), 0)
    keys = cuts[:, 0].astype(np.int64) * (1 << 32) + cuts[:, 1]
    assert np.all(np.diff(keys) >= 0), "share bounds must be non-decreasing"
    for e, c in enumerate(walk(cuts.tolist(), items.tolist())):
        assert np.all(c == 1), f"layer {e}: items visited {np.unique(c)} times"
    for e, i in cuts[:-1]:
        assert e == len(LAYERS) or i < items[e], "a bound at the end of a layer is written as the start of the next"


def test_single_layer_and_odd_pair_counts():
    h = [header_of(300, 384, 3, 1, 128, 20)]           # 9 global units -> 5 pairs: odd, one-pair kernel only
    cuts, items = fluxbin.debug_cut_shares(h, 1, 1, 50, 50)
    assert all(np.all(c == 1) for c in walk(cuts.tolist(), items.tolist()))
    with pytest.raises(fluxbin.FluxBinError):
        fluxbin.debug_cut_shares(h, 1, 2, 50, 50)


def test_static_shares_are_balanced_by_cost():
    """With one share per CTA every share's item count stays within one table build (22 plain items) plus one row
    block of the mean when all items cost the same (no salient region)."""
    headers = [header_of(2048, 1024, 2, 0, 128, 0), header_of(4096, 512, 2, 0, 128, 0)]
    grid = 64
    cuts, items = fluxbin.debug_cut_shares(headers, 1, 1, grid, grid)
    pos = np.concatenate([[0], np.cumsum(items)])
    flat = np.array([pos[e] + i for e, i in cuts])
    per_share = np.diff(flat)
    assert per_share.sum() == items.sum()
    # a share that starts a new pair pays one build (= 22 items); layers end with an epilogue of a few items
    assert per_share.max() - per_share.min() <= 2 * 22 + 8, per_share


def test_rejects_bad_arguments():
    h = [header_of(64, 128, 2, 0, 128, 0)]
    lib = fluxbin.library()
    import ctypes
    out = np.zeros((5, 2), np.int32)
    hp = (ctypes.c_void_p * 1)(h[0].ctypes.data)
    assert lib.fluxbin_debug_cut_shares(1, hp, 3, 1, 4, 4, 100, out.ctypes.data, None) == 3       # no such mode
    assert lib.fluxbin_debug_cut_shares(1, hp, 1, 1, 4, 2, 100, out.ctypes.data, None) == 3       # nshares < grid
    assert lib.fluxbin_debug_cut_shares(1, hp, 1, 1, 4, 4, 100, None, None) == 1
    bad = h[0].copy()
    bad[0] ^= 0xFF
    hp = (ctypes.c_void_p * 1)(bad.ctypes.data)
    assert lib.fluxbin_debug_cut_shares(1, hp, 1, 1, 4, 4, 100, out.ctypes.data, None) == 9       # not a packed layer

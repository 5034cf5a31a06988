"""CPU tests of the host side of the library: symbols, validation, byte model, bit-exact
pack/unpack round trip, and the packed layout walked by a numpy emulator against the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from oracle import models
from paper_2608_15602_b200 import build, fluxbin, synth
from packed_emulator import emulate_linear, parse_header

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FIELDS = ["bits", "row_scale", "col_scale", "sal_idx", "sal_bits", "sal_row_scale", "sal_col_scale"]


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def layer(seed, M, N, Kb, Ks, g, n_sal, pattern="random"):
    idx = None
    if Ks and n_sal:
        rng = np.random.default_rng(seed)
        if pattern == "random":
            idx = np.sort(rng.choice(N, n_sal, replace=False))
        elif pattern == "one_group":
            idx = np.arange(n_sal) + (N // g - 1) * g
        elif pattern == "first":
            idx = np.arange(n_sal)
        idx = idx.astype(np.int32)
    return synth.make_linear(seed, 3, M, N, Kb, Ks, g, idx)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "fluxbin.h")).read()
    declared = set(re.findall(r"\b(fluxbin_[a-z_]+)\s*\(", header))
    assert {"fluxbin_pack", "fluxbin_linear", "fluxbin_unpack", "fluxbin_packed_size"} <= declared
    lib = ctypes.CDLL(build.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in include/fluxbin.h but not exported"
    for name in fluxbin.EXPORTS:
        assert name in declared


CASES = [(1, 32, 1, 0, 32, 0), (5, 128, 2, 1, 32, 7), (33, 384, 3, 2, 128, 40), (100, 256, 1, 1, 256, 19),
         (64, 1024, 2, 1, 128, 51), (7, 96, 2, 2, 96, 50), (9, 160, 4, 3, 32, 160), (40, 512, 2, 1, 512, 1),
         (31, 256, 2, 2, 64, 9), (65, 640, 2, 1, 128, 640), (127, 128, 4, 4, 64, 128)]


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", CASES)
def test_pack_unpack_round_trip_is_bit_exact(M, N, Kb, Ks, g, n_sal):
    L = layer(M + N, M, N, Kb, Ks, g, n_sal)
    # exercise special fp16 patterns: zeros, negative zero, subnormals, max finite
    L.row_scale.flat[::7] = 0x0001
    L.row_scale.flat[1::11] = 0x8000
    L.col_scale.flat[::5] = 0x7BFF
    if L.Ks:
        L.sal_row_scale.flat[::3] = 0x03FF
        L.sal_col_scale.flat[::2] = 0x0000
    buf = fluxbin.pack_host(L)
    assert buf.size == fluxbin.packed_size(L)
    assert buf.size <= fluxbin.packed_size(L, with_map=False)
    U = fluxbin.unpack_host(buf)
    for f in FIELDS:
        assert np.array_equal(getattr(L, f), getattr(U, f)), f
    assert np.array_equal(buf, fluxbin.pack_host(L))          # deterministic bytes


@pytest.mark.parametrize("pattern", ["one_group", "first"])
def test_round_trip_degenerate_salient_maps(pattern):
    L = layer(5, 37, 512, 2, 2, 128, 100, pattern)
    U = fluxbin.unpack_host(fluxbin.pack_host(L))
    for f in FIELDS:
        assert np.array_equal(getattr(L, f), getattr(U, f)), f


@pytest.mark.parametrize("M,N,Kb,Ks,g,n_sal", CASES)
def test_packed_layout_walk_matches_oracle(M, N, Kb, Ks, g, n_sal):
    """The documented addressing (slot = lane ^ step, segment scales, fused column table) applied
    to the packed bytes gives the oracle's y: pins the packer's layout on the CPU."""
    L = layer(2 * M + N, M, N, Kb, Ks, g, n_sal)
    x = synth.make_activations(9, M, 2, N)
    want = oracle.linear_direct(L, x)
    got = emulate_linear(fluxbin.pack_host(L), x)
    W = np.abs(oracle.dense_weight(L))
    bound = np.abs(x.view(np.float16).astype(np.float64)) @ W.T
    assert np.all(np.abs(got - want) <= 1e-12 * bound + 1e-300)


def test_widest_layer_layout_walk():
    """N = 65536 (the limit of the 16-bit column indices), salient columns at both ends of the index range."""
    N = 65536
    idx = np.array([0, 1, 127, 128, 40000, 65407, 65408, 65534, 65535], dtype=np.int32)
    L = synth.make_linear(91, 5, 70, N, 1, 2, 128, idx)
    x = synth.make_activations(91, 6, 2, N)
    want = oracle.linear_direct(L, x)
    buf = fluxbin.pack_host(L)
    got = emulate_linear(buf, x)
    bound = np.abs(x.view(np.float16).astype(np.float64)) @ np.abs(oracle.dense_weight(L)).T
    assert np.all(np.abs(got - want) <= 1e-12 * bound + 1e-300)
    U = fluxbin.unpack_host(buf)
    for f in FIELDS:
        assert np.array_equal(getattr(L, f), getattr(U, f)), f


def test_validation_statuses():
    L = layer(1, 8, 128, 2, 1, 32, 5)
    assert fluxbin.validate(L) == 0
    bad = layer(1, 8, 128, 2, 1, 32, 5)
    bad.sal_idx[1] = bad.sal_idx[0]
    assert fluxbin.status_string(fluxbin.validate(bad)).startswith("salient map")
    assert fluxbin.packed_size(bad) == 0
    bad.sal_idx[:] = np.arange(5) + 200
    assert fluxbin.validate(bad) == 4
    for field, val, status in [("N", 100, 2), ("g", 48, 2), ("M", 0, 2), ("Kb", 0, 3), ("Kb", 5, 3), ("Ks", 5, 3),
                               ("g", 96, 2), ("N", 131072, 2)]:
        b = layer(1, 8, 128, 2, 1, 32, 5)
        setattr(b, field, val)
        assert fluxbin.validate(b) == status, (field, val)
        assert fluxbin.packed_size(b) == 0
    b = layer(1, 8, 128, 2, 1, 32, 5)
    b.row_scale = np.zeros(0, np.uint16)
    assert fluxbin.validate(b) == 1
    buf = fluxbin.pack_host(L)
    d = fluxbin.make_desc(L)
    lib = fluxbin.library()
    assert lib.fluxbin_pack_host(ctypes.byref(d), buf.ctypes.data, buf.size - 1) == 5
    corrupt = buf.copy()
    corrupt[0] ^= 1
    assert lib.fluxbin_packed_dims(corrupt.ctypes.data, corrupt.size, ctypes.byref(fluxbin.LayerDesc())) == 9
    corrupt = buf.copy()
    corrupt[16] ^= 1                # Kb changed: header no longer self-consistent
    assert lib.fluxbin_packed_dims(corrupt.ctypes.data, corrupt.size, ctypes.byref(fluxbin.LayerDesc())) == 9
    assert lib.fluxbin_linear(None, None, 1, 0, None, 0, 0, None, 0, None) == 1
    assert lib.fluxbin_workspace_size(None, 1) == 0
    assert lib.fluxbin_set_table_format(None, 1) == 1 and lib.fluxbin_get_table_format(None) == -1
    assert lib.fluxbin_num_launches(None, 4) == -1


def test_packed_bytes_track_the_storage_model():
    """Padding and the 16-bit column index table are the only bytes above S_base + S_sal: nothing without salient
    columns; with them, the per-group padding of the virtual columns to whole sub-vectors (about 77 sub-vectors
    where the storage model counts 52 bytes of bits and 64 scales per row at N = 8192, 5 % salient) plus at most 15
    unused table slots in the last, narrow salient pair."""
    for (M, N, Kb, Ks, g, n_sal, bound) in [(4096, 4096, 2, 0, 128, 0, 1.005), (1024, 8192, 2, 1, 128, 410, 1.045),
                                            (28672, 8192, 2, 1, 128, 410, 1.03), (8192, 28672, 2, 1, 128, 1434, 1.03)]:
        L = synth.make_linear(1, 1, 32, N, Kb, Ks, g, synth.salient_random(1, 1, N, n_sal / N) if n_sal else None)
        L.M = M                                # dims only: packed_size does not read the arrays
        size = fluxbin.packed_size(L)
        model = models.storage_bits(M, N, Kb, Ks, g, n_sal) / 8
        assert model <= size <= bound * model, (size, model)


@pytest.mark.parametrize("n_sal,Ks,want_w", [(8, 1, 8), (70, 1, 16), (130, 1, 32), (260, 1, 8), (40, 2, 16), (100, 3, 16),
                                             (128, 4, 32)])
def test_last_salient_pair_is_stored_narrow(n_sal, Ks, want_w):
    """All salient sub-vectors of all bases share one flat list of table slots; a last pair with at most 8 / 16
    live slots carries 8 / 16 steps per item (96 bytes per step and 32 rows) instead of 32."""
    M, N, g = 70, 1024, 1024 // 8                      # 8 row-scale groups
    idx = (np.arange(n_sal) * (N // n_sal)).astype(np.int32) if n_sal <= 128 else np.arange(n_sal, dtype=np.int32)
    L = synth.make_linear(3, 3, M, N, 2, Ks, g, idx)
    buf = fluxbin.pack_host(L)
    h = parse_header(buf)
    groups, counts = np.unique(idx // g, return_counts=True)
    n_sv = int(((counts + 7) // 8).sum())
    want_pairs = -(-n_sv * Ks // 32)
    last = n_sv * Ks - 32 * (want_pairs - 1)
    assert h["n_sal_svec"] == n_sv and h["npairs1"] == want_pairs
    assert h["sal_last_w"] == (8 if last <= 8 else 16 if last <= 16 else 32) == want_w, (n_sv, last)
    nrb = h["nrb"]
    assert h["off_sal_idx"] - h["off_items1"] == (want_pairs - 1) * nrb * 3072 + nrb * (3072 if want_w == 32 else 96 * want_w)
    U = fluxbin.unpack_host(buf)
    for f in FIELDS:
        assert np.array_equal(getattr(L, f), getattr(U, f)), f
    x = synth.make_activations(9, M, 2, N)
    want = oracle.linear_direct(L, x)
    got = emulate_linear(buf, x)
    assert np.allclose(got, want, rtol=1e-11, atol=1e-12 * np.abs(want).max())

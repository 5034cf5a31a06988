"""fluxbin_linear_noalloc: the entry point for callers that cannot allocate device memory (guests of a
host application that owns the allocator and hands them only input and output buffers).

Collected last on purpose (see `pytest --collect-only`): it shares one fixed scratch array per device
with every other call of that entry point, so a failure here cannot hide behind an earlier test.
The new entry point is called through the C-ABI twice in a row -- different layer, different batch --
and each result is compared with what the existing fluxbin_linear gives for the same inputs, at the
tolerance the parity tests use.
"""
import numpy as np
import pytest

from paper_2608_15602_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

REL_L2 = 1e-3
MAX_REL = 5e-3


def _close(got, want, what):
    for b in range(want.shape[0]):
        rms = np.sqrt(np.mean(want[b] ** 2))
        l2 = np.linalg.norm(got[b] - want[b]) / max(np.linalg.norm(want[b]), 1e-300)
        rel = np.abs(got[b] - want[b]) / np.maximum(np.abs(want[b]), 1e-2 * rms + 1e-300)
        assert l2 <= REL_L2, f"{what} row {b}: rel L2 {l2:.3e}"
        assert rel.max() <= MAX_REL, f"{what} row {b}: max rel {rel.max():.3e}"


def test_noalloc_matches_workspace_entry_point_on_two_calls_in_a_row():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import fluxbin, layer

    cases = [(2100, 1024, 2, 1, 128, 51, 1), (777, 512, 2, 2, 128, 40, 6)]      # (M, N, Kb, Ks, g, n_sal, B)
    for call, (M, N, Kb, Ks, g, n_sal, B) in enumerate(cases):
        idx = np.sort(np.random.default_rng(call).choice(N, n_sal, replace=False)).astype(np.int32)
        L = synth.make_linear(900 + call, 1, M, N, Kb, Ks, g, idx)
        x = synth.make_activations(900 + call, 2, B, N)
        lin = layer.FluxBinLinear(L)
        xt = torch.from_numpy(x.view(np.float16)).cuda()
        want = lin.forward(xt, lin.workspace(B), fp32_out=True)                  # existing entry point
        got = torch.full((B, M), float("nan"), dtype=torch.float32, device="cuda")
        fluxbin.linear_noalloc(lin.weight, xt.data_ptr(), B, xt.stride(0), got.data_ptr(), True, got.stride(0),
                               int(torch.cuda.current_stream().cuda_stream))
        torch.cuda.synchronize()
        _close(got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64), f"call {call}")


def test_noalloc_rejects_layers_beyond_the_fixed_scratch():
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import fluxbin, layer
    cap = fluxbin.noalloc_capacity()
    assert cap == 1 << 20
    L = synth.make_linear(5, 5, 140000, 32, 1, 0, 32)                            # 140,000 rows: needs > 1 MiB at batch 2
    lin = layer.FluxBinLinear(L)
    assert lin.weight.workspace_size(2) > cap
    x = torch.zeros((2, 32), dtype=torch.float16, device="cuda")
    y = torch.zeros((2, 140000), dtype=torch.float16, device="cuda")
    st = fluxbin.linear_noalloc_status(lin.weight, x.data_ptr(), 2, 32, y.data_ptr(), False, 140000)
    assert st == 5 and "too small" in fluxbin.status_string(st)
    assert fluxbin.linear_noalloc_status(lin.weight, x.data_ptr(), 1, 32, y.data_ptr(), False, 140000) == 0  # batch 1 fits
    torch.cuda.synchronize()


def test_noalloc_row_limits_follow_the_accumulator_rows_of_the_batch():
    """The scratch holds one fp32 accumulator row per vector of a chunk: four rows from batch 3 with fp32 table
    entries, eight from batch 5 with fp16 entries.  Status checks only: calls just above a limit are rejected
    before anything is put on the stream, calls just below it are accepted."""
    from paper_2608_15602_b200 import build
    build.build()
    from paper_2608_15602_b200 import fluxbin, layer
    cap = fluxbin.noalloc_capacity()
    for rows, B, fp16_tables, fits in [(65000, 4, False, True), (66000, 4, False, False),
                                       (32400, 8, True, True), (33000, 8, True, False), (65000, 8, False, True)]:
        lin = layer.FluxBinLinear(synth.make_linear(6, rows, rows, 32, 1, 0, 32), fp16_tables=fp16_tables)
        assert (lin.weight.workspace_size(B) <= cap) == fits, (rows, B, fp16_tables)
        x = torch.zeros((B, 32), dtype=torch.float16, device="cuda")
        y = torch.zeros((B, rows), dtype=torch.float16, device="cuda")
        st = fluxbin.linear_noalloc_status(lin.weight, x.data_ptr(), B, 32, y.data_ptr(), False, rows)
        assert st == (0 if fits else 5), (rows, B, fp16_tables, st)
        # argument errors are reported before the scratch is cleared
        assert fluxbin.linear_noalloc_status(lin.weight, x.data_ptr(), B, 16, y.data_ptr(), False, rows) == 3
        assert fluxbin.linear_noalloc_status(lin.weight, x.data_ptr() + 2, B, 32, y.data_ptr(), False, rows) == 6
    torch.cuda.synchronize()

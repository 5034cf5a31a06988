"""Device-resident FluxBin linear layer: torch owns the memory and the stream, the C-ABI library
does all the work (argument marshalling only on this side)."""
from __future__ import annotations

import numpy as np
import torch

from . import fluxbin


def _stream_ptr(stream=None) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


class Workspace:
    """Zero-initialised scratch for fluxbin_linear; any number of stream-ordered calls may share it."""

    def __init__(self, nbytes: int, device="cuda"):
        self.nbytes = max(256, int(nbytes))
        self.tensor = torch.empty(self.nbytes, dtype=torch.uint8, device=device)
        fluxbin.workspace_init(self.tensor.data_ptr(), self.nbytes, _stream_ptr())


class FluxBinLinear:
    """y = x @ What^T for a packed layer held in a torch uint8 CUDA tensor."""

    def __init__(self, L, device="cuda", packed: np.ndarray | None = None, fp16_tables: bool = False):
        """Pack canonical layer `L` (synth.Linear-like) into device memory.  If `packed` (the result
        of fluxbin.pack_host) is given it is uploaded as is and a handle attached.  `fp16_tables`: batched
        calls (B >= 2) keep their lookup tables in fp16 (twice the batched throughput, about 3e-4 relative
        error; see fluxbin_set_table_format)."""
        self.device = torch.device(device)
        if packed is None:
            nbytes = fluxbin.packed_size(L)
            self.buffer = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self.weight = fluxbin.pack(L, self.buffer.data_ptr(), nbytes, _stream_ptr(), buffer=self.buffer)
        else:
            self.buffer = torch.from_numpy(packed).to(self.device)
            self.weight = fluxbin.attach(packed[:256], self.buffer.data_ptr(), packed.size, buffer=self.buffer)
        self.M, self.N = self.weight.M, self.weight.N
        if fp16_tables:
            self.weight.set_table_format(fluxbin.TABLES_FP16)
        self.packed_bytes = int(self.buffer.numel())

    def clone(self) -> "FluxBinLinear":
        """The same packed layer in a device buffer of its own (a device-to-device copy plus fluxbin_attach)."""
        c = object.__new__(FluxBinLinear)
        c.device = self.device
        c.buffer = self.buffer.clone()
        header = self.buffer[:256].cpu().numpy()
        c.weight = fluxbin.attach(header, c.buffer.data_ptr(), int(c.buffer.numel()), buffer=c.buffer)
        c.weight.set_table_format(self.weight.table_format())
        c.M, c.N, c.packed_bytes = self.M, self.N, self.packed_bytes
        return c

    def workspace(self, B: int) -> Workspace:
        return Workspace(self.weight.workspace_size(B), self.device)

    def forward(self, x: torch.Tensor, ws: Workspace, out: torch.Tensor | None = None, fp32_out: bool = False,
                stream=None) -> torch.Tensor:
        """x: fp16 [B][>=N] (row stride = x.stride(0)); returns y [B][M] (fp16, or fp32 if fp32_out)."""
        assert x.dtype == torch.float16 and x.is_cuda and x.dim() == 2 and x.stride(1) == 1
        B = x.shape[0]
        if out is None:
            out = torch.empty((B, self.M), dtype=torch.float32 if fp32_out else torch.float16, device=x.device)
        fluxbin.linear(self.weight, x.data_ptr(), B, x.stride(0), out.data_ptr(), out.dtype == torch.float32,
                       out.stride(0), ws.tensor.data_ptr(), ws.nbytes, _stream_ptr(stream))
        return out

    def unpack(self):
        return fluxbin.unpack(self.weight, _stream_ptr())


class FluxBinPlan:
    """Several independent layers run in one persistent launch (fluxbin_plan_*).

    `members` is a list of (FluxBinLinear, x, y) with x fp16 [B][>=N] and y [B][M] CUDA tensors that
    stay alive and in place for the life of the plan (the pointers are captured at creation).
    `gate_up`: list of (gate member, up member) index pairs whose outputs are combined as silu(gate) * up into the
    gate member's y (fluxbin_plan_create_gated); the y of an up member may be None."""

    def __init__(self, members, device="cuda", gate_up=None):
        self.members = list(members)
        lins = [m[0] for m in self.members]
        xs = [m[1] for m in self.members]
        ys = [m[2] for m in self.members]
        B = xs[0].shape[0]
        assert all(x.shape[0] == B and x.dtype == torch.float16 and x.stride(1) == 1 for x in xs)
        first_y = next(y for y in ys if y is not None)
        fp32 = first_y.dtype == torch.float32
        assert all(y is None or ((y.dtype == torch.float32) == fp32 and y.shape[0] == B) for y in ys)
        weights = [l.weight for l in lins]
        tbytes = fluxbin.plan_table_bytes(len(lins), B)
        self.table = torch.empty(max(tbytes, 16), dtype=torch.uint8, device=device)
        self.ws = Workspace(fluxbin.plan_workspace_bytes(weights, B), device)
        self.plan = fluxbin.plan_create(weights, [x.data_ptr() for x in xs], [x.stride(0) for x in xs],
                                        [None if y is None else y.data_ptr() for y in ys],
                                        [0 if y is None else y.stride(0) for y in ys], B, fp32,
                                        self.table.data_ptr(), tbytes, self.ws.tensor.data_ptr(), self.ws.nbytes,
                                        _stream_ptr(), keep=(self.members, self.table, self.ws), gate_up=gate_up)
        self.B = B

    def run(self, stream=None):
        self.plan.run(_stream_ptr(stream))

    def num_launches(self) -> int:
        return self.plan.num_launches()

    def pairs_per_row_block(self) -> int:
        return self.plan.pairs_per_row_block()


def rc_decompose(W: torch.Tensor, g: int, K: int, T: int, eps: float = 1e-8, stream=None, col_live: torch.Tensor | None = None):
    """fluxbin_rc_decomp on a CUDA fp32 matrix W [M][N] (last dimension contiguous).  Returns a dict of CUDA tensors:
    bits uint32-as-int32 [K][M][N/32], row_scale / col_scale fp16 [K][M][N/g] / [K][N] (the canonical layout of a
    layer description) and their fp32 originals row_scale_f32 / col_scale_f32."""
    assert W.is_cuda and W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    M, N = W.shape
    dev = W.device
    out = {"bits": torch.empty((K, M, N // 32), dtype=torch.int32, device=dev),
           "row_scale": torch.empty((K, M, N // g), dtype=torch.float16, device=dev),
           "col_scale": torch.empty((K, N), dtype=torch.float16, device=dev),
           "row_scale_f32": torch.empty((K, M, N // g), dtype=torch.float32, device=dev),
           "col_scale_f32": torch.empty((K, N), dtype=torch.float32, device=dev)}
    ws = Workspace(max(fluxbin.rc_decomp_workspace_size(M, N, g, K), 256), device=dev)
    fluxbin.rc_decomp(W.data_ptr(), W.stride(0), M, N, g, K, T, eps, out["bits"].data_ptr(), out["row_scale"].data_ptr(),
                      out["col_scale"].data_ptr(), out["row_scale_f32"].data_ptr(), out["col_scale_f32"].data_ptr(),
                      ws.tensor.data_ptr(), ws.tensor.numel() * ws.tensor.element_size(), _stream_ptr(stream),
                      d_col_live=None if col_live is None else col_live.data_ptr())
    out["_workspace"] = ws
    return out


def _pad_width(s_max: int) -> int:
    for w in (32, 64, 128, 256):
        if s_max <= w:
            return w
    raise ValueError("more than 256 salient columns in one row-scale group")


def hybrid_decompose(W: torch.Tensor, g: int, Kb: int, Ks: int, sal_idx, T: int, eps: float = 1e-8):
    """Global bases plus a refinement on given salient columns (Algorithm 2 without the saliency search and the
    Hessian compensation): fluxbin_rc_decomp on W, then on the residual of every group's salient columns, each
    group's block padded with zero columns to a common width (the padding marked in the live mask), then
    fluxbin_rc_salient_collect.  Only index arithmetic for the padded layout happens here; the decompositions, the
    residual, the gathers of the result and every rounding run in the library.
    Returns a dict of CUDA tensors in the canonical layout of a layer description (sal_idx also as a host array)."""
    assert W.is_cuda and W.dtype == torch.float32
    W = W.contiguous()
    M, N = W.shape
    dev = W.device
    out = rc_decompose(W, g, Kb, T, eps)
    sal_host = np.ascontiguousarray(np.asarray(sal_idx, np.int32))
    n_sal = int(sal_host.size)
    res = {"bits": out["bits"], "row_scale": out["row_scale"], "col_scale": out["col_scale"],
           "row_scale_f32": out["row_scale_f32"], "col_scale_f32": out["col_scale_f32"], "sal_idx_host": sal_host}
    if Ks == 0 or n_sal == 0:
        return res
    # one padded block per group that has salient columns (index arithmetic for the layout only, on the host)
    grp = sal_host // g
    groups, first, counts = np.unique(grp, return_index=True, return_counts=True)
    width = _pad_width(int(counts.max()))
    slot = np.repeat(np.arange(len(groups)), counts)                        # block of each virtual column
    pos = (slot * width + (np.arange(n_sal) - first[slot])).astype(np.int32)  # its column in the padded matrix
    nblocks = len(groups)
    ncols_p = nblocks * width
    idx32 = torch.from_numpy(sal_host).to(dev)
    pos32 = torch.from_numpy(pos).to(dev)
    block_group = torch.from_numpy(groups.astype(np.int32)).to(dev)
    P = torch.empty((M, ncols_p), dtype=torch.float32, device=dev)
    live = torch.empty(ncols_p, dtype=torch.float32, device=dev)
    # the residual of the global part on the salient columns, written into the padded layout by the library
    fluxbin.rc_salient_residual(W.data_ptr(), W.stride(0), M, N, g, Kb, out["bits"].data_ptr(), out["row_scale_f32"].data_ptr(),
                                out["col_scale_f32"].data_ptr(), idx32.data_ptr(), pos32.data_ptr(), n_sal, P.data_ptr(),
                                P.stride(0), ncols_p, live.data_ptr(), _stream_ptr())
    so = rc_decompose(P, width, Ks, T, eps, col_live=live)
    # back to the canonical salient arrays, on the device
    res["sal_idx"] = idx32
    res["sal_bits"] = torch.empty((Ks, M, (n_sal + 31) // 32), dtype=torch.int32, device=dev)
    res["sal_row_scale"] = torch.empty((Ks, M, N // g), dtype=torch.float16, device=dev)
    res["sal_col_scale"] = torch.empty((Ks, n_sal), dtype=torch.float16, device=dev)
    res["sal_row_scale_f32"] = torch.empty((Ks, M, N // g), dtype=torch.float32, device=dev)
    res["sal_col_scale_f32"] = torch.empty((Ks, n_sal), dtype=torch.float32, device=dev)
    fluxbin.rc_salient_collect(so["bits"].data_ptr(), so["row_scale_f32"].data_ptr(), so["col_scale_f32"].data_ptr(),
                               pos32.data_ptr(), block_group.data_ptr(), M, N, g, Ks, n_sal, width, nblocks,
                               res["sal_bits"].data_ptr(), res["sal_row_scale"].data_ptr(), res["sal_col_scale"].data_ptr(),
                               res["sal_row_scale_f32"].data_ptr(), res["sal_col_scale_f32"].data_ptr(), _stream_ptr())
    res["_keep"] = (so, P, live, pos32, block_group)
    return res


def pack_device(r: dict, M: int, N: int, g: int, Kb: int, Ks: int) -> "FluxBinLinear":
    """fluxbin_pack_device on the device-resident canonical arrays of hybrid_decompose: a packed layer without the
    arrays crossing host memory."""
    dev = r["bits"].device
    sal_host = r.get("sal_idx_host", np.zeros(0, np.int32))
    has_sal = Ks > 0 and sal_host.size > 0 and "sal_bits" in r
    if not has_sal:
        Ks, sal_host = 0, np.zeros(0, np.int32)
    n_sal = int(sal_host.size)
    nbytes = fluxbin.packed_size_of(M, N, Kb, Ks, g, sal_host)
    lin = object.__new__(FluxBinLinear)
    lin.device = torch.device(dev)
    lin.buffer = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    ws = torch.empty(max(fluxbin.pack_device_workspace_size(N, g, n_sal), 256), dtype=torch.uint8, device=dev)
    ptrs = [r["bits"].data_ptr(), r["row_scale"].data_ptr(), r["col_scale"].data_ptr()]
    ptrs += [r[k].data_ptr() for k in ("sal_idx", "sal_bits", "sal_row_scale", "sal_col_scale")] if has_sal else [None] * 4
    lin.weight = fluxbin.pack_device((M, N, Kb, Ks, g, n_sal), ptrs, sal_host, lin.buffer.data_ptr(), nbytes, ws.data_ptr(),
                                     int(ws.numel()), _stream_ptr(), buffer=lin.buffer)
    lin.M, lin.N, lin.packed_bytes = M, N, nbytes
    return lin


def quantize_dense(W: torch.Tensor, g: int = 128, K: int = 2, T: int = 10, eps: float = 1e-8, sal_idx=None,
                   Ks: int = 0) -> "FluxBinLinear":
    """Dense fp32 CUDA matrix -> packed FluxBin layer: K global bases and, if `sal_idx` (ascending column indices)
    and Ks > 0 are given, Ks further bases on those columns.  Decomposition, collection of the salient arrays and
    packing all run on the GPU (fluxbin_rc_decomp, fluxbin_rc_salient_collect, fluxbin_pack_device); only the salient
    map itself is host data."""
    M, N = W.shape
    r = hybrid_decompose(W, g, K, Ks if sal_idx is not None else 0, [] if sal_idx is None else sal_idx, T, eps)
    return pack_device(r, M, N, g, K, Ks if sal_idx is not None else 0)

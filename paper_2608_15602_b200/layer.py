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

    def __init__(self, L, device="cuda", packed: np.ndarray | None = None):
        """Pack canonical layer `L` (synth.Linear-like) into device memory.  If `packed` (the result
        of fluxbin.pack_host) is given it is uploaded as is and a handle attached."""
        self.device = torch.device(device)
        if packed is None:
            nbytes = fluxbin.packed_size(L)
            self.buffer = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            self.weight = fluxbin.pack(L, self.buffer.data_ptr(), nbytes, _stream_ptr(), buffer=self.buffer)
        else:
            self.buffer = torch.from_numpy(packed).to(self.device)
            self.weight = fluxbin.attach(packed[:256], self.buffer.data_ptr(), packed.size, buffer=self.buffer)
        self.M, self.N = self.weight.M, self.weight.N
        self.packed_bytes = int(self.buffer.numel())

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
    stay alive and in place for the life of the plan (the pointers are captured at creation)."""

    def __init__(self, members, device="cuda"):
        self.members = list(members)
        lins = [m[0] for m in self.members]
        xs = [m[1] for m in self.members]
        ys = [m[2] for m in self.members]
        B = xs[0].shape[0]
        assert all(x.shape[0] == B and x.dtype == torch.float16 and x.stride(1) == 1 for x in xs)
        fp32 = ys[0].dtype == torch.float32
        assert all((y.dtype == torch.float32) == fp32 and y.shape[0] == B for y in ys)
        weights = [l.weight for l in lins]
        tbytes = fluxbin.plan_table_bytes(len(lins), B)
        self.table = torch.empty(max(tbytes, 16), dtype=torch.uint8, device=device)
        self.ws = Workspace(fluxbin.plan_workspace_bytes(weights, B), device)
        self.plan = fluxbin.plan_create(weights, [x.data_ptr() for x in xs], [x.stride(0) for x in xs],
                                        [y.data_ptr() for y in ys], [y.stride(0) for y in ys], B, fp32,
                                        self.table.data_ptr(), tbytes, self.ws.tensor.data_ptr(), self.ws.nbytes,
                                        _stream_ptr(), keep=(self.members, self.table, self.ws))
        self.B = B

    def run(self, stream=None):
        self.plan.run(_stream_ptr(stream))

    def num_launches(self) -> int:
        return self.plan.num_launches()

    def pairs_per_row_block(self) -> int:
        return self.plan.pairs_per_row_block()


def rc_decompose(W: torch.Tensor, g: int, K: int, T: int, eps: float = 1e-8, stream=None):
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
                      ws.tensor.data_ptr(), ws.tensor.numel() * ws.tensor.element_size(), _stream_ptr(stream))
    out["_workspace"] = ws
    return out


def quantize_dense(W: torch.Tensor, g: int = 128, K: int = 2, T: int = 10, eps: float = 1e-8) -> "FluxBinLinear":
    """Dense fp32 CUDA matrix -> packed FluxBin layer with K global bases and no salient refinement: the GPU
    decomposition (fluxbin_rc_decomp), then the packer.  The canonical arrays pass through host memory because
    fluxbin_pack takes host pointers."""
    from . import synth
    M, N = W.shape
    out = rc_decompose(W.contiguous(), g, K, T, eps)
    torch.cuda.synchronize(W.device)
    L = synth.Linear(M, N, K, 0, g, 0,
                     np.ascontiguousarray(out["bits"].cpu().numpy().view(np.uint32)),
                     np.ascontiguousarray(out["row_scale"].cpu().numpy().view(np.uint16)),
                     np.ascontiguousarray(out["col_scale"].cpu().numpy().view(np.uint16)),
                     np.zeros(0, np.int32), np.zeros((0, M, 0), np.uint32), np.zeros((0, M, N // g), np.uint16),
                     np.zeros((0, 0), np.uint16))
    return FluxBinLinear(L, device=W.device)

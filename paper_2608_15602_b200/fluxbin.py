"""ctypes binding of the FluxBin C-ABI (include/fluxbin.h).  Argument marshalling only.

Every step of the layer runs in the CUDA library; there is no Python or CPU fallback.  The
library must have been built (python -m paper_2608_15602_b200.build); loading fails loudly
otherwise.  Device buffers are passed as integer addresses (e.g. torch.Tensor.data_ptr()).
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from .build import LIB_PATH

STATUS_OK = 0


class FluxBinError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().fluxbin_status_string(status).decode()
        extra = f" (cudaError {_lib().fluxbin_last_cuda_error()})" if status == 8 else ""
        super().__init__(f"{where}: {msg}{extra}")


class LayerDesc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int32), ("N", ctypes.c_int32), ("Kb", ctypes.c_int32), ("Ks", ctypes.c_int32),
                ("g", ctypes.c_int32), ("n_sal", ctypes.c_int32),
                ("bits", ctypes.c_void_p), ("row_scale", ctypes.c_void_p), ("col_scale", ctypes.c_void_p),
                ("sal_idx", ctypes.c_void_p), ("sal_bits", ctypes.c_void_p), ("sal_row_scale", ctypes.c_void_p),
                ("sal_col_scale", ctypes.c_void_p)]


EXPORTS = ["fluxbin_packed_size", "fluxbin_validate", "fluxbin_pack_host", "fluxbin_unpack_host",
           "fluxbin_packed_dims", "fluxbin_pack", "fluxbin_attach", "fluxbin_unpack", "fluxbin_weight_dims",
           "fluxbin_weight_device", "fluxbin_debug_cut_shares",
           "fluxbin_workspace_size", "fluxbin_workspace_init", "fluxbin_linear", "fluxbin_debug_tables",
           "fluxbin_num_table_sets", "fluxbin_num_launches", "fluxbin_free", "fluxbin_status_string",
           "fluxbin_last_cuda_error", "fluxbin_plan_table_bytes", "fluxbin_plan_workspace_bytes",
           "fluxbin_plan_create", "fluxbin_plan_create_gated", "fluxbin_plan_run", "fluxbin_plan_num_launches", "fluxbin_plan_pairs_per_row_block",
           "fluxbin_plan_free",
           "fluxbin_linear_noalloc", "fluxbin_noalloc_capacity", "fluxbin_set_table_format", "fluxbin_get_table_format",
           "fluxbin_rc_decomp", "fluxbin_rc_decomp_workspace_size", "fluxbin_rc_decomp_passes",
           "fluxbin_rc_salient_collect", "fluxbin_pack_device", "fluxbin_pack_device_workspace_size", "fluxbin_rc_salient_residual"]

_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_15602_b200.build` "
                              "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, sz, i32, i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32, ctypes.c_int64
        dp = ctypes.POINTER(LayerDesc)
        lib.fluxbin_packed_size.restype, lib.fluxbin_packed_size.argtypes = sz, [dp]
        lib.fluxbin_validate.restype, lib.fluxbin_validate.argtypes = ctypes.c_int, [dp]
        lib.fluxbin_pack_host.restype, lib.fluxbin_pack_host.argtypes = ctypes.c_int, [dp, vp, sz]
        lib.fluxbin_unpack_host.restype, lib.fluxbin_unpack_host.argtypes = ctypes.c_int, [vp, sz, dp]
        lib.fluxbin_packed_dims.restype, lib.fluxbin_packed_dims.argtypes = ctypes.c_int, [vp, sz, dp]
        lib.fluxbin_pack.restype, lib.fluxbin_pack.argtypes = ctypes.c_int, [dp, vp, sz, vp, ctypes.POINTER(vp)]
        lib.fluxbin_attach.restype, lib.fluxbin_attach.argtypes = ctypes.c_int, [vp, sz, vp, sz, ctypes.POINTER(vp)]
        lib.fluxbin_unpack.restype, lib.fluxbin_unpack.argtypes = ctypes.c_int, [vp, dp, vp]
        lib.fluxbin_weight_dims.restype, lib.fluxbin_weight_dims.argtypes = ctypes.c_int, [vp, dp]
        lib.fluxbin_weight_device.restype, lib.fluxbin_weight_device.argtypes = i32, [vp]
        lib.fluxbin_workspace_size.restype, lib.fluxbin_workspace_size.argtypes = sz, [vp, i32]
        lib.fluxbin_workspace_init.restype, lib.fluxbin_workspace_init.argtypes = ctypes.c_int, [vp, sz, vp]
        lib.fluxbin_linear.restype = ctypes.c_int
        lib.fluxbin_linear.argtypes = [vp, vp, i32, i64, vp, i32, i64, vp, sz, vp]
        lib.fluxbin_debug_tables.restype = ctypes.c_int
        lib.fluxbin_debug_tables.argtypes = [vp, vp, i32, vp, vp, vp, vp]
        lib.fluxbin_debug_cut_shares.restype = ctypes.c_int
        lib.fluxbin_debug_cut_shares.argtypes = [i32, ctypes.POINTER(vp), i32, i32, i32, i32, i32, vp, vp]
        lib.fluxbin_num_table_sets.restype, lib.fluxbin_num_table_sets.argtypes = i32, [vp]
        lib.fluxbin_num_launches.restype, lib.fluxbin_num_launches.argtypes = i32, [vp, i32]
        lib.fluxbin_set_table_format.restype, lib.fluxbin_set_table_format.argtypes = ctypes.c_int, [vp, i32]
        lib.fluxbin_get_table_format.restype, lib.fluxbin_get_table_format.argtypes = i32, [vp]
        lib.fluxbin_free.restype, lib.fluxbin_free.argtypes = None, [vp]
        lib.fluxbin_status_string.restype, lib.fluxbin_status_string.argtypes = ctypes.c_char_p, [ctypes.c_int]
        lib.fluxbin_last_cuda_error.restype, lib.fluxbin_last_cuda_error.argtypes = ctypes.c_int, []
        lib.fluxbin_plan_table_bytes.restype, lib.fluxbin_plan_table_bytes.argtypes = sz, [i32, i32]
        lib.fluxbin_plan_workspace_bytes.restype = sz
        lib.fluxbin_plan_workspace_bytes.argtypes = [i32, ctypes.POINTER(vp), i32]
        lib.fluxbin_plan_create.restype = ctypes.c_int
        lib.fluxbin_plan_create.argtypes = [i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(i64),
                                            ctypes.POINTER(vp), ctypes.POINTER(i64), i32, i32, vp, sz, vp, sz, vp,
                                            ctypes.POINTER(vp)]
        lib.fluxbin_plan_create_gated.restype = ctypes.c_int
        lib.fluxbin_plan_create_gated.argtypes = [i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(i64),
                                                  ctypes.POINTER(vp), ctypes.POINTER(i64), ctypes.POINTER(i32), i32, i32, i32, vp, sz,
                                                  vp, sz, vp, ctypes.POINTER(vp)]
        lib.fluxbin_plan_run.restype, lib.fluxbin_plan_run.argtypes = ctypes.c_int, [vp, vp]
        lib.fluxbin_plan_num_launches.restype, lib.fluxbin_plan_num_launches.argtypes = i32, [vp]
        lib.fluxbin_plan_pairs_per_row_block.restype, lib.fluxbin_plan_pairs_per_row_block.argtypes = i32, [vp]
        lib.fluxbin_plan_free.restype, lib.fluxbin_plan_free.argtypes = None, [vp]
        lib.fluxbin_linear_noalloc.restype = ctypes.c_int
        lib.fluxbin_linear_noalloc.argtypes = [vp, vp, i32, i64, vp, i32, i64, vp]
        lib.fluxbin_noalloc_capacity.restype, lib.fluxbin_noalloc_capacity.argtypes = sz, []
        lib.fluxbin_rc_decomp_workspace_size.restype = sz
        lib.fluxbin_rc_decomp_workspace_size.argtypes = [i32, i32, i32, i32]
        lib.fluxbin_rc_decomp_passes.restype, lib.fluxbin_rc_decomp_passes.argtypes = i32, [i32, i32]
        lib.fluxbin_rc_decomp.restype = ctypes.c_int
        lib.fluxbin_rc_decomp.argtypes = [vp, i64, vp, i32, i32, i32, i32, i32, ctypes.c_float, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.fluxbin_rc_salient_residual.restype = ctypes.c_int
        lib.fluxbin_rc_salient_residual.argtypes = [vp, i64, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, vp, i64, i32, vp, vp]
        lib.fluxbin_rc_salient_collect.restype = ctypes.c_int
        lib.fluxbin_rc_salient_collect.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        lib.fluxbin_pack_device_workspace_size.restype, lib.fluxbin_pack_device_workspace_size.argtypes = sz, [i32, i32, i32]
        lib.fluxbin_pack_device.restype = ctypes.c_int
        lib.fluxbin_pack_device.argtypes = [dp, vp, vp, sz, vp, sz, vp, ctypes.POINTER(vp)]
        _LIB = lib
    return _LIB


def library():
    """The loaded ctypes library (for symbol checks)."""
    return _lib()


def _check(status: int, where: str):
    if status != STATUS_OK:
        raise FluxBinError(status, where)


def _ptr(a):
    return None if a is None or a.size == 0 else a.ctypes.data


def make_desc(L) -> LayerDesc:
    """LayerDesc borrowing the numpy arrays of a canonical layer object (keep `L` alive)."""
    return LayerDesc(L.M, L.N, L.Kb, L.Ks, L.g, L.n_sal, _ptr(L.bits), _ptr(L.row_scale), _ptr(L.col_scale),
                     _ptr(L.sal_idx), _ptr(L.sal_bits), _ptr(L.sal_row_scale), _ptr(L.sal_col_scale))


def status_string(status: int) -> str:
    return _lib().fluxbin_status_string(status).decode()


def validate(L) -> int:
    d = make_desc(L)
    return int(_lib().fluxbin_validate(ctypes.byref(d)))


def packed_size(L, with_map: bool = True) -> int:
    d = make_desc(L)
    if not with_map:
        d.sal_idx = None
    return int(_lib().fluxbin_packed_size(ctypes.byref(d)))


def pack_host(L) -> np.ndarray:
    """Packed layer as a uint8 numpy array (host)."""
    n = packed_size(L)
    if n == 0:
        _check(validate(L) or 2, "fluxbin_packed_size")
    buf = np.empty(n, np.uint8)
    d = make_desc(L)
    _check(_lib().fluxbin_pack_host(ctypes.byref(d), buf.ctypes.data, n), "fluxbin_pack_host")
    return buf


def _empty_canonical(M, N, Kb, Ks, g, n_sal):
    from types import SimpleNamespace
    ng, nws = N // g, (n_sal + 31) // 32
    return SimpleNamespace(
        M=M, N=N, Kb=Kb, Ks=Ks, g=g, n_sal=n_sal,
        bits=np.zeros((Kb, M, N // 32), np.uint32), row_scale=np.zeros((Kb, M, ng), np.uint16),
        col_scale=np.zeros((Kb, N), np.uint16), sal_idx=np.zeros(n_sal, np.int32),
        sal_bits=np.zeros((Ks, M, nws), np.uint32), sal_row_scale=np.zeros((Ks, M, ng), np.uint16),
        sal_col_scale=np.zeros((Ks, n_sal), np.uint16))


def unpack_host(buf: np.ndarray):
    """Inverse of pack_host: a namespace with the canonical arrays."""
    d = LayerDesc()
    _check(_lib().fluxbin_packed_dims(buf.ctypes.data, buf.size, ctypes.byref(d)), "fluxbin_packed_dims")
    out = _empty_canonical(d.M, d.N, d.Kb, d.Ks, d.g, d.n_sal)
    dd = make_desc(out)
    _check(_lib().fluxbin_unpack_host(buf.ctypes.data, buf.size, ctypes.byref(dd)), "fluxbin_unpack_host")
    return out


TABLES_FP32, TABLES_FP16, TABLES_FP32_MU4 = 0, 1, 2


class Weight:
    """A packed layer resident in device memory (the caller's buffer) plus its handle."""

    def __init__(self, handle: int, dims, buffer=None):
        self.handle = handle
        self.M, self.N, self.Kb, self.Ks, self.g, self.n_sal = dims
        self.buffer = buffer          # keeps the caller's device tensor alive, if given

    def close(self):
        if self.handle:
            _lib().fluxbin_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_size(self, B: int) -> int:
        return int(_lib().fluxbin_workspace_size(self.handle, B))

    def device(self) -> int:
        return int(_lib().fluxbin_weight_device(self.handle))

    def num_table_sets(self) -> int:
        return int(_lib().fluxbin_num_table_sets(self.handle))

    def num_launches(self, B: int) -> int:
        return int(_lib().fluxbin_num_launches(self.handle, B))

    def set_table_format(self, fmt: int) -> None:
        """TABLES_FP32 (default) or TABLES_FP16 entries for batched launches, or TABLES_FP32_MU4 (16-entry tables of
        sub-vectors of four columns, every launch); size workspaces afterwards."""
        _check(_lib().fluxbin_set_table_format(self.handle, fmt), "fluxbin_set_table_format")

    def table_format(self) -> int:
        return int(_lib().fluxbin_get_table_format(self.handle))


def pack(L, d_packed: int, d_bytes: int, stream: int = 0, buffer=None) -> Weight:
    """fluxbin_pack: pack canonical layer L into the device buffer at address d_packed."""
    d = make_desc(L)
    h = ctypes.c_void_p()
    _check(_lib().fluxbin_pack(ctypes.byref(d), d_packed, d_bytes, stream, ctypes.byref(h)), "fluxbin_pack")
    return Weight(h.value, (L.M, L.N, L.Kb, L.Ks if L.n_sal else 0, L.g, L.n_sal if L.Ks else 0), buffer)


def attach(header: np.ndarray, d_packed: int, d_bytes: int, buffer=None) -> Weight:
    h = ctypes.c_void_p()
    _check(_lib().fluxbin_attach(header.ctypes.data, header.size, d_packed, d_bytes, ctypes.byref(h)), "fluxbin_attach")
    d = LayerDesc()
    _check(_lib().fluxbin_weight_dims(h.value, ctypes.byref(d)), "fluxbin_weight_dims")
    return Weight(h.value, (d.M, d.N, d.Kb, d.Ks, d.g, d.n_sal), buffer)


def unpack(w: Weight, stream: int = 0):
    out = _empty_canonical(w.M, w.N, w.Kb, w.Ks, w.g, w.n_sal)
    dd = make_desc(out)
    _check(_lib().fluxbin_unpack(w.handle, ctypes.byref(dd), stream), "fluxbin_unpack")
    return out


def workspace_init(d_ws: int, nbytes: int, stream: int = 0):
    _check(_lib().fluxbin_workspace_init(d_ws, nbytes, stream), "fluxbin_workspace_init")


def linear(w: Weight, d_x: int, B: int, ldx: int, d_y: int, y_is_fp32: bool, ldy: int, d_ws: int, ws_bytes: int,
           stream: int = 0):
    """fluxbin_linear: y[B][ldy] = x[B][ldx] * What^T on `stream` (asynchronous)."""
    _check(_lib().fluxbin_linear(w.handle, d_x, B, ldx, d_y, 1 if y_is_fp32 else 0, ldy, d_ws, ws_bytes, stream),
           "fluxbin_linear")


def linear_status(w: Weight, d_x, B, ldx, d_y, y_is_fp32, ldy, d_ws, ws_bytes, stream=0) -> int:
    """Same call, returning the raw status (for argument-validation tests)."""
    return int(_lib().fluxbin_linear(w.handle if w else None, d_x, B, ldx, d_y, 1 if y_is_fp32 else 0, ldy, d_ws,
                                     ws_bytes, stream))


def linear_noalloc_status(w: Weight, d_x: int, B: int, ldx: int, d_y: int, y_is_fp32: bool, ldy: int, stream: int = 0) -> int:
    """fluxbin_linear_noalloc (no workspace argument: the scratch is a fixed array inside the library)."""
    return int(_lib().fluxbin_linear_noalloc(w.handle if w else None, d_x, B, ldx, d_y, 1 if y_is_fp32 else 0, ldy, stream))


def linear_noalloc(w: Weight, d_x: int, B: int, ldx: int, d_y: int, y_is_fp32: bool, ldy: int, stream: int = 0):
    _check(linear_noalloc_status(w, d_x, B, ldx, d_y, y_is_fp32, ldy, stream), "fluxbin_linear_noalloc")


def noalloc_capacity() -> int:
    return int(_lib().fluxbin_noalloc_capacity())


def rc_decomp_workspace_size(M: int, N: int, g: int, K: int) -> int:
    return int(_lib().fluxbin_rc_decomp_workspace_size(M, N, g, K))


def rc_decomp_passes(K: int, T: int) -> int:
    return int(_lib().fluxbin_rc_decomp_passes(K, T))


def rc_decomp_status(d_W, ldw, M, N, g, K, T, eps, d_bits, d_row_scale, d_col_scale, d_row_f32, d_col_f32, d_ws, ws_bytes,
                     stream=0, d_col_live=None) -> int:
    """fluxbin_rc_decomp (argument marshalling only; every pointer is a device address or None)."""
    return int(_lib().fluxbin_rc_decomp(d_W, ldw, d_col_live, M, N, g, K, T, eps, d_bits, d_row_scale, d_col_scale,
                                        d_row_f32, d_col_f32, d_ws, ws_bytes, stream))


def rc_salient_residual(d_W, ldw, M, N, g, Kb, d_bits, d_row_f32, d_col_f32, d_sal_idx, d_pos, n_sal, d_P, ldp, ncols_p,
                        d_live, stream=0):
    _check(int(_lib().fluxbin_rc_salient_residual(d_W, ldw, M, N, g, Kb, d_bits, d_row_f32, d_col_f32, d_sal_idx, d_pos,
                                                  n_sal, d_P, ldp, ncols_p, d_live, stream)), "fluxbin_rc_salient_residual")


def rc_salient_collect(d_bits_p, d_row_f32_p, d_col_f32_p, d_pos, d_block_group, M, N, g, Ks, n_sal, width, nblocks, d_sal_bits,
                       d_sal_row_scale, d_sal_col_scale, d_sal_row_f32=None, d_sal_col_f32=None, stream=0):
    _check(int(_lib().fluxbin_rc_salient_collect(d_bits_p, d_row_f32_p, d_col_f32_p, d_pos, d_block_group, M, N, g, Ks, n_sal,
                                                 width, nblocks, d_sal_bits, d_sal_row_scale, d_sal_col_scale, d_sal_row_f32,
                                                 d_sal_col_f32, stream)), "fluxbin_rc_salient_collect")


def pack_device_workspace_size(N: int, g: int, n_sal: int) -> int:
    return int(_lib().fluxbin_pack_device_workspace_size(N, g, n_sal))


def packed_size_of(M, N, Kb, Ks, g, sal_idx: np.ndarray) -> int:
    """fluxbin_packed_size from the dimensions and the (host) salient map alone."""
    d = LayerDesc(M, N, Kb, Ks, g, int(sal_idx.size), None, None, None, _ptr(sal_idx), None, None, None)
    return int(_lib().fluxbin_packed_size(ctypes.byref(d)))


def pack_device_status(dims, dev_ptrs, h_sal_idx: np.ndarray, d_packed: int, d_bytes: int, d_ws: int, ws_bytes: int, stream: int = 0):
    """fluxbin_pack_device returning (status, handle).  dims = (M, N, Kb, Ks, g, n_sal); dev_ptrs = device addresses of
    bits, row_scale, col_scale, sal_idx, sal_bits, sal_row_scale, sal_col_scale (None where absent)."""
    d = LayerDesc(*dims, *dev_ptrs)
    h = ctypes.c_void_p()
    st = _lib().fluxbin_pack_device(ctypes.byref(d), _ptr(h_sal_idx), d_packed, d_bytes, d_ws, ws_bytes, stream, ctypes.byref(h))
    return int(st), h.value


def pack_device(dims, dev_ptrs, h_sal_idx, d_packed, d_bytes, d_ws, ws_bytes, stream=0, buffer=None) -> Weight:
    st, h = pack_device_status(dims, dev_ptrs, h_sal_idx, d_packed, d_bytes, d_ws, ws_bytes, stream)
    _check(st, "fluxbin_pack_device")
    M, N, Kb, Ks, g, n_sal = dims
    return Weight(h, (M, N, Kb, Ks if n_sal else 0, g, n_sal if Ks else 0), buffer)


def rc_decomp(*args, **kw):
    _check(rc_decomp_status(*args, **kw), "fluxbin_rc_decomp")


def debug_tables(w: Weight, d_x: int, pair: int, d_tables: int, stream: int = 0):
    cols = np.zeros(256, np.int32)
    alpha = np.zeros(256, np.uint16)
    _check(_lib().fluxbin_debug_tables(w.handle, d_x, pair, d_tables, cols.ctypes.data, alpha.ctypes.data, stream),
           "fluxbin_debug_tables")
    return cols, alpha


def debug_cut_shares(headers, mode: int, pairs_per_row_block: int, grid: int, nshares: int, static_percent: int = 100):
    """fluxbin_debug_cut_shares: (cuts int32 [nshares + 1][2], work items per layer) for packed-layer headers
    (uint8 arrays of at least 256 bytes each).  Host only."""
    n = len(headers)
    cuts = np.zeros((nshares + 1, 2), np.int32)
    items = np.zeros(n, np.int32)
    hp = _arr(ctypes.c_void_p, [h.ctypes.data for h in headers])
    _check(_lib().fluxbin_debug_cut_shares(n, hp, mode, pairs_per_row_block, grid, nshares, static_percent,
                                           cuts.ctypes.data, items.ctypes.data), "fluxbin_debug_cut_shares")
    return cuts, items


class Plan:
    """Handle of fluxbin_plan_create: n layers, each with its own x and y, run in one launch."""

    def __init__(self, handle: int, keep):
        self.handle = handle
        self._keep = keep            # weights and buffers the plan points into

    def run(self, stream: int = 0):
        _check(_lib().fluxbin_plan_run(self.handle, stream), "fluxbin_plan_run")

    def num_launches(self) -> int:
        return int(_lib().fluxbin_plan_num_launches(self.handle))

    def pairs_per_row_block(self) -> int:
        return int(_lib().fluxbin_plan_pairs_per_row_block(self.handle))

    def close(self):
        if self.handle:
            _lib().fluxbin_plan_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _arr(ctype, values):
    return (ctype * len(values))(*values)


def plan_table_bytes(n: int, B: int) -> int:
    return int(_lib().fluxbin_plan_table_bytes(n, B))


def plan_workspace_bytes(weights, B: int) -> int:
    hs = _arr(ctypes.c_void_p, [w.handle for w in weights])
    return int(_lib().fluxbin_plan_workspace_bytes(len(weights), hs, B))


def plan_create_status(weights, d_x, ldx, d_y, ldy, B, y_is_fp32, d_table, table_bytes, d_ws, ws_bytes, stream=0):
    """fluxbin_plan_create returning (status, handle)."""
    n = len(weights)
    h = ctypes.c_void_p()
    st = _lib().fluxbin_plan_create(n, _arr(ctypes.c_void_p, [w.handle for w in weights]),
                                    _arr(ctypes.c_void_p, list(d_x)), _arr(ctypes.c_int64, list(ldx)),
                                    _arr(ctypes.c_void_p, list(d_y)), _arr(ctypes.c_int64, list(ldy)),
                                    B, 1 if y_is_fp32 else 0, d_table, table_bytes, d_ws, ws_bytes, stream,
                                    ctypes.byref(h))
    return int(st), h.value


def plan_create_gated_status(weights, d_x, ldx, d_y, ldy, gate_up, B, y_is_fp32, d_table, table_bytes, d_ws, ws_bytes, stream=0):
    """fluxbin_plan_create_gated returning (status, handle); gate_up = list of (gate member, up member)."""
    n = len(weights)
    h = ctypes.c_void_p()
    flat = [int(v) for pair in gate_up for v in pair]
    st = _lib().fluxbin_plan_create_gated(n, _arr(ctypes.c_void_p, [w.handle for w in weights]),
                                          _arr(ctypes.c_void_p, list(d_x)), _arr(ctypes.c_int64, list(ldx)),
                                          _arr(ctypes.c_void_p, list(d_y)), _arr(ctypes.c_int64, list(ldy)),
                                          _arr(ctypes.c_int32, flat) if flat else None, len(gate_up),
                                          B, 1 if y_is_fp32 else 0, d_table, table_bytes, d_ws, ws_bytes, stream, ctypes.byref(h))
    return int(st), h.value


def plan_create(weights, d_x, ldx, d_y, ldy, B, y_is_fp32, d_table, table_bytes, d_ws, ws_bytes, stream=0, keep=None, gate_up=None):
    if gate_up:
        st, h = plan_create_gated_status(weights, d_x, ldx, d_y, ldy, gate_up, B, y_is_fp32, d_table, table_bytes, d_ws, ws_bytes, stream)
        _check(st, "fluxbin_plan_create_gated")
    else:
        st, h = plan_create_status(weights, d_x, ldx, d_y, ldy, B, y_is_fp32, d_table, table_bytes, d_ws, ws_bytes, stream)
        _check(st, "fluxbin_plan_create")
    return Plan(h, (list(weights), keep))

"""Seeded synthetic inputs for the FluxBin decode linear layer.

This module only draws random numbers and lays them out in the canonical
interchange format of the C-ABI (see include/fluxbin.h).  It contains none of
the method's arithmetic: no scale products, no table, no sum.  Both the CPU
oracle's tests and the CUDA path's tests/benchmarks draw their inputs here so
that the two sides see identical bytes.

Canonical layout (all arrays C-contiguous numpy):
  bits           uint32 [Kb][M][N/32]     bit (j % 32) of word j/32 is 1 <=> B_ij = +1
  row_scale      uint16 [Kb][M][N/g]      IEEE fp16 bit patterns
  col_scale      uint16 [Kb][N]
  sal_idx        int32  [n_sal]           strictly ascending
  sal_bits       uint32 [Ks][M][ceil(n_sal/32)]   virtual column v = bit v (pad bits are 0)
  sal_row_scale  uint16 [Ks][M][N/g]
  sal_col_scale  uint16 [Ks][n_sal]       already gathered to virtual-column order

Value distributions follow the workload statement this build is measured on:
bits i.i.d. uniform; row scales |N(0, 0.02^2)|; column scales |N(1, 0.1^2)|;
activations N(0, 1) with optional outlier channels multiplied by 20; all
rounded to fp16 (round-to-nearest-even, numpy's float16 cast).

Every tensor is regenerable on its own from (seed, linear_id, tensor name), so
a large stack can be produced one linear at a time.
"""
from __future__ import annotations

import dataclasses
import zlib

import numpy as np

BASE_SEED = 260815602

# LLaMA-2 decode linear shapes (out rows M x in columns N), with multiplicity per layer.
LLAMA2_7B = [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
             ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)]
LLAMA2_13B = [("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
              ("gate", 13824, 5120), ("up", 13824, 5120), ("down", 5120, 13824)]
LLAMA2_70B = [("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
              ("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)]
LLAMA2_70B_LAYERS = 80


@dataclasses.dataclass
class Linear:
    """One synthetic layer in canonical layout (numpy arrays, host memory)."""
    M: int
    N: int
    Kb: int
    Ks: int
    g: int
    n_sal: int
    bits: np.ndarray
    row_scale: np.ndarray
    col_scale: np.ndarray
    sal_idx: np.ndarray
    sal_bits: np.ndarray
    sal_row_scale: np.ndarray
    sal_col_scale: np.ndarray

    def nbytes(self) -> int:
        return sum(a.nbytes for a in (self.bits, self.row_scale, self.col_scale, self.sal_idx,
                                      self.sal_bits, self.sal_row_scale, self.sal_col_scale))


def _rng(seed: int, linear_id: int, tensor: str) -> np.random.Generator:
    """Counter-based stream (Philox) keyed by (seed, linear_id, tensor name)."""
    key = (np.uint64(seed) << np.uint64(20)) ^ np.uint64(linear_id & 0xFFFFF)
    ctr = zlib.crc32(tensor.encode())
    return np.random.Generator(np.random.Philox(key=int(key), counter=[0, 0, 0, ctr]))


def _random_words(rng: np.random.Generator, shape) -> np.ndarray:
    """Uniform uint32 words straight from the raw Philox stream (fast path for GBs of bits)."""
    n = int(np.prod(shape))
    raw = rng.bit_generator.random_raw((n + 1) // 2)
    return raw.view(np.uint32)[:n].reshape(shape)


def _half_bits(a: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(a.astype(np.float16)).view(np.uint16)


def _abs_normal_fp16(rng, mean: float, std: float, shape) -> np.ndarray:
    v = rng.standard_normal(size=shape, dtype=np.float32)
    v *= np.float32(std)
    v += np.float32(mean)
    np.abs(v, out=v)
    return _half_bits(v)


def salient_random(seed: int, linear_id: int, N: int, frac: float) -> np.ndarray:
    """round(frac*N) distinct columns, uniform over [0, N), ascending."""
    n_sal = int(round(frac * N))
    if n_sal <= 0:
        return np.zeros(0, np.int32)
    rng = _rng(seed, linear_id, "sal_idx")
    idx = rng.choice(N, size=n_sal, replace=False)
    return np.sort(idx).astype(np.int32)


def salient_per_group(seed: int, linear_id: int, N: int, g: int, s: int) -> np.ndarray:
    """Exactly s columns in every group of g columns (the paper's structured pattern)."""
    rng = _rng(seed, linear_id, "sal_idx_grouped")
    out = []
    for G in range(N // g):
        out.append(G * g + np.sort(rng.choice(g, size=s, replace=False)))
    return np.concatenate(out).astype(np.int32) if out else np.zeros(0, np.int32)


def make_linear(seed: int, linear_id: int, M: int, N: int, Kb: int = 2, Ks: int = 0,
                g: int = 128, sal_idx: np.ndarray | None = None) -> Linear:
    """Draw one layer.  `sal_idx` (ascending int32) selects the salient columns; Ks bases on them."""
    assert N % 32 == 0 and g % 32 == 0 and N % g == 0
    if sal_idx is None or Ks == 0:
        sal_idx = np.zeros(0, np.int32)
    sal_idx = np.ascontiguousarray(sal_idx, dtype=np.int32)
    n_sal = int(sal_idx.size)
    ng = N // g

    bits = _random_words(_rng(seed, linear_id, "bits"), (Kb, M, N // 32))
    row_scale = _abs_normal_fp16(_rng(seed, linear_id, "row_scale"), 0.0, 0.02, (Kb, M, ng))
    col_scale = _abs_normal_fp16(_rng(seed, linear_id, "col_scale"), 1.0, 0.1, (Kb, N))

    nw = (n_sal + 31) // 32
    if Ks > 0 and n_sal > 0:
        sal_bits = np.ascontiguousarray(_random_words(_rng(seed, linear_id, "sal_bits"), (Ks, M, nw)))
        tail = n_sal % 32
        if tail:
            sal_bits[:, :, -1] &= np.uint32((1 << tail) - 1)
        sal_row_scale = _abs_normal_fp16(_rng(seed, linear_id, "sal_row_scale"), 0.0, 0.02, (Ks, M, ng))
        sal_col_scale = _abs_normal_fp16(_rng(seed, linear_id, "sal_col_scale"), 1.0, 0.1, (Ks, n_sal))
    else:
        Ks = 0
        sal_bits = np.zeros((0, M, nw), np.uint32)
        sal_row_scale = np.zeros((0, M, ng), np.uint16)
        sal_col_scale = np.zeros((0, n_sal), np.uint16)
    return Linear(M, N, Kb, Ks, g, n_sal, bits, row_scale, col_scale, sal_idx,
                  sal_bits, sal_row_scale, sal_col_scale)


def make_activations(seed: int, linear_id: int, B: int, N: int, outlier_frac: float = 0.0,
                     outlier_scale: float = 20.0) -> np.ndarray:
    """fp16 bit patterns [B][N]; x ~ N(0,1); round(outlier_frac*N) channels (same for every
    batch row, drawn independently of the salient set) are multiplied by outlier_scale."""
    x = _rng(seed, linear_id, "x").standard_normal(size=(B, N), dtype=np.float32)
    n_out = int(round(outlier_frac * N))
    if n_out > 0:
        ch = _rng(seed, linear_id, "x_outliers").choice(N, size=n_out, replace=False)
        x[:, ch] *= np.float32(outlier_scale)
    return _half_bits(x)


def config_linears(config: int):
    """(name, M, N) of the linears of one layer of a workload, plus the layer count."""
    if config in (0, 1):
        return [("lin", 4096, 4096)], 1
    if config == 2:
        return LLAMA2_7B, 1
    if config == 3:
        return LLAMA2_13B, 1
    if config == 4:
        return LLAMA2_70B, LLAMA2_70B_LAYERS
    raise ValueError(config)


def make_config_linear(config: int, layer: int, li: int, g: int = 128) -> Linear:
    """Linear number `li` of layer `layer` of workload `config` (2 global bases; configs 1-4
    add one extra base on a seeded random 5 % of the input columns)."""
    lins, _ = config_linears(config)
    _, M, N = lins[li]
    seed = BASE_SEED + config
    lid = layer * 16 + li
    if config == 0:
        return make_linear(seed, lid, M, N, 2, 0, g)
    idx = salient_random(seed, lid, N, 0.05)
    return make_linear(seed, lid, M, N, 2, 1, g, idx)


def make_config_activations(config: int, layer: int, li: int, B: int) -> np.ndarray:
    lins, _ = config_linears(config)
    _, _, N = lins[li]
    seed = BASE_SEED + config
    return make_activations(seed, layer * 16 + li, B, N, 0.01 if config == 1 else 0.0)


def make_dense_weight(seed: int, matrix_id: int, M: int, N: int, outlier_col_frac: float = 0.0) -> np.ndarray:
    """A dense fp32 weight matrix for the decomposition step: entries N(0, 0.02^2) times a per-row and a per-column
    gain |N(1, 0.25^2)| (the anisotropy the row-column scales are meant to capture); a fraction of the columns
    may be multiplied by 8 (outlier columns).  Random numbers only: none of the method's arithmetic."""
    w = _rng(seed, matrix_id, "dense_w").standard_normal(size=(M, N), dtype=np.float32)
    w *= np.float32(0.02)
    w *= np.abs(_rng(seed, matrix_id, "dense_row_gain").normal(1.0, 0.25, size=(M, 1))).astype(np.float32)
    w *= np.abs(_rng(seed, matrix_id, "dense_col_gain").normal(1.0, 0.25, size=(1, N))).astype(np.float32)
    n_out = int(round(outlier_col_frac * N))
    if n_out > 0:
        cols = _rng(seed, matrix_id, "dense_outlier_cols").choice(N, size=n_out, replace=False)
        w[:, cols] *= np.float32(8.0)
    return np.ascontiguousarray(w)

"""The paper's analytic cost models, written out (test infrastructure only).

storage_bits / abw   storage model of the appendix (S_base, S_sal, S_idx, ABW)
smem_bytes           shared-memory footprint model of the paper's own kernel (S_LUT + S_acc)
effective_tflops     the "effective TFLOPS" metric of the tile-sweep tables
complexity           LUT build / read operation counts (C_build, C_read)
algorithmic_bytes    bytes one decode call must move: storage model + activations in/out
"""
from __future__ import annotations


def storage_bits(M: int, N: int, Kb: int, Ks: int, g: int, n_sal: int) -> int:
    """S_total in bits.  S_base = Kb*(M*N + 16*N + 16*M*N/g);
    S_sal = Ks*(M*N_sal + 16*N_sal + 16*M*N/g) + 16*N_sal (index metadata)."""
    s_base = Kb * (M * N + 16 * N + 16 * M * (N // g))
    s_sal = 0
    if Ks > 0 and n_sal > 0:
        s_sal = Ks * (M * n_sal + 16 * n_sal + 16 * M * (N // g)) + 16 * n_sal
    return s_base + s_sal


def abw(M: int, N: int, Kb: int, Ks: int, g: int, s: int) -> float:
    """Average bit-width for s salient columns per group of g (N_sal = N/g*s)."""
    return storage_bits(M, N, Kb, Ks, g, (N // g) * s) / (M * N)


def smem_bytes(B_tile: int, Kb: int, M_tile: int, K_tile: int, mu: int) -> int:
    """S_LUT + S_acc of the paper's kernel, fp32."""
    s_lut = B_tile * Kb * (K_tile // mu) * (1 << mu) * 4
    s_acc = B_tile * Kb * M_tile * 4
    return s_lut + s_acc


def effective_tflops(M: int, N: int, n_sal: int, latency_s: float, B: int = 1) -> float:
    return 2.0 * M * (N + n_sal) * B / latency_s / 1e12


def complexity(M: int, N: int, Kb: int, Ks: int, n_sal: int, mu: int):
    """(C_build, C_read) summed over both branches."""
    cols = Kb * N + Ks * n_sal
    return (1 << mu) * cols / mu, M * cols / mu


def algorithmic_bytes(M: int, N: int, Kb: int, Ks: int, g: int, n_sal: int, B: int) -> int:
    """Storage model (bits rounded up to bytes per row for the salient matrix) + x in + y out (fp16)."""
    w = Kb * M * N // 8 + 2 * Kb * M * (N // g) + 2 * Kb * N
    if Ks > 0 and n_sal > 0:
        w += Ks * M * ((n_sal + 7) // 8) + 2 * Ks * M * (N // g) + 2 * Ks * n_sal + 2 * n_sal
    return w + 2 * B * N + 2 * B * M

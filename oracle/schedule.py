"""Token-count schedule and multiply-accumulate model of the pruned forward pass.

TEST INFRASTRUCTURE (oracle side).  The only numbers the paper prints that the
hot path can reproduce are its GFLOPs columns (Tables retrieval, qa, deit);
tests/golden/gmacs.txt holds them and tests/test_oracle_pins.py checks this
module against them.  They fix two readings: pruning "at layer l" happens
after block l's MLP, and "[1,4,7]" counts blocks from 1.
"""
from __future__ import annotations

import math


def drops_fixed(N0: int, L: int, r: int, first: int = 1, layers=None):
    """r tokens removed after every block l >= first (1-based), or after the
    listed blocks.  Returns (tokens entering each block, drops per block)."""
    N, Ns, rs = N0, [], []
    for l in range(1, L + 1):
        Ns.append(N)
        on = (l in layers) if layers is not None else (l >= first)
        d = min(r, N - 1) if on else 0
        rs.append(d)
        N -= d
    return Ns, rs


def drops_ratio(N0: int, L: int, ratio: float, layers):
    """floor(ratio * current count) tokens removed after each listed block
    (1-based), progressively (Sec. 4.1 Settings)."""
    N, Ns, rs = N0, [], []
    for l in range(1, L + 1):
        Ns.append(N)
        d = int(math.floor(ratio * N)) if l in layers else 0
        rs.append(d)
        N -= d
    return Ns, rs


def block_macs(N: int, D: int, mlp_ratio: int = 4) -> int:
    """Eq. sa's O(N^2 C + N C^2) with constants: qkv 3ND^2, proj ND^2,
    MLP 2*ratio*ND^2, QK^T and PV N^2 D each."""
    return (4 + 2 * mlp_ratio) * N * D * D + 2 * N * N * D


def model_gmacs(Ns, D: int, patch_tokens: int, patch_in: int) -> float:
    """Sum over blocks plus the patch embedding (patch_tokens x patch_in x D)."""
    return (sum(block_macs(n, D) for n in Ns) + patch_tokens * patch_in * D) / 1e9

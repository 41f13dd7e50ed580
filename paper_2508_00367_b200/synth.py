"""Seeded synthetic inputs with the shapes and statistics of the paper's workloads.

This module holds no arithmetic of the method: it only draws tokens and
weights.  Both the CUDA path and the CPU checker are fed from the arrays made
here (the checker receives fp64 copies), so no random stream is duplicated.

Image workloads (ImageNet-shaped, Sec. 4.2): CLS + a 14x14 or 24x24 patch grid,
iid N(0,1) token embeddings.  Video workloads (Sec. 4.1): CLS + frames x
patches tokens, frame-major, with a stationary AR(1) process (rho = 0.9) across
frames at every (patch position, channel) -- the frame-to-frame redundancy that
makes pruning pay for video.  Weights and biases N(0, 0.02); LayerNorm gain
1 + N(0, 0.02).  Values are rounded to the storage type so that every consumer
sees exactly the same numbers.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch

WEIGHT_NAMES = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
                "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    N: int
    D: int
    H: int
    D_mlp: int
    L: int
    dtype: str                 # "f32" | "bf16"
    drops: tuple               # tokens removed after block l (index l-1)
    frames: int = 0            # > 0: video, AR(1) across frames
    rho: float = 0.9
    has_cls: bool = True

    def tokens_per_block(self) -> List[int]:
        n, out = self.N, []
        for d in self.drops:
            out.append(n)
            n -= d
        return out

    def final_tokens(self) -> int:
        return self.N - sum(self.drops)


def _fixed(N, L, r):
    out, n = [], N
    for _ in range(L):
        d = min(r, n - 1)
        out.append(d)
        n -= d
    return tuple(out)


def _ratio(N, L, ratio, layers):
    out, n = [], N
    for l in range(1, L + 1):
        d = int(math.floor(ratio * n)) if l in layers else 0
        out.append(d)
        n -= d
    return tuple(out)


WORKLOADS = {
    # one ViT-S/16 block, fp32, r = 16
    "vit_s_block": Workload("vit_s_block", 2, 197, 384, 6, 1536, 1, "f32", _fixed(197, 1, 16)),
    # ViT-B/16, 12 blocks, r = 16 after every block
    "vit_b16": Workload("vit_b16", 64, 197, 768, 12, 3072, 12, "bf16", _fixed(197, 12, 16)),
    # ViT-L/16 at 384 px, 24 blocks, r = 20 after every block
    "vit_l16_384": Workload("vit_l16_384", 32, 577, 1024, 16, 4096, 24, "bf16", _fixed(577, 24, 20)),
    # video ViT-B/16, 8 frames, 30 % dropped after blocks 3, 6, 9
    "video_vit_b16": Workload("video_vit_b16", 16, 1569, 768, 12, 3072, 12, "bf16",
                              _ratio(1569, 12, 0.30, (3, 6, 9)), frames=8),
    # video ViT-L/14, 16 frames, 25 % dropped after blocks 4, 8, 12, 16
    "video_vit_l14": Workload("video_vit_l14", 4, 4097, 1024, 16, 4096, 24, "bf16",
                              _ratio(4097, 24, 0.25, (4, 8, 12, 16)), frames=16),
}


def _store(t: torch.Tensor, dtype: str) -> torch.Tensor:
    """fp32 tensor holding values representable in the storage type."""
    if dtype == "bf16":
        return t.to(torch.bfloat16).to(torch.float32)
    return t.to(torch.float32)


def make_tokens(B, N, D, dtype="bf16", frames=0, rho=0.9, has_cls=True,
                gen: Optional[torch.Generator] = None, seed=0) -> torch.Tensor:
    """[B, N, D] fp32 tensor (values representable in `dtype`)."""
    if gen is None:
        gen = torch.Generator().manual_seed(seed)
    if frames <= 0:
        x = torch.randn(B, N, D, generator=gen)
        return _store(x, dtype)
    ncls = 1 if has_cls else 0
    P = (N - ncls) // frames
    assert ncls + frames * P == N, "N must be (cls +) frames * patches"
    cls = torch.randn(B, ncls, D, generator=gen)
    fr = torch.empty(B, frames, P, D)
    fr[:, 0] = torch.randn(B, P, D, generator=gen)
    c = math.sqrt(1.0 - rho * rho)
    for f in range(1, frames):
        fr[:, f] = rho * fr[:, f - 1] + c * torch.randn(B, P, D, generator=gen)
    x = torch.cat([cls, fr.reshape(B, frames * P, D)], dim=1)
    return _store(x, dtype)


def make_block_weights(D, D_mlp, dtype="bf16", gen: Optional[torch.Generator] = None, seed=0):
    """Dict of fp32 tensors, draw order = WEIGHT_NAMES.  Matrices are [out, in]."""
    if gen is None:
        gen = torch.Generator().manual_seed(seed)
    shapes = dict(ln1_g=(D,), ln1_b=(D,), w_qkv=(3 * D, D), b_qkv=(3 * D,), w_o=(D, D), b_o=(D,),
                  ln2_g=(D,), ln2_b=(D,), w_fc1=(D_mlp, D), b_fc1=(D_mlp,), w_fc2=(D, D_mlp),
                  b_fc2=(D,))
    w = {}
    for name in WEIGHT_NAMES:
        t = 0.02 * torch.randn(*shapes[name], generator=gen)
        if name in ("ln1_g", "ln2_g"):
            t = 1.0 + t
        w[name] = _store(t, dtype)
    return w


def make_workload(wl: Workload, seed=0, B: Optional[int] = None, L: Optional[int] = None):
    """Tokens and per-block weights for a workload.  Draw order: x, then the
    blocks in order.  `B` / `L` override the batch / depth (smaller test cases
    draw a prefix of the same stream only when B is unchanged)."""
    gen = torch.Generator().manual_seed(seed)
    x = make_tokens(B or wl.B, wl.N, wl.D, wl.dtype, wl.frames, wl.rho, wl.has_cls, gen=gen)
    blocks = [make_block_weights(wl.D, wl.D_mlp, wl.dtype, gen=gen) for _ in range(L or wl.L)]
    return x, blocks

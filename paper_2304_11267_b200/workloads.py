"""Seeded synthetic inputs for the attention workloads of the Stable Diffusion 1.4 UNet.

This module serves both the CUDA library's callers and the CPU oracle's tests, and holds
none of the method's arithmetic: it only draws numbers and names shapes.  The same bytes
go to both sides.

The paper measures a real SD 1.4 UNet at 512x512 (Sec. 4); its weights and activations are
not available offline, so the values are i.i.d. N(0,1) draws rounded to binary16 while the
shapes carry the structure of the workload: 8 heads, self-attention at 4096/1024/256/64
latent tokens with head dims 40/80/160/160, cross-attention against 77 text tokens whose
last 20 rows are identical (padding tokens), and a batch of 2 (a guidance pair).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np

SEED_BASE = 23041126700
TEXT_TOKENS = 77
PADDING_ROWS = 20

Q_IDX, K_IDX, V_IDX = 0, 1, 2


@dataclass(frozen=True)
class Call:
    """One attention call: q [B,H,Nq,d], k/v [B,H,Nk,d]."""
    name: str
    B: int
    H: int
    Nq: int
    Nk: int
    d: int
    config_index: int          # 1..5, the workload list's numbering
    call_index: int = 0        # position inside a multi-call config
    peaked: bool = False       # Q multiplied by 4 before rounding (logit std about 4)
    padded_text: bool = False  # last PADDING_ROWS rows of K and of V identical

    @property
    def kind(self) -> str:
        return "cross" if self.Nk == TEXT_TOKENS and self.Nq != self.Nk else "self"

    @property
    def flops(self) -> int:
        """Algorithmic FLOPs: 2d for q.k and 2d for p.v per score element."""
        return 4 * self.B * self.H * self.Nq * self.Nk * self.d

    def io_bytes(self, elem_size: int = 2) -> int:
        """Algorithmic HBM bytes: read Q, K, V once, write O once."""
        return elem_size * self.B * self.H * self.d * (2 * self.Nq + 2 * self.Nk)

    def seed(self, tensor_index: int) -> int:
        return SEED_BASE + 10 * self.config_index + tensor_index + 100 * self.call_index

    def scale(self) -> np.float32:
        """The binary32 multiplier handed to the library: 1/sqrt(d) with the true head dim."""
        return np.float32(1.0 / np.sqrt(np.float64(self.d)))


def _normal(seed: int, shape, dtype, mult: float = 1.0) -> np.ndarray:
    x = np.random.default_rng(seed).standard_normal(shape, dtype=np.float32)
    if mult != 1.0:
        x *= np.float32(mult)
    return x.astype(dtype)


def make_inputs(call: Call, dtype=np.float16) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Draw (q, k, v) for a call.  Deterministic in ``call`` and ``dtype``."""
    q = _normal(call.seed(Q_IDX), (call.B, call.H, call.Nq, call.d), dtype,
                4.0 if call.peaked else 1.0)
    k = _normal(call.seed(K_IDX), (call.B, call.H, call.Nk, call.d), dtype)
    v = _normal(call.seed(V_IDX), (call.B, call.H, call.Nk, call.d), dtype)
    if call.padded_text and call.Nk > PADDING_ROWS:
        first = call.Nk - PADDING_ROWS
        k[:, :, first:, :] = k[:, :, first:first + 1, :]
        v[:, :, first:, :] = v[:, :, first:first + 1, :]
    return q, k, v


# --- the five workloads ---------------------------------------------------------------

def config1() -> List[Call]:
    return [Call("c1_self_1024_d40", 1, 8, 1024, 1024, 40, 1)]


def config2() -> List[Call]:
    return [Call("c2_self_4096_d40", 2, 8, 4096, 4096, 40, 2),
            Call("c2_self_4096_d40_peaked", 2, 8, 4096, 4096, 40, 2, call_index=1, peaked=True)]


CROSS_SHAPES = [(4096, 40), (1024, 80), (256, 160), (64, 160)]


def config3() -> List[Call]:
    return [Call("c3_cross_%d_d%d" % (nq, d), 2, 8, nq, TEXT_TOKENS, d, 3, call_index=i,
                 padded_text=True) for i, (nq, d) in enumerate(CROSS_SHAPES)]


# (tokens, head dim, number of transformer blocks at that resolution) for a 512x512 image
UNET_BLOCKS = [(4096, 40, 5), (1024, 80, 5), (256, 160, 5), (64, 160, 1)]


def config4() -> List[Call]:
    """One denoising step: 16 transformer blocks, each a self- and a cross-attention call."""
    calls: List[Call] = []
    for tokens, d, blocks in UNET_BLOCKS:
        for _ in range(blocks):
            i = len(calls)
            calls.append(Call("c4_%02d_self_%d_d%d" % (i, tokens, d), 2, 8, tokens, tokens, d, 4,
                              call_index=i))
            calls.append(Call("c4_%02d_cross_%d_d%d" % (i + 1, tokens, d), 2, 8, tokens,
                              TEXT_TOKENS, d, 4, call_index=i + 1, padded_text=True))
    return calls


def config5() -> List[Call]:
    return [Call("c5_self_9216_d40", 4, 8, 9216, 9216, 40, 5),
            Call("c5_self_9216_d40_peaked", 4, 8, 9216, 9216, 40, 5, call_index=1, peaked=True),
            Call("c5_cross_9216_d40", 4, 8, 9216, TEXT_TOKENS, 40, 5, call_index=2,
                 padded_text=True)]


def all_configs():
    return {1: config1(), 2: config2(), 3: config3(), 4: config4(), 5: config5()}


def shard_units(n_units: int, rank: int, world_size: int) -> Tuple[int, int]:
    """Contiguous [begin, end) range of flattened (batch, head) units owned by ``rank``.

    Attention has no exchange step between (batch, head) pairs, so a multi-GPU job is a
    plain partition of them; the first ``n_units % world_size`` ranks take one extra unit.
    """
    if world_size <= 0 or not (0 <= rank < world_size) or n_units < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_units, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)

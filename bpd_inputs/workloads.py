"""Seeded workloads: five model/input shapes and the controlled-acceptance
schedule.  Everything is synthetic; the shapes follow the paper's translation
setting (tens of subword ids over a ~32k vocabulary) and its super-resolution
setting (8x8x3 intensities in, 32x32x3 intensities out).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np
import torch

from .blob import (DTYPE_BF16, DTYPE_F32, HEAD_BLOCKDIAG, HEAD_DENSE, ModelConfig,
                   tensor_specs, write_blob)


@dataclass(frozen=True)
class Workload:
    name: str
    cfg: ModelConfig
    sigma: float          # std of the normal weight draws
    weight_seed: int
    input_seed: int
    accept_seed: int
    batch: int
    src_lo: int           # source length drawn uniformly in [src_lo, src_hi]
    src_hi: int
    n_decode: int         # tokens to decode per row (fixed-length termination)
    kind: str = "mt"      # "mt": ids in [2, V); "sr": blurred intensities 0..255

    @property
    def max_src(self) -> int:
        return self.src_hi

    def with_layout(self, head_layout: int) -> "Workload":
        return replace(self, cfg=replace(self.cfg, head_layout=head_layout))


def _wl(name, c, cfg, sigma, batch, lo, hi, n, kind="mt"):
    return Workload(name, cfg, sigma, 1000 + c, 2000 + c, 3000 + c, batch, lo, hi, n, kind)


WORKLOADS: Dict[str, Workload] = {
    "C1": _wl("C1", 1, ModelConfig(2, 2, 64, 4, 256, 512, 4, 256, dtype=DTYPE_F32), 0.08, 1, 16, 16, 32),
    "C2": _wl("C2", 2, ModelConfig(6, 6, 512, 8, 2048, 32768, 4, 2048), 0.02, 1, 32, 32, 64),
    "C3": _wl("C3", 3, ModelConfig(6, 6, 1024, 16, 4096, 32768, 8, 4096), 0.02, 1, 40, 40, 128),
    "C4": _wl("C4", 4, ModelConfig(6, 6, 1024, 16, 4096, 32768, 10, 4096), 0.02, 32, 10, 80, 128),
    "C5": _wl("C5", 5, ModelConfig(6, 6, 512, 8, 2048, 256, 10, 2048), 0.02, 1, 192, 192, 3072, "sr"),
    # C5 with 1D local self-attention in the decoder: query blocks of 256 positions, 256 positions of memory
    "C5L": _wl("C5L", 5, ModelConfig(6, 6, 512, 8, 2048, 256, 10, 2048, local_q=256, local_m=256), 0.02, 1, 192, 192,
               3072, "sr"),
}


def make_weights(cfg: ModelConfig, seed: int, sigma: float,
                 overrides: Optional[Dict[str, np.ndarray]] = None) -> np.ndarray:
    """Draw every tensor from a seeded CPU generator and pack the blob.

    Matrices and biases are N(0, sigma) drawn in float32 (then rounded to
    bfloat16, round-to-nearest-even, for bf16 models); layer-norm gains are 1
    and shifts 0.  ``overrides`` replaces named tensors (float32 arrays; they
    are rounded the same way) -- tests use it to plant special cases.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    tensors: Dict[str, np.ndarray] = {}
    for name, shape, kind in tensor_specs(cfg):
        if overrides is not None and name in overrides:
            t = torch.from_numpy(np.ascontiguousarray(overrides[name], dtype=np.float32)).reshape(shape)
        elif kind in ("matrix", "bias"):
            t = torch.randn(shape, generator=gen, dtype=torch.float32) * sigma
        elif kind == "gain":
            t = torch.ones(shape, dtype=torch.float32)
        else:
            t = torch.zeros(shape, dtype=torch.float32)
        if cfg.dtype == DTYPE_F32:
            tensors[name] = t.numpy()
        else:
            tensors[name] = t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    return write_blob(cfg, tensors)


def _box_blur_3x3(img: np.ndarray) -> np.ndarray:
    """3x3 mean per channel with edge replication, rounded to nearest."""
    h, w, _ = img.shape
    pad = np.pad(img.astype(np.int64), ((1, 1), (1, 1), (0, 0)), mode="edge")
    acc = np.zeros_like(img, dtype=np.int64)
    for dy in range(3):
        for dx in range(3):
            acc += pad[dy:dy + h, dx:dx + w, :]
    return ((2 * acc + 9) // 18).astype(np.int32)   # round(acc / 9), halves up


def make_source(w: Workload) -> Tuple[np.ndarray, np.ndarray]:
    """Source ids ``[batch, max_src]`` int32 (zero padded) and lengths ``[batch]``."""
    rng = np.random.default_rng(w.input_seed)
    src = np.zeros((w.batch, w.max_src), dtype=np.int32)
    lens = rng.integers(w.src_lo, w.src_hi + 1, size=w.batch).astype(np.int32)
    for b in range(w.batch):
        if w.kind == "sr":
            side = int(round((int(lens[b]) // 3) ** 0.5))
            assert side * side * 3 == int(lens[b])
            img = rng.integers(0, 256, size=(side, side, 3))
            src[b, :lens[b]] = _box_blur_3x3(img).reshape(-1)
        else:
            src[b, :lens[b]] = rng.integers(2, w.cfg.vocab, size=int(lens[b]))
    return src, lens


def geometric_schedule(seed: int, mean: float, n: int) -> Tuple[np.ndarray, np.ndarray]:
    """``n`` draws G >= 1 from a geometric law with success probability
    1/mean, plus ``n`` corruption offsets r >= 0 (used by ``corrupt_token``)."""
    rng = np.random.default_rng(seed)
    g = rng.geometric(1.0 / mean, size=n).astype(np.int64)
    r = rng.integers(0, 1 << 30, size=n).astype(np.int64)
    return g, r


def corrupt_token(token: int, r: int, vocab: int) -> int:
    """A token id guaranteed to differ from ``token``."""
    return int((token + 1 + (r % (vocab - 1))) % vocab)


def forced_tail(greedy: np.ndarray, j: int, k: int, g: int, r: int, vocab: int) -> np.ndarray:
    """Proposals 2..k for an iteration that starts with ``j`` tokens accepted.

    ``greedy`` is the base model's own greedy continuation (output tokens
    0..N-1).  Proposal i (1-based) targets output index j+i-1; it carries the
    greedy token while i <= g and a corrupted one after, so exactly
    min(k, g, N-j) proposals can be verified.
    """
    n = len(greedy)
    tail = np.zeros(k - 1, dtype=np.int32)
    for i in range(2, k + 1):
        idx = j + i - 1
        base = int(greedy[idx]) if idx < n else (i * 7919) % vocab
        tail[i - 2] = base if (i <= g and idx < n) else corrupt_token(base, r + i, vocab)
    return tail

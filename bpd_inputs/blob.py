"""The weight blob: a self-describing, little-endian container of tensors.

Layout
------
header (128 bytes)::

    0   char[8]  magic "BPDW0001"
    8   int32    version (1)
    12  int32    dtype            0 = float32, 1 = bfloat16 (all tensors)
    16  int32    n_enc            encoder layers
    20  int32    n_dec            decoder layers
    24  int32    d_model
    28  int32    n_heads
    32  int32    d_ff             feed-forward width inside the layers
    36  int32    vocab            shared by source, target and output
    40  int32    k_model          number of proposal heads the model carries
    44  int32    d_hidden         hidden units per proposal head
    48  int32    head_layout      0 = dense second layer, 1 = block diagonal
    52  int32    p1_identity      1 = head 1 is the identity (plain decoder output)
    56  float32  ln_eps
    60  int32    n_tensors
    64  uint64   dir_offset       (= 128)
    72  uint64   data_offset
    80  uint64   total_bytes
    88  int32    local_q          decoder self-attention: 0 = every earlier position; > 0 = 1D local attention
                                  with query blocks of this length ...
    92  int32    local_m          ... and this many positions of memory before the query's block
    96  zero padding to 128

directory: ``n_tensors`` entries of 96 bytes::

    char[64] name (NUL padded) | int32 ndim | int32 dims[3] | uint64 offset | uint64 nbytes

data: every tensor starts on a 256-byte boundary, row-major, innermost
dimension last.  Every projection matrix is stored ``[out_features,
in_features]`` so that one output feature's weights are contiguous.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass
from typing import Dict, List, Tuple

import numpy as np

BLOB_MAGIC = b"BPDW0001"
DTYPE_F32 = 0
DTYPE_BF16 = 1
HEAD_DENSE = 0
HEAD_BLOCKDIAG = 1
HEADER_BYTES = 128
DIRENT_BYTES = 96
ALIGN = 256


@dataclass(frozen=True)
class ModelConfig:
    n_enc: int
    n_dec: int
    d_model: int
    n_heads: int
    d_ff: int
    vocab: int
    k_model: int
    d_hidden: int
    dtype: int = DTYPE_BF16
    head_layout: int = HEAD_DENSE
    p1_identity: int = 0
    ln_eps: float = 1e-6
    local_q: int = 0
    local_m: int = 0

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == DTYPE_F32 else 2


def tensor_specs(cfg: ModelConfig) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, kind) for every tensor, in blob order.

    kind is one of "matrix" (random normal), "bias" (random normal),
    "gain" (ones), "shift" (zeros) and only tells the generator how to
    fill it.
    """
    d, f, V = cfg.d_model, cfg.d_ff, cfg.vocab
    k, fh = cfg.k_model, cfg.d_hidden
    specs: List[Tuple[str, Tuple[int, ...], str]] = [
        ("src_embed", (V, d), "matrix"),
        ("tgt_embed", (V, d), "matrix"),
        ("out_proj", (V, d), "matrix"),
    ]

    def ln(prefix):
        return [(prefix + ".g", (d,), "gain"), (prefix + ".b", (d,), "shift")]

    def ffn(prefix):
        return [(prefix + ".w1", (f, d), "matrix"), (prefix + ".b1", (f,), "bias"),
                (prefix + ".w2", (d, f), "matrix"), (prefix + ".b2", (d,), "bias")]

    for l in range(cfg.n_enc):
        p = f"enc.{l}"
        specs += ln(p + ".ln1")
        specs += [(p + ".attn.wqkv", (3 * d, d), "matrix"), (p + ".attn.wo", (d, d), "matrix")]
        specs += ln(p + ".ln2")
        specs += ffn(p + ".ffn")
    specs += ln("enc.lnf")
    for l in range(cfg.n_dec):
        p = f"dec.{l}"
        specs += ln(p + ".ln1")
        specs += [(p + ".self.wqkv", (3 * d, d), "matrix"), (p + ".self.wo", (d, d), "matrix")]
        specs += ln(p + ".ln2")
        specs += [(p + ".cross.wq", (d, d), "matrix"), (p + ".cross.wkv", (2 * d, d), "matrix"),
                  (p + ".cross.wo", (d, d), "matrix")]
        specs += ln(p + ".ln3")
        specs += ffn(p + ".ffn")
    specs += ln("dec.lnf")
    specs += [("head.w1", (k * fh, d), "matrix"), ("head.b1", (k * fh,), "bias")]
    if cfg.head_layout == HEAD_DENSE:
        specs += [("head.w2", (k * d, k * fh), "matrix")]
    else:
        specs += [("head.w2", (k, d, fh), "matrix")]
    specs += [("head.b2", (k * d,), "bias")]
    return specs


def _round_up(x: int, a: int) -> int:
    return (x + a - 1) // a * a


def blob_layout(cfg: ModelConfig) -> Tuple[List[Tuple[str, Tuple[int, ...], str, int, int]], int, int]:
    """Offsets of every tensor.  Returns (entries, data_offset, total_bytes)."""
    specs = tensor_specs(cfg)
    data_offset = _round_up(HEADER_BYTES + DIRENT_BYTES * len(specs), ALIGN)
    off = data_offset
    entries = []
    for name, shape, kind in specs:
        nbytes = int(np.prod(shape)) * cfg.elem_bytes
        entries.append((name, shape, kind, off, nbytes))
        off = _round_up(off + nbytes, ALIGN)
    return entries, data_offset, off


def write_blob(cfg: ModelConfig, tensors: Dict[str, np.ndarray]) -> np.ndarray:
    """Pack ``tensors`` (name -> array already in storage dtype: float32, or
    uint16 holding bfloat16 bit patterns) into one uint8 array."""
    entries, data_offset, total = blob_layout(cfg)
    buf = np.zeros(total, dtype=np.uint8)
    hdr = struct.pack(
        "<8s12ifiQQQ2i", BLOB_MAGIC, 1, cfg.dtype, cfg.n_enc, cfg.n_dec, cfg.d_model, cfg.n_heads,
        cfg.d_ff, cfg.vocab, cfg.k_model, cfg.d_hidden, cfg.head_layout, cfg.p1_identity,
        cfg.ln_eps, len(entries), HEADER_BYTES, data_offset, total, cfg.local_q, cfg.local_m)
    buf[:len(hdr)] = np.frombuffer(hdr, dtype=np.uint8)
    pos = HEADER_BYTES
    want = np.float32 if cfg.dtype == DTYPE_F32 else np.uint16
    for name, shape, _kind, off, nbytes in entries:
        arr = tensors[name]
        if arr.dtype != want or tuple(arr.shape) != tuple(shape):
            raise ValueError(f"tensor {name}: got {arr.dtype}{arr.shape}, want {want}{shape}")
        dims = list(shape) + [1] * (3 - len(shape))
        ent = struct.pack("<64si3iQQ", name.encode(), len(shape), *dims, off, nbytes)
        buf[pos:pos + DIRENT_BYTES] = np.frombuffer(ent, dtype=np.uint8)
        pos += DIRENT_BYTES
        buf[off:off + nbytes] = np.ascontiguousarray(arr).view(np.uint8).reshape(-1)
    return buf

"""Oracle model: blob parser and the combined scoring-and-proposal Transformer
in float64 numpy.  Test infrastructure only (see the package docstring).

The paper defers the scorer to the cited encoder-decoder Transformer
(Section 3, last paragraph) and adds the multi-output head of Section 6 /
Figure 3.  Conventions the paper leaves open are fixed here and recorded in
the blob header: pre-norm residual blocks with a final layer norm, sinusoidal
positions added to sqrt(d)-scaled embeddings, no biases on attention and
vocabulary projections, ReLU feed-forward layers with biases, argmax ties to
the lowest id.
"""
from __future__ import annotations

import struct
from dataclasses import dataclass
from typing import Dict, List, Optional

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- blob

@dataclass
class OracleModel:
    n_enc: int
    n_dec: int
    d: int
    H: int
    d_ff: int
    V: int
    k_model: int
    d_hidden: int
    dtype: int
    head_layout: int      # 0 dense, 1 block diagonal
    p1_identity: int
    eps: float
    w: Dict[str, np.ndarray]   # float64 tensors
    local_q: int = 0           # decoder self-attention: 0 = full causal, else 1D local attention (query block,
    local_m: int = 0           # memory length)


def parse_blob(blob: np.ndarray) -> OracleModel:
    """Decode the weight container (format: 128-byte header, 96-byte
    directory entries, 256-byte aligned row-major tensors)."""
    raw = np.ascontiguousarray(blob).view(np.uint8)
    if bytes(raw[:8]) != b"BPDW0001":
        raise ValueError("bad magic")
    (version, dtype, n_enc, n_dec, d, H, d_ff, V, k_model, d_hidden, layout,
     p1id) = struct.unpack_from("<12i", raw, 8)
    (eps,) = struct.unpack_from("<f", raw, 56)
    (n_tensors,) = struct.unpack_from("<i", raw, 60)
    dir_off, _data_off, total = struct.unpack_from("<3Q", raw, 64)
    local_q, local_m = struct.unpack_from("<2i", raw, 88)
    if version != 1 or total != raw.size:
        raise ValueError("bad version or size")
    w: Dict[str, np.ndarray] = {}
    for t in range(n_tensors):
        base = dir_off + 96 * t
        name = bytes(raw[base:base + 64]).split(b"\0")[0].decode()
        ndim, d0, d1, d2 = struct.unpack_from("<4i", raw, base + 64)
        off, nbytes = struct.unpack_from("<2Q", raw, base + 80)
        shape = (d0, d1, d2)[:ndim]
        seg = raw[off:off + nbytes]
        if dtype == 0:
            arr = seg.view(np.float32).astype(F64)
        else:  # bfloat16 = upper half of a float32
            arr = (seg.view(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(F64)
        w[name] = arr.reshape(shape)
    return OracleModel(n_enc, n_dec, d, H, d_ff, V, k_model, d_hidden, dtype, layout, p1id,
                       float(eps), w, int(local_q), int(local_m))


# --------------------------------------------------------------------------- primitives

def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray, eps: float) -> np.ndarray:
    """(x - mean) / sqrt(var + eps) * g + b over the last axis (biased variance)."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * g + b


def softmax_masked(scores: np.ndarray, allowed: np.ndarray) -> np.ndarray:
    """Row softmax over allowed entries; disallowed entries get weight exactly 0."""
    s = np.where(allowed, scores, -np.inf)
    m = s.max(axis=-1, keepdims=True)
    e = np.where(allowed, np.exp(s - m), 0.0)
    return e / e.sum(axis=-1, keepdims=True)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, allowed: np.ndarray, H: int) -> np.ndarray:
    """Multi-head scaled dot-product attention.

    q [n, d], k and v [m, d], allowed [n, m] bool.  Head h uses feature
    columns h*d_h:(h+1)*d_h of q, k and v; scores are q.k / sqrt(d_h).
    """
    n, d = q.shape
    dh = d // H
    out = np.empty((n, d), dtype=F64)
    for h in range(H):
        sl = slice(h * dh, (h + 1) * dh)
        scores = q[:, sl] @ k[:, sl].T / np.sqrt(F64(dh))
        out[:, sl] = softmax_masked(scores, allowed) @ v[:, sl]
    return out


def positional(pos: np.ndarray, d: int) -> np.ndarray:
    """Sinusoidal signal: PE(p, 2i) = sin(p / 10000^(2i/d)), PE(p, 2i+1) = cos(same)."""
    i = np.arange(d // 2, dtype=F64)
    ang = np.asarray(pos, dtype=F64)[:, None] / np.power(F64(10000.0), 2.0 * i / d)[None, :]
    pe = np.empty((len(pos), d), dtype=F64)
    pe[:, 0::2] = np.sin(ang)
    pe[:, 1::2] = np.cos(ang)
    return pe


def embed(table: np.ndarray, ids, first_pos: int) -> np.ndarray:
    ids = np.asarray(ids, dtype=np.int64)
    d = table.shape[1]
    return table[ids] * np.sqrt(F64(d)) + positional(np.arange(first_pos, first_pos + len(ids)), d)


def ffn(x, w1, b1, w2, b2):
    return np.maximum(x @ w1.T + b1, 0.0) @ w2.T + b2


# --------------------------------------------------------------------------- encoder

def encode(m: OracleModel, src_ids, src_len: Optional[int] = None) -> np.ndarray:
    """Encoder memory [S, d] for one row.  Keys at positions >= src_len are
    masked (weight 0); rows past src_len are computed but meaningless."""
    w = m.w
    S = len(src_ids)
    src_len = S if src_len is None else int(src_len)
    x = embed(w["src_embed"], src_ids, 0)
    allowed = np.broadcast_to(np.arange(S)[None, :] < src_len, (S, S))
    for l in range(m.n_enc):
        p = f"enc.{l}"
        y = layer_norm(x, w[p + ".ln1.g"], w[p + ".ln1.b"], m.eps)
        qkv = y @ w[p + ".attn.wqkv"].T
        a = attention(qkv[:, :m.d], qkv[:, m.d:2 * m.d], qkv[:, 2 * m.d:], allowed, m.H)
        x = x + a @ w[p + ".attn.wo"].T
        y = layer_norm(x, w[p + ".ln2.g"], w[p + ".ln2.b"], m.eps)
        x = x + ffn(y, w[p + ".ffn.w1"], w[p + ".ffn.b1"], w[p + ".ffn.w2"], w[p + ".ffn.b2"])
    return layer_norm(x, w["enc.lnf.g"], w["enc.lnf.b"], m.eps)


# --------------------------------------------------------------------------- decoder

def self_attention_allowed(m: OracleModel, query_pos: np.ndarray, n_keys: int) -> np.ndarray:
    """Which keys (positions 0..n_keys-1) each decoder query may attend to.

    Causal: key j <= query position t.  With 1D local attention (Section 7.2
    names it for the super-resolution model; the block lengths are this
    build's choice, carried in the blob header) the target sequence is cut
    into query blocks of local_q positions, and a query also sees only the
    local_m positions before its own block: j >= (t // local_q) * local_q - local_m."""
    t = np.asarray(query_pos)[:, None]
    j = np.arange(n_keys)[None, :]
    ok = j <= t
    if m.local_q > 0:
        ok &= j >= (t // m.local_q) * m.local_q - m.local_m
    return ok


def decoder_full(m: OracleModel, memory: np.ndarray, src_len: int, dec_inputs, trace: Optional[list] = None) -> np.ndarray:
    """Uncached decoder: final-layer-norm output h [n, d] for decoder inputs
    u_0..u_{n-1} (position of u_t is t).  Causal self-attention, cross-attention
    over memory rows < src_len.  ``trace``, if given, receives a copy of the
    residual stream [n, d] after every layer (for comparing intermediates)."""
    w = m.w
    n = len(dec_inputs)
    S = memory.shape[0]
    x = embed(w["tgt_embed"], dec_inputs, 0)
    causal = self_attention_allowed(m, np.arange(n), n)
    cross_ok = np.broadcast_to(np.arange(S)[None, :] < src_len, (n, S))
    for l in range(m.n_dec):
        p = f"dec.{l}"
        y = layer_norm(x, w[p + ".ln1.g"], w[p + ".ln1.b"], m.eps)
        qkv = y @ w[p + ".self.wqkv"].T
        a = attention(qkv[:, :m.d], qkv[:, m.d:2 * m.d], qkv[:, 2 * m.d:], causal, m.H)
        x = x + a @ w[p + ".self.wo"].T
        y = layer_norm(x, w[p + ".ln2.g"], w[p + ".ln2.b"], m.eps)
        q = y @ w[p + ".cross.wq"].T
        kv = memory @ w[p + ".cross.wkv"].T
        a = attention(q, kv[:, :m.d], kv[:, m.d:], cross_ok, m.H)
        x = x + a @ w[p + ".cross.wo"].T
        y = layer_norm(x, w[p + ".ln3.g"], w[p + ".ln3.b"], m.eps)
        x = x + ffn(y, w[p + ".ffn.w1"], w[p + ".ffn.b1"], w[p + ".ffn.w2"], w[p + ".ffn.b2"])
        if trace is not None:
            trace.append(x.copy())
    return layer_norm(x, w["dec.lnf.g"], w["dec.lnf.b"], m.eps)


class DecoderCache:
    """Key/value cache for one row.  Self-attention K/V of positions < length
    are live; anything at or beyond ``length`` is dead storage that the next
    pass overwrites (rollback = not advancing ``length``)."""

    def __init__(self, m: OracleModel, memory: np.ndarray, src_len: int, capacity: int):
        self.m, self.src_len, self.length = m, int(src_len), 0
        self.k = np.zeros((m.n_dec, capacity, m.d), dtype=F64)
        self.v = np.zeros((m.n_dec, capacity, m.d), dtype=F64)
        self.cross = []
        for l in range(m.n_dec):
            kv = memory @ m.w[f"dec.{l}.cross.wkv"].T
            self.cross.append((kv[:, :m.d].copy(), kv[:, m.d:].copy()))

    def extend(self, tokens) -> np.ndarray:
        """Run the decoder over ``tokens`` placed at positions length..length+n-1,
        writing their K/V speculatively (length is NOT advanced).  Returns h [n, d]."""
        m, w, T, n = self.m, self.m.w, self.length, len(tokens)
        x = embed(w["tgt_embed"], tokens, T)
        allowed = self_attention_allowed(m, T + np.arange(n), T + n)
        S = self.cross[0][0].shape[0]
        cross_ok = np.broadcast_to(np.arange(S)[None, :] < self.src_len, (n, S))
        for l in range(m.n_dec):
            p = f"dec.{l}"
            y = layer_norm(x, w[p + ".ln1.g"], w[p + ".ln1.b"], m.eps)
            qkv = y @ w[p + ".self.wqkv"].T
            self.k[l, T:T + n] = qkv[:, m.d:2 * m.d]
            self.v[l, T:T + n] = qkv[:, 2 * m.d:]
            a = attention(qkv[:, :m.d], self.k[l, :T + n], self.v[l, :T + n], allowed, m.H)
            x = x + a @ w[p + ".self.wo"].T
            y = layer_norm(x, w[p + ".ln2.g"], w[p + ".ln2.b"], m.eps)
            q = y @ w[p + ".cross.wq"].T
            a = attention(q, self.cross[l][0], self.cross[l][1], cross_ok, m.H)
            x = x + a @ w[p + ".cross.wo"].T
            y = layer_norm(x, w[p + ".ln3.g"], w[p + ".ln3.b"], m.eps)
            x = x + ffn(y, w[p + ".ffn.w1"], w[p + ".ffn.b1"], w[p + ".ffn.w2"], w[p + ".ffn.b2"])
        return layer_norm(x, w["dec.lnf.g"], w["dec.lnf.b"], m.eps)

    def commit(self, n_accept: int) -> None:
        self.length += int(n_accept)


# --------------------------------------------------------------------------- heads

def head_outputs(m: OracleModel, h: np.ndarray, k: int) -> np.ndarray:
    """Section 6: one feed-forward layer with hidden size k_model*d_hidden and
    output size k_model*d_model between the decoder output h and the vocabulary
    projection, with a residual from h to each of the k outputs.  Returns
    o [n, k, d] for the first k heads."""
    w, d, fh = m.w, m.d, m.d_hidden
    u = np.maximum(h @ w["head.w1"].T + w["head.b1"], 0.0)           # [n, k_model*fh]
    n = h.shape[0]
    o = np.empty((n, k, d), dtype=F64)
    for i in range(k):
        if m.head_layout == 0:
            oi = u @ w["head.w2"][i * d:(i + 1) * d].T
        else:
            oi = u[:, i * fh:(i + 1) * fh] @ w["head.w2"][i].T
        o[:, i, :] = oi + w["head.b2"][i * d:(i + 1) * d] + h
    if m.p1_identity:
        o[:, 0, :] = h
    return o


def head_logits(m: OracleModel, h: np.ndarray, k: int) -> np.ndarray:
    """The original vocabulary projection applied identically to each of the k
    outputs: logits [n, k, V]."""
    return head_outputs(m, h, k) @ m.w["out_proj"].T


def argmax_lowest(logits: np.ndarray) -> np.ndarray:
    """Top-1 over the last axis, ties to the lowest id."""
    return np.argmax(logits, axis=-1).astype(np.int64)

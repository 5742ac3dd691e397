"""Oracle decode loops: greedy (Section 2), blockwise parallel decoding in
its two-call form (Section 3) and in its merged form (Section 4).  Test
infrastructure only (see the package docstring).

Every loop is written against an ``invoke(dec_inputs, n_new)`` callable -- one
*model invocation*: given decoder inputs u_0..u_t (u_0 the start token,
u_t = y_t) it returns, for each of the last ``n_new`` positions, the argmax
token of each of the k models p_1..p_k: an integer table [n_new][k].  Entry
[r][i-1] for the position holding u_t is argmax p_i(y_{t+i} | y_<=t, x).
Tests drive the loops with hand-made tables; ``TransformerScorer`` supplies
the real model.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np

from .model import DecoderCache, OracleModel, argmax_lowest, decoder_full, encode, head_logits

START_ID = 0


@dataclass
class DecodeResult:
    ids: List[int]
    khats: List[int] = field(default_factory=list)   # accepted block size per iteration
    invocations: int = 0

    @property
    def iterations(self) -> int:
        return len(self.khats)

    @property
    def mean_block(self) -> float:
        """Mean accepted block size: tokens per decoding iteration (the
        priming invocation is not an iteration)."""
        return len(self.ids) / max(1, len(self.khats))


# --------------------------------------------------------------------------- acceptance

class P1View:
    """What the Verify substep may ask about p_1 at one position: its argmax and,
    when the logits are known, the rank of any token (number of tokens that beat
    it; larger logit wins, equal logits go to the lower id)."""

    def __init__(self, argmax: Optional[int] = None, logits: Optional[np.ndarray] = None):
        self.logits = None if logits is None else np.asarray(logits)
        self._argmax = int(np.argmax(self.logits)) if argmax is None else int(argmax)

    @property
    def argmax(self) -> int:
        return self._argmax

    def rank(self, token: int) -> int:
        if self.logits is None:
            return 0 if token == self._argmax else 1 << 30
        lg = self.logits
        return int(np.sum(lg > lg[token]) + np.sum(lg[:token] == lg[token]))


def _view(x) -> "P1View":
    return x if isinstance(x, P1View) else P1View(argmax=x[0])


def accept_exact(proposal: int, p1) -> bool:
    """Section 3, Verify: the proposal must equal the base model's argmax."""
    return proposal == _view(p1).argmax


def accept_topn(n: int):
    """Section 5.1: the proposal must lie within the n highest-scoring tokens of p_1."""
    return lambda proposal, p1: _view(p1).rank(proposal) < n


def accept_distance(eps: int):
    """Section 5.2 with d(u, v) = |u - v| (intensities): the proposal must be within
    eps of p_1's argmax."""
    return lambda proposal, p1: abs(int(proposal) - _view(p1).argmax) <= eps


def verify_prefix(block: Sequence[int], p1_of: Callable[[int], Sequence[int]],
                  accept: Callable[[int, Sequence[int]], bool] = accept_exact, min_block: int = 1) -> int:
    """Largest khat such that proposal i is accepted for all 1 <= i <= khat.

    ``block[i-1]`` is the proposal for y_{j+i}; ``p1_of(i)`` gives what the
    acceptance test needs about p_1(y_{j+i} | y_<=j+i-1): a P1View, or a sequence
    whose first entry is its argmax.  Proposal 1 is p_1's own argmax on the same
    prefix, so khat >= 1 without testing it.  ``min_block`` (Section 5.3) forces at
    least that many proposals to be taken.  Whatever the criterion, the token kept
    is the proposal (Section 3, Accept), not p_1's argmax.
    """
    khat = 1
    while khat < len(block) and (khat < min_block or accept(block[khat], p1_of(khat + 1))):
        khat += 1
    return khat


def p1_views(invoke, table) -> Callable[[int], "P1View"]:
    """p_1 for y_{j+i} sits at the position of proposal i-1 (row i-2 of the table).
    Uses the scorer's logits when it keeps them, the argmax ids otherwise."""
    logits = getattr(invoke, "last_logits", None)

    def of(i: int) -> P1View:
        if logits is not None:
            return P1View(argmax=int(table[i - 2][0]), logits=logits[i - 2, 0])
        return P1View(argmax=int(table[i - 2][0]))
    return of


def clip_termination(block: Sequence[int], khat: int, j: int, n_max: int, eos: int):
    """Fixed-length termination clips the accepted count to the tokens still
    wanted; with an end-of-sequence id the block is cut after the first
    accepted EOS.  Returns (khat, finished)."""
    khat = min(khat, n_max - j)
    finished = (j + khat >= n_max)
    if eos >= 0:
        for i in range(khat):
            if block[i] == eos:
                return i + 1, True
    return khat, finished


# --------------------------------------------------------------------------- loops

def greedy(invoke, n_max: int, eos: int = -1) -> DecodeResult:
    """Section 2: extend with argmax p_1 one token at a time."""
    res = DecodeResult(ids=[])
    inputs = [START_ID]
    while len(res.ids) < n_max:
        tok = int(invoke(inputs, 1)[0][0])
        res.invocations += 1
        res.ids.append(tok)
        res.khats.append(1)
        inputs.append(tok)
        if eos >= 0 and tok == eos:
            break
    return res


TailFn = Callable[[int, int], Sequence[int]]   # (j accepted so far, iteration index) -> proposals 2..k


def blockwise_twocall(invoke, k: int, n_max: int, eos: int = -1,
                      tail_fn: Optional[TailFn] = None, accept=accept_exact, min_block: int = 1) -> DecodeResult:
    """Section 3 literally: a Predict invocation on the accepted prefix, then a
    Verify invocation on prefix + block; two invocations per iteration."""
    res = DecodeResult(ids=[])
    inputs = [START_ID]
    while True:
        j = len(res.ids)
        block = [int(t) for t in invoke(inputs, 1)[0][:k]]                 # Predict
        if tail_fn is not None:
            block[1:] = [int(t) for t in tail_fn(j, res.iterations)]
        table = invoke(inputs + block, k)                                  # Verify
        res.invocations += 2
        # p_1 for y_{j+i} is conditioned on y_<=j+i-1, i.e. sits at the position of proposal i-1
        khat = verify_prefix(block, p1_views(invoke, table), accept, min_block)
        khat, finished = clip_termination(block, khat, j, n_max, eos)
        res.ids += block[:khat]
        res.khats.append(khat)
        inputs += block[:khat]
        if finished:
            return res


def blockwise_merged(invoke, k: int, n_max: int, eos: int = -1,
                     tail_fn: Optional[TailFn] = None, accept=accept_exact, min_block: int = 1) -> DecodeResult:
    """Section 4: the combined model returns all k heads at all k block
    positions, so the row of the last accepted position is the next Predict;
    one priming invocation, then one invocation per iteration."""
    res = DecodeResult(ids=[])
    inputs = [START_ID]
    block = [int(t) for t in invoke(inputs, 1)[0][:k]]                     # priming pass
    res.invocations = 1
    while True:
        j = len(res.ids)
        if tail_fn is not None:
            block[1:] = [int(t) for t in tail_fn(j, res.iterations)]
        table = invoke(inputs + block, k)
        res.invocations += 1
        khat = verify_prefix(block, p1_views(invoke, table), accept, min_block)
        khat, finished = clip_termination(block, khat, j, n_max, eos)
        res.ids += block[:khat]
        res.khats.append(khat)
        inputs += block[:khat]
        if finished:
            return res
        block = [int(t) for t in table[khat - 1][:k]]                      # reuse row khat


# --------------------------------------------------------------------------- the real model

class TransformerScorer:
    """``invoke`` backed by the oracle Transformer for one source row.

    cached=False recomputes the whole decoder over the prefix at every call
    (the plain definition); cached=True keeps self-attention K/V of accepted
    positions and only runs the new ones.  ``last_logits`` / ``last_hidden``
    hold the [n_new, k, V] logits and [n_new, d] decoder outputs of the latest
    call."""

    def __init__(self, m: OracleModel, src_ids, src_len: Optional[int] = None, k: Optional[int] = None,
                 cached: bool = False, capacity: int = 0):
        self.m = m
        self.k = m.k_model if k is None else k
        self.src_len = len(src_ids) if src_len is None else int(src_len)
        self.memory = encode(m, src_ids, self.src_len)
        self.cached = cached
        self.cache = DecoderCache(m, self.memory, self.src_len, capacity) if cached else None
        self.inputs_seen: List[int] = []
        self.last_logits = None
        self.last_hidden = None

    def logits(self, dec_inputs: Sequence[int], n_new: int) -> np.ndarray:
        if not self.cached:
            h = decoder_full(self.m, self.memory, self.src_len, dec_inputs)[-n_new:]
        else:
            keep = len(dec_inputs) - n_new
            c = self.cache
            # positions already run and now part of the accepted prefix become live
            if keep < c.length or list(dec_inputs[:c.length]) != self.inputs_seen[:c.length]:
                raise ValueError("cache does not hold this prefix")
            if list(dec_inputs[c.length:keep]) != self.inputs_seen[c.length:keep]:
                raise ValueError("prefix extends beyond what the last pass computed")
            c.commit(keep - c.length)
            h = c.extend(dec_inputs[keep:])
            self.inputs_seen = list(dec_inputs)
        self.last_hidden = h
        self.last_logits = head_logits(self.m, h, self.k)
        return self.last_logits

    def layer_outputs(self, dec_inputs: Sequence[int], n_new: int) -> np.ndarray:
        """Residual stream after every decoder layer for the last ``n_new`` inputs, [n_dec, n_new, d]
        (uncached forward; for comparing intermediates)."""
        trace: list = []
        decoder_full(self.m, self.memory, self.src_len, dec_inputs, trace)
        return np.stack([x[-n_new:] for x in trace])

    def __call__(self, dec_inputs: Sequence[int], n_new: int) -> np.ndarray:
        return argmax_lowest(self.logits(dec_inputs, n_new))

"""Lock-step comparison of the CUDA library with the CPU oracle.

Both sides are driven one iteration at a time from the same state.  Random
weights give many near-ties between the two best logits, where bf16 rounding
may legitimately pick either token; so for every entry of the k x k table:

  * oracle margin (top-1 minus top-2 logit) >= MARGIN: the ids must be equal;
  * otherwise the GPU's id must score within 2*TOL of the oracle's maximum,
    and the oracle adopts the GPU's id for that entry.

After adoption both sides hold the same table, so the accepted block size,
the accepted tokens and the next block must match exactly.  Logits and decoder
outputs must agree within TOL (bf16 weights, fp32 accumulation on the GPU,
float64 in the oracle).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional

import numpy as np

from oracle.decode import TransformerScorer, clip_termination, verify_prefix
from oracle.model import OracleModel

MARGIN = 0.1
TOL = 2e-2


@dataclass
class LockstepReport:
    iterations: int = 0
    adopted: int = 0
    entries: int = 0
    max_logit_err: float = 0.0
    max_hidden_err: float = 0.0
    khats: List[List[int]] = field(default_factory=list)


def _reconcile(gpu_ids: np.ndarray, logits: np.ndarray, rep: LockstepReport, what: str) -> np.ndarray:
    """gpu_ids [...], logits [..., V] (oracle).  Returns the table both sides agree on."""
    flat_ids = gpu_ids.reshape(-1)
    flat = logits.reshape(-1, logits.shape[-1])
    out = np.empty_like(flat_ids)
    for e in range(flat.shape[0]):
        row = flat[e]
        top = int(np.argmax(row))
        best = row[top]
        second = np.partition(row, -2)[-2] if row.size > 1 else -np.inf
        g = int(flat_ids[e])
        if g == -1:                      # not evaluated (lazy heads): nothing to compare, the oracle keeps its own
            out[e] = top
            continue
        rep.entries += 1
        if best - second >= MARGIN:
            assert g == top, f"{what}: entry {e}: GPU id {g} != oracle id {top} at margin {best - second:.4f}"
            out[e] = top
        else:
            assert 0 <= g < row.size and best - row[g] <= 2 * TOL, (
                f"{what}: entry {e}: GPU id {g} scores {best - row[g]:.4f} below the oracle maximum")
            if g != top:
                rep.adopted += 1
            out[e] = g
    return out.reshape(gpu_ids.shape)


def _decision(kind, param, proposal: int, top: int, row: np.ndarray):
    """Oracle's accept decision for one proposal and how far (in logits) it is from flipping."""
    if kind == "exact":
        return proposal == top, np.inf
    if kind == "distance":
        return abs(proposal - top) <= param, np.inf          # integers once the argmax is agreed
    # top-n: rank under (logit desc, id asc); the boundary is between the n-th and the (n+1)-th entry
    order = sorted(range(row.size), key=lambda v: (-row[v], v))
    rank = order.index(proposal)
    if rank < param:
        other = row[order[param]] if param < row.size else -np.inf
        return True, row[proposal] - other
    return False, row[order[param - 1]] - row[proposal]


def near_miss_tail(scorer_factory, inputs: List[int], p1: int, k: int, it: int, kind: str, vocab: int) -> np.ndarray:
    """Proposals 2..k that sit around the acceptance boundary: each is chosen from the
    oracle's p_1 at the position before it -- a cycling rank (top-n tests) or a cycling
    offset from the argmax (distance tests)."""
    ranks = [1, 0, 2, 3, 0, 1, 2, 0]
    offsets = [1, -2, 0, 3, 2, -1, 0, -3]
    seq = list(inputs) + [int(p1)]
    tail = []
    sc = scorer_factory()
    for i in range(2, k + 1):
        row = sc.logits(seq, 1)[0, 0]
        order = sorted(range(row.size), key=lambda v: (-row[v], v))
        if kind == "distance":
            tok = min(max(order[0] + offsets[(it + i) % len(offsets)], 0), vocab - 1)
        else:
            tok = order[ranks[(it + i) % len(ranks)]]
        tail.append(tok)
        seq.append(tok)
    return np.array(tail, dtype=np.int32)


def lockstep(sess, om: OracleModel, src: np.ndarray, src_len: np.ndarray, k: int, n_max: int,
             max_iters: int, tail_fn: Optional[Callable[[int, int, int], np.ndarray]] = None,
             eos: int = -1, rows: Optional[List[int]] = None, check_values: bool = True,
             tol: float = TOL, accept=("exact", 0), accept_mode: int = 0, min_block: int = 1,
             near_miss: bool = False) -> LockstepReport:
    """Drive ``sess`` (a freshly created binding Session) and the oracle together.

    tail_fn(row, j, iteration) -> proposals 2..k for that row, or None.
    rows: batch rows the oracle follows (default: all).
    accept / accept_mode / min_block: the Verify criterion as the oracle names it and as
    the C ABI encodes it.  near_miss: build the forced tails from the oracle's own p_1 so
    that they straddle the acceptance boundary.
    """
    B = sess.B
    rows = list(range(B)) if rows is None else rows
    rep = LockstepReport()
    sess.bpd_encode(src, src_len)
    scorers = {b: TransformerScorer(om, src[b, :src_len[b]], k=k, cached=True, capacity=n_max + 2 * k + 2)
               for b in rows}
    inputs = {b: [0] for b in rows}
    done = {b: False for b in rows}
    emitted = {b: [] for b in rows}
    blocks = {}
    prime_logits = {b: scorers[b].logits(inputs[b], 1)[0] for b in rows}      # [k, V]
    j_all = np.zeros(B, dtype=np.int64)
    for it in range(max_iters):
        tails = None
        if near_miss and k > 1:
            tails = np.zeros((B, k - 1), dtype=np.int32)
            for b in rows:
                if done[b]:
                    continue
                p1 = int(np.argmax(prime_logits[b][0])) if it == 0 else blocks[b][0]
                tails[b] = near_miss_tail(lambda: TransformerScorer(om, src[b, :src_len[b]], k=1), inputs[b], p1, k, it,
                                          accept[0], om.V)
        elif tail_fn is not None and k > 1:
            tails = np.zeros((B, k - 1), dtype=np.int32)
            for b in range(B):
                tails[b] = tail_fn(b, int(j_all[b]), it)
        res = sess.bpd_iteration(k, n_max, eos_id=eos, forced_tail=tails, want_logits=check_values,
                                 want_hidden=check_values, accept_mode=accept_mode)
        if check_values:
            g_logits = res["logits"].cpu().numpy()
            g_hidden = res["hidden"].cpu().numpy()
        kh_row = []
        for b in rows:
            if done[b]:
                assert res["khat"][b] == 0
                kh_row.append(0)
                continue
            if it == 0:
                # the priming pass: the block's first entry is p_1's argmax on the start token
                first = _reconcile(res["block"][b, :1] if tails is not None else res["block"][b],
                                   prime_logits[b][:1] if tails is not None else prime_logits[b], rep, "prime")
                blocks[b] = [int(t) for t in (list(first) + list(tails[b]) if tails is not None else first)]
            elif tails is not None:
                blocks[b] = [blocks[b][0]] + [int(t) for t in tails[b]]
            assert list(res["block"][b]) == blocks[b], f"row {b} iteration {it}: scored block differs"
            sc = scorers[b]
            lg = sc.logits(inputs[b] + blocks[b], k)                 # [k, k, V]
            if check_values:
                herr = float(np.abs(g_hidden[b] - sc.last_hidden).max())
                lerr = float(np.abs(g_logits[b] - lg).max())
                rep.max_hidden_err = max(rep.max_hidden_err, herr)
                rep.max_logit_err = max(rep.max_logit_err, lerr)
                assert herr <= tol, f"row {b} iteration {it}: decoder output differs by {herr}"
                assert lerr <= tol, f"row {b} iteration {it}: logits differ by {lerr}"
            table = _reconcile(res["table"][b], lg, rep, f"row {b} iteration {it}")
            j = len(emitted[b])
            # walk the block as Section 3's Verify does; where the oracle's decision is within MARGIN of
            # flipping, follow the GPU (its accepted count tells its decision for every proposal it reached)
            kg = int(res["khat"][b])
            khat = 1
            while khat < k:
                d, m = _decision(accept[0], accept[1], blocks[b][khat], int(table[khat - 1][0]), lg[khat - 1, 0])
                d = d or khat < min_block
                cut = khat >= n_max - j or (eos >= 0 and eos in blocks[b][:khat])   # the GPU stopped for another reason
                g = True if kg > khat else (False if (kg == khat and not cut) else None)
                if g is not None and g != d:
                    assert m < MARGIN, (f"row {b} iteration {it}: proposal {khat + 1} GPU {'accepts' if g else 'rejects'}, "
                                        f"oracle disagrees at margin {m:.4f}")
                    rep.adopted += 1
                    d = g
                if not d:
                    break
                khat += 1
            khat, fin = clip_termination(blocks[b], khat, j, n_max, eos)
            assert khat == int(res["khat"][b]), f"row {b} iteration {it}: khat {res['khat'][b]} != oracle {khat}"
            acc = blocks[b][:khat]
            assert list(res["accepted"][b, :khat]) == acc and np.all(res["accepted"][b, khat:] == -1)
            nxt = [int(t) for t in table[khat - 1]]
            if not fin:                      # a finished row has no next block to speak of
                assert list(res["next_block"][b]) == nxt, f"row {b} iteration {it}: next block differs"
            emitted[b] += acc
            inputs[b] += acc
            blocks[b] = nxt
            done[b] = fin
            kh_row.append(khat)
        for b in range(B):
            j_all[b] += int(res["khat"][b])
        rep.khats.append(kh_row)
        rep.iterations += 1
        if all(done.values()):
            break
    rep.emitted = emitted
    return rep

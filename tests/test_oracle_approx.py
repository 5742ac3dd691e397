"""Pins for the oracle's approximate acceptance criteria (Section 5 of the
paper): top-n membership, distance to the argmax, minimum block size.  CPU only."""
import itertools

import numpy as np
import pytest

from bpd_inputs import DTYPE_F32, ModelConfig, make_weights
from oracle.decode import (P1View, TransformerScorer, accept_distance, accept_exact, accept_topn,
                           blockwise_merged, blockwise_twocall, greedy, verify_prefix)
from oracle.model import parse_blob


def test_rank_is_position_in_a_stable_descending_sort():
    rng = np.random.default_rng(0)
    lg = rng.integers(0, 6, size=40).astype(np.float64)       # many exact ties
    order = sorted(range(40), key=lambda v: (-lg[v], v))       # larger logit first, then lower id
    view = P1View(logits=lg)
    assert view.argmax == order[0]
    for pos, tok in enumerate(order):
        assert view.rank(tok) == pos
    for n in (1, 2, 3, 7):
        acc = accept_topn(n)
        assert [t for t in range(40) if acc(t, view)] == sorted(order[:n])
    # ids only (no logits): the argmax is rank 0, nothing else is in any top-n
    ids_only = P1View(argmax=9)
    assert accept_topn(3)(9, ids_only) and not accept_topn(3)(8, ids_only)


def test_distance_criterion_on_intensities():
    view = P1View(argmax=100)
    assert [u for u in range(95, 106) if accept_distance(2)(u, view)] == [98, 99, 100, 101, 102]
    assert [u for u in range(95, 106) if accept_distance(0)(u, view)] == [100]
    # through verify_prefix: proposals 103, 99 against argmaxes 101, 104
    table = [[101], [104], [0]]
    assert verify_prefix([7, 103, 99], lambda i: table[i - 2], accept_distance(2)) == 2
    assert verify_prefix([7, 103, 102], lambda i: table[i - 2], accept_distance(2)) == 3
    assert verify_prefix([7, 103, 102], lambda i: table[i - 2], accept_exact) == 1


def test_minimum_block_size_forces_proposals_in():
    table = [[50], [60], [70]]
    block = [1, 2, 3, 70]
    assert verify_prefix(block, lambda i: table[i - 2], accept_exact) == 1
    assert verify_prefix(block, lambda i: table[i - 2], accept_exact, min_block=2) == 2
    assert verify_prefix(block, lambda i: table[i - 2], accept_exact, min_block=3) == 4   # 4th matches 70
    assert verify_prefix(block, lambda i: table[i - 2], accept_exact, min_block=9) == 4   # never beyond the block


def _tiny(V=29, k=4, seed=5):
    cfg = ModelConfig(1, 2, 16, 2, 32, V, k, 24, dtype=DTYPE_F32)
    return parse_blob(make_weights(cfg, seed, 0.5))


def test_top1_and_zero_distance_reduce_to_exact():
    m = _tiny()
    src, n, k = [3, 4, 5, 6], 16, 4
    ref = blockwise_merged(TransformerScorer(m, src), k, n)
    for acc in (accept_topn(1), accept_distance(0)):
        got = blockwise_merged(TransformerScorer(m, src), k, n, accept=acc)
        assert got.ids == ref.ids and got.khats == ref.khats
    assert ref.ids == greedy(TransformerScorer(m, src), n).ids


def test_relaxing_the_criterion_never_shortens_a_block_and_keeps_the_proposal():
    m = _tiny(V=11)
    src, k = [1, 2, 3], 4
    sc = TransformerScorer(m, src)
    prefix = greedy(sc, 5).ids
    inputs = [0] + prefix
    first = int(sc(inputs, 1)[0][0])
    for tail in itertools.product(range(11), repeat=2):
        block = [first] + list(tail) + [0]
        table = sc(inputs + block, k)
        logits = sc.last_logits
        views = lambda i: P1View(argmax=int(table[i - 2][0]), logits=logits[i - 2, 0])
        kh = [verify_prefix(block, views, accept_topn(n)) for n in (1, 2, 3, 11)]
        assert kh[0] <= kh[1] <= kh[2] <= kh[3] == k                 # top-V accepts everything
        assert kh[0] == verify_prefix(block, views, accept_exact)
        kd = [verify_prefix(block, views, accept_distance(e)) for e in (0, 1, 2, 10)]
        assert kd[0] <= kd[1] <= kd[2] <= kd[3] == k
        # by definition: proposal 2 is accepted under top-n iff fewer than n tokens beat it
        row = logits[0, 0]
        beats = sum(1 for v in range(11) if (row[v], -v) > (row[tail[0]], -tail[0]))
        for n, got in zip((1, 2, 3), kh):
            assert (got >= 2) == (beats < n)
    # a decode under top-3: every emitted token is a proposal that ranked < 3 (or a p_1 argmax), and the
    # merged and two-call forms agree
    tails = list(itertools.product(range(11), repeat=3))
    fn = lambda j, it: tails[(7 * it + j) % len(tails)]
    a = blockwise_merged(TransformerScorer(m, src), k, 14, tail_fn=fn, accept=accept_topn(3))
    b = blockwise_twocall(TransformerScorer(m, src), k, 14, tail_fn=fn, accept=accept_topn(3))
    assert a.ids == b.ids and a.khats == b.khats
    sc2 = TransformerScorer(m, src)
    for t in range(14):
        lg = sc2.logits([0] + a.ids[:t], 1)[0, 0]
        assert P1View(logits=lg).rank(a.ids[t]) < 3

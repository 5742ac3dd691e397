"""Pins for the oracle's decode loops: what Sections 2-4 and 7.4 of the paper
fix (greedy equivalence, khat >= 1, invocation counts, the figures' narratives,
the worked trace) plus brute force on tiny vocabularies.  CPU only."""
import itertools
import os

import numpy as np
import pytest

from bpd_inputs import (DTYPE_F32, ModelConfig, forced_tail, geometric_schedule, make_weights)
from oracle.decode import (TransformerScorer, blockwise_merged, blockwise_twocall, clip_termination,
                           greedy, verify_prefix)
from oracle.model import parse_blob

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    rows = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            if parts[0].lstrip("-").isdigit():
                rows.append([int(p) for p in parts])
            else:
                out[parts[0]] = [int(p) for p in parts[1:]]
    out["rows"] = rows
    return out


class HashModel:
    """A toy autoregressive 'model': p_1's argmax is a hash of the whole prefix
    (so any bookkeeping slip changes the continuation); head i proposes the true
    i-step-ahead greedy token with probability ``agree`` and a wrong one otherwise."""

    def __init__(self, vocab, k, agree, seed):
        self.V, self.k, self.agree, self.seed = vocab, k, agree, seed
        self.calls = 0

    def _p1(self, prefix):
        h = self.seed
        for t in prefix:
            h = (h * 1000003 + t + 12345) % 2147483647
        return h % self.V

    def _row(self, prefix):
        row, ext = [], list(prefix)
        for i in range(self.k):
            true = self._p1(ext)
            coin = (self._p1(list(prefix) + [977 + i]) % 1000) / 1000.0
            row.append(true if (i == 0 or coin < self.agree) else (true + 1 + i) % self.V)
            ext.append(true)
        return row

    def __call__(self, dec_inputs, n_new):
        self.calls += 1
        n = len(dec_inputs)
        return [self._row(dec_inputs[:t + 1]) for t in range(n - n_new, n)]


# ---------------------------------------------------------------- figures and trace

def test_figures_1_and_2_replay():
    g = _read_golden("figures_1_2_tables.txt")
    block, table = g["block"], [g["row1"], g["row2"], g["row3"]]
    khat = verify_prefix(block, lambda i: [table[i - 2][0]])
    assert khat == g["khat"][0] == 2
    assert table[khat - 1] == g["next_block"]
    # through the loop: a scripted model that answers exactly these tables
    calls = []

    def invoke(inputs, n_new):
        calls.append((list(inputs), n_new))
        if n_new == 1:
            return [block]
        return table

    res = blockwise_merged(invoke, 3, n_max=2)
    assert res.ids == block[:2] and res.khats == [2] and res.invocations == 2
    assert calls[1] == ([0] + block, 3)


def test_section_7_4_trace_bookkeeping():
    g = _read_golden("trace_section_7_4.txt")
    k, plan = g["k"][0], g["accepted"]
    EOS = 1
    total = sum(plan)
    seq = [2 + t for t in range(total - 1)] + [EOS] + [500 + t for t in range(2 * k)]
    starts = list(itertools.accumulate([0] + plan))[:-1]
    # at the position that starts step n, heads 1..L_n are right, the rest wrong; the
    # last step's heads are right beyond the EOS so only the EOS rule can stop it
    right = {s: (L if n < len(plan) - 1 else k) for n, (s, L) in enumerate(zip(starts, plan))}

    def invoke(inputs, n_new):
        rows = []
        for t in range(len(inputs) - n_new, len(inputs)):
            L = right.get(t, 1)
            rows.append([seq[t + i] if i < L else 9000 + i for i in range(k)])
        return rows

    res = blockwise_merged(invoke, k, n_max=1000, eos=EOS)
    assert res.khats == plan
    assert len(res.ids) == g["total_tokens"][0] == 34
    assert res.iterations == g["steps"][0] == 6
    assert res.invocations == 7
    assert res.ids[-1] == EOS and res.ids == seq[:total]
    assert round(res.mean_block, 2) == 5.67
    assert plan[g["eos_step"][0] - 1] == g["eos_index_in_block"][0]


def test_invocation_counts_with_perfect_proposals():
    for m_len, k, n_greedy, n_two, n_merged in _read_golden("invocation_counts.txt")["rows"]:
        model = HashModel(vocab=97, k=k, agree=1.1, seed=m_len)
        g = greedy(model, m_len)
        assert g.invocations == n_greedy == m_len
        two = blockwise_twocall(HashModel(97, k, 1.1, m_len), k, m_len)
        mer = blockwise_merged(HashModel(97, k, 1.1, m_len), k, m_len)
        assert two.ids == g.ids and mer.ids == g.ids
        assert two.invocations == n_two and mer.invocations == n_merged
        assert mer.iterations == -(-m_len // k)


# ---------------------------------------------------------------- guarantees of Section 3

@pytest.mark.parametrize("k", [1, 2, 4, 8, 10])
@pytest.mark.parametrize("agree", [0.0, 0.5, 0.9])
def test_blockwise_equals_greedy_for_arbitrary_heads(k, agree):
    for seed in range(6):
        n = 37 + seed
        g = greedy(HashModel(50, k, agree, seed), n)
        mer = blockwise_merged(HashModel(50, k, agree, seed), k, n)
        two = blockwise_twocall(HashModel(50, k, agree, seed), k, n)
        assert mer.ids == g.ids and two.ids == g.ids
        assert mer.khats == two.khats                      # merging changes cost, not behaviour
        assert all(1 <= x <= k for x in mer.khats) and mer.iterations <= n
        assert sum(mer.khats) == n
        assert two.invocations == 2 * two.iterations and mer.invocations == mer.iterations + 1
        if k == 1:
            assert mer.khats == [1] * n
        if agree == 0.0:
            assert mer.khats == [1] * n


def test_eos_and_length_clipping():
    assert clip_termination([5, 6, 7, 8], 4, j=10, n_max=12, eos=-1) == (2, True)
    assert clip_termination([5, 6, 7, 8], 3, j=0, n_max=12, eos=7) == (3, True)
    assert clip_termination([5, 6, 7, 8], 2, j=0, n_max=12, eos=7) == (2, False)   # EOS not accepted
    assert clip_termination([7, 6, 7, 8], 4, j=0, n_max=12, eos=7) == (1, True)
    for eos_at in (0, 3, 11):
        m = HashModel(30, 4, 0.8, seed=eos_at)
        g = greedy(m, 12)
        eos = g.ids[eos_at]
        first = g.ids.index(eos)
        ge = greedy(HashModel(30, 4, 0.8, eos_at), 12, eos=eos)
        be = blockwise_merged(HashModel(30, 4, 0.8, eos_at), 4, 12, eos=eos)
        assert ge.ids == g.ids[:first + 1] == be.ids


# ---------------------------------------------------------------- the real (tiny) Transformer

def _tiny(V, k, seed=21, layout=0):
    cfg = ModelConfig(1, 2, 16, 2, 32, V, k, 24, dtype=DTYPE_F32, head_layout=layout)
    return parse_blob(make_weights(cfg, seed, 0.5))


@pytest.mark.parametrize("layout", [0, 1])
def test_transformer_blockwise_equals_greedy_and_cached_equals_uncached(layout):
    m = _tiny(23, 4, layout=layout)
    src = [3, 9, 4, 11, 2]
    n = 14
    g = greedy(TransformerScorer(m, src), n)
    gc = greedy(TransformerScorer(m, src, cached=True, capacity=n + 8), n)
    mer = blockwise_merged(TransformerScorer(m, src), 4, n)
    merc = blockwise_merged(TransformerScorer(m, src, cached=True, capacity=n + 8), 4, n)
    two = blockwise_twocall(TransformerScorer(m, src, cached=True, capacity=n + 8), 4, n)
    assert g.ids == gc.ids == mer.ids == merc.ids == two.ids
    assert mer.khats == merc.khats == two.khats
    k2 = blockwise_merged(TransformerScorer(m, src, k=2), 2, n)
    assert k2.ids == g.ids


@pytest.mark.parametrize("V,k", [(3, 2), (3, 3), (5, 2), (5, 3)])
def test_brute_force_all_tails_tiny_vocab(V, k):
    m = _tiny(V, k, seed=40 + V + k)
    src = [1, 2, 0, 1]
    n = 6
    sc = TransformerScorer(m, src)
    g = greedy(sc, n + k).ids           # continuation long enough for every block
    for j in range(n):
        inputs = [0] + g[:j]
        full = 0
        for tail in itertools.product(range(V), repeat=k - 1):
            block = [g[j]] + list(tail)
            table = sc(inputs + block, k)
            khat = verify_prefix(block, lambda i: [table[i - 2][0]])
            lcp = 0
            while lcp < k - 1 and tail[lcp] == g[j + 1 + lcp]:
                lcp += 1
            assert khat == 1 + lcp
            full += (khat == k)
        assert full == 1                  # exactly one tail is accepted whole
    # and a decode that cycles through the tails still ends at the greedy output
    tails = list(itertools.product(range(V), repeat=k - 1))
    res = blockwise_merged(TransformerScorer(m, src), k, n, tail_fn=lambda j, it: tails[(3 * it + j) % len(tails)])
    assert res.ids == g[:n]


def test_controlled_acceptance_schedule_is_exact():
    m = _tiny(23, 4, seed=77)
    src = [5, 6, 7]
    n, k = 20, 4
    g = np.array(greedy(TransformerScorer(m, src), n).ids)
    G, R = geometric_schedule(3001, 2.0, 64)
    res = blockwise_merged(TransformerScorer(m, src), k, n,
                           tail_fn=lambda j, it: forced_tail(g, j, k, int(G[it]), int(R[it]), m.V))
    assert res.ids == list(g)
    j = 0
    for it, kh in enumerate(res.khats):
        assert kh == min(k, int(G[it]), n - j)
        j += kh
    # closed form E[min(k, G)] = (1 - (1-p)^k) / p
    for mean, kk, want in [(2.0, 4, 1.875), (2.0, 8, 1.992), (5.0, 8, 4.161), (5.0, 10, 4.463)]:
        GG, _ = geometric_schedule(9, mean, 400000)
        p = 1.0 / mean
        assert abs((1 - (1 - p) ** kk) / p - want) < 6e-4
        assert abs(np.minimum(GG, kk).mean() - want) < 0.02

"""GPU parity: the CUDA library against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from bpd_inputs import (DTYPE_BF16, DTYPE_F32, HEAD_BLOCKDIAG, HEAD_DENSE, WORKLOADS, ModelConfig, Workload,
                        forced_tail, geometric_schedule, make_source, make_weights)

pytestmark = pytest.mark.gpu

MINI = Workload("mini", ModelConfig(2, 2, 128, 2, 256, 1000, 4, 256, dtype=DTYPE_BF16), 0.05,
                11, 12, 13, batch=1, src_lo=9, src_hi=9, n_decode=24)
MINI_BLOCK = MINI.with_layout(HEAD_BLOCKDIAG)
MINI_BATCH = Workload("mini3", MINI.cfg, 0.05, 11, 22, 23, batch=3, src_lo=3, src_hi=11, n_decode=20)
# shapes the three-launches-per-layer decoder path takes (head width 64, d_model a multiple of 256)
MIDI = Workload("midi", ModelConfig(2, 2, 256, 4, 512, 1000, 4, 256, dtype=DTYPE_BF16), 0.05,
                41, 42, 43, batch=1, src_lo=9, src_hi=9, n_decode=24)
MIDI_BATCH = Workload("midi3", MIDI.cfg, 0.05, 41, 52, 53, batch=3, src_lo=3, src_hi=11, n_decode=20)
MINI_F32 = Workload("minif", ModelConfig(1, 2, 96, 6, 200, 333, 3, 136, dtype=DTYPE_F32), 0.1,
                    31, 32, 33, batch=2, src_lo=2, src_hi=7, n_decode=15)


LAYER_PATHS = {
    "persistent": {"persistent_layers": 1},                       # one kernel for the whole layer stack
    "cluster": {"persistent_layers": 0},                          # three cluster launches per layer
    "per-projection": {"persistent_layers": 0, "cluster_layers": 0},
}


@pytest.fixture(scope="module")
def bpd():
    import paper_1811_03115_b200 as pkg
    return pkg


def _setup(bpd, w, extra_tgt=0):
    from oracle.model import parse_blob
    blob = make_weights(w.cfg, w.weight_seed, w.sigma)
    model = bpd.Model(blob)
    src, src_len = make_source(w)
    return blob, model, src, src_len, parse_blob(blob)


def _tail_fn(w, greedy_ids, k, mean):
    sched = [geometric_schedule(w.accept_seed * 1000 + b, mean, w.n_decode + 1) for b in range(w.batch)]

    def fn(b, j, it):
        G, R = sched[b]
        jj = min(j, w.n_decode)
        return forced_tail(greedy_ids[b], jj, k, int(G[jj]), int(R[jj]), w.cfg.vocab)
    return fn, sched


def _plan(w, greedy_ids, k, mean):
    fn, sched = _tail_fn(w, greedy_ids, k, mean)
    plan = np.zeros((w.batch, w.n_decode, k - 1), dtype=np.int32)
    for b in range(w.batch):
        for j in range(w.n_decode):
            plan[b, j] = fn(b, j, 0)
    return plan, sched


def _expected_khats(sched_b, k, n):
    G, _ = sched_b
    j, out = 0, []
    while j < n:
        kh = min(k, int(G[j]), n - j)
        out.append(kh)
        j += kh
    return out


# ---------------------------------------------------------------- single operators

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,in_f,out_f", [(1, 64, 50), (8, 1024, 3072), (13, 520, 77), (64, 256, 129), (64, 256, 384),
                                             (100, 512, 1024), (40, 2048, 132)])
def test_op_linear_matches_definition(bpd, dtype, rows, in_f, out_f):
    import torch
    g = torch.Generator().manual_seed(rows * 1000 + in_f)
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    x = (torch.randn(rows, in_f, generator=g)).to(td)
    w = (torch.randn(out_f, in_f, generator=g) * 0.05).to(td)
    b = (torch.randn(out_f, generator=g) * 0.1).to(td)
    want = x.double().numpy() @ w.double().numpy().T + b.double().numpy()
    y = bpd.bpd_op_linear(x.cuda(), w.cuda(), b.cuda(), relu=False).cpu().numpy()
    np.testing.assert_allclose(y, want, atol=2e-4 * np.sqrt(in_f / 64))
    y = bpd.bpd_op_linear(x.cuda(), w.cuda(), None, relu=True).cpu().numpy()
    np.testing.assert_allclose(y, np.maximum(want - b.double().numpy(), 0), atol=2e-4 * np.sqrt(in_f / 64))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,d,vocab", [(1, 64, 5), (16, 512, 1000), (64, 1024, 32768), (9, 128, 257)])
def test_op_vocab_argmax_matches_definition(bpd, dtype, rows, d, vocab):
    import torch
    from oracle.model import argmax_lowest
    g = torch.Generator().manual_seed(rows + d + vocab)
    td = torch.float32 if dtype == "f32" else torch.bfloat16
    x = torch.randn(rows, d, generator=g).to(td)
    w = (torch.randn(vocab, d, generator=g) * 0.02).to(td)
    if vocab > 8:
        w[7] = w[3]                      # an exact tie: the lower id must win if it is the maximum
        x[0] = (w[3].float() * 50).to(td)
    logits = x.double().numpy() @ w.double().numpy().T
    idx, val = bpd.bpd_op_vocab_argmax(x.cuda(), w.cuda(), want_val=True)
    idx, val = idx.cpu().numpy(), val.cpu().numpy()
    want = argmax_lowest(logits)
    best = logits.max(-1)
    for r in range(rows):
        second = np.partition(logits[r], -2)[-2] if vocab > 1 else -np.inf
        if best[r] - second > 1e-3:
            assert idx[r] == want[r]
        assert abs(logits[r, idx[r]] - best[r]) <= 1e-3
        assert abs(val[r] - best[r]) <= 1e-3
    if vocab > 8:
        assert idx[0] == 3
    # a second call on the same scratch-free path gives the same answer (counters were reset)
    idx2 = bpd.bpd_op_vocab_argmax(x.cuda(), w.cuda()).cpu().numpy()
    assert np.array_equal(idx, idx2)


# ---------------------------------------------------------------- whole path, small models

@pytest.mark.parametrize("w", [WORKLOADS["C1"], MINI, MINI_BLOCK, MINI_BATCH, MINI_F32, MIDI, MIDI_BATCH],
                         ids=lambda w: w.name)
def test_greedy_blockwise_and_lockstep(bpd, w):
    from harness import lockstep
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    # greedy, then blockwise: identical ids (the guarantee of Section 3), on the GPU alone
    s.bpd_encode(src, src_len)
    g_ids, g_len, g_st = s.bpd_decode_greedy(N)
    assert np.all(g_len == N) and g_st.tokens == N * w.batch and g_st.invocations == N
    for kk in sorted({1, 2, k}):
        s.bpd_encode(src, src_len)
        b_ids, b_len, b_st = s.bpd_decode_blockwise(kk, N)
        assert np.array_equal(b_ids, g_ids), f"k={kk}: blockwise differs from greedy"
        assert b_st.tokens == N * w.batch and b_st.invocations == b_st.iterations + 1
        assert sum(c * n for c, n in enumerate(b_st.khat_hist)) == N * w.batch
        if kk == 1:
            assert b_st.iterations == N
    # controlled acceptance through the device-resident plan: khat is known in advance
    for mean in (2.0, 5.0):
        plan, sched = _plan(w, g_ids, k, mean)
        s.bpd_encode(src, src_len)
        s.bpd_set_forced_plan(plan, k)
        p_ids, _, p_st = s.bpd_decode_blockwise(k, N)
        assert np.array_equal(p_ids, g_ids)
        want = [_expected_khats(sched[b], k, N) for b in range(w.batch)]
        hist = np.zeros(17, dtype=np.int64)
        for row in want:
            for kh in row:
                hist[kh] += 1
        assert list(hist) == list(p_st.khat_hist)
        assert p_st.iterations == max(len(r) for r in want)
        assert p_st.row_iterations == sum(len(r) for r in want)
    # lock-step against the oracle: free-running, then with forced tails
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N)
    for b in range(w.batch):
        assert rep.emitted[b] == list(g_ids[b]), "lock-step output differs from the GPU's greedy decode"
    if w.cfg.dtype == DTYPE_F32:
        assert rep.adopted == 0
    fn, sched = _tail_fn(w, g_ids, k, 2.0)
    rep2 = lockstep(s, om, src, src_len, k, N, max_iters=N, tail_fn=fn)
    for b in range(w.batch):
        assert [r[b] for r in rep2.khats if r[b] > 0] == _expected_khats(sched[b], k, N)
    s.close()
    model.close()


def test_c1_ids_equal_oracle_greedy(bpd):
    """fp32 weights: the GPU's greedy and blockwise ids are the oracle's greedy ids."""
    from oracle.decode import TransformerScorer, blockwise_merged, greedy
    w = WORKLOADS["C1"]
    blob, model, src, src_len, om = _setup(bpd, w)
    s = bpd.Session(model, 1, w.max_src, w.n_decode)
    s.bpd_encode(src, src_len)
    ids, _, _ = s.bpd_decode_blockwise(4, w.n_decode)
    sc = TransformerScorer(om, src[0, :src_len[0]], cached=True, capacity=w.n_decode + 12)
    want = greedy(sc, w.n_decode)
    assert list(ids[0]) == want.ids
    ob = blockwise_merged(TransformerScorer(om, src[0, :src_len[0]], cached=True, capacity=w.n_decode + 12),
                          4, w.n_decode)
    s.bpd_encode(src, src_len)
    _, _, st = s.bpd_decode_blockwise(4, w.n_decode)
    assert st.iterations == ob.iterations and st.invocations == ob.invocations
    s.close()
    model.close()


def test_eos_terminates_inside_a_block(bpd):
    w = MINI
    blob, model, src, src_len, om = _setup(bpd, w)
    N, k = w.n_decode, 4
    s = bpd.Session(model, 1, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    eos_at = 6
    eos = int(g_ids[0, eos_at])
    first = list(g_ids[0]).index(eos)
    plan = np.zeros((1, N, k - 1), dtype=np.int32)
    for j in range(N):
        plan[0, j] = forced_tail(g_ids[0], j, k, k, 0, w.cfg.vocab)     # always-right proposals
    s.bpd_encode(src, src_len)
    s.bpd_set_forced_plan(plan, k)
    ids, ln, st = s.bpd_decode_blockwise(k, N, eos_id=eos)
    assert ln[0] == first + 1 and list(ids[0, :first + 1]) == list(g_ids[0, :first + 1])
    assert np.all(ids[0, first + 1:] == -1)
    assert st.iterations == -(-(first + 1) // k)
    s.bpd_encode(src, src_len)
    ids2, ln2, _ = s.bpd_decode_greedy(N, eos_id=eos)
    assert ln2[0] == first + 1 and np.array_equal(ids2, ids)
    s.close()
    model.close()


def test_a_smaller_max_new_later_on_finishes_the_row(bpd):
    """bpd_iteration takes max_new per call.  A later call with max_new at or below what a row already holds must
    mark the row finished and change nothing else (no negative block size, no writes before the tables)."""
    w = MINI_BATCH
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    s.bpd_encode(src, src_len)
    for _ in range(4):
        s.bpd_iteration(k, N)
    ids0, len0, st0 = s.bpd_fetch_output(N)
    assert np.all(len0 >= 4)
    r = s.bpd_iteration(k, 2)                      # every row already holds more than 2 tokens
    assert np.all(r["khat"] == 0)
    ids1, len1, st1 = s.bpd_fetch_output(N)
    assert np.array_equal(ids1, ids0) and np.array_equal(len1, len0)
    assert st1.tokens == st0.tokens and st1.khat_hist == st0.khat_hist
    r = s.bpd_iteration(k, N)                      # finished rows stay finished
    assert np.all(r["khat"] == 0)
    s.close()
    model.close()


def test_state_and_argument_errors(bpd):
    w = MINI
    blob, model, src, src_len, _ = _setup(bpd, w)
    s = bpd.Session(model, 1, w.max_src, 16)
    with pytest.raises(bpd.BpdError) as e:
        s.bpd_decode_greedy(8)
    assert e.value.status == -5
    s.bpd_encode(src, src_len)
    with pytest.raises(bpd.BpdError) as e:
        s.bpd_decode_blockwise(5, 8)          # k above k_model
    assert e.value.status == -1
    with pytest.raises(bpd.BpdError) as e:
        s.bpd_decode_greedy(17)               # above max_tgt
    assert e.value.status == -2
    bad = src.copy()
    bad[0, 0] = w.cfg.vocab
    with pytest.raises(bpd.BpdError) as e:
        s.bpd_encode(bad, src_len)
    assert e.value.status == -1
    s.bpd_encode(src, src_len)
    s.bpd_decode_greedy(8)
    with pytest.raises(bpd.BpdError) as e:
        s.bpd_iteration(4, 8)                 # greedy session cannot continue blockwise
    assert e.value.status == -5
    s.close()
    model.close()


# ---------------------------------------------------------------- paper-sized configurations

def _full_size(bpd, name, iters, rows=None, layout=HEAD_DENSE, mean=2.0, free_iters=2, layer_path=None):
    from harness import lockstep
    w = (WORKLOADS[name] if isinstance(name, str) else name).with_layout(layout)
    blob, model, src, src_len, om = _setup(bpd, w)
    del blob
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    if layer_path is not None:
        assert s.layer_path == layer_path, f"expected layer path {layer_path}, got {s.layer_path}"
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    s.bpd_encode(src, src_len)
    b_ids, _, b_st = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(b_ids, g_ids)
    plan, sched = _plan(w, g_ids, k, mean)
    s.bpd_encode(src, src_len)
    s.bpd_set_forced_plan(plan, k)
    p_ids, _, p_st = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(p_ids, g_ids)
    want = [_expected_khats(sched[b], k, N) for b in range(w.batch)]
    assert p_st.row_iterations == sum(len(r) for r in want)
    assert p_st.iterations == max(len(r) for r in want)
    rep = lockstep(s, om, src, src_len, k, N, max_iters=free_iters, rows=rows)
    fn, _ = _tail_fn(w, g_ids, k, mean)
    rep2 = lockstep(s, om, src, src_len, k, N, max_iters=iters, tail_fn=fn, rows=rows)
    for b in (rows if rows is not None else range(w.batch)):
        got = [r[i] for r in rep2.khats for i, bb in enumerate(rows if rows is not None else range(w.batch)) if bb == b]
        assert got == want[b][:len(got)]
    s.close()
    model.close()
    return rep, rep2


def test_c2_base_model(bpd):
    _full_size(bpd, "C2", iters=6)


def test_c2_base_model_blockdiag(bpd):
    _full_size(bpd, "C2", iters=3, layout=HEAD_BLOCKDIAG)


def test_c3_big_model(bpd):
    _full_size(bpd, "C3", iters=3, mean=5.0, free_iters=1)


def test_c3_model_two_sequences_sixteen_rows(bpd):
    """The big model with two sequences of different source lengths: 16 rows per pass, the widest pass of the
    few-row layer paths (two token tiles of 8 rows, 16 heads; the working buffers of two token tiles leave the
    persistent kernel no room beside a second CTA on the SM, so such a session runs the cluster launches)."""
    c3 = WORKLOADS["C3"]
    w = Workload("c3x2", c3.cfg, c3.sigma, c3.weight_seed, 2103, 3103, batch=2, src_lo=23, src_hi=40, n_decode=40)
    _full_size(bpd, w, iters=4, mean=5.0, free_iters=1, layer_path=1)


def test_c5_super_resolution_shape(bpd):
    _full_size(bpd, "C5", iters=3, mean=5.0, free_iters=1)


def test_c5_local_attention_deep_into_the_sequence(bpd):
    """The super-resolution shape with 1D local attention (query blocks of 256, memory 256), followed in lock-step
    with every proposal accepted until position 1100: by then the window starts at 768 and 24 chunks of 32 keys
    lie outside it."""
    from harness import lockstep
    w = WORKLOADS["C5L"]
    blob, model, src, src_len, om = _setup(bpd, w)
    del blob
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    s.bpd_encode(src, src_len)
    b_ids, _, _ = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(b_ids, g_ids)

    def all_accepted(b, j, it):
        return forced_tail(g_ids[b], min(j, N), k, k, 0, w.cfg.vocab)
    rep = lockstep(s, om, src, src_len, k, N, max_iters=110, tail_fn=all_accepted)
    assert sum(r[0] for r in rep.khats) == 1100 and rep.emitted[0] == list(g_ids[0][:1100])
    wf = WORKLOADS["C5"]
    model_f = bpd.Model(make_weights(wf.cfg, wf.weight_seed, wf.sigma))
    sf = bpd.Session(model_f, 1, w.max_src, N)
    sf.bpd_encode(src, src_len)
    f_ids, _, _ = sf.bpd_decode_greedy(N)
    assert np.array_equal(f_ids[0][:256], g_ids[0][:256]) and not np.array_equal(f_ids, g_ids)
    sf.close(); model_f.close(); s.close(); model.close()


def test_c4_batch32_ragged(bpd):
    w = WORKLOADS["C4"]
    _, src_len = make_source(w)
    rows = sorted({int(np.argmin(src_len)), int(np.argmax(src_len)), 0, w.batch - 1})
    _full_size(bpd, "C4", iters=2, rows=rows, mean=2.0, free_iters=1)


# ---------------------------------------------------------------- paper-sized configurations, whole decodes

def _whole_decode(bpd, name, mean, rows=None, check_values=True, all_accepted=False):
    """Lock-step with the oracle from the first iteration to the last token of the configuration's decode, under
    controlled acceptance (or with every proposal accepted): ids under the margin rule, accepted block sizes and
    next blocks exact in every iteration, hidden states and logits within tolerance where they are compared."""
    from harness import lockstep
    w = WORKLOADS[name]
    blob, model, src, src_len, om = _setup(bpd, w)
    del blob
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    if all_accepted:
        def fn(b, j, it):
            return forced_tail(g_ids[b], min(j, N), k, k, 0, w.cfg.vocab)
        want = None
    else:
        fn, sched = _tail_fn(w, g_ids, k, mean)
        want = [_expected_khats(sched[b], k, N) for b in range(w.batch)]
    sel = list(range(w.batch)) if rows is None else rows
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N, tail_fn=fn, rows=rows, check_values=check_values)
    for i, b in enumerate(sel):
        assert rep.emitted[b] == list(g_ids[b]), f"row {b}: lock-step output differs from the GPU's greedy decode"
        got = [r[i] for r in rep.khats if r[i] > 0]
        if want is not None:
            assert got == want[b]
        else:
            assert got == [k] * (N // k) + ([N % k] if N % k else [])
    s.close()
    model.close()
    return rep


@pytest.mark.parametrize("mean", [5.0, 2.0])
def test_c3_whole_decode_in_lockstep(bpd, mean):
    """The headline configuration, all 128 tokens, every iteration compared with the oracle (values too)."""
    rep = _whole_decode(bpd, "C3", mean)
    assert rep.max_logit_err <= 2e-2 and rep.max_hidden_err <= 2e-2


def test_c4_whole_decode_in_lockstep(bpd):
    """Batch 32 with ragged source lengths and per-row acceptance: four rows (shortest and longest source, first and
    last row) followed through all 128 tokens in the launch configuration the benchmark times (two-stage heads)."""
    w = WORKLOADS["C4"]
    _, src_len = make_source(w)
    rows = sorted({int(np.argmin(src_len)), int(np.argmax(src_len)), 0, w.batch - 1})
    _whole_decode(bpd, "C4", 5.0, rows=rows, check_values=False)


def test_c5_whole_image_in_lockstep(bpd):
    """The super-resolution shape through all 3072 positions with every proposal accepted: the self-attention
    schedule switches from one CTA per row to shared keys at 256 visible keys and folds several chunks per lump
    beyond 2048; hidden states and logits are compared with the oracle in every iteration."""
    rep = _whole_decode(bpd, "C5", 0.0, all_accepted=True)
    assert rep.iterations == -(-3072 // 10)


def test_full_attention_beyond_2048_keys(bpd):
    """A small model decoded to 2320 positions with full causal attention: past key 2048 a rank's lumps wrap
    around and hold several chunks each.  Greedy and blockwise agree, and the lock-step against the oracle (values
    in every iteration) runs across the wrap."""
    from harness import lockstep
    w = Workload("midi-2k", MIDI.cfg, 0.05, 41, 42, 43, batch=1, src_lo=9, src_hi=9, n_decode=2320)
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    for path in ("cluster", "persistent"):
        s = bpd.Session(model, w.batch, w.max_src, N, options=LAYER_PATHS[path])
        assert s.layer_path == (2 if path == "persistent" else 1)
        s.bpd_encode(src, src_len)
        g_ids, _, _ = s.bpd_decode_greedy(N)
        s.bpd_encode(src, src_len)
        b_ids, _, _ = s.bpd_decode_blockwise(k, N)
        assert np.array_equal(b_ids, g_ids), path

        def all_accepted(b, j, it):
            return forced_tail(g_ids[b], min(j, N), k, k, 0, w.cfg.vocab)
        rep = lockstep(s, om, src, src_len, k, N, max_iters=N, tail_fn=all_accepted)
        assert rep.emitted[0] == list(g_ids[0]) and rep.iterations == N // k, path
        s.close()
    model.close()


# ---------------------------------------------------------------- approximate acceptance (Section 5)

@pytest.mark.parametrize("accept", [("topn", 2), ("topn", 3), ("distance", 2)], ids=lambda a: f"{a[0]}{a[1]}")
@pytest.mark.parametrize("w", [WORKLOADS["C1"], MINI, MINI_BATCH], ids=lambda w: w.name)
def test_approximate_acceptance_lockstep(bpd, w, accept):
    """Top-n and distance acceptance against the oracle, with forced proposals that straddle the
    acceptance boundary (taken from the oracle's own p_1 ranking)."""
    from harness import lockstep
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    mode = bpd.BPD_ACCEPT_TOPN(accept[1]) if accept[0] == "topn" else bpd.BPD_ACCEPT_DISTANCE(accept[1])
    s = bpd.Session(model, w.batch, w.max_src, N)
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N, accept=accept, accept_mode=mode, near_miss=True)
    flat = [kh for row in rep.khats for kh in row if kh > 0]
    assert max(flat) > 1 and min(flat) < k, "the forced tails should produce both acceptances and rejections"
    for b in range(w.batch):
        assert len(rep.emitted[b]) == N
    s.close()
    model.close()


def test_acceptance_modes_that_reduce_to_exact_and_minimum_block(bpd):
    w = MINI
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, 1, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    for mode in (bpd.BPD_ACCEPT_TOPN(1), bpd.BPD_ACCEPT_DISTANCE(0), bpd.BPD_ACCEPT_MIN_BLOCK(1)):
        s.bpd_encode(src, src_len)
        ids, _, st = s.bpd_decode_blockwise(k, N, accept_mode=mode)
        assert np.array_equal(ids, g_ids)
    # the whole vocabulary as "top n" (n = 255 is the largest the encoding carries): free-running heads on
    # random weights are then accepted far more often than under exact matching
    s.bpd_encode(src, src_len)
    _, _, st_exact = s.bpd_decode_blockwise(k, N)
    s.bpd_encode(src, src_len)
    _, _, st_top = s.bpd_decode_blockwise(k, N, accept_mode=bpd.BPD_ACCEPT_TOPN(255))
    assert st_top.iterations < st_exact.iterations and st_top.tokens == N
    # minimum block size k = fixed-size blocks (Section 5.3): ceil(N / k) iterations whatever the heads say
    s.bpd_encode(src, src_len)
    ids, ln, st = s.bpd_decode_blockwise(k, N, accept_mode=bpd.BPD_ACCEPT_MIN_BLOCK(k))
    assert st.iterations == -(-N // k) and ln[0] == N and st.khat_hist[k] == N // k
    with pytest.raises(bpd.BpdError):
        s.bpd_encode(src, src_len)
        s.bpd_decode_blockwise(k, N, accept_mode=bpd.BPD_ACCEPT_MIN_BLOCK(k + 1))
    with pytest.raises(bpd.BpdError):
        s.bpd_decode_blockwise(k, N, accept_mode=3 << 8)
    s.close()
    model.close()


def test_minimum_block_lockstep(bpd):
    from harness import lockstep
    w = MINI_F32
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N, accept=("topn", 2), near_miss=True, min_block=2,
                   accept_mode=bpd.BPD_ACCEPT_TOPN(2) | bpd.BPD_ACCEPT_MIN_BLOCK(2))
    assert all(kh >= 2 or kh == 0 for row in rep.khats[:-1] for kh in row)
    s.close()
    model.close()


# ---------------------------------------------------------------- lazy (two-stage) head evaluation

@pytest.mark.parametrize("w", [MINI, MINI_BLOCK, MINI_BATCH], ids=lambda w: w.name)
def test_lazy_heads_give_the_same_decode(bpd, w):
    """p_1 at every position first, all heads only at the accepted position: same ids, same accepted
    block sizes, same next blocks as the one-stage evaluation and as the oracle."""
    from harness import lockstep
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s0 = bpd.Session(model, w.batch, w.max_src, N)
    s0.bpd_encode(src, src_len)
    g_ids, _, _ = s0.bpd_decode_greedy(N)
    plan, sched = _plan(w, g_ids, k, 2.0)
    s0.bpd_encode(src, src_len)
    s0.bpd_set_forced_plan(plan, k)
    _, _, st0 = s0.bpd_decode_blockwise(k, N)
    s0.close()
    s = bpd.Session(model, w.batch, w.max_src, N, options={"lazy_heads": 1})
    s.bpd_encode(src, src_len)
    ids, _, _ = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(ids, g_ids)
    s.bpd_encode(src, src_len)
    s.bpd_set_forced_plan(plan, k)
    ids, _, st = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(ids, g_ids) and st.khat_hist == st0.khat_hist and st.iterations == st0.iterations
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N, check_values=False)
    for b in range(w.batch):
        assert rep.emitted[b] == list(g_ids[b])
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N, check_values=False, accept=("topn", 2),
                   accept_mode=bpd.BPD_ACCEPT_TOPN(2), near_miss=True)
    assert max(kh for row in rep.khats for kh in row) > 1
    s.close()
    model.close()



@pytest.mark.parametrize("w", [MIDI, MIDI_BATCH], ids=lambda w: w.name)
def test_layer_paths_agree(bpd, w):
    """Sessions with few rows run each decoder layer as three cluster launches (one cluster per head); the same
    sessions can also run all layers in one persistent kernel or one kernel per projection.  The sums are split
    differently, so the three agree to fp32 rounding of bf16-weight products, far inside the oracle tolerance --
    hidden states after every layer, decoder outputs and logits."""
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode

    def run(options, path):
        s = bpd.Session(model, w.batch, w.max_src, N, options=options)
        assert s.layer_path == path, f"asked for {options}, got layer path {s.layer_path}"
        s.bpd_encode(src, src_len)
        steps = []
        for _ in range(4):
            r = s.bpd_iteration(k, N, want_logits=True, want_hidden=True, want_layers=True)
            steps.append((r["hidden"].cpu().numpy().copy(), r["logits"].cpu().numpy().copy(),
                          r["layers"].cpu().numpy().copy()))
        s.close()
        return steps

    ref = run(LAYER_PATHS["per-projection"], 0)
    for name, path in (("persistent", 2), ("cluster", 1)):
        got = run(LAYER_PATHS[name], path)
        for it, ((ha, la, xa), (hb, lb, xb)) in enumerate(zip(got, ref)):
            assert np.abs(xa - xb).max() <= 2e-3, f"{name}, iteration {it}: residual stream differs"
            assert np.abs(ha - hb).max() <= 2e-3 and np.abs(la - lb).max() <= 2e-3, f"{name}, iteration {it}"
    model.close()


def test_layer_dump_matches_the_oracle(bpd):
    """The residual stream after every decoder layer (the debug dump of bpd_iteration) against the oracle's."""
    from oracle.decode import TransformerScorer
    w = MIDI
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    for name, options in LAYER_PATHS.items():
        s = bpd.Session(model, 1, w.max_src, N, options=options)
        assert s.layer_path == {"persistent": 2, "cluster": 1, "per-projection": 0}[name]
        s.bpd_encode(src, src_len)
        s.bpd_iteration(k, N)
        r = s.bpd_iteration(k, N, want_layers=True)
        ids, _, _ = s.bpd_fetch_output(N)
        sc = TransformerScorer(om, src[0, :src_len[0]], k=k)
        n_prev = int(np.sum(ids[0] >= 0)) - int(r["khat"][0])
        inputs = [0] + [int(t) for t in ids[0][:n_prev]] + [int(t) for t in r["block"][0]]
        want = sc.layer_outputs(inputs, k)                                  # [n_dec, k, d]
        got = r["layers"].cpu().numpy()[:, 0]
        assert got.shape == want.shape
        err = np.abs(got - want).max(axis=-1)
        assert err.max() <= 2e-2, (f"{name}: layer outputs differ, per (layer, row): {err.round(4).tolist()}; inputs {inputs}, "
                                   f"khat {r['khat']}")
        s.close()
    model.close()


@pytest.mark.parametrize("path", ["persistent", "cluster"])
@pytest.mark.parametrize("w", [MIDI, MIDI_BATCH, MINI_BATCH], ids=lambda w: w.name)
def test_staged_encoder_rows_change_nothing(bpd, w, path):
    """Cross-attention normally reads the encoder's keys and values from shared memory, where they were copied
    ahead of time; sources too long for that are read from L2.  Both routes do the same arithmetic in the same
    order: same hidden states, logits and ids."""
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode

    def run(extra):
        s = bpd.Session(model, w.batch, w.max_src, N, options=dict(LAYER_PATHS[path], **extra))
        s.bpd_encode(src, src_len)
        r = s.bpd_iteration(k, N, want_logits=True, want_hidden=True)
        r = s.bpd_iteration(k, N, want_logits=True, want_hidden=True)
        hidden, logits = r["hidden"].cpu().numpy().copy(), r["logits"].cpu().numpy().copy()
        s.bpd_encode(src, src_len)
        ids, _, _ = s.bpd_decode_blockwise(k, N)
        s.close()
        return hidden, logits, ids
    h_a, l_a, ids_a = run({})
    h_b, l_b, ids_b = run({"stage_encoder_rows": 0})
    assert np.array_equal(h_a, h_b) and np.array_equal(l_a, l_b) and np.array_equal(ids_a, ids_b)
    model.close()


def test_one_session_per_device_takes_the_persistent_kernel(bpd):
    """Two persistent layer kernels running at once could keep each other's clusters off the SMs, so the library
    gives that kernel to one live session per device: a second session created meanwhile runs the cluster launches,
    decodes the same ids, and the kernel is free again once its holder is closed."""
    w = MIDI
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    a = bpd.Session(model, w.batch, w.max_src, N)
    b = bpd.Session(model, w.batch, w.max_src, N)
    assert (a.layer_path, b.layer_path) == (2, 1)
    forced = bpd.Session(model, w.batch, w.max_src, N, options=LAYER_PATHS["persistent"])
    assert forced.layer_path == 2                 # an explicit request is honoured
    forced.close()
    ids = []
    for s in (a, b, a, b):                        # decodes of the two sessions follow one another on one stream
        s.bpd_encode(src, src_len)
        ids.append(s.bpd_decode_blockwise(k, N)[0])
    assert np.array_equal(ids[0], ids[2]) and np.array_equal(ids[1], ids[3])
    b.bpd_encode(src, src_len)
    assert np.array_equal(b.bpd_decode_greedy(N)[0], ids[1])
    a.close()
    c = bpd.Session(model, w.batch, w.max_src, N)
    assert c.layer_path == 2
    c.close(); b.close(); model.close()


def test_same_decode_twice_gives_identical_ids(bpd):
    """Every reduction has a fixed order: decoding the same input twice gives bit-identical hidden states and ids
    (an order-dependent reduction -- a race between CTAs -- would show up as a difference)."""
    for w in (MIDI_BATCH, MINI_BATCH):
        blob, model, src, src_len, om = _setup(bpd, w)
        k, N = w.cfg.k_model, w.n_decode
        s = bpd.Session(model, w.batch, w.max_src, N)
        outs = []
        for _ in range(3):
            s.bpd_encode(src, src_len)
            r = s.bpd_iteration(k, N, want_hidden=True, want_logits=True)
            hid, lg = r["hidden"].cpu().numpy().copy(), r["logits"].cpu().numpy().copy()
            s.bpd_encode(src, src_len)
            ids, _, _ = s.bpd_decode_blockwise(k, N)
            outs.append((hid, lg, ids))
        for hid, lg, ids in outs[1:]:
            assert np.array_equal(hid, outs[0][0]) and np.array_equal(lg, outs[0][1]) and np.array_equal(ids, outs[0][2])
        s.close()
        model.close()


# 1D local attention (query blocks of local_q positions + local_m positions of memory), one model per attention kernel
_LOC = dict(local_q=8, local_m=20)
LOCAL_MODELS = [
    Workload("local-fused", ModelConfig(2, 2, 256, 4, 512, 1000, 4, 256, dtype=DTYPE_BF16, **_LOC), 0.05,
             61, 62, 63, batch=1, src_lo=9, src_hi=9, n_decode=72),
    Workload("local-split", ModelConfig(2, 2, 128, 2, 256, 1000, 4, 256, dtype=DTYPE_BF16, **_LOC), 0.05,
             64, 65, 66, batch=2, src_lo=5, src_hi=9, n_decode=72),
    Workload("local-generic", ModelConfig(1, 2, 96, 4, 200, 333, 3, 136, dtype=DTYPE_F32, local_q=5, local_m=9), 0.1,
             67, 68, 69, batch=2, src_lo=2, src_hi=7, n_decode=48),
    Workload("local-seq", ModelConfig(1, 2, 128, 2, 256, 500, 4, 128, dtype=DTYPE_BF16, **_LOC), 0.05,
             70, 71, 72, batch=8, src_lo=3, src_hi=8, n_decode=44),
    Workload("local-rows", ModelConfig(1, 2, 128, 1, 256, 500, 4, 128, dtype=DTYPE_BF16, **_LOC), 0.05,
             73, 74, 75, batch=8, src_lo=3, src_hi=8, n_decode=44),
]


@pytest.mark.parametrize("w", LOCAL_MODELS, ids=lambda w: w.name)
def test_local_attention_lockstep(bpd, w):
    """Section 7.2's model class: decoder self-attention restricted to the query's block and a fixed memory
    before it.  Every attention kernel (cluster path, split, generic, per-sequence, per-row) against the oracle,
    decoding far enough that whole 32-key chunks fall out of the window."""
    from harness import lockstep
    blob, model, src, src_len, om = _setup(bpd, w)
    assert om.local_q == w.cfg.local_q and om.local_m == w.cfg.local_m
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    s.bpd_encode(src, src_len)
    b_ids, _, _ = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(b_ids, g_ids)
    fn, sched = _tail_fn(w, g_ids, k, 3.0)
    rows = sorted({0, w.batch - 1})
    rep = lockstep(s, om, src, src_len, k, N, max_iters=N, tail_fn=fn, rows=rows)
    for i, b in enumerate(rows):
        assert rep.emitted[b] == list(g_ids[b])
        assert [r[i] for r in rep.khats if r[i] > 0] == _expected_khats(sched[b], k, N)
    # the window matters: the same weights with full attention decode differently
    import dataclasses
    w_full = dataclasses.replace(w, cfg=dataclasses.replace(w.cfg, local_q=0, local_m=0))
    model_f = bpd.Model(make_weights(w_full.cfg, w.weight_seed, w.sigma))
    sf = bpd.Session(model_f, w.batch, w.max_src, N)
    sf.bpd_encode(src, src_len)
    f_ids, _, _ = sf.bpd_decode_greedy(N)
    assert not np.array_equal(f_ids, g_ids)
    sf.close(); model_f.close(); s.close(); model.close()



LONG_MODELS = [
    Workload("midi-long", MIDI.cfg, 0.05, 41, 42, 43, batch=1, src_lo=9, src_hi=9, n_decode=420),
    Workload("midi3-long", MIDI.cfg, 0.05, 41, 52, 53, batch=3, src_lo=3, src_hi=11, n_decode=330),
]


@pytest.mark.parametrize("w", LONG_MODELS, ids=lambda w: w.name)
def test_long_sequences_share_their_keys(bpd, w):
    """Full causal attention far into a sequence on the cluster path: once a row sees more than eight chunks of
    32 keys the self-attention block switches from one CTA per row to keys fetched once for all rows of a
    sequence.  Both schedules must give the same ids (greedy passes carry one row per sequence, blockwise
    passes k), and the lock-step against the oracle runs across the switch with every proposal accepted."""
    from harness import lockstep
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    s.bpd_encode(src, src_len)
    b_ids, _, _ = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(b_ids, g_ids)
    plan, sched = _plan(w, g_ids, k, 3.0)
    s.bpd_encode(src, src_len)
    s.bpd_set_forced_plan(plan, k)
    p_ids, _, _ = s.bpd_decode_blockwise(k, N)
    assert np.array_equal(p_ids, g_ids)

    def all_accepted(b, j, it):
        return forced_tail(g_ids[b], min(j, N), k, k, 0, w.cfg.vocab)
    rows = sorted({0, w.batch - 1})
    rep = lockstep(s, om, src, src_len, k, N, max_iters=(N + k - 1) // k, tail_fn=all_accepted, rows=rows)
    for b in rows:
        assert rep.emitted[b] == list(g_ids[b])
    s.close(); model.close()


def test_bounded_wait_expires_and_the_context_survives(bpd):
    """Failure detection without a fault: a wait on a barrier nobody signals, and a wait for tagged words nobody
    writes, give up after their limit; the call reports BPD_E_TIMEOUT and the same process keeps computing
    correctly afterwards."""
    import torch
    assert bpd.bpd_debug_wait_timeout(2000) == -7
    msg = bpd.lib.bpd_last_error().decode()
    assert "expired" in msg and "104" in msg          # both kinds of wait: the mbarrier and the tagged words
    x = torch.randn(4, 64).cuda()
    w = torch.randn(10, 64).cuda()
    y = bpd.bpd_op_linear(x, w).cpu()
    assert torch.allclose(y, x.cpu() @ w.cpu().T, atol=1e-4)


# ---------------------------------------------------------------- the two-call form (Section 3)

@pytest.mark.parametrize("w", [WORKLOADS["C1"], MINI, MINI_BATCH, MIDI], ids=lambda w: w.name)
def test_two_call_form_gives_the_merged_decode(bpd, w):
    """Predict and Verify as separate invocations: the same ids and the same accepted block sizes as the
    merged form and as the oracle's two-call loop, at two invocations per iteration instead of one per
    iteration plus the priming pass."""
    from oracle.decode import TransformerScorer, blockwise_twocall
    blob, model, src, src_len, om = _setup(bpd, w)
    k, N = w.cfg.k_model, w.n_decode
    s = bpd.Session(model, w.batch, w.max_src, N)
    s.bpd_encode(src, src_len)
    g_ids, _, _ = s.bpd_decode_greedy(N)
    # free running: whatever the heads propose
    s.bpd_encode(src, src_len)
    m_ids, m_len, m_st = s.bpd_decode_blockwise(k, N)
    s.bpd_encode(src, src_len)
    t_ids, t_len, t_st = s.bpd_decode_blockwise_twocall(k, N)
    assert np.array_equal(t_ids, g_ids) and np.array_equal(t_ids, m_ids) and np.array_equal(t_len, m_len)
    assert t_st.khat_hist == m_st.khat_hist and t_st.row_iterations == m_st.row_iterations
    assert m_st.invocations == m_st.iterations + 1
    assert t_st.invocations == 2 * t_st.iterations          # Section 4: 2m/k against m/k + 1
    # controlled acceptance: the same schedule through both forms, and through the oracle's two-call loop on row 0
    plan, sched = _plan(w, g_ids, k, 2.0)
    s.bpd_encode(src, src_len)
    s.bpd_set_forced_plan(plan, k)
    _, _, m_st = s.bpd_decode_blockwise(k, N)
    s.bpd_encode(src, src_len)
    s.bpd_set_forced_plan(plan, k)
    t_ids, _, t_st = s.bpd_decode_blockwise_twocall(k, N)
    assert np.array_equal(t_ids, g_ids) and t_st.khat_hist == m_st.khat_hist
    assert t_st.invocations == 2 * t_st.iterations and t_st.iterations == m_st.iterations
    if w.batch == 1:
        G, R = sched[0]
        sc = TransformerScorer(om, src[0, :src_len[0]], cached=True, capacity=N + 2 * k + 2)
        want = blockwise_twocall(sc, k, N, tail_fn=lambda j, it: forced_tail(g_ids[0], j, k, int(G[j]), int(R[j]), w.cfg.vocab))
        assert want.ids == list(t_ids[0])
        assert want.invocations == t_st.invocations
        hist = [0] * 17
        for kh in want.khats:
            hist[kh] += 1
        assert list(t_st.khat_hist) == hist
    # an end-of-sequence id inside a block ends the row in both forms at the same place
    eos = int(g_ids[0][min(5, N - 1)])
    s.bpd_encode(src, src_len)
    m_ids, m_len, _ = s.bpd_decode_blockwise(k, N, eos_id=eos)
    s.bpd_encode(src, src_len)
    t_ids, t_len, _ = s.bpd_decode_blockwise_twocall(k, N, eos_id=eos)
    assert np.array_equal(t_ids, m_ids) and np.array_equal(t_len, m_len)
    s.close()
    model.close()

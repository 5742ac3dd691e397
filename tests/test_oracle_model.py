"""Pins for the oracle's Transformer: library cross-checks in float64, closed
forms and invariants.  None of these call the CUDA library."""
import numpy as np
import pytest
import torch

from bpd_inputs import (DTYPE_BF16, DTYPE_F32, HEAD_BLOCKDIAG, HEAD_DENSE, ModelConfig,
                        make_weights, tensor_specs)
from oracle.model import (DecoderCache, attention, decoder_full, embed, encode, head_logits,
                          head_outputs, layer_norm, parse_blob, positional, softmax_masked)

CFG = ModelConfig(n_enc=2, n_dec=2, d_model=32, n_heads=4, d_ff=64, vocab=50, k_model=3,
                  d_hidden=48, dtype=DTYPE_F32)


def _model(cfg=CFG, seed=7, sigma=0.3, overrides=None, random_ln=True):
    ov = dict(overrides or {})
    if random_ln:
        rng = np.random.default_rng(seed + 1)
        for name, shape, kind in tensor_specs(cfg):
            if kind == "gain" and name not in ov:
                ov[name] = 1.0 + 0.2 * rng.standard_normal(shape)
            if kind == "shift" and name not in ov:
                ov[name] = 0.2 * rng.standard_normal(shape)
    return parse_blob(make_weights(cfg, seed, sigma, ov))


# ---------------------------------------------------------------- blob

def test_blob_roundtrip_f32_and_bf16():
    for dtype in (DTYPE_F32, DTYPE_BF16):
        cfg = ModelConfig(1, 1, 16, 2, 32, 11, 2, 24, dtype=dtype, head_layout=HEAD_BLOCKDIAG)
        ov = {"out_proj": np.arange(11 * 16, dtype=np.float32).reshape(11, 16) / 7.0}
        m = parse_blob(make_weights(cfg, 3, 0.1, ov))
        assert (m.n_enc, m.n_dec, m.d, m.H, m.d_ff, m.V, m.k_model, m.d_hidden) == (1, 1, 16, 2, 32, 11, 2, 24)
        assert m.head_layout == HEAD_BLOCKDIAG and m.w["head.w2"].shape == (2, 16, 24)
        want = torch.from_numpy(ov["out_proj"])
        if dtype == DTYPE_BF16:
            want = want.to(torch.bfloat16).to(torch.float32)
        np.testing.assert_array_equal(m.w["out_proj"], want.double().numpy())
        assert abs(m.eps - 1e-6) < 1e-12


# ---------------------------------------------------------------- primitives vs torch float64

def test_layer_norm_and_softmax_match_torch():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 32)) * 3 + 1
    g, b = rng.standard_normal(32), rng.standard_normal(32)
    want = torch.nn.functional.layer_norm(torch.from_numpy(x), (32,), torch.from_numpy(g),
                                          torch.from_numpy(b), eps=1e-6).numpy()
    np.testing.assert_allclose(layer_norm(x, g, b, 1e-6), want, atol=1e-12)
    y = layer_norm(x, np.ones(32), np.zeros(32), 1e-6)
    np.testing.assert_allclose(y.mean(-1), 0, atol=1e-12)
    np.testing.assert_allclose(y.var(-1), 1, atol=1e-5)
    s = rng.standard_normal((4, 9)) * 5
    allowed = rng.random((4, 9)) < 0.6
    allowed[:, 0] = True
    p = softmax_masked(s, allowed)
    assert np.all(p[~allowed] == 0.0)
    np.testing.assert_allclose(p.sum(-1), 1, atol=1e-14)
    want = torch.softmax(torch.from_numpy(np.where(allowed, s, -np.inf)), -1).numpy()
    np.testing.assert_allclose(p, want, atol=1e-14)


def test_attention_matches_torch_sdpa_and_single_key():
    rng = np.random.default_rng(1)
    n, m_, d, H = 5, 7, 32, 4
    q, k, v = rng.standard_normal((n, d)), rng.standard_normal((m_, d)), rng.standard_normal((m_, d))
    allowed = rng.random((n, m_)) < 0.7
    allowed[:, 0] = True
    got = attention(q, k, v, allowed, H)
    tq = torch.from_numpy(q).view(n, H, d // H).transpose(0, 1)
    tk = torch.from_numpy(k).view(m_, H, d // H).transpose(0, 1)
    tv = torch.from_numpy(v).view(m_, H, d // H).transpose(0, 1)
    want = torch.nn.functional.scaled_dot_product_attention(
        tq, tk, tv, attn_mask=torch.from_numpy(allowed)).transpose(0, 1).reshape(n, d).numpy()
    np.testing.assert_allclose(got, want, atol=1e-12)
    # one visible key: the output is that key's value row, whatever the scores
    one = np.zeros((n, m_), dtype=bool)
    one[:, 3] = True
    np.testing.assert_allclose(attention(q, k, v, one, H), np.tile(v[3], (n, 1)), atol=1e-14)


def test_positional_closed_forms():
    d = 32
    pe = positional(np.arange(6), d)
    np.testing.assert_allclose(pe[0, 0::2], 0, atol=0)
    np.testing.assert_allclose(pe[0, 1::2], 1, atol=0)
    np.testing.assert_allclose(pe[:, 0], np.sin(np.arange(6)), atol=1e-15)
    np.testing.assert_allclose(pe[:, 1], np.cos(np.arange(6)), atol=1e-15)
    np.testing.assert_allclose(pe[5, d - 2], np.sin(5 / 10000 ** ((d - 2) / d)), atol=1e-15)
    np.testing.assert_allclose(pe[5, 7], np.cos(5 / 10000 ** (6 / d)), atol=1e-15)
    table = np.random.default_rng(2).standard_normal((9, d))
    x = embed(table, [4, 2], first_pos=3)
    np.testing.assert_allclose(x[1], table[2] * np.sqrt(d) + positional(np.array([4]), d)[0], atol=1e-14)


# ---------------------------------------------------------------- whole stack vs torch.nn.Transformer

def _torch_transformer(m):
    t = torch.nn.Transformer(d_model=m.d, nhead=m.H, num_encoder_layers=m.n_enc,
                             num_decoder_layers=m.n_dec, dim_feedforward=m.d_ff, dropout=0.0,
                             activation="relu", layer_norm_eps=m.eps, batch_first=True,
                             norm_first=True, dtype=torch.float64)
    T = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    w = m.w
    with torch.no_grad():
        def ln(mod, p):
            mod.weight.copy_(T(w[p + ".g"])); mod.bias.copy_(T(w[p + ".b"]))

        def ff(layer, p):
            layer.linear1.weight.copy_(T(w[p + ".w1"])); layer.linear1.bias.copy_(T(w[p + ".b1"]))
            layer.linear2.weight.copy_(T(w[p + ".w2"])); layer.linear2.bias.copy_(T(w[p + ".b2"]))

        for l, layer in enumerate(t.encoder.layers):
            p = f"enc.{l}"
            layer.self_attn.in_proj_weight.copy_(T(w[p + ".attn.wqkv"])); layer.self_attn.in_proj_bias.zero_()
            layer.self_attn.out_proj.weight.copy_(T(w[p + ".attn.wo"])); layer.self_attn.out_proj.bias.zero_()
            ln(layer.norm1, p + ".ln1"); ln(layer.norm2, p + ".ln2"); ff(layer, p + ".ffn")
        ln(t.encoder.norm, "enc.lnf")
        for l, layer in enumerate(t.decoder.layers):
            p = f"dec.{l}"
            layer.self_attn.in_proj_weight.copy_(T(w[p + ".self.wqkv"])); layer.self_attn.in_proj_bias.zero_()
            layer.self_attn.out_proj.weight.copy_(T(w[p + ".self.wo"])); layer.self_attn.out_proj.bias.zero_()
            layer.multihead_attn.in_proj_weight.copy_(T(np.concatenate([w[p + ".cross.wq"], w[p + ".cross.wkv"]])))
            layer.multihead_attn.in_proj_bias.zero_()
            layer.multihead_attn.out_proj.weight.copy_(T(w[p + ".cross.wo"])); layer.multihead_attn.out_proj.bias.zero_()
            ln(layer.norm1, p + ".ln1"); ln(layer.norm2, p + ".ln2"); ln(layer.norm3, p + ".ln3")
            ff(layer, p + ".ffn")
        ln(t.decoder.norm, "dec.lnf")
    return t.eval()


@pytest.mark.parametrize("src_len", [9, 6])
def test_encoder_decoder_match_torch_transformer(src_len):
    m = _model()
    t = _torch_transformer(m)
    rng = np.random.default_rng(5)
    S, n = 9, 7
    src = rng.integers(0, m.V, S)
    tgt = rng.integers(0, m.V, n)
    pad = torch.arange(S)[None, :] >= src_len
    with torch.no_grad():
        mem = t.encoder(torch.from_numpy(embed(m.w["src_embed"], src, 0))[None], src_key_padding_mask=pad)
        causal = torch.triu(torch.ones(n, n, dtype=torch.bool), diagonal=1)
        out = t.decoder(torch.from_numpy(embed(m.w["tgt_embed"], tgt, 0))[None], mem, tgt_mask=causal,
                        memory_key_padding_mask=pad)
    mine_mem = encode(m, src, src_len)
    np.testing.assert_allclose(mine_mem[:src_len], mem[0, :src_len].numpy(), atol=1e-10)
    mine = decoder_full(m, mine_mem, src_len, tgt)
    np.testing.assert_allclose(mine, out[0].numpy(), atol=1e-10)


def test_padding_does_not_change_the_row():
    m = _model()
    rng = np.random.default_rng(6)
    src = rng.integers(2, m.V, 6)
    padded = np.concatenate([src, np.zeros(10, dtype=src.dtype)])
    tgt = [0, 3, 4, 5]
    a = decoder_full(m, encode(m, src), 6, tgt)
    b = decoder_full(m, encode(m, padded, 6), 6, tgt)
    np.testing.assert_allclose(a, b, atol=1e-12)


# ---------------------------------------------------------------- cache, rollback, causality

def test_cached_equals_uncached_with_rejections_and_poison():
    m = _model()
    rng = np.random.default_rng(8)
    src = rng.integers(0, m.V, 8)
    mem = encode(m, src)
    cache = DecoderCache(m, mem, 8, capacity=40)
    accepted = []
    for step in range(8):
        block = list(rng.integers(0, m.V, 4))
        # stale storage beyond the live length must have no effect
        cache.k[:, cache.length:] = np.nan
        cache.v[:, cache.length:] = np.nan
        h = cache.extend(block)
        full = decoder_full(m, mem, 8, accepted + block)[-4:]
        np.testing.assert_allclose(h, full, atol=1e-10)
        keep = int(rng.integers(1, 5))
        accepted += block[:keep]
        cache.commit(keep)
    assert cache.length == len(accepted)


def test_causality_bitwise():
    m = _model()
    mem = encode(m, [3, 4, 5])
    a = decoder_full(m, mem, 3, [0, 7, 8, 9, 10])
    b = decoder_full(m, mem, 3, [0, 7, 8, 11, 12])
    assert np.array_equal(a[:3], b[:3]) and not np.array_equal(a[3], b[3])


# ---------------------------------------------------------------- proposal heads (Section 6)

def test_heads_zero_second_layer_gives_identical_columns():
    d, k, fh = CFG.d_model, CFG.k_model, CFG.d_hidden
    m = _model(overrides={"head.w2": np.zeros((k * d, k * fh)), "head.b2": np.zeros(k * d)})
    h = np.random.default_rng(9).standard_normal((4, d))
    lg = head_logits(m, h, k)
    want = h @ m.w["out_proj"].T
    for i in range(k):
        np.testing.assert_allclose(lg[:, i], want, atol=1e-12)


def test_heads_formula_by_hand_and_identity_flag():
    m = _model()
    d, k, fh = m.d, m.k_model, m.d_hidden
    h = np.random.default_rng(10).standard_normal((2, d))
    o = head_outputs(m, h, k)
    # scalar loops, head 2, row 1, straight from the definition
    i, r = 1, 1
    u = [max(0.0, sum(h[r, c] * m.w["head.w1"][j, c] for c in range(d)) + m.w["head.b1"][j])
         for j in range(k * fh)]
    for c in (0, 5, d - 1):
        val = sum(u[j] * m.w["head.w2"][i * d + c, j] for j in range(k * fh)) + m.w["head.b2"][i * d + c] + h[r, c]
        assert abs(o[r, i, c] - val) < 1e-12
    from dataclasses import replace
    cfg = replace(CFG, p1_identity=1)
    mi = _model(cfg)
    lg = head_logits(mi, h, k)
    np.testing.assert_allclose(lg[:, 0], h @ mi.w["out_proj"].T, atol=1e-12)
    np.testing.assert_allclose(lg[:, 1:], head_logits(m, h, k)[:, 1:], atol=1e-12)


def test_dense_with_block_structure_equals_blockdiag_layout():
    from dataclasses import replace
    d, k, fh = CFG.d_model, CFG.k_model, CFG.d_hidden
    rng = np.random.default_rng(11)
    blocks = rng.standard_normal((k, d, fh)).astype(np.float32) * 0.3
    dense = np.zeros((k * d, k * fh), dtype=np.float32)
    for i in range(k):
        dense[i * d:(i + 1) * d, i * fh:(i + 1) * fh] = blocks[i]
    md = _model(overrides={"head.w2": dense})
    mb = _model(replace(CFG, head_layout=HEAD_BLOCKDIAG), overrides={"head.w2": blocks})
    h = rng.standard_normal((3, d))
    np.testing.assert_allclose(head_logits(md, h, k), head_logits(mb, h, k), atol=1e-12)
    # fewer heads than the model carries: the first k of them
    np.testing.assert_allclose(head_logits(md, h, 2), head_logits(md, h, k)[:, :2], atol=0)


# ---------------------------------------------------------------- 1D local attention (Section 7.2's model class)

def test_local_attention_window_by_enumeration():
    """The visible keys of a query, enumerated from the definition for every (query block, memory) pair and
    every position: its own block up to itself plus local_m positions before the block's first one."""
    from dataclasses import replace
    from oracle.model import self_attention_allowed
    base = _model()
    for q_len in (1, 2, 3, 5, 8):
        for mem in (0, 1, 4, 7):
            m = replace(base, local_q=q_len, local_m=mem)
            ok = self_attention_allowed(m, np.arange(20), 20)
            for t in range(20):
                block_start = (t // q_len) * q_len
                want = [j for j in range(20) if block_start - mem <= j <= t]
                assert list(np.nonzero(ok[t])[0]) == want
    full = self_attention_allowed(base, np.arange(9), 9)
    assert np.array_equal(full, np.tril(np.ones((9, 9), dtype=bool)))


def test_local_attention_special_cases_and_cache():
    """(i) memory at least as long as the sequence: identical to full causal attention; (ii) blocks of one
    position without memory: every query sees only itself, softmax over one key is 1, so a decoder layer's
    self-attention returns the value row and positions stop influencing each other; (iii) the cached decoder
    (blocks, rejections) equals the uncached one under local attention."""
    from dataclasses import replace
    base = _model()
    rng = np.random.default_rng(5)
    src = rng.integers(2, base.V, size=6)
    memory = encode(base, src, 6)
    toks = [0] + [int(t) for t in rng.integers(2, base.V, size=11)]
    full = decoder_full(base, memory, 6, toks)
    wide = replace(base, local_q=3, local_m=64)
    np.testing.assert_array_equal(decoder_full(wide, memory, 6, toks), full)
    alone = replace(base, local_q=1, local_m=0)
    h_alone = decoder_full(alone, memory, 6, toks)
    for t in (0, 4, 11):           # a position computed with nothing before it, at its own position: same row
        solo = replace(base, local_q=1, local_m=0)
        other = list(toks)
        for j in range(t):
            other[j] = 2 + (other[j] + 7) % (base.V - 2)     # change every earlier token
        np.testing.assert_array_equal(decoder_full(solo, memory, 6, other)[t], h_alone[t])
    assert not np.allclose(h_alone, full)
    loc = replace(base, local_q=4, local_m=3)
    want = decoder_full(loc, memory, 6, toks)
    assert not np.allclose(want[8:], full[8:])
    cache = DecoderCache(loc, memory, 6, capacity=32)
    got = np.zeros_like(want)
    pos = 0
    for n, acc in ((1, 1), (4, 2), (3, 3), (4, 1), (5, 5)):
        n = min(n, len(toks) - pos)
        h = cache.extend(toks[pos:pos + n])
        got[pos:pos + n] = h
        acc = min(acc, n)
        cache.commit(acc)
        pos += acc
        if pos >= len(toks):
            break
    np.testing.assert_allclose(got[:pos], want[:pos], rtol=0, atol=1e-12)

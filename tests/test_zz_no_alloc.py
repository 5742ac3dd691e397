"""The allocation-free top-1 entry point against the workspace-taking one.

Some embedders of this library cannot allocate device memory at call time (the
whole GPU belongs to a framework's pool, or an allocation's device-wide
synchronisation is not acceptable in their serving loop).  For them
bpd_op_vocab_argmax_noalloc keeps its reduction workspace in a fixed array
inside the library.  This test calls it through the C ABI twice in a row -- the
array keeps the first call's contents, so the second call proves the clearing --
and compares with bpd_op_vocab_argmax on the same inputs.  It runs last so that
a failure here cannot hide any other test's result.
"""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_workspace_variant_twice(dtype):
    import torch
    import paper_1811_03115_b200 as bpd
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    g = torch.Generator().manual_seed(5)
    w = (torch.randn(32768, 512, generator=g) * 0.02).to(td).cuda()
    out_idx = torch.empty(64, dtype=torch.int32, device="cuda")
    out_val = torch.empty(64, dtype=torch.float32, device="cuda")
    for call, rows in enumerate((64, 37)):          # second call: fewer rows over the used workspace
        x = torch.randn(rows, 512, generator=g).to(td).cuda()
        want_idx, want_val = bpd.bpd_op_vocab_argmax(x, w, want_val=True)
        out_idx.fill_(-7)
        out_val.fill_(0)
        before = torch.cuda.memory_allocated()
        bpd.bpd_op_vocab_argmax_noalloc(x, w, out_idx[:rows], out_val[:rows])
        assert torch.cuda.memory_allocated() == before
        torch.cuda.synchronize()
        assert torch.equal(out_idx[:rows], want_idx), f"call {call}: ids differ"
        assert torch.allclose(out_val[:rows], want_val, atol=1e-3), f"call {call}: values differ"
        if rows < 64:
            assert bool((out_idx[rows:] == -7).all())   # nothing written past the rows asked for


def test_noalloc_rejects_sizes_beyond_its_workspace():
    import torch
    import paper_1811_03115_b200 as bpd
    x = torch.zeros(257, 64, device="cuda")
    w = torch.zeros(100, 64, device="cuda")
    out = torch.full((257,), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(bpd.BpdError) as e:
        bpd.bpd_op_vocab_argmax_noalloc(x, w, out)
    assert e.value.status == -4 and "256 rows" in str(e.value)
    x = torch.zeros(4, 64, device="cuda")
    w = torch.zeros(65537, 64, device="cuda")
    with pytest.raises(bpd.BpdError) as e:
        bpd.bpd_op_vocab_argmax_noalloc(x, w, out[:4])
    assert e.value.status == -4
    torch.cuda.synchronize()
    assert bool((out == -7).all())

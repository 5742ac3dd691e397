"""The allocation-free top-1 entry point.

Some embedders of this library cannot allocate device memory at call time (the
whole GPU belongs to a framework's pool, or an allocation's device-wide
synchronisation is not acceptable in their serving loop).  For them
bpd_op_vocab_argmax_noalloc keeps its reduction workspace in a fixed array
inside the library.  These tests call it through the C ABI twice in a row -- the
array keeps the first call's contents, so the second call proves the clearing --
and check the result against the definition (float64 logits, ties to the lowest
id, near-ties allowed either way) and against bpd_op_vocab_argmax on the same
inputs.  They run last so that a failure here cannot hide any other test's
result.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

MARGIN = 1e-3      # a top-1 / top-2 gap below this may be decided either way by fp32 summation order


def _check_against_definition(x, w, idx, val, what):
    logits = x.double().cpu().numpy() @ w.double().cpu().numpy().T
    idx, val = idx.cpu().numpy(), val.cpu().numpy()
    best = logits.max(-1)
    for r in range(logits.shape[0]):
        second = np.partition(logits[r], -2)[-2]
        if best[r] - second > MARGIN:
            assert idx[r] == int(np.argmax(logits[r])), f"{what}: row {r}"
        assert abs(logits[r, idx[r]] - best[r]) <= MARGIN, f"{what}: row {r} picked a value {best[r] - logits[r, idx[r]]} below the maximum"
        assert abs(val[r] - best[r]) <= MARGIN, f"{what}: row {r} value"


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_noalloc_matches_definition_and_workspace_variant_twice(dtype):
    import torch
    import paper_1811_03115_b200 as bpd
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    g = torch.Generator().manual_seed(5)
    w = (torch.randn(32768, 512, generator=g) * 0.02).to(td)
    w[7] = w[3]                                     # an exact tie: the lower id must win where it is the maximum
    w = w.cuda()
    out_idx = torch.empty(64, dtype=torch.int32, device="cuda")
    out_val = torch.empty(64, dtype=torch.float32, device="cuda")
    # The first call on a device is the set-up call: the library looks up its array's address, and the CUDA driver
    # loads the kernel's code when it is first launched (the driver's own memory, 2 MiB in a fresh process; nothing
    # when other tests have launched that kernel before).  Embedders make it once at start-up; the calls after it
    # must leave the device's free memory exactly as it was.
    x0 = torch.randn(1, 512, generator=g).to(td).cuda()
    bpd.bpd_op_vocab_argmax_noalloc(x0, w, out_idx[:1], out_val[:1])
    torch.cuda.synchronize()
    _check_against_definition(x0, w, out_idx[:1], out_val[:1], "set-up call")
    for call, rows in enumerate((64, 37)):          # second call: fewer rows over the used workspace
        x = torch.randn(rows, 512, generator=g).to(td)
        x[0] = (w[3].float().cpu() * 50).to(td)
        x = x.cuda()
        want_idx, want_val = bpd.bpd_op_vocab_argmax(x, w, want_val=True)
        out_idx.fill_(-7)
        out_val.fill_(0)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()  # the driver's own count: sees an allocation by anybody
        bpd.bpd_op_vocab_argmax_noalloc(x, w, out_idx[:rows], out_val[:rows])
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, f"call {call}: device memory changed by {free_before - free_after} bytes"
        _check_against_definition(x, w, out_idx[:rows], out_val[:rows], f"call {call}")
        assert int(out_idx[0]) == 3                 # the planted tie
        # second check, against the workspace-taking entry point: equal wherever the answer is not a near-tie
        same = out_idx[:rows] == want_idx
        near = (out_val[:rows] - want_val).abs() <= MARGIN
        assert bool((same | near).all()), f"call {call}: ids differ from bpd_op_vocab_argmax beyond a near-tie"
        assert torch.allclose(out_val[:rows], want_val, atol=MARGIN), f"call {call}: values differ"
        if rows < 64:
            assert bool((out_idx[rows:] == -7).all())   # nothing written past the rows asked for


def test_noalloc_at_its_limits():
    """256 rows, vocabulary 65536, d = 1024: the largest sizes the built-in workspace takes."""
    import torch
    import paper_1811_03115_b200 as bpd
    g = torch.Generator().manual_seed(9)
    w = (torch.randn(65536, 1024, generator=g) * 0.02).to(torch.bfloat16).cuda()
    x = torch.randn(256, 1024, generator=g).to(torch.bfloat16).cuda()
    out_idx = torch.full((256,), -7, dtype=torch.int32, device="cuda")
    out_val = torch.zeros(256, dtype=torch.float32, device="cuda")
    for call in range(2):
        bpd.bpd_op_vocab_argmax_noalloc(x, w, out_idx, out_val)
        torch.cuda.synchronize()
        _check_against_definition(x, w, out_idx, out_val, f"call {call}")


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
    x = torch.zeros(4, 1032, device="cuda")         # d above the kernel's limit: a shape error, as in bpd_op_vocab_argmax
    w = torch.zeros(100, 1032, device="cuda")
    with pytest.raises(bpd.BpdError) as e:
        bpd.bpd_op_vocab_argmax_noalloc(x, w, out[:4])
    assert e.value.status == -2
    launches = bpd.bpd_kernel_launches()
    x = torch.zeros(4, 64, device="cuda")
    w = torch.zeros(100, 64, device="cuda")
    bpd.bpd_op_vocab_argmax_noalloc(x, w, out[:4])
    assert bpd.bpd_kernel_launches() == launches + 1   # the call is counted like every other launch
    torch.cuda.synchronize()
    assert bool((out[4:] == -7).all())

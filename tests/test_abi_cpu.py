"""Host-side checks of the C ABI that need no GPU: every symbol the header
declares is exported, and malformed input is turned into error codes."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from bpd_inputs import DTYPE_BF16, DTYPE_F32, ModelConfig, WORKLOADS, make_weights

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1811_03115_b200.build import build_library
    build_library()
    from paper_1811_03115_b200 import binding
    return binding


def _declared():
    text = open(os.path.join(ROOT, "include", "bpd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bpd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert "bpd_load_weights" in names and "bpd_encode" in names and "bpd_decode_greedy" in names
    assert "bpd_decode_blockwise" in names and "bpd_iteration" in names
    for n in names:
        assert hasattr(lib.lib, n), f"{n} declared in bpd.h but not exported"
    assert set(lib.EXPORTED) == set(names)


def test_struct_layouts_match_header(lib):
    assert C.sizeof(lib.bpd_stats) == 8 * 4 + 8 * 17 + 8
    assert C.sizeof(lib.bpd_iter_out) == 8 * C.sizeof(C.c_void_p)
    assert C.sizeof(lib.bpd_session_options) == 10 * 4
    opt = lib.bpd_session_options()
    lib.lib.bpd_session_options_init(C.byref(opt))
    assert opt.struct_bytes == 40 and all(getattr(opt, n) == -1 for n in lib.OPTION_FIELDS)
    # the header declares the same fields in the same order
    text = open(os.path.join(ROOT, "include", "bpd.h")).read()
    body = text[text.index("typedef struct {\n  int32_t struct_bytes"):text.index("} bpd_session_options;")]
    assert re.findall(r"int32_t (\w+);", body) == ["struct_bytes"] + list(lib.OPTION_FIELDS)


def _sizes(lib, blob, batch=1, max_src=8, max_tgt=8):
    wb, sb = C.c_size_t(0), C.c_size_t(0)
    rc = lib.lib.bpd_query_sizes(blob.ctypes.data_as(C.c_void_p), blob.nbytes, batch, max_src, max_tgt,
                                 C.byref(wb), C.byref(sb))
    return rc, wb.value, sb.value, lib.lib.bpd_last_error().decode()


def test_query_sizes_and_blob_validation(lib):
    cfg = ModelConfig(1, 1, 32, 2, 64, 40, 3, 48, dtype=DTYPE_F32)
    blob = make_weights(cfg, 1, 0.1)
    rc, wb, sb, _ = _sizes(lib, blob)
    assert rc == 0 and wb >= blob.nbytes and sb > 0
    rc2, _, sb2, _ = _sizes(lib, blob, batch=4, max_src=8, max_tgt=100)
    assert rc2 == 0 and sb2 > sb
    # malformed blobs
    bad = blob.copy(); bad[0] = ord("X")
    assert _sizes(lib, bad)[0] == -3
    assert _sizes(lib, blob[:100])[0] == -3
    assert _sizes(lib, blob[:-256])[0] == -3                   # size disagrees with the header
    bad = blob.copy(); bad[8] = 9                                # version
    assert _sizes(lib, bad)[0] == -3
    bad = blob.copy(); bad[24:28] = np.frombuffer(np.int32(33).tobytes(), np.uint8)   # d_model not a multiple of 8
    assert _sizes(lib, bad)[0] == -3
    bad = blob.copy(); bad[40:44] = np.frombuffer(np.int32(17).tobytes(), np.uint8)   # k_model above the limit
    rc, _, _, msg = _sizes(lib, bad)
    assert rc == -8 and "k_model" in msg
    bad = blob.copy(); bad[128 + 80:128 + 88] = np.frombuffer(np.uint64(blob.nbytes).tobytes(), np.uint8)  # tensor past the end
    assert _sizes(lib, bad)[0] == -3
    # arguments
    assert _sizes(lib, blob, batch=0)[0] == -1
    assert lib.lib.bpd_query_sizes(None, 0, 1, 1, 1, None, None) == -1
    # null handles never crash
    assert lib.lib.bpd_encode(None, None, None) == -1
    assert lib.lib.bpd_decode_greedy(None, 1, -1, None, None, None) == -1
    assert lib.lib.bpd_iteration(None, 1, 0, 1, -1, None, None) == -1
    assert lib.lib.bpd_session_destroy(None) == 0 and lib.lib.bpd_model_destroy(None) == 0


def test_session_size_accounts_for_cache_and_workspace(lib):
    """The session of the headline configuration holds the paged cache for
    max_tgt + k + 1 positions per row and fits comfortably in device memory."""
    w = WORKLOADS["C2"]
    cfg = w.cfg
    blob = make_weights(ModelConfig(1, 1, 64, 2, 64, 64, 2, 64, dtype=DTYPE_BF16), 1, 0.1)
    _, _, small, _ = _sizes(lib, blob, batch=1, max_src=8, max_tgt=64)
    _, _, big, _ = _sizes(lib, blob, batch=1, max_src=8, max_tgt=64 + 640)
    pages = 640 // 64
    assert big - small >= pages * 64 * 64 * 2 * 2          # K and V, one decoder layer, bf16
    assert cfg.k_model <= 16

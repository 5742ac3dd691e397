"""ctypes binding of libbpd.so: the same calls as include/bpd.h, with argument
marshalling only.  Device buffers come from torch (uint8 tensors); every step
of the decoding path runs inside the library's CUDA kernels.  There is no
fallback: if the library is missing or fails to load, importing this module
raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np

from .build import LIB_PATH

BPD_MAX_K = 16
BPD_OK = 0
STATUS_NAMES = {0: "BPD_OK", -1: "BPD_E_INVALID", -2: "BPD_E_SHAPE", -3: "BPD_E_FORMAT", -4: "BPD_E_NOMEM",
                -5: "BPD_E_STATE", -6: "BPD_E_CUDA", -7: "BPD_E_TIMEOUT", -8: "BPD_E_UNSUPPORTED"}


class BpdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class bpd_stats(C.Structure):
    _fields_ = [("tokens", C.c_int64), ("iterations", C.c_int64), ("invocations", C.c_int64),
                ("row_iterations", C.c_int64), ("khat_hist", C.c_int64 * (BPD_MAX_K + 1)),
                ("device_ms", C.c_double)]


class bpd_iter_out(C.Structure):
    _fields_ = [("khat", C.c_void_p), ("accepted", C.c_void_p), ("table", C.c_void_p),
                ("next_block", C.c_void_p), ("block", C.c_void_p), ("logits_dev", C.c_void_p),
                ("hidden_dev", C.c_void_p), ("layers_dev", C.c_void_p)]


OPTION_FIELDS = ("tensor_cores", "cuda_graphs", "dependent_launch", "lazy_heads", "fold_layer_norms", "cluster_layers",
                 "persistent_layers", "stage_encoder_rows", "l2_stream_hints")


class bpd_session_options(C.Structure):
    _fields_ = [("struct_bytes", C.c_int32)] + [(name, C.c_int32) for name in OPTION_FIELDS]


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it first (python -m paper_1811_03115_b200.build "
                      "or __graft_entry__.build()); there is no CPU fallback")
lib = C.CDLL(LIB_PATH)

_vp, _sz, _i = C.c_void_p, C.c_size_t, C.c_int
_SIGS = {
    "bpd_last_error": (C.c_char_p, []),
    "bpd_query_sizes": (_i, [_vp, _sz, _i, _i, _i, C.POINTER(_sz), C.POINTER(_sz)]),
    "bpd_session_bytes": (_i, [_vp, _i, _i, _i, C.POINTER(_sz)]),
    "bpd_session_layer_path": (_i, [_vp]),
    "bpd_load_weights": (_i, [_vp, _sz, _vp, _sz, _vp, C.POINTER(_vp)]),
    "bpd_session_create": (_i, [_vp, _i, _i, _i, _vp, _sz, _vp, C.POINTER(_vp)]),
    "bpd_session_options_init": (None, [C.POINTER(bpd_session_options)]),
    "bpd_session_create_opt": (_i, [_vp, _i, _i, _i, _vp, _sz, _vp, C.POINTER(bpd_session_options), C.POINTER(_vp)]),
    "bpd_session_destroy": (_i, [_vp]),
    "bpd_model_destroy": (_i, [_vp]),
    "bpd_encode": (_i, [_vp, _vp, _vp]),
    "bpd_decode_greedy": (_i, [_vp, _i, C.c_int32, _vp, _vp, C.POINTER(bpd_stats)]),
    "bpd_decode_blockwise": (_i, [_vp, _i, _i, _i, C.c_int32, _vp, _vp, C.POINTER(bpd_stats)]),
    "bpd_decode_blockwise_twocall": (_i, [_vp, _i, _i, _i, C.c_int32, _vp, _vp, C.POINTER(bpd_stats)]),
    "bpd_iteration": (_i, [_vp, _i, _i, _i, C.c_int32, _vp, C.POINTER(bpd_iter_out)]),
    "bpd_set_forced_plan": (_i, [_vp, _vp, _i, _i]),
    "bpd_rewind": (_i, [_vp]),
    "bpd_kernel_launches": (C.c_longlong, []),
    "bpd_profile": (_i, [_vp, _i]),
    "bpd_profile_read": (_i, [_vp, _i, C.POINTER(C.c_int64), C.POINTER(C.c_double)]),
    "bpd_fetch_output": (_i, [_vp, _i, _vp, _vp, C.POINTER(bpd_stats)]),
    "bpd_debug_wait_timeout": (_i, [_vp, _i, _vp]),
    "bpd_op_vocab_argmax_scratch_bytes": (_sz, [_i, _i, _i, _i]),
    "bpd_op_vocab_argmax": (_i, [_vp, _vp, _i, _i, _i, _i, _vp, _sz, _vp, _vp, _vp]),
    "bpd_op_vocab_argmax_noalloc": (_i, [_vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp]),
    "bpd_op_linear_scratch_bytes": (_sz, [_i, _i, _i, _i]),
    "bpd_op_linear": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _sz, _vp, _vp]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(lib, _name)          # AttributeError here = a declared symbol is not exported
    _fn.restype, _fn.argtypes = _res, _args
EXPORTED = tuple(_SIGS)


def BPD_ACCEPT_TOPN(n: int) -> int:
    return (1 << 8) | (n & 0xff)


def BPD_ACCEPT_DISTANCE(eps: int) -> int:
    return (2 << 8) | (eps & 0xff)


def BPD_ACCEPT_MIN_BLOCK(l: int) -> int:
    return (l & 0xff) << 16


def _check(rc: int) -> None:
    if rc != BPD_OK:
        raise BpdError(rc, lib.bpd_last_error().decode(errors="replace"))


def _host_i32(a, shape=None) -> np.ndarray:
    arr = np.ascontiguousarray(a, dtype=np.int32)
    if shape is not None and tuple(arr.shape) != tuple(shape):
        raise ValueError(f"expected int32 array of shape {shape}, got {arr.shape}")
    return arr


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


@dataclass
class Stats:
    tokens: int
    iterations: int
    invocations: int
    row_iterations: int
    khat_hist: list
    device_ms: float

    @property
    def mean_block(self) -> float:
        return self.tokens / max(1, self.row_iterations)


def _stats(st: bpd_stats) -> Stats:
    return Stats(st.tokens, st.iterations, st.invocations, st.row_iterations, list(st.khat_hist), st.device_ms)


def bpd_query_sizes(blob: np.ndarray, batch: int, max_src: int, max_tgt: int):
    wb, sb = _sz(0), _sz(0)
    _check(lib.bpd_query_sizes(_ptr(blob), blob.nbytes, batch, max_src, max_tgt, C.byref(wb), C.byref(sb)))
    return wb.value, sb.value


class Model:
    """bpd_load_weights / bpd_model_destroy.  Owns the torch buffer that holds the weights."""

    def __init__(self, blob: np.ndarray, device: str = "cuda:0"):
        import torch
        blob = np.ascontiguousarray(blob).view(np.uint8)
        wb = _sz(0)
        _check(lib.bpd_query_sizes(_ptr(blob), blob.nbytes, 1, 1, 1, C.byref(wb), None))
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.buf = torch.empty(wb.value, dtype=torch.uint8, device=self.device)
            self.handle = _vp(0)
            _check(lib.bpd_load_weights(_ptr(blob), blob.nbytes, self.buf.data_ptr(), wb.value, _stream(),
                                        C.byref(self.handle)))
        self.blob_header = bytes(blob[:128])

    def close(self):
        if self.handle:
            lib.bpd_model_destroy(self.handle)
            self.handle = _vp(0)


class Session:
    """bpd_session_create_opt and the calls that take a session.  ``options`` maps the field names of
    bpd_session_options to 0 / 1 (anything left out keeps the library's default)."""

    def __init__(self, model: Model, batch: int, max_src: int, max_tgt: int, options: Optional[dict] = None):
        import torch
        opt = bpd_session_options()
        lib.bpd_session_options_init(C.byref(opt))
        for name, value in (options or {}).items():
            if name not in OPTION_FIELDS:
                raise ValueError(f"unknown session option {name!r}")
            setattr(opt, name, int(value))
        self.model, self.B, self.max_src, self.max_tgt = model, batch, max_src, max_tgt
        nb = _sz(0)
        _check(lib.bpd_session_bytes(model.handle, batch, max_src, max_tgt, C.byref(nb)))
        sb = nb.value
        with torch.cuda.device(model.device):
            self.buf = torch.empty(sb, dtype=torch.uint8, device=model.device)
            # a stream of its own: the library replays each decoder pass as a CUDA graph, which the
            # default stream cannot capture.  Time it with events recorded on ``self.stream``.
            self.stream = torch.cuda.Stream(device=model.device)
            self.stream.wait_stream(torch.cuda.current_stream())
            self.handle = _vp(0)
            _check(lib.bpd_session_create_opt(model.handle, batch, max_src, max_tgt, self.buf.data_ptr(), sb,
                                              self.stream.cuda_stream, C.byref(opt), C.byref(self.handle)))
        self.session_bytes = sb

    def close(self):
        if self.handle:
            lib.bpd_session_destroy(self.handle)
            self.handle = _vp(0)

    def bpd_encode(self, src_ids, src_len):
        src = _host_i32(src_ids, (self.B, self.max_src))
        ln = _host_i32(src_len, (self.B,))
        _check(lib.bpd_encode(self.handle, _ptr(src), _ptr(ln)))

    def _decode(self, fn, args, max_new, fetch):
        st = bpd_stats()
        if not fetch:
            _check(fn(self.handle, *args, None, None, None))
            return None
        ids = np.empty((self.B, max_new), dtype=np.int32)
        ln = np.empty(self.B, dtype=np.int32)
        _check(fn(self.handle, *args, _ptr(ids), _ptr(ln), C.byref(st)))
        return ids, ln, _stats(st)

    def bpd_decode_greedy(self, max_new: int, eos_id: int = -1, fetch: bool = True):
        return self._decode(lib.bpd_decode_greedy, (max_new, eos_id), max_new, fetch)

    def bpd_decode_blockwise(self, k: int, max_new: int, eos_id: int = -1, accept_mode: int = 0, fetch: bool = True):
        return self._decode(lib.bpd_decode_blockwise, (k, accept_mode, max_new, eos_id), max_new, fetch)

    def bpd_decode_blockwise_twocall(self, k: int, max_new: int, eos_id: int = -1, accept_mode: int = 0, fetch: bool = True):
        return self._decode(lib.bpd_decode_blockwise_twocall, (k, accept_mode, max_new, eos_id), max_new, fetch)

    def bpd_fetch_output(self, max_new: int):
        st = bpd_stats()
        ids = np.empty((self.B, max_new), dtype=np.int32)
        ln = np.empty(self.B, dtype=np.int32)
        _check(lib.bpd_fetch_output(self.handle, max_new, _ptr(ids), _ptr(ln), C.byref(st)))
        return ids, ln, _stats(st)

    def bpd_rewind(self):
        _check(lib.bpd_rewind(self.handle))

    def bpd_profile(self, enable: bool):
        _check(lib.bpd_profile(self.handle, int(enable)))

    def bpd_profile_read(self, phase: int):
        n, ms = C.c_int64(0), C.c_double(0.0)
        _check(lib.bpd_profile_read(self.handle, phase, C.byref(n), C.byref(ms)))
        return n.value, ms.value

    def bpd_set_forced_plan(self, plan, k: int):
        if plan is None:
            _check(lib.bpd_set_forced_plan(self.handle, None, 0, 0))
            return
        p = _host_i32(plan)
        if p.ndim != 3 or p.shape[0] != self.B or p.shape[2] != k - 1:
            raise ValueError(f"plan must be [batch, plan_len, k-1], got {p.shape}")
        _check(lib.bpd_set_forced_plan(self.handle, _ptr(p), p.shape[1], k))

    def bpd_iteration(self, k: int, max_new: int, eos_id: int = -1, forced_tail=None, accept_mode: int = 0,
                      want_logits: bool = False, want_hidden: bool = False, want_layers: bool = False):
        import torch
        B = self.B
        out = bpd_iter_out()
        khat = np.empty(B, np.int32)
        acc = np.empty((B, k), np.int32)
        table = np.empty((B, k, k), np.int32)
        nxt = np.empty((B, k), np.int32)
        blk = np.empty((B, k), np.int32)
        out.khat, out.accepted, out.table, out.next_block, out.block = (_ptr(khat), _ptr(acc), _ptr(table),
                                                                        _ptr(nxt), _ptr(blk))
        logits = hidden = layers = None
        V, d = self.vocab, self.d_model
        if want_layers:
            layers = torch.empty((self.n_dec, B, k, d), dtype=torch.float32, device=self.model.device)
            out.layers_dev = layers.data_ptr()
        if want_logits:
            logits = torch.empty((B, k, k, V), dtype=torch.float32, device=self.model.device)
            out.logits_dev = logits.data_ptr()
        if want_hidden:
            hidden = torch.empty((B, k, d), dtype=torch.float32, device=self.model.device)
            out.hidden_dev = hidden.data_ptr()
        tail = None if forced_tail is None else _host_i32(forced_tail, (B, k - 1))
        _check(lib.bpd_iteration(self.handle, k, accept_mode, max_new, eos_id, _ptr(tail), C.byref(out)))
        res = {"khat": khat, "accepted": acc, "table": table, "next_block": nxt, "block": blk}
        if logits is not None:
            res["logits"] = logits
        if hidden is not None:
            res["hidden"] = hidden
        if layers is not None:
            res["layers"] = layers
        return res

    @property
    def layer_path(self) -> int:
        """0: one kernel per projection, 1: three cluster launches per layer, 2: one persistent kernel per pass."""
        return int(lib.bpd_session_layer_path(self.handle))

    @property
    def n_dec(self) -> int:
        return int(np.frombuffer(self.model.blob_header[20:24], np.int32)[0])

    @property
    def vocab(self) -> int:
        return int(np.frombuffer(self.model.blob_header[36:40], np.int32)[0])

    @property
    def d_model(self) -> int:
        return int(np.frombuffer(self.model.blob_header[24:28], np.int32)[0])


def bpd_debug_wait_timeout(limit_us: int = 2000) -> int:
    """Runs the bounded-wait self test and returns the status code (BPD_E_TIMEOUT = -7 is the expected outcome)."""
    import torch
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    return int(lib.bpd_debug_wait_timeout(word.data_ptr(), limit_us, _stream()))


def bpd_kernel_launches() -> int:
    return int(lib.bpd_kernel_launches())


def bpd_op_vocab_argmax(x, w, want_val: bool = False):
    """x [rows, d], w [vocab, d]: CUDA tensors, both float32 or both bfloat16.  Returns idx (and val)."""
    import torch
    rows, d = x.shape
    vocab = w.shape[0]
    dtype = 0 if x.dtype == torch.float32 else 1
    nbytes = lib.bpd_op_vocab_argmax_scratch_bytes(rows, d, vocab, dtype)
    scratch = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=x.device)
    idx = torch.empty(rows, dtype=torch.int32, device=x.device)
    val = torch.empty(rows, dtype=torch.float32, device=x.device) if want_val else None
    _check(lib.bpd_op_vocab_argmax(x.data_ptr(), w.data_ptr(), rows, d, vocab, dtype, scratch.data_ptr(), nbytes,
                                   idx.data_ptr(), None if val is None else val.data_ptr(), _stream()))
    return (idx, val) if want_val else idx


def bpd_op_vocab_argmax_noalloc(x, w, out_idx, out_val=None):
    """Top-1 of x w^T using the library's built-in workspace: nothing is allocated
    here or in the library, the caller passes the outputs (int32 [rows] and,
    optionally, float32 [rows] CUDA tensors).  For callers that cannot allocate:
    see include/bpd.h for the limits and the sharing rule."""
    import torch
    rows, d = x.shape
    dtype = 0 if x.dtype == torch.float32 else 1
    _check(lib.bpd_op_vocab_argmax_noalloc(x.data_ptr(), w.data_ptr(), rows, d, w.shape[0], dtype,
                                           out_idx.data_ptr(), None if out_val is None else out_val.data_ptr(),
                                           _stream()))


def bpd_op_linear(x, w, bias=None, relu: bool = False):
    """y = act(x w^T + bias) as float32.  x [rows, in], w [out, in], bias [out] or None."""
    import torch
    rows, in_f = x.shape
    out_f = w.shape[0]
    dtype = 0 if x.dtype == torch.float32 else 1
    nbytes = lib.bpd_op_linear_scratch_bytes(rows, in_f, out_f, dtype)
    scratch = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=x.device)
    y = torch.empty((rows, out_f), dtype=torch.float32, device=x.device)
    _check(lib.bpd_op_linear(x.data_ptr(), w.data_ptr(), None if bias is None else bias.data_ptr(), rows, in_f,
                             out_f, dtype, int(relu), scratch.data_ptr(), nbytes, y.data_ptr(), _stream()))
    return y

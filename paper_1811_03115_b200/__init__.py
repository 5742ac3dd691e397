"""Blockwise parallel decoding on NVIDIA B200: hand-written CUDA behind a C ABI
(include/bpd.h), with a thin ctypes binding of the same names.

``paper_1811_03115_b200.build`` compiles the library; everything else lives in
``paper_1811_03115_b200.binding`` and is re-exported here on first use (so the
build module can be imported before the library exists).  There is no CPU
fallback: touching any binding name without a built library raises.
"""
_BINDING_NAMES = ("BpdError", "Model", "Session", "Stats", "bpd_op_linear", "bpd_op_vocab_argmax", "bpd_op_vocab_argmax_noalloc",
                  "bpd_kernel_launches", "bpd_debug_wait_timeout", "BPD_ACCEPT_TOPN", "BPD_ACCEPT_DISTANCE", "BPD_ACCEPT_MIN_BLOCK", "bpd_query_sizes", "lib", "EXPORTED")


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)

"""Seeded synthetic inputs for blockwise parallel decoding experiments.

This package only *produces data*: model hyper-parameters, random weights
packed into a self-describing blob, source token ids, and acceptance
schedules.  It holds none of the decoding method's arithmetic (no attention,
no projections, no argmax, no verification) so that the CPU oracle and the
CUDA library can both consume its output without sharing any code.
"""
from .blob import (BLOB_MAGIC, DTYPE_BF16, DTYPE_F32, HEAD_BLOCKDIAG, HEAD_DENSE,
                   ModelConfig, tensor_specs, write_blob)
from .workloads import (WORKLOADS, Workload, corrupt_token, forced_tail,
                        geometric_schedule, make_source, make_weights)

__all__ = [
    "BLOB_MAGIC", "DTYPE_BF16", "DTYPE_F32", "HEAD_BLOCKDIAG", "HEAD_DENSE",
    "ModelConfig", "tensor_specs", "write_blob",
    "WORKLOADS", "Workload", "corrupt_token", "forced_tail",
    "geometric_schedule", "make_source", "make_weights",
]

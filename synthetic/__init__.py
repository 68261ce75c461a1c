"""Seeded synthetic inputs (videos, weight blobs, workload configurations).

This package holds no arithmetic of the method itself: it only produces the
inputs that both the CPU oracle and the CUDA library consume, so that both see
bit-identical fp32 arrays.  numpy only.
"""
from .configs import EncoderShape, MergeParams, VideoSpec, Workload, WORKLOADS, workload  # noqa: F401
from .videos import make_video, make_batch  # noqa: F401
from .weights import make_weights, weight_layout, blob_size  # noqa: F401

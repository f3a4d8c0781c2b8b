"""Seeded synthetic inputs (partitions, class masks, logits) shared by the tests and the bench.

This package holds input recipes only; it imports neither the CPU oracle nor
the CUDA library, and contains none of the masking path's arithmetic.
"""
from . import rng  # noqa: F401
from . import grammars  # noqa: F401
from .workloads import (  # noqa: F401
    CONFIGS,
    Partition,
    Workload,
    class_mask_bernoulli,
    class_mask_n_classes,
    heavy_tail_partition,
    identity_partition,
    logits_normal,
    make_workload,
    pack_bits,
    unpack_bits,
    zipf_partition,
)

"""Fused + pruned residual-network inference on B200 (FuPruner's inference hot path).

``workloads`` builds seeded synthetic networks and inputs; ``binding`` is the thin ctypes
layer over the C-ABI library (``fp_fuse`` / ``fp_prune`` / ``fp_forward`` ...).  The
binding is imported lazily so that describing a workload does not need the CUDA library.
"""

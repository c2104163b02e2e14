"""B200-native rollout step (MoE-transformer decode / chunked prefill over a paged KV cache).

The CUDA library is loaded lazily by :mod:`paper_2511_11373_b200.binding`; importing the package
itself (for example to reach :mod:`paper_2511_11373_b200.workloads`) needs no GPU and no build.
"""
__all__ = ["binding", "workloads", "build"]

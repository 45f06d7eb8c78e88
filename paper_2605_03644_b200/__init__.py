"""B200-native AdapShot KV-reuse hot path.

`binding` loads the CUDA C-ABI library and raises if it is missing (there is no
CPU fallback); `workloads` holds the seeded synthetic input generators.
"""
__all__ = ["binding", "workloads", "build"]

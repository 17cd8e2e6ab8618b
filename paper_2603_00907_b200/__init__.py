"""B200-native KV-merge pass (KVSlimmer): CUDA kernels behind a C ABI plus a thin binding.

`workloads` holds the seeded input generators; `binding` loads the shared library.
The compute entry points are imported lazily so that the generators can be used on a
machine without the built library.
"""
__all__ = ["workloads", "binding"]

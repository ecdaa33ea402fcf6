"""B200-native paged GQA decode attention + KV append (the decode iteration's hot path).

`workloads` draws seeded inputs and needs nothing else; `binding` loads the CUDA shared library
and raises if it has not been built -- there is no CPU fallback.
"""

__all__ = ["workloads", "binding"]

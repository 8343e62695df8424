"""B200-native KV-Fold fold step: thin Python binding over the C-ABI library.

`workloads` (synthetic inputs) imports nothing else; `binding` loads libkvfold.so and
raises if it is missing - there is no fallback path.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding", "build"]

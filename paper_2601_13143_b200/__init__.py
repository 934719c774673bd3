"""B200-native FastAV prune step: score -> select -> compact behind a C-ABI CUDA library.

``workloads`` (seeded synthetic inputs) imports nothing else from the package.  The binding
(``fastav``) loads ``libfastav.so`` on first use and raises if it is missing: there is no CPU
fallback.
"""
__all__ = ["workloads", "fastav", "flops", "build"]

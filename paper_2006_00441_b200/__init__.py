"""DaSGD (Local SGD with Delayed Averaging) hot path for NVIDIA B200 (sm_100a).

``inputs`` (seeded synthetic workloads) imports without the native library;
everything else goes through ``binding``, which loads ``libdasgd.so`` and raises
if it is missing -- there is no fallback implementation.
"""

__all__ = ["inputs", "binding", "build"]

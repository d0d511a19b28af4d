"""B200-native per-chunk hot path of the OmniTide streaming loop.

``workloads`` (seeded synthetic inputs) imports without the CUDA library;
everything in ``binding`` needs ``libomnitide.so`` and fails loudly without it.
"""
__all__ = ["workloads", "binding"]

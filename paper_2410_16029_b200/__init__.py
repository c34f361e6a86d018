"""Natural GaLore optimizer step for B200 (sm_100a).

``workload`` describes the synthetic matrix sets; ``ngalore`` is the thin
binding over the C-ABI library (it raises at import when the library is
missing: there is no CPU fallback).
"""
__all__ = ["workload"]

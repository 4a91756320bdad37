"""B200-native execution of one pipeline stage of a decoder-only LLM (prefill + paged-KV decode)
and the HypSplit-DP / HypSched-RT host algorithms, behind a C-ABI library.

`from paper_2511_14450_b200 import hyperion` gives the thin ctypes binding; the shared library is
loaded on first use and a missing build raises immediately (there is no CPU fallback).
"""
__all__ = ["hyperion", "inputs"]

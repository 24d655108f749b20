"""B200-native hot path of the CHELA token mixer: chunked causal linear attention with its
short-conv / long-conv prologue stages, as a C-ABI CUDA library plus a thin Python binding.

The binding (``paper_2406_08128_b200.chela``) loads ``libchela.so`` lazily and fails loudly
when it is missing; there is no CPU fallback.
"""
__all__ = ["chela", "inputs"]

"""B200-native StructKV prefill-time KV-compression hot path.

``paper_2604_06746_b200.binding`` is the thin ctypes layer over the C-ABI
library (it raises at import if the CUDA library has not been built);
``paper_2604_06746_b200.synth`` draws the seeded synthetic workloads.
"""
__all__ = ["binding", "synth"]

"""B200-native per-fragment merge of the Decoupled DiLoCo syncer.

``paper_2604_21428_b200.ddmerge`` is the binding of the C-ABI library (CUDA,
sm_100a); ``paper_2604_21428_b200.synth`` draws seeded synthetic inputs.  The
binding is imported lazily so that drawing inputs needs no CUDA library; any
call into the merge raises if the library has not been built.
"""
__all__ = ["ddmerge", "synth"]

"""ipkv — sequence-split decode attention over a write-time-partitioned KV cache (sm_100a).

``paper_2609_14507_b200.binding`` is the thin ctypes layer over the C-ABI library
(``include/ipkv.h``); ``paper_2609_14507_b200.synth`` draws the seeded synthetic inputs.
Importing the package loads nothing native; the binding loads ``libipkv.so`` on first use and
raises if it is missing.
"""
__all__ = ["binding", "synth", "build"]

"""TEST INFRASTRUCTURE — the float64 CPU oracle of the sequence-split decode-attention path.

Two independent statements of the same mathematics live here:

* ``ipkv_oracle.cpp`` (loaded through ctypes by :mod:`oracle.c_oracle`): plain C++ loops;
* :mod:`oracle.np_oracle`: NumPy float64, vectorised differently.

Nothing in the product imports this package; the CUDA library and the oracle share no code.
Only tests, the smoke check and the benchmark's CPU-baseline leg may use it.
"""

"""B200-native emulated oneshot all-reduce with dual buffering and speculative reduction.

``paper_2607_08973_b200.binding`` is the thin ctypes layer over ``libsifar.so``
(the CUDA library); ``paper_2607_08973_b200.synth`` holds the seeded input
generators.  Importing the package does not load the CUDA library; the first
call into the binding does, and raises if the library has not been built.
"""

"""B200-native FP-Sketch verifier: hand-written sm_100a kernels behind a C ABI.

``paper_2609_19758_b200.fpsk`` is the thin binding over the shared library
(it raises if the library has not been built); ``workloads`` holds the seeded
synthetic input generators.  Nothing is loaded at package import.
"""

"""B200-native hot path of Chiplet-Contiguous Layout (CCL).

``paper_2606_11718_b200.binding`` is the thin ctypes layer over the C-ABI library
(``include/ccl.h``); ``paper_2606_11718_b200.synth`` holds the seeded synthetic inputs.
Nothing is imported eagerly: the CUDA library is loaded on first use of the
binding and fails loudly if it has not been built.
"""

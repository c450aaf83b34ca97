"""B200-native Q4_K layer-window decoding (the GPU hot path of pipelined-ring inference).

``paper_2504_08791_b200.binding`` is the thin ctypes layer over the C-ABI library built from
``csrc/``; ``paper_2504_08791_b200.synth`` produces seeded synthetic inputs.  Importing the package
does not load the CUDA library; the first use of ``binding`` does, and fails loudly if it is absent.
"""

"""B200-native Sali-Cache pre-attention filter and mixed-precision K/V store.

``paper_2602_14236_b200.binding`` is the ctypes binding over the C-ABI library
(``libsalicache.so``); ``paper_2602_14236_b200.synth`` holds the seeded inputs.
"""

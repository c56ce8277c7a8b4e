"""Feature whitening by gradient transformation -- B200-native hot path.

`paper_2010_01546_b200.binding` is the thin ctypes layer over the C-ABI library
(include/fw.h); `paper_2010_01546_b200.synth` holds the seeded input
generators.  Importing the package does not load the CUDA library; the first
call into `binding` does, and raises if it is missing.
"""
__all__ = ["binding", "synth", "build"]

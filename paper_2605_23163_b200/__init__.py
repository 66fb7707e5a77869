"""B200-native decode hot path of block-diffusion driving VLAs (Fast-dDrive).

`paper_2605_23163_b200.fdd` is the thin binding over the C-ABI CUDA library
(csrc/, declared in include/fdd.h); `paper_2605_23163_b200.synth` makes the
seeded synthetic inputs.  There is no CPU fallback: using the binding without
the built library raises.
"""
__all__ = ["synth"]

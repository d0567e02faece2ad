"""B200-native (sm_100a) Key-Value Means attention layer.

`paper_2605_09877_b200.kvm` is the thin ctypes binding over the C-ABI CUDA library
(`include/kvm.h`); importing it fails loudly if the library has not been built.
`paper_2605_09877_b200.synth` holds the seeded input generators only.
"""
__all__ = ["synth"]

"""B200-native verify / accept / commit for gated-delta-rule speculative decoding.

The compute path is the CUDA library ``libspeca.so`` (C-ABI, ``include/speca.h``);
``binding`` marshals torch tensors into it and does nothing else.  There is no
CPU fallback: calling any operation without the built library raises.
``synth`` holds the seeded synthetic input generators (no method arithmetic).
"""
__all__ = ["binding", "synth", "build"]

"""B200-native MuLo-SD draft-and-verify round: CUDA kernels behind a C ABI.

``binding`` loads ``libmulo.so`` (built in-tree by ``build``) and exposes the
same calls the header declares.  There is no CPU fallback: using the binding
without the built library raises.
"""
__all__ = ["binding", "build", "synth"]

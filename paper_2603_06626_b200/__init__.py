"""B200-native routed SwiGLU expert layer under preemptive (frozen, cached) routing.

The product is the CUDA library under `csrc/` behind the C ABI declared in
`include/grouter.h`; `binding` marshals arguments to it and `synth` draws the
seeded synthetic inputs.  There is no CPU fallback: importing `binding` without
the built library raises.
"""
__all__ = ["synth"]

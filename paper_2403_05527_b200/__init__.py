"""B200-native GEAR hot path: KV-cache compression and decode attention over the
compressed cache (arXiv 2403.05527), as hand-written sm_100a CUDA behind a C ABI.

`paper_2403_05527_b200.binding` loads the shared library (lazily, on first use)
and exposes the C entry points under the same names; `synth` holds the seeded
input generators.  There is no CPU fallback: without the built library every
call raises."""
__all__ = ["binding", "synth"]

"""One EAGLE-3 speculative step (draft head + dynamic tree, tree-masked target
verification, greedy acceptance, KV compaction) as hand-written sm_100a CUDA
kernels behind a C-ABI library.

Sub-modules:
  synth    seeded synthetic inputs (weights, prompts, id maps); no method arithmetic
  binding  ctypes binding of the C-ABI library (argument marshalling only)

Nothing is imported eagerly: `synth` must stay usable on machines without the
compiled CUDA library, while `binding` fails loudly when the library is absent.
"""

__all__ = ["synth", "binding"]

"""B200-native speculative semantic-ID decode (NEZHA hot path).

Sub-modules:
  synth   -- seeded synthetic workloads (configs, weights, catalogues, histories); no method arithmetic.
  binding -- ctypes binding of the C-ABI library ``libnezha.so`` (argument marshalling only).

Nothing is imported eagerly so that ``synth`` stays usable without the CUDA library.
"""

__all__ = ["synth", "binding"]

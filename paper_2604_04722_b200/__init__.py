"""B200-native adaptive mixed-precision KV cache: controller decision, quantize-append and
decode attention over a segregated packed store, as hand-written CUDA behind a C ABI.

``synth`` (seeded inputs) imports nothing heavy; the CUDA library is loaded on first use of
``binding`` and raises if it has not been built -- there is no CPU fallback.
"""
__all__ = ["synth", "binding", "build"]

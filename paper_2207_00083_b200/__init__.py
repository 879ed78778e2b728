"""B200-native masked linear algebra (DarKnight's encode / linear / decode /
verify / wgrad path).  ``synth`` draws seeded inputs; ``binding`` is the thin
ctypes layer over the C-ABI library ``libdk.so`` built from ``csrc/``."""

__all__ = ["synth", "binding"]

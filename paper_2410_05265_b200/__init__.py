"""B200-native W4A4KV4 inference hot path of PrefixQuant (static per-tensor activations,
per-head static KV, prefixed outlier tokens kept in full precision).

``paper_2410_05265_b200.binding`` is the thin ctypes layer over the C-ABI CUDA library;
``paper_2410_05265_b200.inputs`` holds the seeded synthetic input recipes.
"""

__all__ = ["binding", "inputs", "build"]

"""B200-native verify step of Speech Speculative Decoding (SSD).

`synth` holds the seeded input generators; `binding` is the thin ctypes layer over the C-ABI
library built from `csrc/` (imported lazily: nothing here needs a GPU until it is called).
"""
__all__ = ["synth", "binding"]

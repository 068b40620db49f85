"""B200-native Ulysses attention prologue (QK RMSNorm + 2D RoPE, V-first
sequence-shard -> head-shard exchange, V-Major selection / compaction /
unpack) behind a C ABI.

`synth` is the seeded input recipe; `binding` is the thin ctypes layer over
libcocodiff.so (argument marshalling only).  Importing the package does not
load the CUDA library; `binding.lib()` does and raises if it is missing.
"""
__all__ = ["synth", "binding"]

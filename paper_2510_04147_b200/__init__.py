"""B200-native Self Speculative Decoding (SSD) verification path for masked-diffusion LMs.

`workloads` draws the seeded synthetic inputs; `binding` is the thin ctypes layer over the
C-ABI library built from `csrc/` (imported lazily: it fails loudly if the library is missing).
"""
__all__ = ["workloads"]

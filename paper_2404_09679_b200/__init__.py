"""B200-native BSP sparse-ranking hot path (AntDT, arXiv 2404.09679) behind a C-ABI library.

`binding` holds the thin ctypes layer over libantdt.so (same names as the C entry points);
`synth` holds the seeded input generators.  The CUDA library is loaded on first use and a
missing or unbuilt library is an error, never a fallback.
"""
__all__ = ["binding", "synth", "build"]

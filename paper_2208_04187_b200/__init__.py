"""B200-native DIVISION activation compress / decompress (hand-written sm_100a CUDA behind a C ABI).

`paper_2208_04187_b200.binding` is the thin ctypes layer over the shared library;
`paper_2208_04187_b200.synth` makes the seeded synthetic workloads.  There is no CPU fallback:
every call fails loudly if the CUDA library has not been built.
"""
__all__ = ["binding", "synth", "build"]

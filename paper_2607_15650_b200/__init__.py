"""B200-native (sm_100a) selective attention-state path of DiTango.

`paper_2607_15650_b200.binding` is the thin ctypes layer over the C-ABI library
(libditango.so); `paper_2607_15650_b200.inputs` holds the seeded synthetic workloads.
Importing the package loads nothing; the library is loaded on first use and its absence is
an error, never a fallback.
"""
__all__ = ["binding", "inputs"]

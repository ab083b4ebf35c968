"""B200-native 2:4-sparse ternary BitLinear (Sparse-BitNet hot path).

`paper_2603_05168_b200.binding` is the thin ctypes layer over the C-ABI library `libsbn.so`
(hand-written sm_100a CUDA); `paper_2603_05168_b200.inputs` holds the seeded input generators.
Importing this package loads nothing heavy; the library is loaded on first use of the binding.
"""
__all__ = ["binding", "inputs", "build"]

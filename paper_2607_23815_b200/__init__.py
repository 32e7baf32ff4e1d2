"""B200-native attention over a paged KV-cache pool (C-ABI library + thin binding).

Importing the package loads nothing heavy; ``paper_2607_23815_b200.kvattn`` loads
the CUDA shared library on first use and fails loudly if it is missing.
"""

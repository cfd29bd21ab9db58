"""B200-native verification step of judge decoding (arXiv 2501.19309).

``paper_2501_19309_b200.jd`` is the thin ctypes binding over the C-ABI library
built from ``csrc/``; ``paper_2501_19309_b200.inputs`` draws the seeded synthetic
workloads.  Importing the package loads nothing native; the library is loaded on
first use of the binding and its absence is an error, never a fallback.
"""
__version__ = "0.1.0"

"""Incremental depth-first CNN inference (Binas & Bengio, arXiv 1804.10727) on B200.

``paper_1804_10727_b200.idf`` is the thin binding over the C-ABI library
(``include/idf.h``); ``paper_1804_10727_b200.workloads`` holds the seeded
synthetic workloads.  The CUDA library is loaded on first use and there is no
CPU fallback: using the binding without the built library raises.
"""

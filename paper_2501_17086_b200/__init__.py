"""Highway backpropagation hot path on B200: Python binding over the C-ABI library.

``workloads`` (seeded synthetic inputs) imports without the CUDA library;
everything in ``binding`` needs ``libhbp.so`` and raises if it is missing.
"""

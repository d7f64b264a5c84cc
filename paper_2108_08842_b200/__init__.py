"""EDEN (arXiv 2108.08842) sender and receiver hot path as CUDA kernels for sm_100a.

``paper_2108_08842_b200.eden``   ctypes binding over libeden.so (needs the built library)
``paper_2108_08842_b200.synth``  seeded synthetic workloads (inputs only)
``paper_2108_08842_b200.build``  in-tree nvcc build of libeden.so
"""

"""B200-native GDN draft-tree verify + commit (tree-structured WY transform).

``binding`` wraps the C-ABI library ``libtreewy.so`` (hand-written sm_100a CUDA
kernels); ``workloads`` draws the seeded synthetic inputs; ``footprint`` holds the
byte accounting used by the bench.  Importing the package does not load CUDA.
"""
__all__ = ["binding", "workloads", "footprint"]

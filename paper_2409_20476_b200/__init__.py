"""B200-native GPU-initiated OpenSHMEM data path (after Intel SHMEM, arXiv 2409.20476).

``paper_2409_20476_b200.binding`` is the ctypes binding of the C-ABI library
``libishmem.so`` (built from ``csrc/`` for sm_100a); ``inputs`` holds the seeded
synthetic workloads.  Nothing here falls back to the CPU: using the binding
without the built library raises.
"""
__all__ = ["binding", "inputs", "build"]

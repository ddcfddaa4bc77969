"""B200-native receive-side data path of the Dynamic Bounded-Loss Protocol (DBLP).

The product is the C-ABI library built from ``csrc/`` (declared in ``include/dblp.h``); ``binding`` marshals
arguments to it, ``workloads`` states the seeded synthetic inputs.  Nothing here computes on the CPU: without the
CUDA library every call fails loudly.
"""

"""B200-native verified sparse-attention decode (vAttention, arXiv 2510.05688).

`binding` loads the C-ABI library (hand-written sm_100a kernels) and exposes the same entry
points; `synth` draws the seeded synthetic workloads.  Nothing here computes on the CPU:
using the decode path without the built CUDA library raises.
"""

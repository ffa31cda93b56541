"""Gradient dropping (Aji & Heafield 2017, Algorithm 1) as a CUDA library for B200 (sm_100a).

`binding` mirrors the C ABI of include/gd.h; `session` allocates the buffers the calls need;
`workloads` draws the seeded synthetic gradients used by the tests and the benchmark; `build`
compiles libgd.so in-tree.  Nothing here computes on the CPU.
"""
__all__ = ["binding", "session", "workloads", "build"]

"""Quantized GBDT training hot path for NVIDIA B200: C-ABI CUDA library + thin Python binding.

`binding` exposes the calls of include/qgbdt.h; `synth` generates the seeded synthetic
workloads; `build` compiles the library in-tree.  There is no CPU implementation here.
"""

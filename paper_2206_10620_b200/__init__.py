"""Pattern-pruned 3x3 convolution for NVIDIA B200: Python face of libpatconv.

`binding` wraps the C ABI (ctypes); `workloads` draws seeded synthetic layers;
`build` compiles the CUDA library in-tree.  Nothing here computes on the CPU.
"""

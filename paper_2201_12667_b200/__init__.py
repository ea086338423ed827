"""libdslide: a B200-native SLIDE adaptive-sparse training step.

`paper_2201_12667_b200.binding` is the thin ctypes layer over the C ABI in
include/dslide.h (it fails loudly when the CUDA library is missing);
`paper_2201_12667_b200.workloads` draws the seeded synthetic inputs.
Nothing is imported eagerly so that the input generators can be used
without the CUDA library.
"""
__all__ = ["binding", "workloads", "build"]

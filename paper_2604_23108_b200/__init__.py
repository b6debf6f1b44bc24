"""B200-native MoHGE expert layer (forward + backward) as a C-ABI CUDA library.

`paper_2604_23108_b200.binding` loads the shared library and exposes the same
entry points as `include/mohge.h`; `paper_2604_23108_b200.inputs` draws the
seeded synthetic workloads.  Importing the package itself loads nothing.
"""

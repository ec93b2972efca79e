"""B200-native DropCompute threshold-sweep simulator.

``paper_2306_10598_b200.api`` is the thin binding over the C-ABI library (it raises if the CUDA
library is missing); ``paper_2306_10598_b200.workloads`` holds the seeded synthetic inputs;
``paper_2306_10598_b200.build`` compiles the library in-tree.
"""
__all__ = ["api", "workloads", "build"]

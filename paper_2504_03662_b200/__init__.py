"""B200-native strategy search: batched cost model, layer-wise min-plus DP, plan backtrack.

`binding` wraps the C library (libgalv.so, CUDA sm_100a); `search` holds device
buffers for a workload and runs the path; `inputs` generates seeded workloads.
Importing the package loads nothing heavy; the CUDA library is opened on first use.
"""

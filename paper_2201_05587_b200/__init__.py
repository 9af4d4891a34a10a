"""Transfer-tuning's hot path on B200: fused DNN operators run under schedule records.

The CUDA library is loaded on first use of :mod:`paper_2201_05587_b200.binding`;
importing the package itself (for the input generators or the workload
inventories) needs no GPU.
"""

"""B200 (sm_100a) implementation of the PermuQuant per-group quantized linear layer.

`binding` exposes the C ABI of include/pq.h one to one; `pipeline` sequences those calls into
the offline calibration pass and the runtime linear; `inputs` draws the seeded synthetic
workloads.  Importing the package loads nothing: the CUDA library is opened on first use and
there is no fallback if it is missing.
"""
__all__ = ["binding", "inputs", "pipeline", "build"]

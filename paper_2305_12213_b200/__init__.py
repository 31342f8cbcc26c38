"""libdynbatch: the parameter-server step of dynamic-batching BSP training on B200.

`paper_2305_12213_b200.binding` wraps the C-ABI library (CUDA kernels for
sm_100a); `paper_2305_12213_b200.inputs` holds the seeded synthetic workloads.
Nothing is loaded at import time; the binding loads the shared library on
first use and raises if it has not been built.
"""
__all__ = ["binding", "inputs", "build"]

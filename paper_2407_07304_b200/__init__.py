"""SlimAttention over an INT8 KV cache: CUDA kernels for sm_100a behind a C ABI.

The kernels live in csrc/ and are built into libslim.so; `binding` is the
ctypes front end with the same entry-point names; `workloads` draws the seeded
synthetic inputs.  There is no CPU implementation here: calling an entry point
without the built library raises.
"""
__all__ = ["binding", "workloads"]

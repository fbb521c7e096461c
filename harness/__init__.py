"""Closed-loop harness around the C-ABI library: the device-side backend that bench.py, the smoke
run and the GPU tests drive, and the launcher that starts one process per GPU.

Nothing here computes any step of the method: the backend only owns torch buffers and forwards
them to the library; the launcher only starts processes.
"""
from .cuda_backend import CudaBackend, bits_to_device  # noqa: F401
from .launcher import rank_env, spawn_ranks  # noqa: F401

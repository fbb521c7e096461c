"""Seeded synthetic inputs shaped like multi-session agent memory.

This package only *generates inputs* (token corpora, per-stream scripts, bf16
noise logits, planting decisions).  It holds none of the method's arithmetic:
no automaton, no walk, no argmax, no accept.  Both the CPU oracle and the CUDA
path consume the bytes produced here; neither is imported from here.
"""
from .agent_memory import (  # noqa: F401
    CONFIGS,
    WorkloadConfig,
    ClosedLoopFeeder,
    f32_to_bf16_bits,
    bf16_bits_to_f32,
    make_corpus,
    make_noise_logits,
    make_open_loop_feed,
    make_scripts,
    zipf_cdf,
)
from .closed_loop import HostLogits, run_closed_loop, trace_stats  # noqa: F401,E402
from .device_noise import device_bits_to_host, make_noise_logits_device  # noqa: F401,E402

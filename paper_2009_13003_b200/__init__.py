"""LC-Checkpoint compress / recover passes for NVIDIA B200 (sm_100a).

``binding`` wraps the C ABI of ``liblc.so`` (see ``include/lc.h``); ``synth`` holds the seeded synthetic
workloads. Importing the package does not load the CUDA library; the first call into ``binding`` does.
"""
__all__ = ["binding", "synth", "build"]

"""Block-rotated MXFP4 W4A4 linear layer for NVIDIA B200 (sm_100a).

``binding`` wraps the C ABI of ``libbro.so`` (hand-written CUDA kernels); ``synth`` draws the
seeded synthetic inputs.  Importing ``binding`` fails loudly if the shared library has not been
built — there is no fallback implementation.
"""
__all__ = ["binding", "synth", "build"]

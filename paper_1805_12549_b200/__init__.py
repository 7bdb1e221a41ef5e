"""Channel-gated convolution (Channel Gating Neural Networks, arXiv 1805.12549) for NVIDIA B200.

`binding` wraps the C-ABI CUDA library (include/cgconv.h); `synth` draws the
seeded synthetic workloads.  Nothing is loaded until it is used.
"""
__all__ = ["binding", "synth", "build"]

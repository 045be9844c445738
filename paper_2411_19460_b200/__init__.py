"""libssd for B200: the Mamba-2 SSD selective-scan layer, forward and backward, driven under
Multi-Axis Gradient Checkpointing (sequence-axis state checkpoints at segment boundaries).

The arithmetic lives in hand-written sm_100a CUDA kernels behind a C ABI (include/ssd.h);
`paper_2411_19460_b200.libssd` is the thin ctypes binding.  There is no CPU fallback:
calling an op without the built shared library raises.
"""
__version__ = "0.1.0"

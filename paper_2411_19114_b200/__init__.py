"""Fused vision preprocessing for B200: ragged uint8 HWC batch -> dense NCHW fp32/fp16.

The work is done by a C-ABI CUDA library (``libpreba.so``, built from ``csrc/``);
``binding`` marshals arguments to it and nothing else.  ``workloads`` holds the
seeded synthetic inputs.  Importing the package does not load the library; the
first call does, and fails loudly if it has not been built.
"""
__all__ = ["binding", "workloads"]

"""B200-native training step (forward + backward) of a T5.1.1-style Transformer.

The compute lives in a C-ABI shared library built from `csrc/` (hand-written
sm_100a CUDA); `binding` marshals arguments to it.  Importing this package
does not load the library; `binding.lib()` does, and raises if it is missing.
"""
__all__ = ["binding", "workloads", "build"]

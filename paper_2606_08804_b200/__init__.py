"""B200-native (sm_100a) Q-Delta kernels: chunkwise forward/backward and the decode step.

The compute lives in ``libqdelta.so`` (hand-written CUDA behind a C ABI, declared in
``include/qdelta.h``); ``paper_2606_08804_b200.binding`` marshals torch device
pointers into it.  Importing the package does not load the library; the first call
does, and raises if the library has not been built.  ``inputs`` is the seeded
synthetic-input generator (numpy only).
"""
__all__ = ["binding", "inputs"]

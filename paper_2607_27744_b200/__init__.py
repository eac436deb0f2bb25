"""B200-native In-Kernel Broadcast Optimization (IKBO) kernels for ROCS request-candidate layers.

The compute lives in ``librocs.so`` (hand-written sm_100a CUDA behind a C ABI, see
``include/rocs.h``); :mod:`.binding` marshals torch device pointers into it and
:mod:`.workloads` draws the seeded synthetic inputs.  Importing the package does not load
the library; the first call does, and raises if it is missing.
"""

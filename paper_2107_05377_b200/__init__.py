"""Merged multi-task BERT forward pass on B200 (sm_100a).

The compute lives in the C-ABI library built from ``csrc/`` (see
``include/mt_bert.h``); ``binding`` is a thin ctypes wrapper with the same
names.  Importing this package does not load the library, so the seeded
generators in ``synth`` are usable on machines without CUDA.
"""

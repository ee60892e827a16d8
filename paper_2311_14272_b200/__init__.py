"""CRISP hybrid-sparse (block + N:M) weight format, mask projection and SpMM for B200.

The compute lives in ``libcrisp.so`` (hand-written CUDA for sm_100a, built from
``csrc/``); ``binding`` marshals arguments to its C ABI and nothing else.
"""
__all__ = ["binding", "workloads", "build"]

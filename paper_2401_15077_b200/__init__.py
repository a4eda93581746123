"""B200-native tree verification for EAGLE speculative decoding (tree-masked attention + acceptance).

The compute lives in ``libeagle_verify.so`` (hand-written CUDA for sm_100a behind a C ABI, see
``include/eagle_verify.h``); ``binding`` marshals torch device tensors into it.  Importing this
package does not load the library; the first call does, and raises if it is missing (there is no
CPU or PyTorch fallback).
"""
__all__ = ["binding", "workloads"]

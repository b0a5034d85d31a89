"""B200-native post-prefill KV-cache compression pass of ReFreeKV (arXiv 2502.16886).

The compute lives in a C-ABI CUDA library (``csrc/``); ``binding`` marshals
torch tensors into it and ``workloads`` draws the seeded synthetic caches.
Importing the package does not load the CUDA library; the first call into
``binding`` does, and raises if it has not been built.
"""

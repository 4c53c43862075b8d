"""B200-native flash-attention forward (bf16, causal / GQA, log-sum-exp output).

The compute path is a CUDA library for sm_100a behind a C ABI
(``include/ave_attn.h``); ``binding`` marshals torch tensors into it and
``inputs`` generates the seeded synthetic workloads.  Importing the package
does not load the CUDA library; the first call into ``binding`` does, and it
raises if the library has not been built.
"""
__version__ = "0.1.0"

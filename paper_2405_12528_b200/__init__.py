"""B200-native retention pass of SirLLM (token entropy, decay, top-k selection, KV compaction).

The work is done by hand-written CUDA kernels behind a C ABI (``include/sirllm.h``);
``paper_2405_12528_b200.binding`` marshals torch device tensors into those calls.
Importing the package does not load the CUDA library; the first call does, and it
raises if the library has not been built (there is no CPU fallback).
"""

__all__ = ["binding", "workloads", "build"]

"""KeepKV hot path for NVIDIA B200 (sm_100a): Electoral-Votes decode attention and
periodic ZIP-merge compression of a bf16 KV cache, as hand-written CUDA behind a
small C ABI (``include/keepkv.h``).

``paper_2504_09936_b200.binding`` marshals torch tensors into that C ABI;
``paper_2504_09936_b200.workloads`` draws the seeded synthetic inputs.  Nothing
here computes on the CPU: without the compiled CUDA library every call raises.
"""

__all__ = ["binding", "workloads"]

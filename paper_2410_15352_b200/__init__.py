"""B200-native CompAct compressed linear layer (arxiv 2410.15352).

`binding` wraps the C-ABI library libcompact.so; `workloads` draws the seeded
synthetic inputs.  Nothing here computes on the CPU: if the CUDA library is
missing, loading it raises.
"""
__all__ = ["binding", "workloads", "build"]

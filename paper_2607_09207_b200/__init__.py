"""libpdattn: paged decode attention for RL rollout on B200 (sm_100a).

`paper_2607_09207_b200.pdattn` is the ctypes binding of the C-ABI library (it raises if the
CUDA library has not been built: there is no CPU fallback); `paper_2607_09207_b200.workloads`
makes seeded synthetic inputs and imports neither the library nor the oracle.
"""
__all__ = ["pdattn", "workloads"]

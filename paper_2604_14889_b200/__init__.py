"""MemoSight per-step attention hot path for B200 (sm_100a).

The CUDA library is loaded on first use of :mod:`paper_2604_14889_b200.binding`;
importing the package itself touches neither CUDA nor the oracle.
"""
__all__ = ["binding", "synth", "build"]

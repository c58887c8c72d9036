"""BlockFFN chunk-verify FFN forward for B200 (sm_100a).

The CUDA library is loaded lazily by :mod:`paper_2507_08771_b200.binding`; importing
the package (for example to reach :mod:`paper_2507_08771_b200.inputs`) loads nothing.
"""
__all__ = ["binding", "inputs"]

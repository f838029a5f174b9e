"""B200-native semi-naive fixpoint engine for tagged Datalog rules.

``paper_2609_27203_b200.xlog`` is the thin ctypes binding over ``libxlog.so`` (the C ABI
in ``include/xlog.h``); ``synth`` / ``workloads`` generate the seeded benchmark inputs.
The CUDA library is loaded on first use and its absence is an error: there is no CPU path.
"""
__all__ = ["xlog", "synth", "workloads"]

"""B200-native LocMoE router path: GrAP gate, capacity rule, capacity-bounded
routing into an All-to-All shaped buffer, dispatch and gate-weighted combine.

``paper_2401_13920_b200.binding`` is the Python face of the C-ABI library
(``include/locmoe.h``); ``paper_2401_13920_b200.workloads`` draws the seeded
synthetic inputs.  There is no CPU fallback: calling the binding without the
compiled CUDA library raises.
"""
__all__ = ["binding", "workloads", "build"]

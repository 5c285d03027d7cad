"""B200-native per-layer path of distributed auto-differentiation (dAD / rank-dAD).

`libdad` (C ABI, hand-written sm_100a CUDA) is reached through :mod:`paper_2102_09631_b200.binding`;
:mod:`paper_2102_09631_b200.workloads` holds the seeded synthetic input generators.
"""
__all__ = ["binding", "workloads"]

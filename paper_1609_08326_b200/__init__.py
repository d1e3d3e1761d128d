"""DC-ASGD parameter-server update for NVIDIA B200 (sm_100a).

`binding`  - the `dcasgd_*` calls of the C-ABI server library (CUDA kernels)
`synth`    - seeded synthetic inputs (vectors, gradient pools, worker event logs)
`build`    - in-tree build of the native parts
"""
__all__ = ["binding", "synth", "build"]

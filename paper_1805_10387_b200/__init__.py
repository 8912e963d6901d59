"""Mixed-precision training step of a stack of linear layers on B200 (sm_100a).

`paper_1805_10387_b200.mp` binds the C-ABI library (CUDA kernels);
`paper_1805_10387_b200.synth` draws the seeded synthetic workloads.
Nothing is imported eagerly, so that drawing inputs needs no CUDA library.
"""

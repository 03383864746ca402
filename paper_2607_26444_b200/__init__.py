"""B200-native MoE routing layout, token dispatch and gate-weighted combine.

The CUDA path lives in ``csrc/`` behind a C-ABI shared library; ``binding``
marshals arguments to it and nothing more.  ``workloads`` only generates
seeded inputs.  Nothing here falls back to a CPU implementation: calling the
binding without the built library raises.
"""

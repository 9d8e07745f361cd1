"""SharePrefill prefill-attention hot path for NVIDIA B200 (sm_100a).

`synth` makes seeded synthetic workloads; `binding` marshals arguments into the
C-ABI shared library built from `csrc/` (there is no CPU fallback: calling the
binding without the built library raises).
"""

"""B200-native LASAD operator: causal linear attention with Spatial-Aware Decay.

The product is the C-ABI library built from ``csrc/`` (``lasad_forward`` for chunked prefill,
``lasad_decode_step`` for one-token generation against a persistent fp32 state).  ``binding``
is the thin argument-marshalling layer over it; ``workloads`` draws seeded synthetic inputs.
Nothing here falls back to a CPU implementation: a missing or stale library raises.
"""
__all__ = ["binding", "workloads", "build"]

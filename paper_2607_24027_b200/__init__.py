"""B200 (sm_100a) implementation of the Sol-Attn fused sparse-attention forward pass.

The compute lives in ``libsol_attn.so`` (hand-written CUDA, C ABI declared in
``include/sol_attn.h``); ``binding`` marshals torch tensors into it.  There is no CPU
fallback: importing ``binding`` without the built library raises.
"""
__all__ = ["binding", "configs", "synth", "build"]

"""HiFA4 hot path for B200 (sm_100a): Smooth-QK + HIF4 quantization of Q/K/V and a fused
4-bit-operand prefill attention forward, behind a C-ABI library (see include/hifa4.h).

Importing the package does not load the CUDA library; `paper_2607_04302_b200.binding`
loads it on first use and raises if it is missing (there is no CPU fallback)."""

__all__ = ["binding", "synth"]

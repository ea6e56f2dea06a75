"""Seeded synthetic inputs shaped like the paper's 35B-class MoE workloads.

This package only draws random tensors and formats them (bf16 / fp16 bit
patterns, packed int4 bytes).  It holds none of the method's arithmetic:
no routing, no dequantisation, no FFN.  Both the CPU oracle's tests and the
CUDA path's tests and benchmark take their inputs from here.
"""

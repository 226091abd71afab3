"""B200-native batch LoRA inference (EdgeLoRA, Section 3.4): a LoRA-augmented linear
layer over a mixed batch of tokens, each token carrying its own adapter slot id.

``binding`` wraps the C-ABI library (CUDA kernels for sm_100a); ``workloads`` holds the
seeded synthetic input generators.  Nothing here computes on the CPU.
"""
__all__ = ["binding", "workloads"]

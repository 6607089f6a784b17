"""B200-native hot path of the LVSpec verify step: verification attention with
fused visual mass, and the loose acceptance pass (Sec. 3 of the paper).

Importing the package does not load the CUDA library; ``binding`` does, and it
raises if the library is missing."""
__all__ = ["workloads"]

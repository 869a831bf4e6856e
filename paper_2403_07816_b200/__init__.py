"""B200-native MoE feed-forward hot path of Branch-Train-MiX (arXiv 2403.07816).

The compute lives in a C-ABI CUDA library (csrc/, built in-tree as libbtx.so); `binding`
marshals torch tensors into it.  Importing the package does not load the library, so the
input generators in `synth` can be used on machines without a GPU.
"""
__all__ = ["synth", "binding"]

"""B200-native run-time path of Binarized Neural Networks (binary GEMM and the layers fused around it).

The compute lives in a C-ABI CUDA library (``csrc/``, built in-tree as ``libbnn_b200.so``);
``binding`` marshals arguments to it and nothing else.  Importing this package does not load
the library; the first call does, and fails loudly if it has not been built.
"""
__all__ = ["binding", "workloads", "build"]

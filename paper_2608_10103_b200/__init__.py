"""B200-native dense GEMM C = A * B^T in FP16, INT8 and packed INT4.

The compute lives in libb200gemm.so (hand-written CUDA for sm_100a, built by
`python -m paper_2608_10103_b200.build`); `binding` marshals arguments to its
C entry points, `synth` draws seeded synthetic operands.
"""
__all__ = ["binding", "build", "synth"]

"""B200-native deterministic fused-upcast linear layer (hand-written CUDA for sm_100a behind a C ABI).

The CUDA library is loaded lazily by `paper_2609_25624_b200.binding`; importing the package or its
`inputs` module does not touch CUDA.
"""
__all__ = ["binding", "inputs", "build"]

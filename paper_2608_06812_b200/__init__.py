"""FP64 GEMM emulated on B200 FP4 tensor cores (Ozaki scheme II, base-13 E2M1 limbs).

The CUDA library is loaded lazily by `paper_2608_06812_b200.binding`; importing
this package or its `inputs` module does not need a GPU.
"""
__all__ = ["binding", "inputs"]

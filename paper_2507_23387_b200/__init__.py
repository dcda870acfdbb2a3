"""SGEMM-cube for NVIDIA B200 (sm_100a): FP32 GEMM rebuilt from three FP16 tensor-core products.

The public names are the C-ABI entry points of libsgemm_cube.so, re-exported by the thin
binding in `paper_2507_23387_b200.binding` (argument marshalling only).  The CUDA library is loaded on
first use; there is no CPU fallback: without the library every call raises.
"""
__all__ = ["binding", "inputs"]

"""B200-native folded quantized linear layer (FWHT + per-token quantization +
integer GEMM + dequant epilogue) behind a C-ABI shared library.

``paper_2609_24433_b200.fq`` is the ctypes binding (loads the CUDA library on
first use and raises if it is missing); ``paper_2609_24433_b200.synth`` holds
the seeded input generators; ``paper_2609_24433_b200.replicas`` the host-side
bookkeeping for one-process-per-GPU replicas.
"""
__all__ = ["fq", "synth", "replicas"]

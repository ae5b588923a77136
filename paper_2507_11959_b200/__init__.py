"""B200-native PoT-PTQ inference kernels: packed power-of-two weight codes -> FP16/BF16,
standalone and fused into GEMV / GEMM.  The CUDA library is loaded on first use by
``paper_2507_11959_b200.binding``; importing the package itself touches no GPU code."""

"""CPU oracle for the quantized adaptive-subgradient step (QCMD / QRDA adagrad).

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only the
tests, the smoke check and the benchmark's CPU-baseline leg call it.  It is a plain,
slow, single-threaded numpy restatement of the paper's definitions (fp64 wherever the
method is floating point; fp32 only where a floating-point comparison decides an
integer code, so that the decision is taken in the precision the kernels use).
It shares no code, tables or helpers with the CUDA path.
"""

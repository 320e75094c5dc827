"""B200-native library for the per-iteration hot path of QCMD adagrad / QRDA adagrad:
quantize each worker's gradient to 2-bit codes + scale, decode and average, update the
diagonal AdaGrad accumulator, apply the closed-form L1-proximal update.

`libqasg`  - thin ctypes binding of the C-ABI shared library (argument marshalling only;
             every step runs in the CUDA kernels; there is no CPU fallback).
`inputs`   - seeded synthetic inputs (no arithmetic of the method).
"""
__all__ = ["libqasg", "inputs"]

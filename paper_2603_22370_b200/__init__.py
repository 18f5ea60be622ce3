"""B200-native kernels for one FAAR layer-wise rounding-optimisation step
(NVFP4 soft-quantisation, forward GEMM + MSE, dW GEMM + dV + update, harden
and pack).  The compute lives in the CUDA library `libfaar.so` behind a C ABI;
`paper_2603_22370_b200.faar` is the thin ctypes binding.  Importing this
package does not load the library; `faar.lib()` does, and raises if it is
missing."""

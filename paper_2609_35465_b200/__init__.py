"""B200-native fused decode-and-multiply GEMV for 48-bit Tetra (Leech-lattice) codes.

Submodules:
  synth   seeded synthetic inputs (no method arithmetic)
  shapes  workload shapes and byte accounting
  tetra   ctypes binding of the C-ABI CUDA library (loaded on first use; raises
          if the library has not been built -- there is no CPU fallback)
"""
__all__ = ["synth", "shapes", "tetra"]

"""B200-native hot path of full-graph GCN training (sparse aggregation + dense update).

Sub-modules:
  synth    seeded synthetic inputs (no arithmetic of the method; no native code needed)
  build    compiles the CUDA library ``libmixgcn.so`` for sm_100a in-tree
  binding  thin ctypes binding of the C-ABI in ``include/mixgcn.h`` (argument marshalling only)

Importing ``binding`` fails loudly when the CUDA library has not been built: there is no CPU
or PyTorch fallback for any step of the path.
"""
__all__ = ["synth", "build", "binding"]

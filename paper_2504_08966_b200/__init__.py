"""B200-native PACT visual-token reduction (EUTI pruning + DBDPC clustering + merge).

The product is the CUDA library `libpact.so` (C ABI in include/pact.h); `binding` is a thin
ctypes layer with the same call names that only marshals arguments.  Importing the package
does not load the library; `binding.lib()` does, and fails loudly if it is missing.
"""
__all__ = ["binding", "workloads", "build"]

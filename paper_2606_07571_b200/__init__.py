"""B200-native BiCache attention hot path: a C-ABI CUDA library plus a thin
ctypes binding.  Importing the package is cheap; the shared library is loaded
on first use of `binding` and a missing library is a hard error (there is no
CPU fallback)."""

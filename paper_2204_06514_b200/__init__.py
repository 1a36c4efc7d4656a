"""B200 (sm_100a) CUDA library for the single-device decoder-only Transformer
training step, with its ctypes binding.  Importing the package does not load
the library; `binding.load_library()` does, and raises if libfax.so is absent
(there is no CPU or framework fallback)."""

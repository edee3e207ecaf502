"""B200-native SparseLoCo outer step: C-ABI CUDA library + thin Python binding.

`inputs` holds the seeded synthetic generators; `binding` (imported on demand) wraps the
C-ABI of the CUDA shared library and raises if that library is missing -- there is no CPU
fallback.
"""

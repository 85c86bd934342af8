"""B200-native best-matching-unit (BMU) search for sparse-binary self-organizing maps.

Sub-modules (imported on demand, nothing heavy happens at package import):

* ``som``    - thin ctypes binding over the C-ABI CUDA library (``include/som.h``).
               It raises if the compiled library is missing: there is no CPU fallback.
* ``synth``  - seeded synthetic workload generators (codebook fill, Zipf CSR batches).
               Pure data generation; contains none of the search arithmetic.
* ``build``  - compiles the CUDA library in-tree for sm_100a with nvcc.
"""

__all__ = ["som", "synth", "build"]

"""B200-native RegTop-k sparsification step (arXiv 2501.05633, Algorithm 2) behind a C ABI.

`binding` marshals torch tensors into the C calls of include/regtopk.h; every step of the method runs
in the CUDA library (csrc/regtopk.cu).  `synth` holds the seeded synthetic input generators; it
contains none of the method's arithmetic.
"""
from .binding import RegTopK, aggregate_pairs_static, build, load_library, library_path  # noqa: F401

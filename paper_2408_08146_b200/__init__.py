"""B200-native draft-then-verify step of speculative decoding with K-layer draft heads.

The product is libkoala.so (CUDA, sm_100a; sources under csrc/, C ABI in include/koala.h);
`binding` marshals arguments to it.
"""
from .binding import (KOALA_BF16, KOALA_EAGLE, KOALA_F_NO_PDL, KOALA_F_NO_TENSOR_CORES, KOALA_FP32,  # noqa: F401
                      KOALA_MEDUSA, Koala, KoalaError, koala_gemm_bf16, koala_workspace_bytes, load_library)

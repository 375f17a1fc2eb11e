"""B200-native Encode stage (micro-batched encoder forward pass) behind a C ABI.

`binding` mirrors the entry points declared in include/eas_encoder.h; every step of the forward
pass runs in the CUDA library.  There is no CPU fallback: loading fails loudly when the library
has not been built (python -m paper_2609_31551_b200.build)."""
from .binding import (Encoder, EasError, load_library, pack_items, kernel_gemm, kernel_norm,  # noqa: F401
                      kernel_attention, weights_to_device, SmPartition)

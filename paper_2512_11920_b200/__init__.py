"""speckv: B200-native KV-cache page codec (compress, decompress+gather, translate).

The compute lives in libspeckv.so (hand-written CUDA for sm_100a behind a C ABI, see
include/speckv.h); `binding` marshals torch tensors into it.  There is no CPU fallback: if
the library is missing or the device is not a B200-class GPU, calls raise.
"""
from .binding import (Context, SpeckvError, PREFETCH_DTYPE, VADDR_DTYPE, PADDR_DTYPE, load_library,  # noqa: F401
                      RAW, INT8, INT8_DELTA, INT8_DELTA_RLE, AUTO, GROUPED, compress_static, STATIC_MAX_PAGES, CTL_BLOCK_BYTES,
                      probe_pages, select_scheme, PROBE_DTYPE, CANDIDATE_SCHEMES)

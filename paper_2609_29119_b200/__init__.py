"""B200-native invertible constant-Q transform: thin Python binding over the C-ABI CUDA library."""
from .binding import (CqtError, Plan, SliCQ, lib_path, load_library, multires_bands,  # noqa: F401
                      WIN_HANN, WIN_BLACKMAN_HARRIS, M_MULT4, M_SMOOTH, M_POW2)

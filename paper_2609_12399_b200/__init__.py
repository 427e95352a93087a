"""B200-native (sm_100a) beam-shared Gated DeltaNet decode: ctypes binding over libonela.so.

The library is loaded on first use (``load_library``), never at import, and there is no fallback if
it is missing.  ``inputs`` holds the seeded synthetic workloads and none of the method's arithmetic.
"""
from . import inputs  # noqa: F401
from .binding import (DTYPE_BF16, DTYPE_F32, FLAG_DRY_RUN, FLAG_FORCE_GENERIC, FLAG_GTR_DELTA, FLAG_SHARED_CHAINS, MAX_BATCH, Onela, OnelaConfig,  # noqa: F401
                      OnelaError, load_library, make_config, onela_select_beams_static, onela_workspace_bytes, status_string)

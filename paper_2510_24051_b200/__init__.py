"""B200-native batched `forward` attention handler (KvPage append + masked paged attention).

The work is done by libpie_b200.so (hand-written sm_100a CUDA behind a C ABI, declared in
include/pie_b200.h); this package only marshals arguments.  Importing it loads the library
and fails loudly if that is impossible: there is no CPU or library fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import LIB_PATH, PieError, lib  # noqa: F401

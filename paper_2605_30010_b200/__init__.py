"""B200-native compressed video vision-encoder (EarlyTom hot path).

The product is the C-ABI shared library built from csrc/ (see include/earlytom.h); this package
is its thin Python binding.  Importing `binding` loads the library and fails loudly if it is
missing; nothing here computes on the CPU.
"""
from . import binding  # noqa: F401
from .binding import (Encoder, EarlyTomError, ForcedPlan, HostBuffers, Result, Trace, ET_BF16, ET_F32)  # noqa: F401

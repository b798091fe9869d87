"""B200-native PowerSGD+ gradient compression: thin Python binding of libpsgd.so.

Every step of the path runs in the CUDA library; this package only marshals
arguments (torch tensors -> device pointers, torch streams -> cudaStream_t).
There is no CPU fallback: using the binding without the built library raises.
"""
from .binding import (  # noqa: F401
    PSGDError,
    PowerSGDPlus,
    StepGroup,
    lib,
    library_path,
    PSGD_W_RANK_DEFICIENT,
    PSGD_W_NOT_CONVERGED,
    PSGD_W_TIMEOUT,
    KERNEL_FAMILIES,
)
from .stack import StreamedStack  # noqa: F401,E402
from .exchange import ExchangedStack, slot_offsets  # noqa: F401,E402

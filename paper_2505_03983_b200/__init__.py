"""B200 (sm_100a) Autospeculative Decoding for DDPMs: thin Python binding over the C ABI
declared in include/asd.h.  All arithmetic runs in the CUDA library; this package only
marshals arguments (torch supplies device memory and the stream)."""
from .binding import (  # noqa: F401
    AsdError, AsdSampler, RoundStats, RunStats, lib_path, load_library, EXPORTED_SYMBOLS, ddpm_schedule,
)

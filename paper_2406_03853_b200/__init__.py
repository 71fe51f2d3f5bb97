"""B200-native EESD decode round: thin Python binding over the C-ABI CUDA library."""
from .binding import (Config, Engine, EesdError, Stats, accept_resample, lib, lib_path, project_rows, sample_rows)  # noqa: F401

"""libsds: speculative sampling for diffusion chains on one B200 (CUDA kernels behind a C ABI)."""
from .binding import *  # noqa: F401,F403
from .binding import Sampler, SdsError, load, lib_path  # noqa: F401
from .presets import sampler_for, schedule_for, drafter_for, picard_for  # noqa: F401
from . import schedules  # noqa: F401
from .schedules import projection_basis  # noqa: F401

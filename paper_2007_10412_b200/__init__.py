"""RAD activation sampling for B200 (sm_100a): Python binding over the C ABI in include/rad.h."""
from .binding import *  # noqa: F401,F403
from .binding import lib, Store, MLPStep, IRNNStep, CNNStep, RadError  # noqa: F401

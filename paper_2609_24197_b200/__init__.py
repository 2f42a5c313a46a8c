"""H-Spec block-parallel draft step for one B200 (sm_100a): Python binding over libhspec.so."""
from .binding import *  # noqa: F401,F403
from .binding import Drafter, HSpecError, EXPORTS, LIB_PATH, load_library, make_config  # noqa: F401

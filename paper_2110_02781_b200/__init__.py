"""B200-native per-stage training library (C ABI in include/ftpipe.h) and its thin Python binding."""
from . import ftpipe          # noqa: F401
from .ftpipe import *         # noqa: F401,F403

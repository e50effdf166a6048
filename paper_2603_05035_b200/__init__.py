"""B200-native GELO obfuscated Q/K/V offload: Python binding of the C-ABI library."""
from . import inputs  # noqa: F401
from .binding import *  # noqa: F401,F403

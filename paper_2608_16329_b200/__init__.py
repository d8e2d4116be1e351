"""B200-native hot path of the small-footprint MLIP: C-ABI CUDA library plus a thin binding."""
from . import binding, decomposition  # noqa: F401
from .binding import *  # noqa: F401,F403

binding.lib()  # fail loudly at import if the CUDA library has not been built

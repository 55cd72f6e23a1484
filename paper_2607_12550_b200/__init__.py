"""B200-native JoLT / FlashJoLT KV-cache compressor: C-ABI CUDA library plus a thin ctypes binding."""
from . import synth  # noqa: F401


def load():
    """Import the binding (raises if the CUDA library has not been built)."""
    from . import binding
    return binding

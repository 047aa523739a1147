"""B200-native corrected low-bit KV-cache chunk attention (libkvq) and its Python binding."""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding", "build"]

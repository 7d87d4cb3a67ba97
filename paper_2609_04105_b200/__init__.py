"""B200-native full-FP4 attention forward with Direct-P (C-ABI library + thin binding)."""
from . import inputs  # noqa: F401

__all__ = ["inputs"]

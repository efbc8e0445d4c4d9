"""CPU oracle of the fused linear operator (test infrastructure, never a product path)."""
from .fused_linear import (act, build, fused_linear, threads)  # noqa: F401

"""Seeded synthetic input generators (no arithmetic of the method lives here)."""
from .gen import *  # noqa: F401,F403
from .gen import CONFIGS, ModelShape  # noqa: F401

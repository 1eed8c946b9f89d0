"""CPU oracle package (test infrastructure; see minicache_oracle.py)."""
from .minicache_oracle import *  # noqa: F401,F403
from . import minicache_oracle  # noqa: F401

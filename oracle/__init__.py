"""CPU checker for the DIVISION compress/decompress pair (test infrastructure, not product code)."""
from .division_oracle import *  # noqa: F401,F403

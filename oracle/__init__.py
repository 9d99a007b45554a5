"""CPU oracle (test infrastructure).  See fls_oracle.py."""
from . import fls_oracle  # noqa: F401

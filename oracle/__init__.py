"""CPU oracle (test infrastructure only): see criticalkv_oracle.py."""
from . import criticalkv_oracle  # noqa: F401

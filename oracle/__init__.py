"""CPU oracle (test infrastructure only; the product library never imports this package)."""
from .oracle import *  # noqa: F401,F403

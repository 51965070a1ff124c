"""CPU oracle (test infrastructure only; never imported by the product path)."""
from .quasar_oracle import *  # noqa: F401,F403
from .build import build_model  # noqa: F401

"""CPU oracle (test infrastructure only; never imported by the product path)."""
from .quasar_oracle import *  # noqa: F401,F403
from .build import build_model, quantize_rows_in_parallel  # noqa: F401

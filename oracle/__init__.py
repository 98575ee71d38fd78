"""CPU oracle (test infrastructure only; the CUDA path never imports this)."""
from .think_oracle import *  # noqa: F401,F403
from .think_oracle import ThinKOracle  # noqa: F401

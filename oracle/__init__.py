"""CPU oracle (test infrastructure only; never imported by the CUDA library)."""
from .litevggt_oracle import *  # noqa: F401,F403
from . import litevggt_oracle  # noqa: F401

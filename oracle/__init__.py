"""CPU oracle (test infrastructure): see mnnllm_oracle.cpp.  Only tests, the smoke check and the
benchmark's CPU-baseline legs may import this package."""
from .oracle import *  # noqa: F401,F403

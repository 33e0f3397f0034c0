"""CPU oracle for the Q-GaLore per-step optimizer update.

TEST INFRASTRUCTURE ONLY. Nothing in the product path may import this package;
it exists so that the CUDA path can be compared, element by element, with a
plain and slow restatement of the method.  It shares no code with the CUDA
path and never imports it.
"""
from .qgalore_oracle import *  # noqa: F401,F403

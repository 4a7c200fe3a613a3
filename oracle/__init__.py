"""TEST INFRASTRUCTURE: the CPU oracle of the Transactional Attention retention step.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package. It shares no code with
the CUDA library and never imports it.
"""
from .ta_oracle import *  # noqa: F401,F403

"""CPU oracle for the DS-MoE layer.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline legs of
``bench.py`` may import this package; the CUDA product path never does.
"""
from .dsmoe_oracle import *  # noqa: F401,F403

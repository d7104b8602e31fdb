"""TEST INFRASTRUCTURE: Python access to the CPU oracle (``sop_oracle.cpp``).

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline / reference legs may
import this package.  It never imports the CUDA binding and the CUDA binding never imports it.
"""
from .binding import *  # noqa: F401,F403

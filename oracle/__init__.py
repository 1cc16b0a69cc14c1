"""CPU oracle for the CATS tree-verification forward (test infrastructure only).

Only the test-suite, ``__graft_entry__.smoke()`` and the benchmark's CPU-baseline
leg may import this package.  It shares no code with the CUDA library.
"""
from .ref import *  # noqa: F401,F403

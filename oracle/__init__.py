"""CPU fp64 oracle for the rotated-MXFP4 linear layer (test infrastructure only).

Nothing in the product package imports this; only the tests, the smoke check and
the benchmark's cpu_baseline / reference legs do.
"""
from .torq_oracle import *  # noqa: F401,F403
from .nvfp4_oracle import *  # noqa: F401,F403,E402
from .givens_oracle import *  # noqa: F401,F403,E402
from .mxint4_oracle import *  # noqa: F401,F403,E402

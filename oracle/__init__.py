"""EOQ oracle (test infrastructure, not product code).

A slow CPU statement of the EOQ 8-bit training layer of arXiv 2105.13890, used
only by the tests, the smoke check and the CPU-baseline leg of the benchmark.
"""
from .eoq_oracle import *  # noqa: F401,F403
from . import eoq_network as network  # noqa: F401,E402

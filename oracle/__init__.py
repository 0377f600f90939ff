"""Reference oracle: a plain, slow, float64 CPU statement of what the training path computes.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports, calls or links this
code; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.  It
shares no code with the CUDA library.

Pin status (see tests/test_oracle_*.py):
  ops forward/backward, loss, SGD, stage split, capacity estimate, partition optimiser,
  redistribution without failure, snapshot, schedules, the state variables of Table I and the
  three outcomes of the fault handler's probe (recovery.py) ........ pinned
  redistribution with a failed index (Algorithm 1, I_fail >= 0) and recovery sources after
  failures (Sec. III-F) ... parity unpinned beyond invariants, the prose rules of Sec. III-F and
  the agreement of the prose plan with Algorithm 1 (the worked figures are not available)
  asynchronous 1F1B schedule with weight stashing, vertical sync and aggregation (schedule.py,
  Sec. III-C) ... the order of passes and the version numbers are pinned on the paper's prose
  example (stage 0 of three); what "aggregate" computes, when, and vertical sync on later stages
  are readings (listed in schedule.py): parity unpinned for those
"""
from .ops import *          # noqa: F401,F403
from .model import OracleModel   # noqa: F401
from .partition import *    # noqa: F401,F403
from . import recovery      # noqa: F401
from . import schedule      # noqa: F401

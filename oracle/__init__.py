"""CPU oracle of the batch-1 decode step (test infrastructure only).

Only tests/, __graft_entry__.smoke() and bench.py's CPU-baseline legs may import this package.
It does not import the CUDA package and shares no code with it.
"""
from .binding import OracleModel, build_oracle, lib  # noqa: F401

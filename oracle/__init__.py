"""CPU oracle of the allocation search.  Test infrastructure only: imported by
``tests/``, by ``__graft_entry__.smoke`` and by the CPU-baseline legs of
``bench.py``; never by the product package."""
from .loki_oracle import build, solve, result_to_dict, OracleResult  # noqa: F401

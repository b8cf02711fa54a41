"""CPU oracle of the verification step.  Test infrastructure only: imported by tests,
the smoke check and the benchmark's CPU-baseline leg, never by the product package."""
from .oracle import Oracle, OracleResult, verify_greedy  # noqa: F401

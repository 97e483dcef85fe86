"""CPU oracle for fused-subgraph execution.  Test infrastructure only: imported by tests/, by the
smoke check and by the benchmark's CPU-baseline leg, never by the product path."""
from .interp import run, Value  # noqa: F401

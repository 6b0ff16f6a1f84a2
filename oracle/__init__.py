"""fp64 CPU oracle of the QA-LoRA layer.  Test infrastructure only: imported by
tests, the smoke check and the benchmark's CPU-baseline leg, never by the
product path."""
from . import qalora_oracle  # noqa: F401

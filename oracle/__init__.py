"""fp64 CPU oracle of the QA-LoRA layer and of the adapter update.  Test infrastructure only: imported by
tests, the smoke check and the benchmark's CPU-baseline leg, never by the
product path."""
from . import optimizer_oracle, qalora_oracle  # noqa: F401

"""fp64 CPU oracle of the SFB minibatch step.  Test infrastructure only: imported by tests/, the smoke check
and the bench's CPU-baseline leg; never by the CUDA product path."""
from .sfb_oracle import *  # noqa: F401,F403

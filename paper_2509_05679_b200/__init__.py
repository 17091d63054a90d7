"""fdg: stale-gradient decoupled training step for sm_100a (see include/fdg.h)."""
from . import synth  # noqa: F401

"""Seeded synthetic repair instances and their plain data model.

Shared by the CPU oracle's wrapper and by the CUDA binding; holds none of the
repair method's arithmetic (no counting, enumeration, ranking or candidate
evaluation)."""
from .model import *          # noqa: F401,F403
from .configs import *        # noqa: F401,F403

"""Synthetic workloads (configurations and seeded input generators). Holds no method arithmetic."""
from .configs import *  # noqa: F401,F403
from .configs import KoalaConfig, CONFIGS, TINY_EAGLE, TINY_MEDUSA, T7_MEDUSA, T7_EAGLE, T13_EAGLE, T33_EAGLE, reduced  # noqa: F401

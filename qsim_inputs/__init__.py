"""Neutral input recipes shared by the CPU oracle wrapper and the CUDA binding.

Holds plain data (`SimInputs`), host-side planning (the fluid LP) and seeded synthetic
workload recipes.  Neither simulator's event arithmetic lives here.
"""
from .spec import *  # noqa: F401,F403
from .spec import SimInputs  # noqa: F401
from . import fluid_lp, lengths, online, presets  # noqa: F401

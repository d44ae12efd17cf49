"""Seeded synthetic inputs shared by the CPU checker and the GPU harness.

Input generation only; nothing of the TSVD forward is computed here.
"""
from .configs import CONFIGS, Case, CaseSpec, laplace_matrix, make_case, make_weights, make_x, scaled, set_entries, widen_x  # noqa: F401
from . import rng  # noqa: F401

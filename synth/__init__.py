"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This package holds data generation only: random tensors, model shapes, weight
tables.  None of the method's arithmetic (schedule algebra, network forward,
acceptance rule) lives here, so both implementations can consume the same bytes
without sharing any code that could hide a common mistake.
"""
from .rng import normal, uniform01, round_to_bf16          # noqa: F401
from .models import (DiTShape, TINY, DIT_S2, DIT_XL2_256, DIT_XL2_512,   # noqa: F401
                     make_target_weights, make_drafter_weights, pos_embed_2d)
from .workloads import verifier_inputs, lambda_profile, pack_states, eps_verifier_inputs     # noqa: F401

"""CPU oracle for the packed parallel-verification path of FREE.

TEST INFRASTRUCTURE ONLY.  A plain, slow, fp64 numpy restatement of what the
paper's method computes: DDPM schedule algebra, the target DiT forward, the
feature-level drafter, the reflection-coupling verifier (strict and relaxed)
and the speculative sampling loop.  It follows the paper's steps and notation
in order, without blocking, fusion or reordering.  It shares no code with the
CUDA path and must only be imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; the product path never calls it.

Pins (see tests/test_oracle_*.py): the verifier, the schedule and every layer
primitive are checked against closed forms, brute force, identities from the
paper's appendix and library routines.  The end-to-end numerical outputs of the
DiT and of the drafter are "parity unpinned" by the paper (it prints no
activations and ships no weights); they are pinned only through their parts.
"""
from . import schedule, dit, verify, drafter, trajectory   # noqa: F401

"""Double-precision CPU oracle for the Rubick scheduler hot path.

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the CPU-baseline leg of the
benchmark may import this package; the CUDA library and its Python binding never do.
"""
from .oracle import (  # noqa: F401
    JOB_FIELDS, ENV_FIELDS, TERM_FIELDS, MEM_FIELDS,
    build, lib, overlap, terms, memory, feas_word, enumerate_plans, eval_candidates,
    best_plan, gain, schedule_round, schedule_round_incremental, bruteforce, min_resources, fit, FIT_NAMES,
)

"""CPU oracle for the multi-LoRA hot path over a unified LoRA/KV block pool.

TEST INFRASTRUCTURE ONLY.  Plain, slow, float64 restatements of what the path computes, written
from the paper's definitions (Eq. 1, Eq. 2, Eq. 3, Section 2.1 prefix reuse, Section 4.3 unified
pool and swapping).  Nothing here is imported by the product package; only the tests, the smoke
check and the benchmark's cpu-baseline leg call it.  It shares no code with the CUDA path.

Pins (tests/test_oracle_*.py): closed forms and invariants listed in each module's header.
"""

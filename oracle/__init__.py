"""CPU oracle: a plain, slow, obviously-correct statement of what the hot path computes.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this; only the
tests, the smoke check and the benchmark's CPU-baseline leg call it.  It shares no code
with the CUDA path: the forward pass (forward.py), the analytic op trace (trace.py), the
prefetch policy (policy.py) and the plan validator (validate.py) are each written here
from the paper's description, in numpy / pure Python.

Parity status of each part:
* forward.py  - pinned by brute-force double-precision loops, closed forms, and
                library cross-checks on tiny shapes (tests/test_oracle_forward.py).
* trace.py    - pinned by hand-computed op counts on a toy shape (tests/test_oracle_policy.py).
* policy.py   - the paper gives prose only (Sections III-B, IV-D, IV-E); classification
                is pinned by hand-computed toy rooflines, the schedule by the invariants
                in validate.py, closed forms and a brute-force pin-set search.  The
                policy *constants* (hold window, zero-copy ratio, ring minimum, alignment,
                tie-breaks) are choices of this build: parity unpinned for those.
"""

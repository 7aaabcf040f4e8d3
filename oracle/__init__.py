"""CPU oracle for one speculative-decoding rollout step (TEST INFRASTRUCTURE ONLY).

A plain, slow, fp64 NumPy restatement of what the hot path computes, written
from the paper's description of the draft-then-verify cycle (Sec. 2.2, Eq. 1;
App. B.1 "MTP Architecture"; App. E, the restart equations).  It shares no code
with the CUDA library and must never be imported by the product path: only the
tests, the smoke check and the benchmark's CPU-baseline leg may use it.

Parity status of each part (what pins it, other than itself):

* philox.py   - pinned: published known-answer vectors of Philox4x32-10.
* sampler.py  - pinned: exhaustive enumeration of all 2^24 uniforms (inverse CDF),
                Eq. 5 closed form for acceptance, chi-square exactness of the
                committed distribution, Eq. 6 expected accepted length.
* model.py    - pinned: closed forms and special cases of RMSNorm / RoPE / attention,
                a scalar-loop brute force, incremental == full recompute,
                paged == contiguous, GQA == MHA with repeated heads.
                The draft head's input order [embedding ; hidden], the use of the
                pre-final-norm hidden state and the head-owned final norm are
                conventions the paper does not fix: PARITY UNPINNED for those three
                choices (they are immaterial under random initialisation).
* step.py     - pinned: cache composition after a restart (App. E), length growth
                on full acceptance, always >= 1 committed token.
"""

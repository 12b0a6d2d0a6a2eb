"""float64 CPU checker for the MLA-Online step (test infrastructure, not product code).

Nothing here is fast, blocked or fused.  It is the plain definition written out so that
a reader can compare it with the paper by eye: full causal MLA attention over the
request-positioned concatenated context (keys re-rotated to their request positions, one
softmax per row, no segments), the grouped output projections, the select-or-artifact
rule and the shared second projection.  It shares no code with the CUDA library and
imports nothing from it; only tests, the smoke check and the benchmark's cpu_baseline /
reference arms may call it.

Pins (tests/test_oracle_pins.py): exact logical-head factorization, relocation
invariance, segmented merge == one softmax, scalar brute force, prefix exactness,
zero-query and one-hot closed forms, packed-order permutation invariance, global shift
invariance, the printed profile ceilings, and torch's scaled_dot_product_attention in
float64 as a library special case.

`reuse_error_report` (how far MLA-Online with honest position-zero artifacts is from full
recomputation) is pinned as arithmetic by a closed form; the quantity itself, on random data, has
no value to compare with -- the paper quantifies reuse quality only through model-level F1/EM --
and no parity claim rests on it.
"""
from .mla_online import *  # noqa: F401,F403
from . import phase  # noqa: F401  (output-phase variant: RestorePhase / R^{-1}; pins in tests/test_oracle_phase_pins.py)
from . import policy  # noqa: F401  (Eq. protected and Eq. moe; pins in tests/test_oracle_policy_pins.py)

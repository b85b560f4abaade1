"""fp64 CPU oracle for tree-causal prefix-shared attention.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only
the tests, the smoke check and the benchmark's CPU-baseline leg call it.  It
shares no code with the CUDA path.

  plan.py       canonical plan of a prefix forest (segments -> pages, block
                table, reference counts), written step by step as an encoding.
  attention.py  the plain definition of the attention result: every sample
                (root-to-end path) is materialised as an unshared causal
                sequence and run through naive softmax attention, forward and
                backward, in fp64; results are scattered back to the shared
                layout.

Pins (what each function is checked against, other than itself) are listed in
the header of each module.
"""
from .plan import oracle_plan, PlanError  # noqa: F401
from .attention import (  # noqa: F401
    oracle_attn,
    oracle_rows,
    sample_paths,
)

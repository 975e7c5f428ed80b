"""CPU oracle for fused operator chains.  TEST INFRASTRUCTURE ONLY.

A plain float64 interpreter of the operator-DAG spec: it walks the nodes in
the order they are written, materialises every node as a numpy float64 array
and applies each operator's textbook definition.  It shares no code with the
CUDA library and must never be imported by it; only tests, the smoke check and
the benchmark's CPU-baseline leg may call it.

Parity pins: every operator here is pinned by closed forms, brute-force loops
and torch float64 library routines in ``tests/test_oracle_pins.py``.  The paper
prints no numeric worked example, so operator conventions it leaves open
(GELU variant, biased variance with eps inside the root, cross-correlation
with zero padding) are fixed by those pins rather than by printed values.
"""
from .interp import run, run_nodes  # noqa: F401
from .graph import parse, Graph, SpecError  # noqa: F401

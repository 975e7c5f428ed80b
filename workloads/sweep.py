"""The graph-augmentation sweep: 200 random operator DAGs, seeds 0..199.

``sweep_specs.json`` records, per seed, which attempt of the generator was kept (graphs that are
numerically ill-conditioned are redrawn, see oracle/make_sweep.py); the spec text itself is
regenerated from (seed, attempt).
"""
from __future__ import annotations

import json
import os

from . import graph_growth, random_dag

_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "sweep_specs.json")


def entries():
    with open(_PATH) as f:
        return json.load(f)["entries"]


def get(seed: int, rows: int | None = None):
    """(spec, laws, meta) of sweep graph ``seed``; ``rows`` overrides the row count."""
    e = entries()[seed]
    assert e["seed"] == seed
    return random_dag.make_dag(seed, e["attempt"], rows=rows)


_GROWN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "growth_specs.json")


def grown_entries():
    with open(_GROWN) as f:
        return json.load(f)["entries"]


def get_grown(seed: int, rows: int | None = None):
    """(spec, laws, meta) of branching multi-output graph ``seed`` (whole Algorithm 1); ``rows`` overrides the row count."""
    e = grown_entries()[seed]
    assert e["seed"] == seed
    return graph_growth.grow_graph(seed, e["attempt"], rows=rows)

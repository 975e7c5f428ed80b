"""Writes workloads/sweep_specs.json: the 200 random operator DAGs of the graph-augmentation sweep,
and workloads/growth_specs.json: 60 branching multi-output DAGs grown with the whole of Algorithm 1.

    python -m oracle.make_sweep

For seed 0..199 the generator (workloads.random_dag, after the paper's Algorithm 1) is asked
for a graph; the graph is then checked for data-flow validity in the numerical sense: it is
evaluated by the oracle on a 64-row proxy twice, once in float64 and once with the same
definitions carried out in float32, and it is rolled back and redrawn (next attempt number)
when any value is non-finite or above 1e30, or when single precision alone already moves the
result by more than 2e-6 of the row's magnitude, i.e. when the graph is too ill-conditioned
for any float32 implementation to be compared at 1e-5 (sums that cancel, exponentials of
large arguments, results that underflow).
Calls only workloads/ and oracle/.
"""
from __future__ import annotations

import json
import os

import numpy as np

from oracle import graph as ograph
from oracle import interp
from workloads import configs, graph_growth, random_dag, tensors

N_SEEDS = 200
PROXY_ROWS = 64
N_GROWN = 60
OUT = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "workloads", "sweep_specs.json")


def gemm_f32_sequential(a, b):
    """Single-precision product accumulated term by term in k order (no blocking, no pairwise
    summation): the least favourable accumulation a float32 implementation may use."""
    acc = np.zeros((a.shape[0], b.shape[1]), dtype=np.float32)
    for k in range(a.shape[1]):
        acc += a[:, k:k + 1] * b[k:k + 1, :]
    return acc


def column_scale(a):
    """Magnitude against which an element's error is judged: the largest value of its row, or of
    the whole tensor when rows have a single element."""
    if a.shape[-1] == 1:
        return np.full_like(a, np.abs(a).max())
    return np.abs(a).max(axis=-1, keepdims=True)


def well_conditioned(spec: str, laws: dict, seed: int) -> bool:
    g = ograph.parse(spec)
    t = configs.draw_inputs(spec, laws, seed)
    ins = {n: tensors.as_float64(t[n], d) for n, d, _ in configs.parse_inputs(spec)}
    with np.errstate(all="ignore"):
        exact = interp.run_nodes(g, ins)
        single = interp.run_nodes(g, ins, dtype=np.float32, gemm_fn=gemm_f32_sequential)
    for name, node in g.nodes.items():
        v = exact[name]
        if not np.all(np.isfinite(v)) or np.abs(v).max() > 1e30:
            return False
    for out, _ in g.outputs:
        a, b = exact[out], single[out].astype(np.float64)
        if not np.all(np.isfinite(b)):
            return False
        rho = column_scale(a)
        if not np.all(np.abs(a - b) <= 2e-6 * np.maximum(np.abs(a), rho)):
            return False
    return True


def main():
    entries = []
    for seed in range(N_SEEDS):
        attempt = 0
        while True:
            proxy_spec, laws, meta = random_dag.make_dag(seed, attempt, rows=PROXY_ROWS)
            if well_conditioned(proxy_spec, laws, seed):
                break
            attempt += 1
            assert attempt < 64, f"seed {seed}: no well-conditioned graph in 64 attempts"
        entries.append({"seed": seed, "attempt": attempt, "rows": meta["rows"], "cols": meta["cols"], "n_ops": meta["n_ops"],
                        "rollbacks": meta["rollbacks"]})
    with open(OUT, "w") as f:
        json.dump({"generator": "workloads.random_dag.make_dag(seed, attempt)", "entries": entries}, f, indent=0)
        f.write("\n")
    rej = sum(e["attempt"] for e in entries)
    print(f"wrote {OUT}: {len(entries)} graphs, {rej} redraws for conditioning")

    grown = []
    for seed in range(N_GROWN):
        attempt = 0
        while True:
            proxy_spec, laws, meta = graph_growth.grow_graph(seed, attempt, rows=PROXY_ROWS)
            if well_conditioned(proxy_spec, laws, seed):
                break
            attempt += 1
            assert attempt < 200, f"grown graph {seed}: no well-conditioned graph in 200 attempts"
        grown.append(meta)
    out2 = os.path.join(os.path.dirname(OUT), "growth_specs.json")
    with open(out2, "w") as f:
        json.dump({"generator": "workloads.graph_growth.grow_graph(seed, attempt)", "entries": grown}, f, indent=0)
        f.write("\n")
    print(f"wrote {out2}: {len(grown)} graphs, {sum(e['attempt'] for e in grown)} redraws for conditioning")


if __name__ == "__main__":
    main()

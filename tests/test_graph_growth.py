"""Host-side checks of the Algorithm 1 graph generator: determinism and the validity rules of Section 3.2."""
import math

import oracle
from workloads import graph_growth, sweep


def _parsed(seed, attempt=0, rows=32):
    spec, laws, meta = graph_growth.grow_graph(seed, attempt, rows=rows)
    return spec, laws, meta, oracle.parse(spec)


def test_same_seed_same_graph_and_rows_only_change_the_row_count():
    a = graph_growth.grow_graph(7, 2, rows=32)
    b = graph_growth.grow_graph(7, 2, rows=32)
    assert a == b
    c = graph_growth.grow_graph(7, 2, rows=96)[0]
    assert c == a[0].replace("[32,", "[96,")
    assert graph_growth.grow_graph(8, 2, rows=32)[0] != a[0]


def test_grown_graphs_are_valid_dags_without_dangling_nodes():
    shapes_seen, multi_output, with_connection, with_branch, with_merge = set(), 0, 0, 0, 0
    for seed in range(60):
        spec, laws, meta, g = _parsed(seed)
        names = list(g.nodes)
        defined = set(g.inputs)
        consumed = set()
        for name in names:
            node = g.nodes[name]
            if node.op == "input":
                continue
            for a in node.args:
                if isinstance(a, str):
                    assert a in defined, (seed, name, a)        # operands come from inputs or earlier nodes: acyclic
                    consumed.add(a)
            defined.add(name)
        outs = {o for o, _ in g.outputs}
        for name in names:                                      # no dangling node: consumed or an output
            assert name in consumed or name in outs, (seed, name)
        assert set(laws) == set(g.inputs)
        assert meta["n_nodes"] > meta["n_max"] or meta["depth"] > meta["d_max"]     # the loop's exit test
        assert meta["max_usage"] <= meta["usage_cap"] == math.ceil(0.25 * len(graph_growth.POOL))
        multi_output += meta["outputs"] > 1
        with_connection += meta["connections"] > 0
        with_branch += meta["branches"] > 0
        with_merge += meta["merges"] > 0
        shapes_seen.add((meta["rows"], meta["cols"]))
    # the three diversity actions and several outputs all occur across the set
    assert multi_output >= 10 and with_connection >= 5 and with_branch >= 20 and with_merge >= 10
    assert len(shapes_seen) >= 4


def test_recorded_attempts_regenerate_the_committed_list():
    entries = sweep.grown_entries()
    assert len(entries) == 60
    for seed in (0, 17, 59):
        spec, laws, meta = sweep.get_grown(seed, rows=64)
        assert meta == entries[seed]

"""The parity harness's own logic (no GPU): table comparison and the margin rule that decides which
differences between the library and the oracle are excused."""
import numpy as np

from oracle import stand_oracle as so
from tests import harness


def _table(entries, K=4):
    """entries: {key tuple: (count, {id: prob})} -> the array form both sides export."""
    M = len(entries)
    keys = np.full((M, 4), -1, np.int32)
    counts = np.zeros(M, np.uint32)
    n_items = np.zeros(M, np.int32)
    ids = np.full((M, K), -1, np.int32)
    probs = np.zeros((M, K), np.float64)
    for i, (key, (cnt, items)) in enumerate(entries.items()):
        keys[i, 4 - len(key):] = key
        counts[i] = cnt
        n_items[i] = len(items)
        for t, (tok, p) in enumerate(items.items()):
            ids[i, t], probs[i, t] = tok, p
    return keys, counts, n_items, ids, probs


def test_table_differences_finds_every_kind_and_nothing_else():
    base = {(1,): (3, {5: 0.5, 6: 0.25}), (1, 2): (1, {7: 1.0}), (9, 9, 9, 9): (2, {1: 0.3, 2: 0.2, 3: 0.1})}
    same = dict(reversed(list(base.items())))  # other slot order, items in another order
    same[(1,)] = (3, {6: 0.25, 5: 0.5})
    assert harness.table_differences(_table(same), _table(base), 1e-5) == {}
    within = dict(base); within[(1, 2)] = (1, {7: 1.0 + 5e-6})
    assert harness.table_differences(_table(within), _table(base), 1e-5) == {}
    g = dict(base)
    g[(1, 2)] = (1, {7: 1.0 + 5e-5})          # outside the tolerance
    g[(1,)] = (4, {5: 0.5, 6: 0.25})          # another count
    g[(9, 9, 9, 9)] = (2, {1: 0.3, 2: 0.2, 4: 0.1})  # another id kept
    g[(8,)] = (1, {1: 1.0})                   # only here
    o = dict(base); o[(7, 7)] = (1, {1: 1.0})  # only in the oracle
    assert harness.table_differences(_table(g), _table(o), 1e-5) == {
        (1, 2): "prob", (1,): "count", (9, 9, 9, 9): "ids", (8,): "missing_oracle", (7, 7): "missing_gpu"}
    assert harness.table_differences(_table({}), _table({}), 1e-5) == {}


PARENT = np.array([-1, 0, 0, 1, 1, 3], np.int32)  # 0 -> 1, 2; 1 -> 3, 4; 3 -> 5


def _judge(gpu, orc, recs, path, old_tail, new_tail, gt, ot):
    ints = np.array([r[0] for r in recs], np.int32).reshape(-1, 8)
    margins = np.array([r[1] for r in recs], np.float64)
    j = harness.StepJudge(PARENT, 2, 1e-5)
    as3 = lambda x: (np.array(x[0], np.int32), np.array(x[1], np.int32), np.array(x[2], np.int32))
    return j.judge(as3(gpu), as3(orc), ints, margins, np.array(path, np.int32), np.array(old_tail, np.int32),
                   np.array(new_tail, np.int32), lambda: (_table(gt), _table(ot)))


def _rec(kind, b, node, aux=0, key=(-1, -1, -1, -1), margin=1e-9):
    return ([kind, b, node, aux, *key], margin)


TREE = [50, 20, 21, 30, 31, 40]


def test_an_emitted_difference_is_excused_only_by_the_decision_that_made_it():
    # oracle: accepted nodes 1 and 3, then sampled 77 at node 3; the library sampled 78 there
    orc = ([[20, 30, 77]], [3], [TREE])
    gpu = ([[20, 30, 78]], [3], [TREE])
    path, old, new = [[0, 1, 3]], [[4, 50]], [[30, 77]]
    t = {(50,): (1, {20: 1.0})}
    args = (path, old, new, t, t)
    # the fed contexts differ after position 2, so the tables differ there: allowed once the decision is excused
    gt = dict(t); gt[(30,)] = (1, {78: 1.0})
    ot = dict(t); ot[(30,)] = (1, {77: 1.0})
    hard, exc, _ = _judge(gpu, orc, [_rec(so.MARGIN_FINAL, 0, 3)], path, old, new, gt, ot)
    assert hard == [] and exc == [("decision", 0, 2)]
    # a low margin of the same sequence at another node, or of another kind, does not explain it
    for rec in (_rec(so.MARGIN_FINAL, 0, 1), _rec(so.MARGIN_ACCEPT, 0, 0), _rec(so.MARGIN_GUMBEL, 0, 3),
                _rec(so.MARGIN_FINAL, 1, 3), _rec(so.MARGIN_FINAL, 0, 3, margin=1e-3)):
        hard, exc, _ = _judge(gpu, orc, [rec], *args)
        assert [h[0] for h in hard] == ["emitted"] and exc == []
    # one walk stopped where the other accepted the same token: the decision sat one node earlier
    gpu2 = ([[20, 30, -1]], [2], [TREE])
    hard, exc, _ = _judge(gpu2, orc, [_rec(so.MARGIN_ACCEPT, 0, 1)], *args)
    assert hard == [] and exc == [("decision", 0, 2)]
    hard, exc, _ = _judge(gpu2, orc, [_rec(so.MARGIN_ACCEPT, 0, 0)], *args)
    assert [h[0] for h in hard] == ["emitted"]
    # an unexplained table difference stays hard even next to an excused sequence
    gt2 = dict(gt); gt2[(99,)] = (1, {1: 1.0})
    hard, exc, _ = _judge(gpu, orc, [_rec(so.MARGIN_FINAL, 0, 3)], path, old, new, gt2, ot)
    assert hard == [("table", (99,), "missing_oracle")]


def test_a_tree_difference_is_excused_by_its_parents_selection_or_by_an_excused_context():
    orc = ([[60, -1, -1]], [1], [TREE])
    other = list(TREE); other[5] = 41            # node 5 (child of node 3) differs
    gpu = ([[60, -1, -1]], [1], [other])
    path, old, new = [[0, -1, -1]], [[4, 5]], [[5, 50]]
    t = {(50,): (1, {20: 1.0})}
    hard, exc, _ = _judge(gpu, orc, [_rec(so.MARGIN_GUMBEL, 0, 3)], path, old, new, t, t)
    assert hard == [] and exc == [("gumbel", 0, 5)]
    for rec in (_rec(so.MARGIN_GUMBEL, 0, 1), _rec(so.MARGIN_GUMBEL, 0, 5), _rec(so.MARGIN_FINAL, 0, 3)):
        hard, exc, _ = _judge(gpu, orc, [rec], path, old, new, t, t)
        assert [h[0] for h in hard] == ["tree"] and exc == []
    # node 3 looked up (20, 30) and (30,): a truncation tie at (20, 30) that left other ids explains the draft ...
    gt = dict(t); gt[(20, 30)] = (2, {40: 0.5, 41: 0.25})
    ot = dict(t); ot[(20, 30)] = (2, {40: 0.5, 42: 0.25})
    tie = _rec(so.MARGIN_MERGE, -1, -1, 2, (-1, -1, 20, 30))
    hard, exc, _ = _judge(gpu, orc, [tie], path, old, new, gt, ot)
    assert hard == [] and ("lookup", 0, 5) in exc
    # ... a tie at a context the node did not look up does not, and neither does a tie whose tables agree
    gt3 = dict(t); gt3[(7, 7)] = (2, {40: 0.5, 41: 0.25})
    ot3 = dict(t); ot3[(7, 7)] = (2, {40: 0.5, 42: 0.25})
    hard, exc, _ = _judge(gpu, orc, [_rec(so.MARGIN_MERGE, -1, -1, 2, (-1, -1, 7, 7))], path, old, new, gt3, ot3)
    assert [h[0] for h in hard] == ["tree"]
    hard, exc, _ = _judge(gpu, orc, [tie], path, old, new, t, t)
    assert [h[0] for h in hard] == ["tree"]
    # a tie excuses "other ids kept" at its context and nothing else there
    gt4 = dict(t); gt4[(20, 30)] = (3, {40: 0.5, 42: 0.25})
    hard, exc, _ = _judge((orc[0], orc[1], orc[2]), orc, [tie], path, old, new, gt4, ot)
    assert hard == [("table", (20, 30), "count")]


def test_a_low_margin_truncation_alone_makes_the_tables_be_compared():
    orc = ([[60, -1, -1]], [1], [TREE])
    t = {(50,): (1, {20: 1.0})}
    tie = _rec(so.MARGIN_MERGE, -1, -1, 1, (-1, -1, -1, 50))
    hard, exc, looked = _judge(orc, orc, [tie], [[0, -1, -1]], [[4, 5]], [[5, 60]], t, t)
    assert hard == [] and exc == [] and looked
    gt = {(50,): (1, {21: 1.0})}
    hard, exc, looked = _judge(orc, orc, [tie], [[0, -1, -1]], [[4, 5]], [[5, 60]], gt, t)
    assert hard == [] and exc == [("merge", [(50,)])]
    hard, exc, looked = _judge(orc, orc, [], [[0, -1, -1]], [[4, 5]], [[5, 60]], gt, t)
    assert not looked  # nothing logged, nothing differed: the tables are left for the periodic whole-table checks

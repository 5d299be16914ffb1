"""Pins of the CPU oracle against what the paper and the mathematics fix.

Every test here checks the oracle against something other than itself: published
known-answer vectors, library routines, closed forms, hand-worked cases, brute
force and statistical laws.  A plausible mistake anywhere in the oracle (a dropped
term, a wrong sign or index, a wrong normalisation) fails at least one of them.
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy import special, stats

from oracle import stand_oracle as so

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- randomness
def test_philox_known_answers():
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        assert list(so.philox(w[0:4], w[4:6])) == w[6:10]


def test_uniform_mapping_and_counter_layout():
    seed = 0x1234_5678_9ABC_DEF0
    word0 = int(so.philox([3, 5, 7, 11], [seed & 0xFFFFFFFF, seed >> 32])[0])
    assert so.uniform(seed, 3, 5, 7, 11) == (word0 >> 8) / 2.0 ** 24
    assert so.uniform(seed, 3, 5, 7, 11, open_interval=True) == ((word0 >> 8) + 0.5) / 2.0 ** 24
    u = np.array([so.uniform(1, 0, 0, 0, s) for s in range(20000)])
    assert 0.0 <= u.min() and u.max() < 1.0
    assert stats.kstest(u, "uniform").pvalue > 1e-3


# ------------------------------------------------------ softmax and top-k (O1, O2)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("T", [1.0, 0.6])
def test_softmax_matches_scipy(dtype, T):
    from paper_2506_04708_b200 import inputs
    rng = np.random.default_rng(1)
    x = (rng.standard_normal(777) * 3).astype(np.float32)
    if dtype == "bf16":
        bits = inputs.f32_to_bf16_bits(x)
        xv = inputs.bf16_bits_to_f32(bits).astype(np.float64)
        row = bits
    else:
        xv, row = x.astype(np.float64), x
    Tf = float(np.float32(T))
    lse, ids, vals, probs, p = so.row_stats(row, Tf, 10, want_p=True)
    ref = special.softmax(xv / Tf)
    assert np.allclose(p, ref, rtol=1e-12, atol=0)
    assert abs(lse - special.logsumexp(xv / Tf)) < 1e-12
    assert abs(p.sum() - 1) < 1e-12
    order = np.lexsort((np.arange(len(xv)), -xv))[:10]
    assert list(ids) == list(order)
    assert np.array_equal(vals, xv[order])
    assert np.allclose(probs, ref[order], rtol=1e-12)


def test_topk_ties_break_by_lower_id():
    x = np.array([1, 5, 5, 3, 5, 0, 3, 3], np.float32)
    _, ids, vals, _, _ = so.row_stats(x, 1.0, 6)
    assert list(ids) == [1, 2, 4, 3, 6, 7]
    # fewer elements than k: padded with -1
    _, ids, _, _, _ = so.row_stats(np.array([2, 9, 4], np.float32), 1.0, 5)
    assert list(ids) == [1, 2, 0, -1, -1]


def test_inverse_cdf_matches_searchsorted():
    rng = np.random.default_rng(2)
    w = rng.random(50)
    w[rng.integers(0, 50, 10)] = 0.0
    cdf = np.cumsum(w)
    for U in list(rng.random(500)) + [0.0, 1 - 2.0 ** -24]:
        y, _ = so.inverse_cdf(w, U)
        assert y == int(np.searchsorted(cdf, U * w.sum(), side="right"))
    # zero-weight tokens are never returned
    assert all(w[so.inverse_cdf(w, U)[0]] > 0 for U in rng.random(200))


# ------------------------------------------------- Gumbel-Top-K (Sec. 4.2) = Plackett-Luce
def _plackett_luce(q, seq):
    pr, rest = 1.0, 1.0
    for i in seq:
        pr *= q[i] / rest
        rest -= q[i]
    return pr


def test_gumbel_top_is_argsort_of_perturbed_logprob():
    rng = np.random.default_rng(3)
    phi = rng.random(9) + 0.01
    U = rng.random(9)
    ids = np.arange(100, 109)
    g = np.log(phi) - np.log(-np.log(U))
    got = so.gumbel_top(ids, phi, U, 4)
    assert list(got) == list(ids[np.argsort(-g)[:4]])
    # fewer candidates than requested
    assert len(so.gumbel_top(ids[:2], phi[:2], U[:2], 5)) == 2


def test_gumbel_top_k_samples_without_replacement():
    """Ordered k-subsets drawn by Gumbel-Top-K follow the sequential
    sampling-without-replacement law prod_j q_ij / (1 - sum_{l<j} q_il)."""
    phi = np.array([0.4, 0.25, 0.2, 0.1, 0.05]) * 0.7  # not normalised on purpose
    q = phi / phi.sum()
    ids = np.array([11, 3, 8, 20, 5])
    n, k, trials = len(ids), 3, 200_000
    pos = {int(t): i for i, t in enumerate(ids)}
    counts = {}
    for t in range(trials):
        U = np.array([so.uniform(9, t & 0xFFFF, t >> 16, 2, so.SLOT_GUMBEL | int(i), True) for i in ids])
        seq = tuple(pos[int(x)] for x in so.gumbel_top(ids, phi, U, k))
        counts[seq] = counts.get(seq, 0) + 1
    seqs = list(itertools.permutations(range(n), k))
    obs = np.array([counts.get(s, 0) for s in seqs], float)
    exp = np.array([_plackett_luce(q, s) for s in seqs]) * trials
    assert abs(exp.sum() - trials) < 1e-6
    assert stats.chisquare(obs, exp).pvalue > 0.01


# ------------------------------------------------ verification is lossless (Sec. 3.2)
def _threshold(fn, lo=0, hi=1 << 24):
    """Smallest integer u in [lo, hi] with fn(u / 2^24) False, fn monotone True -> False."""
    while lo < hi:
        mid = (lo + hi) // 2
        if fn(mid / 2.0 ** 24):
            lo = mid + 1
        else:
            hi = mid
    return lo


def _exact_output_distribution(p, cand_id, cand_phi, m):
    """Output distribution of drafting m children (without replacement from
    q = phi/sum) and verifying them, with the oracle's verification used as a BLACK BOX:
    accept thresholds and resampling boundaries are found by bisection over the
    24-bit uniforms, the draft law is the textbook Plackett-Luce product."""
    V = len(p)
    q = np.asarray(cand_phi) / np.sum(cand_phi)
    out = np.zeros(V)
    n = len(cand_id)
    for seq in itertools.permutations(range(n), m):
        pr_draft = _plackett_luce(q, seq)
        child = [cand_id[i] for i in seq]
        reach = pr_draft
        for j in range(m):
            # uniforms of the earlier children force rejection: find one that rejects
            def accepted_j(U, j=j):
                ua = [1 - 2.0 ** -24] * m
                ua[j] = U
                return so.verify_children(p, cand_id, cand_phi, child[:j + 1], ua[:j + 1], 0.0)[0] == j
            # the earlier children must be rejected at U = 1 - 2^-24 unless their
            # acceptance probability is 1; handle that case by its measured threshold
            a_j = _threshold(accepted_j) / 2.0 ** 24
            out[child[j]] += reach * a_j
            reach *= 1 - a_j
            if reach == 0:
                break
        if reach > 0:
            ua = [1 - 2.0 ** -24] * m
            prev = 0
            for v in range(V):
                def not_past(U, v=v):
                    return so.verify_children(p, cand_id, cand_phi, child, ua, U)[1] <= v
                hi = _threshold(not_past, lo=prev)
                out[v] += reach * (hi - prev) / 2.0 ** 24
                prev = hi
    return out


@pytest.mark.parametrize("case", range(4))
def test_verification_is_lossless_exactly(case):
    rng = np.random.default_rng(100 + case)
    V = [6, 9, 12, 16][case]
    p = rng.random(V) ** 3
    p[rng.integers(0, V)] = 0.0
    p /= p.sum()
    n = [2, 3, 4, 3][case]
    m = [1, 2, 3, 3][case]
    cand_id = list(rng.choice(V, n, replace=False))
    cand_phi = list(rng.random(n) * 0.3 + 0.01)  # unnormalised, unrelated to p
    out = _exact_output_distribution(p, cand_id, cand_phi, m)
    # every boundary is resolved to 2^-24; a handful of them enter each entry
    assert np.abs(out - p).max() < 2e-6, (out, p)


def test_verification_single_draft_rule():
    """One draft: accept iff U*q(x) < p(x); on rejection the resample follows norm(max(0,p-q))."""
    p = np.array([0.1, 0.2, 0.3, 0.4])
    cand_id, cand_phi = [0, 3], [3.0, 1.0]  # q = (0.75, 0, 0, 0.25)
    # x = 0: p/q = 0.1/0.75
    assert so.verify_children(p, cand_id, cand_phi, [0], [0.1333], 0.5)[0] == 0
    assert so.verify_children(p, cand_id, cand_phi, [0], [0.1334], 0.5)[0] == -1
    # x = 3: q <= p, always accepted
    assert so.verify_children(p, cand_id, cand_phi, [3], [1 - 2.0 ** -24], 0.5)[0] == 0
    # residual = max(0, p - q) = (0, .2, .3, .15) / .65
    r = np.array([0, 0.2, 0.3, 0.15]) / 0.65
    cdf = np.cumsum(r)
    for U in [0.0, 0.3, 0.307, 0.308, 0.76, 0.77, 0.999]:
        acc, y = so.verify_children(p, cand_id, cand_phi, [0], [0.9], U)
        assert acc == -1 and y == int(np.searchsorted(cdf, U, side="right"))


def test_verification_chi_square_through_the_tree_walk():
    """1e6 trials through the full oracle (table -> Gumbel-Top-K drafting ->
    tree verification): the first emitted token follows the root's target
    distribution, and the token after an accepted child follows that child's."""
    from paper_2506_04708_b200 import inputs
    V, K = 12, 4
    parent = np.array([-1, 0, 0, 0, 1, 1, 2], np.int32)  # 3 children of the root, 2+1 grandchildren
    N = len(parent)
    rng = np.random.default_rng(5)
    logits = (rng.standard_normal((1, N, V)) * 1.5).astype(np.float32)
    T = 0.8
    B = 1
    trials = 1_000_000 // 250
    first = np.zeros(V)
    second = {}
    # many independent "sequences": B = 250 per oracle call keeps it quick
    Bn = 250
    big = np.ascontiguousarray(np.broadcast_to(logits, (Bn, N, V)))
    for rep in range(trials):
        o = so.Oracle(Bn, N, V, K, 2, 0, T, 1000 + rep, parent)
        # a table whose contexts are hit at every node: unigram context of every token
        ctx = np.array([[-1, t] for t in range(V)], np.int32)
        ids = np.array([[(t + 1 + 2 * i) % V for i in range(K)] for t in range(V)], np.int32)
        probs = np.tile(np.array([0.5, 0.2, 0.2, 0.1], np.float32), (V, 1))
        o.update_bulk(ctx, ids, probs)
        o.reset_sequences(np.tile(np.array([-1, 3], np.int32), (Bn, 1)), np.full(Bn, 1))
        tree = o.draft()
        assert (tree[:, 1:4] >= 0).all()
        em, ne = o.verify(big)
        path = o.path()
        np.add.at(first, em[:, 0], 1)
        for b in np.nonzero(ne >= 2)[0]:
            node = int(path[b, 1])
            second.setdefault(node, np.zeros(V))[em[b, 1]] += 1
        o.close()
    lse, _, _, _, p0 = so.row_stats(logits[0, 0], float(np.float32(T)), K, want_p=True)
    assert first.sum() == Bn * trials
    assert stats.chisquare(first, p0 * first.sum()).pvalue > 0.01
    checked = 0
    for node, cnt in second.items():
        if cnt.sum() < 5000:
            continue
        _, _, _, _, pn = so.row_stats(logits[0, node], float(np.float32(T)), K, want_p=True)
        keep = pn * cnt.sum() >= 5
        assert stats.chisquare(cnt[keep], pn[keep] / pn[keep].sum() * cnt[keep].sum()).pvalue > 0.01
        checked += 1
    assert checked >= 1


# --------------------------------------- deterministic drafting (Sec. 3.2), the variant
def test_deterministic_draft_is_accepted_with_its_target_probability():
    """Sec. 3.2: with a one-hot draft distribution "the drafted token is accepted with p(x_draft)"."""
    p = np.array([0.1, 0.2, 0.3, 0.4])
    for x in range(4):
        thr = _threshold(lambda U, x=x: so.verify_children_deterministic(p, [x], [U], 0.0)[0] == 0)
        assert abs(thr / 2.0 ** 24 - p[x]) < 2.0 ** -23
    # on rejection the resample follows norm(max(0, p - onehot)): x loses its mass
    r = np.array([0.1, 0.2, 0.0, 0.4]) / 0.7
    cdf = np.cumsum(r)
    for U in [0.0, 0.14, 0.15, 0.42, 0.43, 0.999]:
        acc, y = so.verify_children_deterministic(p, [2], [0.9], U)
        assert acc == -1 and y == int(np.searchsorted(cdf, U, side="right")) and y != 2


@pytest.mark.parametrize("case", range(3))
def test_deterministic_verification_is_lossless_exactly(case):
    """Several deterministic drafts tested one after the other: the output still follows p exactly.  The oracle is
    used as a black box (thresholds by bisection over the 24-bit uniforms)."""
    rng = np.random.default_rng(200 + case)
    V = [5, 9, 14][case]
    m = [1, 3, 4][case]
    p = rng.random(V) ** 2
    p /= p.sum()
    child = list(rng.choice(V, m, replace=False))
    out = np.zeros(V)
    reach = 1.0
    for j in range(m):
        def accepted_j(U, j=j):
            ua = [1 - 2.0 ** -24] * m
            ua[j] = U
            return so.verify_children_deterministic(p, child[:j + 1], ua[:j + 1], 0.0)[0] == j
        a_j = _threshold(accepted_j) / 2.0 ** 24
        out[child[j]] += reach * a_j
        reach *= 1 - a_j
    ua = [1 - 2.0 ** -24] * m
    prev = 0
    for v in range(V):
        hi = _threshold(lambda U, v=v: so.verify_children_deterministic(p, child, ua, U)[1] <= v, lo=prev)
        out[v] += reach * (hi - prev) / 2.0 ** 24
        prev = hi
    assert np.abs(out - p).max() < 2e-6, (out, p)


def test_deterministic_drafts_are_the_most_probable_candidates():
    ids = np.array([40, 7, 19, 3, 28])
    phi = np.array([0.1, 0.3, 0.3, 0.05, 0.2])
    assert list(so.most_probable(ids, phi, 3)) == [7, 19, 28]      # equal probabilities: lower id first
    assert list(so.most_probable(ids, phi, 9)) == [7, 19, 28, 40, 3]
    # through the whole oracle: the tree holds the top candidates in order and no randomness enters drafting
    parent = np.array([-1, 0, 0, 0], np.int32)
    trees = []
    for seed in (1, 2):
        o = so.Oracle(1, 4, 50, 5, 2, 0, 1.0, seed, parent, deterministic=True)
        i = np.array([[40, 7, 19, 3, 28]], np.int32)
        o.update_bulk(np.array([[-1, 9]], np.int32), i, phi[None].astype(np.float32))
        o.reset_sequences(np.array([[-1, 9]], np.int32), np.array([1]))
        trees.append(o.draft()[0].tolist())
        o.close()
    assert trees[0] == trees[1] == [9, 7, 19, 28]


def test_deterministic_walk_chi_square():
    """1e5 trials through the full oracle in deterministic mode (table -> top candidates -> tree verification):
    the first emitted token follows the root's target distribution."""
    V, K = 12, 4
    parent = np.array([-1, 0, 0, 0, 1, 1, 2], np.int32)
    N = len(parent)
    rng = np.random.default_rng(6)
    logits = (rng.standard_normal((1, N, V)) * 1.5).astype(np.float32)
    T, Bn, reps = 0.8, 250, 400
    big = np.ascontiguousarray(np.broadcast_to(logits, (Bn, N, V)))
    first = np.zeros(V)
    accepted = 0
    for rep in range(reps):
        o = so.Oracle(Bn, N, V, K, 2, 0, T, 5000 + rep, parent, deterministic=True)
        ctx = np.array([[-1, t] for t in range(V)], np.int32)
        ids = np.array([[(t + 1 + 2 * i) % V for i in range(K)] for t in range(V)], np.int32)
        probs = np.tile(np.array([0.5, 0.2, 0.2, 0.1], np.float32), (V, 1))
        o.update_bulk(ctx, ids, probs)
        o.reset_sequences(np.tile(np.array([-1, 3], np.int32), (Bn, 1)), np.full(Bn, 1))
        tree = o.draft()
        assert (tree == tree[0]).all()  # no randomness in deterministic drafting
        em, ne = o.verify(big)
        np.add.at(first, em[:, 0], 1)
        accepted += int((ne >= 2).sum())
        o.close()
    _, _, _, _, p0 = so.row_stats(logits[0, 0], float(np.float32(T)), K, want_p=True)
    assert accepted > 0
    assert stats.chisquare(first, p0 * first.sum()).pvalue > 0.01


# ------------------------------------------------------ N-gram module (Sec. 4.1)
def test_merge_hand_cases():
    for line in open(os.path.join(GOLD, "merge_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, count, old, fresh, want = [f.strip() for f in line.split("|")]
        k, count = int(k), int(count)
        parse = lambda s: [(int(a), float(b)) for a, b in (t.split(":") for t in s.split())]
        old, fresh, want = parse(old), parse(fresh), parse(want)
        o = so.Oracle(1, 1, 64, k, 1, 0, 1.0, 0, np.array([-1], np.int32))

        def row(items):
            ids = np.full((1, k), -1, np.int32)
            pr = np.zeros((1, k), np.float32)
            for i, (a, b) in enumerate(items):
                ids[0, i], pr[0, i] = a, b
            return ids, pr
        # `count` sightings of the old distribution, then the fresh one
        for _ in range(count):
            o.update_bulk(np.array([[42]], np.int32), *row(old))
        o.update_bulk(np.array([[42]], np.int32), *row(fresh))
        cnt, ids, pr = o.table_get([42])
        assert cnt == count + 1
        assert list(ids) == [a for a, _ in want]
        assert np.allclose(pr, [b for _, b in want], rtol=1e-6)
        o.close()


def test_table_equals_recount_of_the_stream():
    """With one-hot rows the stored values are the empirical next-token frequencies of
    a count-based N-gram model: recount them from the token stream."""
    rng = np.random.default_rng(7)
    Vs, n_max, K = 5, 3, 8  # K >= Vs: nothing is ever truncated
    stream = rng.integers(0, Vs, 400)
    o = so.Oracle(1, 1, Vs, K, n_max, 0, 1.0, 0, np.array([-1], np.int32))
    ctx, ids, pr = [], [], []
    for i in range(len(stream) - 1):
        w = [-1] * n_max
        for t in range(n_max):
            j = i - (n_max - 1 - t)
            if j >= 0:
                w[t] = stream[j]
        ctx.append(w)
        ids.append([stream[i + 1]] + [-1] * (K - 1))
        pr.append([1.0] + [0.0] * (K - 1))
    o.update_bulk(np.array(ctx, np.int32), np.array(ids, np.int32), np.array(pr, np.float32))
    counts = {}
    for n in range(1, n_max + 1):
        for i in range(n - 1, len(stream) - 1):
            key = tuple(int(t) for t in stream[i - n + 1:i + 1])
            counts.setdefault(key, {}).setdefault(int(stream[i + 1]), 0)
            counts[key][int(stream[i + 1])] += 1
    table = o.table()
    assert set(table) == set(counts)
    for key, nxt in counts.items():
        total = sum(nxt.values())
        cnt, items = table[key]
        assert cnt == total
        assert set(items) == set(nxt)
        for t, c in nxt.items():
            assert abs(items[t] - c / total) < 1e-12
    o.close()


def test_truncation_keeps_the_most_probable():
    o = so.Oracle(1, 1, 64, 2, 1, 0, 1.0, 0, np.array([-1], np.int32))
    o.update_bulk(np.array([[1]], np.int32), np.array([[10, 11]], np.int32), np.array([[0.6, 0.4]], np.float32))
    o.update_bulk(np.array([[1]], np.int32), np.array([[12, 11]], np.int32), np.array([[0.9, 0.1]], np.float32))
    cnt, ids, pr = o.table_get([1])
    # 10: .3, 11: .25, 12: .45 -> keep 12, 10
    assert cnt == 2 and list(ids) == [12, 10] and np.allclose(pr, [0.45, 0.3], rtol=1e-6)
    o.close()


# ------------------------------------------------------ lookup order (Sec. 4.2)
def _mk(o, window, ids):
    K = o.K
    i = np.full((1, K), -1, np.int32)
    p = np.zeros((1, K), np.float32)
    i[0, :len(ids)] = ids
    p[0, :len(ids)] = 1.0 / len(ids)
    o.update_bulk(np.array([window], np.int32), i, p)


def test_lookup_prefers_the_longest_order_and_takes_the_first_hit():
    parent = np.array([-1, 0, 0, 1], np.int32)
    V, K, n_max = 50, 4, 3
    # only the unigram (7,) and bigram (6,7) exist after feeding window [-1,6,7]:
    o = so.Oracle(1, 4, V, K, n_max, 0, 1.0, 0, parent)
    _mk(o, [-1, 6, 7], [20, 21])
    # now overwrite the unigram of 7 alone with other ids through a window that only has 7
    _mk(o, [-1, -1, 7], [30, 31, 32])
    t = o.table()
    assert set(t) == {(7,), (6, 7)}
    # unigram of 7: {20,21} at 1/2 merged with {30,31,32} at 1/3 -> .25,.25,1/6,1/6,1/6, cut to 4 (ties: lower id)
    assert t[(7,)][0] == 2 and set(t[(7,)][1]) == {20, 21, 30, 31}
    # sequence ends with ... 6 7: the bigram wins, children come from {20, 21}
    o.reset_sequences(np.array([[5, 6, 7]], np.int32), np.array([3]))
    tree = o.draft()
    assert tree[0, 0] == 7 and set(tree[0, 1:3]) == {20, 21}
    # node 3 hangs under node 1: its context ends with (7, tree[1]) -> no bigram,
    # no unigram for tree[1] -> undrafted
    assert tree[0, 3] == -1
    # sequence ends with 9 7: only the unigram matches
    o.reset_sequences(np.array([[5, 9, 7]], np.int32), np.array([3]))
    tree = o.draft()
    assert set(tree[0, 1:3]) <= {20, 21, 30, 31} and tree[0, 1] != tree[0, 2]
    # a hit with fewer candidates than children: the rest stays undrafted (no fall-through)
    o2 = so.Oracle(1, 4, V, K, n_max, 0, 1.0, 0, parent)
    _mk(o2, [-1, -1, 7], [30, 31, 32])
    _mk(o2, [-1, 6, 7], [20])
    o2.reset_sequences(np.array([[5, 6, 7]], np.int32), np.array([3]))
    tree = o2.draft()
    assert tree[0, 1] == 20 and tree[0, 2] == -1
    o.close(); o2.close()


def test_update_feeds_only_the_accepted_path_in_order():
    """After one step the table holds exactly the contexts of the accepted path."""
    parent = np.array([-1, 0, 1], np.int32)
    V, K, n_max = 20, 3, 2
    rng = np.random.default_rng(11)
    logits = (rng.standard_normal((1, 3, V)) * 2).astype(np.float32)
    o = so.Oracle(1, 3, V, K, n_max, 0, 1.0, 3, parent)
    o.reset_sequences(np.array([[4, 5]], np.int32), np.array([2]))
    em, ne, tree = o.step(logits)
    # nothing was drafted before the first step: one token sampled from the root row
    assert ne[0] == 1
    t = o.table()
    assert set(t) == {(5,), (4, 5)}
    _, ids, _, probs, _ = so.row_stats(logits[0, 0], 1.0, K)
    for key in t:
        assert t[key][0] == 1 and list(t[key][1]) == list(ids)
        assert np.allclose(list(t[key][1].values()), probs)
    st = o.state()
    assert list(st["tail"][0]) == [5, em[0, 0]] and st["len"][0] == 3 and tree[0, 0] == em[0, 0]
    o.close()


def test_sequence_base_offsets_the_counter_of_every_draw():
    """A context that holds sequences seq_base.. of a larger batch draws the random numbers of those sequences
    (counter word 0 = seq_base + b): with a one-node tree every step is one inverse-CDF draw, recomputed here
    from the published uniform of sequence seq_base + b."""
    V, T, seed, base = 64, 0.8, 11, 3
    rng = np.random.default_rng(5)
    parent = np.array([-1], np.int32)
    o = so.Oracle(2, 1, V, 4, 2, 0, T, seed, parent, seq_base=base)
    o.reset_sequences(np.full((2, 2), 1, np.int32), np.full(2, 4, np.int64))
    shifted = 0
    for step in range(1, 21):
        logits = rng.normal(0, 2, size=(2, 1, V)).astype(np.float32)
        em, ne, _ = o.step(logits)
        assert list(ne) == [1, 1]
        for b in range(2):
            z = logits[b, 0].astype(np.float64) / np.float64(np.float32(T))
            p = np.exp(z - z.max())
            cdf = np.cumsum(p)
            pick = lambda seq: int(np.searchsorted(cdf, so.uniform(seed, seq, step, 0, 0x40000000) * cdf[-1], side="right"))
            assert em[b, 0] == pick(base + b)
            shifted += em[b, 0] != pick(b)
    assert shifted > 20  # and not those of sequences 0, 1
    o.take_margins()
    o.close()


# ------------------------------- the update's pairing of rows and context windows (Sec. 4.1, Fig. "Overview")
def _one_hot_logits(parent, streams, lens, V):
    """Row (b, u) puts all its mass on the token that the stream holds at the position the row predicts
    (len_b + depth(u)): exp(-1000) is zero in double precision, so every row is a one-hot distribution."""
    depth = np.zeros(len(parent), int)
    for u in range(1, len(parent)):
        depth[u] = depth[parent[u]] + 1
    x = np.zeros((len(streams), len(parent), V), np.float32)
    for b in range(len(streams)):
        for u in range(len(parent)):
            x[b, u, streams[b][lens[b] + depth[u]]] = 1000.0
    return x


@pytest.mark.parametrize("B", [1, 3])
def test_closed_loop_table_equals_a_recount_of_the_emitted_stream(B):
    """Whole steps (verify -> update -> draft) on one-hot target rows: whatever is drafted, the emitted tokens are
    the stream's, accepted paths are several nodes long once contexts repeat, and the table must hold, under every
    order, exactly the follower frequencies of the emitted text (Sec. 4.1: "when the language model generates
    'I am Bob' we store the distribution" of the token after it).  The recount below knows nothing about trees or
    paths: it pins which row is paired with which context window along an accepted path."""
    rng = np.random.default_rng(40 + B)
    V, K, n_max = 40, 6, 3
    parent = np.array([-1, 0, 0, 1, 1, 2, 3, 3, 6, 8], np.int32)  # branching: a node's index is not its depth
    prompt, total = 5, 700
    # text made of a few recurring phrases over five tokens: inside a phrase a context has one follower and the
    # drafts run deep, at a phrase boundary it has several and drafts are rejected
    phrases = [list(3 + 7 * rng.integers(0, 5, rng.integers(5, 10))) for _ in range(5)]
    streams = []
    for _ in range(B):
        text = []
        while len(text) < total:
            text += phrases[rng.integers(0, len(phrases))]
        streams.append(text)
    o = so.Oracle(B, len(parent), V, K, n_max, 0, 1.0, 17, parent)
    tail = np.array([s[prompt - n_max:prompt] for s in streams], np.int32)
    lens = np.full(B, prompt, np.int64)
    o.reset_sequences(tail, lens)
    deep = 0
    for _ in range(120):
        em, ne, _ = o.step(_one_hot_logits(parent, streams, lens, V))
        for b in range(B):
            assert list(em[b, :ne[b]]) == streams[b][lens[b]:lens[b] + ne[b]]  # lossless on one-hot targets
        deep += int((ne >= 3).sum())
        lens = lens + ne
    o.take_margins()
    assert deep > 20 * B  # accepted paths with j >= 2 are the rule, not the exception
    assert np.array_equal(o.state()["len"], lens)
    want = {}
    for b in range(B):
        for t in range(prompt, int(lens[b])):
            for n in range(1, n_max + 1):
                key = tuple(int(v) for v in streams[b][t - n:t])
                want.setdefault(key, {}).setdefault(int(streams[b][t]), 0)
                want[key][int(streams[b][t])] += 1
    got = o.table()
    assert set(got) == set(want)
    for key, followers in want.items():
        cnt, items = got[key]
        n_seen = sum(followers.values())
        assert cnt == n_seen
        positive = {t: v for t, v in items.items() if v > 0}
        assert set(positive) == set(followers)
        for t, c in followers.items():
            assert abs(positive[t] - c / n_seen) < 1e-12
    o.close()


def test_deep_nodes_are_drafted_from_the_tail_plus_the_tokens_on_their_own_path():
    """Sec. 4.2, "for each position in the draft tree": the context of a node below depth 1 is the sequence
    followed by the tokens drafted on the way from the root to that node.  Here every lookup that matters can only
    hit through such a context, and the two branches of the tree must each continue their own token."""
    parent = np.array([-1, 0, 0, 1, 2, 3, 4], np.int32)  # two children of the root, each heads a chain of three
    V, K, n_max = 100, 4, 2

    def feed(o, window, ids, times=1):
        i = np.full((1, K), -1, np.int32)
        p = np.zeros((1, K), np.float32)
        i[0, :len(ids)] = ids
        p[0, :len(ids)] = 1.0 / len(ids)
        for _ in range(times):
            o.update_bulk(np.array([window], np.int32), i, p)

    orders_seen = set()
    for seed in range(8):
        o = so.Oracle(1, len(parent), V, K, n_max, 0, 1.0, seed, parent)
        feed(o, [6, 7], [20, 21])        # after (6, 7): 20 or 21
        feed(o, [7, 20], [50])           # after (7, 20): 50      after (7, 21): 51
        feed(o, [7, 21], [51])
        feed(o, [20, 50], [60])          # after (20, 50): 60     after (21, 51): 61
        feed(o, [21, 51], [61])
        # the shorter contexts alone point elsewhere: a lookup that loses the path's earlier token is led astray
        for tok, wrong in ((20, 40), (21, 41), (50, 42), (51, 43)):
            feed(o, [9, tok], [wrong], times=5)
        o.reset_sequences(np.array([[6, 7]], np.int32), np.array([2]))
        tree = o.draft()[0]
        assert tree[0] == 7 and sorted(tree[1:3]) == [20, 21]
        orders_seen.add(tuple(tree[1:3]))
        for head, mid, leaf in ((1, 3, 5), (2, 4, 6)):
            assert tree[mid] == {20: 50, 21: 51}[tree[head]]   # context (7, tree[head]): tail + one path token
            assert tree[leaf] == {50: 60, 51: 61}[tree[mid]]   # context (tree[head], tree[mid]): path tokens only
        st = o.state()
        assert st["cand_n"][0, 1] == 1 and st["cand_id"][0, 1, 0] == tree[3]  # the snapshot is the bigram's list
        o.close()
    assert len(orders_seen) == 2  # both Gumbel orders of the root's children occurred

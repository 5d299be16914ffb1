"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest

from oracle import stand_oracle as so
from paper_2506_04708_b200 import inputs
from tests import harness

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


# ------------------------------------------------------------------ row pass (a1)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [2, 13, 16, 1000, 1024, 1032, 5000, 32000, 151936])
def test_row_stats_matches_oracle(dtype, V):
    from paper_2506_04708_b200 import binding
    torch = _torch()
    rng = np.random.default_rng(V)
    rows, k, T = 5, 10, 0.7
    x = (rng.standard_normal((rows, V)) * 2.5).astype(np.float32)
    x[0, rng.integers(0, V)] += 8
    x[1, :] = np.round(x[1, :])          # many exact ties
    x[2, :] = -30.0 - np.abs(x[2, :])    # far from zero: the offset logic must cope
    if V > 1024:
        x[3, :1024] -= 200.0             # first chunk far below the rest: forces a new offset
        x[4] = np.sort(x[4])             # ascending: every vector brings new candidates
    raw = inputs.f32_to_bf16_bits(x) if dtype == "bf16" else x
    dl = harness.to_device_logits(raw)
    lse, ids, vals, probs = (t.cpu().numpy() for t in binding.row_stats(dl, T, k))
    tol = harness.value_tol(inputs.DTYPE_BF16 if dtype == "bf16" else inputs.DTYPE_F32)
    for r in range(rows):
        olse, oids, ovals, oprobs, _ = so.row_stats(raw[r], float(np.float32(T)), k)
        assert np.array_equal(ids[r], oids), (r, ids[r], oids)
        kk = min(k, V)
        assert np.array_equal(vals[r, :kk].astype(np.float64), ovals[:kk])
        assert abs(lse[r] - olse) <= 1e-5 * max(1.0, abs(olse))
        assert np.allclose(probs[r, :kk], oprobs[:kk], rtol=tol, atol=1e-30)


@pytest.mark.parametrize("dtype,V", [("bf16", 151936), ("f32", 128256), ("bf16", 40008)])
def test_row_stats_large_launch_takes_the_streaming_kernel(dtype, V):
    """Launches of more than a couple of waves of chunks go through the bulk-copy ring (smaller ones are read
    directly, one warp per chunk): enough rows to be there, sampled rows against the oracle."""
    from paper_2506_04708_b200 import binding
    torch = _torch()
    rows, k, T = 60000 // ((V + 1023) // 1024) + 1, 10, 0.7  # more chunks than the direct kernel takes on this GPU
    g = torch.Generator(device="cuda:0").manual_seed(V)
    x = torch.randn((rows, V), generator=g, device="cuda:0") * 2.5
    x[torch.arange(rows), torch.randint(0, V, (rows,), generator=g, device="cuda:0")] += 8.0
    dl = x.to(torch.bfloat16) if dtype == "bf16" else x
    host = dl.cpu()
    raw = host.view(torch.int16).numpy().view(np.uint16) if dtype == "bf16" else host.numpy()
    lse, ids, vals, probs = (t.cpu().numpy() for t in binding.row_stats(dl, T, k))
    tol = harness.value_tol(inputs.DTYPE_BF16 if dtype == "bf16" else inputs.DTYPE_F32)
    for r in list(range(0, rows, max(1, rows // 24))) + [rows - 1]:
        olse, oids, ovals, oprobs, _ = so.row_stats(raw[r], float(np.float32(T)), k)
        assert np.array_equal(ids[r], oids), (r, ids[r], oids)
        assert abs(lse[r] - olse) <= 1e-5 * max(1.0, abs(olse))
        assert np.allclose(probs[r], oprobs, rtol=tol, atol=1e-30)


def test_row_stats_unaligned_rows_and_many_rows():
    from paper_2506_04708_b200 import binding
    torch = _torch()
    rng = np.random.default_rng(5)
    rows, V, k = 300, 1001, 8   # V*esize is not a multiple of 16: scalar loads
    x = (rng.standard_normal((rows, V)) * 3).astype(np.float32)
    for raw in (x, inputs.f32_to_bf16_bits(x)):
        lse, ids, vals, probs = (t.cpu().numpy() for t in binding.row_stats(harness.to_device_logits(raw), 1.0, k))
        for r in range(0, rows, 17):
            olse, oids, ovals, oprobs, _ = so.row_stats(raw[r], 1.0, k)
            assert np.array_equal(ids[r], oids)
            assert abs(lse[r] - olse) <= 1e-5 * max(1.0, abs(olse))
            assert np.allclose(probs[r], oprobs, rtol=1e-5 if raw.dtype == np.float32 else 4e-3)


def test_row_stats_degenerate_rows():
    """Rows that defeat the chunk-maximum bound: constant rows (every entry reaches the bound, so the candidate
    buffers overflow and the streaming selection takes over), rows with -inf, and one-entry maxima."""
    from paper_2506_04708_b200 import binding
    V, k = 5000, 10
    x = np.zeros((6, V), np.float32)
    x[0, :] = 1.5                                  # constant: top-k = the first k ids
    x[1, :] = -np.inf; x[1, 4321] = 0.25           # a single finite entry
    x[2, :] = np.arange(V) % 7                     # long runs of equal maxima in every chunk
    x[3, :] = -np.inf; x[3, :3] = [1.0, 2.0, 3.0]  # fewer finite entries than k
    x[4, :] = -1e6; x[4, V - 1] = 1e6              # extreme spread (the documented range is |x| log2(e) / T < 2^24)
    x[5, :] = -0.0; x[5, ::2] = 0.0                # +0 and -0 are one value: ties by id
    for raw in (x, inputs.f32_to_bf16_bits(x)):
        tol = 1e-5 if raw.dtype == np.float32 else 4e-3
        lse, ids, vals, probs = (t.cpu().numpy() for t in binding.row_stats(harness.to_device_logits(raw), 1.0, k))
        for r in range(x.shape[0]):
            olse, oids, ovals, oprobs, _ = so.row_stats(raw[r], 1.0, k)
            assert np.array_equal(ids[r], oids), (r, ids[r], oids)
            assert abs(lse[r] - olse) <= 1e-5 * max(1.0, abs(olse)), (r, lse[r], olse)
            assert np.allclose(probs[r], oprobs, rtol=tol, atol=1e-30), r


def test_maximum_sizes():
    """The largest vocabulary (2^20: 1024 chunks, the general bound search), the largest tree (128 nodes), top-12,
    order 4: a few whole steps against the oracle."""
    parent = inputs.topology(128, 8, 4)
    w = inputs.Workload("max", 2, 128, 8, 4, 1 << 20, inputs.DTYPE_BF16, 0.7, 4, 12, 3, 1 << 14, 2.5, 0.6, 32, 1.05)
    loop = harness.ClosedLoop(w, seed=1, peak_mode="add8", parent=parent, device_logits=True)
    try:
        for _ in range(w.steps):
            loop.step()
        assert loop.hard == [] and loop.check_state_and_table() == []
        assert loop.gpu.stats()["wait_timeouts"] == 0
    finally:
        loop.close()


def test_constant_logits_through_the_whole_step():
    """Every row constant: the uniform target distribution, all top-k ties broken by id, through verify, update,
    draft; every sequence of every step is judged by the margin rule."""
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=2, V=3000, steps=6)
    loop = harness.ClosedLoop(w, seed=3, table_slots=1 << 12, tail=np.array([[1, 2, 3], [4, 5, 6]], np.int32))
    logits = np.full((w.B, w.N, w.V), 0.5, np.float32)
    try:
        for s in range(w.steps):
            loop.step(logits)
        assert loop.hard == [] and loop.tolerated <= 1
        assert loop.check_state_and_table() == []
    finally:
        loop.close()


# ------------------------------------------------------------- whole step, closed loop
def _run(w, steps, peak_mode, seed=0, check_every=0, **kw):
    w = inputs.scaled(w, steps=steps)
    loop = harness.ClosedLoop(w, seed=seed, peak_mode=peak_mode, **kw)
    try:
        for s in range(steps):
            loop.step()
            if check_every and (s + 1) % check_every == 0:
                assert loop.check_state_and_table() == []
        assert loop.hard == [], loop.hard[:3]
        assert loop.check_state_and_table() == []
        st = loop.gpu.stats()
        assert st["drops"] == 0 and st["bad_tokens"] == 0 and st["wait_timeouts"] == 0
        # low-margin decisions are rare: a few per ten thousand verified rows at most
        assert loop.tolerated <= max(2, int(3e-4 * steps * w.B * w.N))
        return loop.emitted_total / (steps * w.B), loop.tolerated, st
    finally:
        loop.close()


@pytest.mark.parametrize("peak_mode", ["add8", "p80"])
def test_cfg1_full_run(peak_mode):
    acc, tolerated, st = _run(inputs.WORKLOADS["cfg1"], 1000, peak_mode, table_slots=1 << 16, check_every=250)
    if peak_mode == "p80":
        assert acc > 1.15  # accept paths deeper than the root are exercised
        assert sum(st["lookup_hits"]) > 0


@pytest.mark.parametrize("peak_mode", ["add8", "p80"])
def test_cfg2_window(peak_mode):
    acc, _, st = _run(inputs.WORKLOADS["cfg2"], 48, peak_mode, table_slots=1 << 16, check_every=16)


@pytest.mark.parametrize("peak_mode", ["add8", "p80"])
def test_cfg3_window(peak_mode):
    _run(inputs.WORKLOADS["cfg3"], 64, peak_mode, table_slots=1 << 18, check_every=32, device_logits=True)


@pytest.mark.parametrize("peak_mode", ["add8", "p80"])
def test_cfg4_window(peak_mode):
    _run(inputs.WORKLOADS["cfg4"], 32, peak_mode, table_slots=1 << 18, check_every=16, device_logits=True)


def test_cfg5_shape_small_vocab():
    # the tree-search shape (256 forked beams, shared prefixes -> many same-step updates of one context)
    w = inputs.scaled(inputs.WORKLOADS["cfg5"], V=4096)
    _run(w, 40, "p80", table_slots=1 << 18, check_every=10)


@pytest.mark.parametrize("peak_mode", ["add8", "p80"])
def test_cfg5_full_size_in_the_benchmark_configuration(peak_mode):
    """The benchmark's workload at full size (256 x 24 rows of 151,936 bf16, 16M-slot table): whole steps against the
    oracle, every emitted token, tree, table entry and state word."""
    w = inputs.WORKLOADS["cfg5"]
    steps = 4
    loop = harness.ClosedLoop(inputs.scaled(w, steps=steps), seed=0, peak_mode=peak_mode, device_logits=True)
    try:
        for _ in range(steps):
            loop.step()
        assert loop.hard == [], loop.hard[:3]
        assert loop.check_state_and_table() == []
        st = loop.gpu.stats()
        assert st["drops"] == 0 and st["bad_tokens"] == 0 and st["wait_timeouts"] == 0
        assert st["records"] >= w.B * steps
        assert loop.tolerated <= 2
    finally:
        loop.close()


@pytest.mark.parametrize("V,N,D,kb", [(16, 1, 0, 1), (13, 4, 2, 2), (50, 7, 3, 2), (1000, 16, 4, 3)])
@pytest.mark.parametrize("dtype", [inputs.DTYPE_F32, inputs.DTYPE_BF16])
def test_tiny_shapes(V, N, D, kb, dtype):
    w = inputs.Workload("tiny", 3, N, D, kb, V, dtype, 0.9, 3, min(6, V), 60, 1 << 12, 2.0, 0.7, 12, 1.1)
    _run(w, 60, "p80", check_every=20)


def test_more_sequences_than_resident_blocks():
    """Many more sequences than the GPU holds thread blocks at once: several waves of every per-sequence kernel."""
    w = inputs.Workload("wide", 700, 4, 2, 2, 200, inputs.DTYPE_F32, 0.9, 2, 6, 12, 1 << 14, 2.0, 0.7, 12, 1.1)
    _run(w, 12, "p80", check_every=6)


# ------------------------------------------------------------ deterministic drafting (Sec. 3.2)
@pytest.mark.parametrize("dtype", [inputs.DTYPE_F32, inputs.DTYPE_BF16])
def test_deterministic_drafting_small(dtype):
    w = inputs.Workload("det", 4, 16, 4, 3, 3000, dtype, 0.8, 3, 8, 120, 1 << 14, 2.0, 0.7, 16, 1.1)
    acc, _, st = _run(w, 120, "p80", check_every=40, deterministic=True)
    assert acc > 1.1 and sum(st["lookup_hits"]) > 0


def test_deterministic_drafting_cfg3_window():
    _run(inputs.WORKLOADS["cfg3"], 8, "p80", table_slots=1 << 16, check_every=4, deterministic=True)


def test_deterministic_and_stochastic_drafting_differ_only_in_the_draft():
    """Same seeds, same logits: before any tree exists both modes emit the same first token; afterwards the
    deterministic tree holds the most probable candidates of each lookup."""
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=2)
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    streams = inputs.token_streams(w, 5, 300)
    a = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 5, 1 << 12, parent)
    b = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 5, 1 << 12, parent, deterministic=True)
    tail = torch.from_numpy(streams[:, 5:8].copy())
    lens = np.full(w.B, 8, np.int64)
    for g in (a, b):
        g.reset_sequences(tail, torch.from_numpy(lens))
    dl = harness.to_device_logits(inputs.logits_numpy(w, streams, lens, depth, 0, 5, "p80"))
    ea, _, ta = (t.cpu().numpy().copy() for t in a.step(dl))
    eb, _, tb = (t.cpu().numpy().copy() for t in b.step(dl))
    assert np.array_equal(ea, eb)              # no tree yet: one token from the root row, same uniform
    st = b.state_dump()
    for s in range(w.B):                        # the first child of the root is the most probable candidate
        n = st["cand_n"][s, 0]
        if n:
            best = st["cand_id"][s, 0, np.lexsort((st["cand_id"][s, 0, :n], -st["cand_phi"][s, 0, :n]))[0]]
            assert tb[s, 1] == best
    a.close(); b.close()


# ------------------------------------------------ acceptance counters and tree optimisation (Sec. 4.2)
def test_node_acceptance_counters_and_tree_optimisation():
    """Data-driven tree optimisation on a synthetic workload: start from (a 128-node prefix of) Algorithm 1's
    tree, count how often each node is accepted, keep the most accepted nodes, run on with the smaller tree."""
    from paper_2506_04708_b200 import binding
    parent, depth, _, total = binding.initial_tree(20, capacity=128)
    assert total == 625
    D = int(depth.max())
    w = inputs.Workload("opt", 6, 128, D, 8, 3000, inputs.DTYPE_F32, 0.9, 3, 8, 50, 1 << 14, 2.0, 0.7, 16, 1.1)
    loop = harness.ClosedLoop(w, seed=2, peak_mode="p80", parent=parent)
    counts = np.zeros(128, np.uint64)
    try:
        for _ in range(w.steps):
            loop.step()
            for row in loop.orc.path():
                for u in row[row >= 0]:
                    counts[u] += 1
        assert loop.hard == [] and loop.tolerated <= 2
        got = loop.gpu.node_accepts()
        if loop.tolerated == 0:
            assert np.array_equal(got, counts)
        assert got[0] == w.B * w.steps and got[1:].sum() > 0
        assert all(got[u] <= got[parent[u]] for u in range(1, 128))
        small, old = binding.prune_tree(parent, got, 24)
        assert loop.gpu.node_accepts(reset=True)[0] == got[0] and loop.gpu.node_accepts().sum() == 0
    finally:
        loop.close()
    # the optimised tree is a valid topology and runs in parity too
    d2 = int(inputs.node_depths(small).max())
    w2 = inputs.Workload("opt24", 6, 24, d2, 8, 3000, inputs.DTYPE_F32, 0.9, 3, 8, 30, 1 << 14, 2.0, 0.7, 16, 1.1)
    loop2 = harness.ClosedLoop(w2, seed=2, peak_mode="p80", parent=small)
    try:
        for _ in range(w2.steps):
            loop2.step()
        assert loop2.hard == [] and loop2.check_state_and_table() == []
    finally:
        loop2.close()


@pytest.mark.parametrize("B", [3, 1])  # a batch, and the paper's own setting: one sequence (the two-launch step)
def test_full_initial_tree_to_eighty_nodes(B):
    """The paper's procedure at its own sizes (Sec. 4.2, App. A.1): all 625 nodes of Algorithm 1's tree, acceptance
    counts over a run, the 80 most accepted nodes kept."""
    from paper_2506_04708_b200 import binding
    parent, depth, _, total = binding.initial_tree()
    assert total == 625 and len(parent) == 625
    w = inputs.Workload("init625", B, 625, int(depth.max()), 8, 2000, inputs.DTYPE_BF16, 0.6, 4, 10, 25, 1 << 14, 2.0, 0.7,
                        24, 1.05)
    loop = harness.ClosedLoop(w, seed=4, peak_mode="p80", parent=parent)
    try:
        for _ in range(w.steps):
            loop.step()
        assert loop.hard == [] and loop.check_state_and_table() == []
        got = loop.gpu.node_accepts()
        assert got[0] == w.B * w.steps
        small, old = binding.prune_tree(parent, got, 80)
    finally:
        loop.close()
    assert len(small) == 80 and small[0] == -1
    w2 = inputs.Workload("opt80", B, 80, int(inputs.node_depths(small).max()), 8, 2000, inputs.DTYPE_BF16, 0.6, 4, 10, 20,
                         1 << 14, 2.0, 0.7, 24, 1.05)
    loop2 = harness.ClosedLoop(w2, seed=4, peak_mode="p80", parent=small)
    try:
        for _ in range(w2.steps):
            loop2.step()
        assert loop2.hard == [] and loop2.check_state_and_table() == []
    finally:
        loop2.close()


# ------------------------------------------------------------------- stages on their own
@pytest.mark.parametrize("B", [1, 4, 16, 20])
def test_stage_calls_equal_the_fused_step(B):
    """stand_step against verify / update / draft called one by one.  A single sequence takes the step's
    two-launch form with its whole tail in one block, a batch of up to 16 the two-launch form with the tail in
    one thread-block cluster, a larger batch the four-launch form."""
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=B, steps=30)
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    streams = inputs.token_streams(w, 3, 400)
    a = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 3, 1 << 14, parent)
    b = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 3, 1 << 14, parent)
    tail = torch.from_numpy(streams[:, 5:8].copy())
    lens = np.full(w.B, 8, np.int64)
    a.reset_sequences(tail, torch.from_numpy(lens))
    b.reset_sequences(tail, torch.from_numpy(lens))
    for s in range(30):
        dl = harness.to_device_logits(inputs.logits_numpy(w, streams, lens, depth, s, 3, "p80"))
        ea, na, ta = (t.cpu().numpy().copy() for t in a.step(dl))
        b.verify_tree(dl)
        b.ngram_update()
        b.draft_tree()
        assert np.array_equal(ea, b.emitted.cpu().numpy()) and np.array_equal(na, b.n_emitted.cpu().numpy())
        assert np.array_equal(ta, b.tree.cpu().numpy())
        lens = a.state_dump()["len"]
    assert a.launch_count() - b.launch_count() == (-30 * 3 if B <= 16 else -30)  # 2 (or 4) launches per step against 5
    ta = a.table_dict()
    assert ta == b.table_dict() and len(ta) > 50
    # update without a pending verification is refused
    from paper_2506_04708_b200.binding import StandError
    with pytest.raises(StandError):
        b.ngram_update()
    a.close(); b.close()


def test_sequence_base_against_the_oracle():
    """A context whose sequences are numbers 5.. of a larger batch (seq_base = 5): its random numbers are those
    of sequences 5.., on both sides; and they are not those of sequences 0..."""
    w = inputs.Workload("tiny", 3, 16, 4, 3, 1000, inputs.DTYPE_BF16, 0.9, 3, 6, 60, 1 << 12, 2.0, 0.7, 12, 1.1)
    emitted = {}
    for base in (5, 0):
        loop = harness.ClosedLoop(w, seed=2, peak_mode="p80", seq_base=base)
        try:
            seen = []
            for _ in range(w.steps):
                seen.append(loop.step()[0].copy())
            assert loop.hard == [] and loop.check_state_and_table() == []
            assert loop.tolerated <= 2
            emitted[base] = np.stack(seen)
        finally:
            loop.close()
    assert not np.array_equal(emitted[5], emitted[0])


@pytest.mark.parametrize("deterministic", [False, True])
def test_sharded_contexts_equal_the_unsharded_one(deterministic):
    """A batch of 6 sequences split 2 + 4 over two contexts (seq_base 0 and 2), each with its own copy of the
    table, the accepted rows exchanged every step and applied in global sequence order: emitted tokens, drafts
    and both tables equal those of one context holding all 6 (which the other tests tie to the oracle)."""
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand, StandError
    from paper_2506_04708_b200 import sharded
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=6, steps=40)
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    streams = inputs.token_streams(w, 5, 500)
    mk = lambda B, base: Stand(B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 5, 1 << 14, parent,
                               deterministic=deterministic, seq_base=base)
    whole = mk(6, 0)
    cuts = [(0, 2), (2, 6)]
    parts = [sharded.ShardedStand(mk(hi - lo, lo)) for lo, hi in cuts]
    tail = torch.from_numpy(streams[:, 5:8].copy())
    lens = np.full(w.B, 8, np.int64)
    whole.reset_sequences(tail, torch.from_numpy(lens))
    for (lo, hi), sh in zip(cuts, parts):
        sh.stand.reset_sequences(tail[lo:hi], torch.from_numpy(lens[lo:hi]))
    for s in range(40):
        dl = harness.to_device_logits(inputs.logits_numpy(w, streams, lens, depth, s, 5, "p80"))
        ew, nw, tw = (t.cpu().numpy().copy() for t in whole.step(dl))
        rows = [sh.verify(dl[lo:hi].contiguous()) for (lo, hi), sh in zip(cuts, parts)]
        all_rows = sharded.concat_rows(rows)
        for (lo, hi), sh in zip(cuts, parts):
            tree = sh.finish(all_rows)
            assert np.array_equal(ew[lo:hi], sh.stand.emitted.cpu().numpy()), s
            assert np.array_equal(nw[lo:hi], sh.stand.n_emitted.cpu().numpy()), s
            assert np.array_equal(tw[lo:hi], tree.cpu().numpy()), s
        lens = whole.state_dump()["len"]
    assert nw.sum() > w.B  # drafts were accepted: the tables matter
    t0 = whole.table_dict()
    assert len(t0) > 100
    for sh in parts:
        assert sh.stand.table_dict() == t0
        assert sh.stand.stats()["drops"] == 0
    # nothing pending any more: neither export nor skip is valid
    with pytest.raises(StandError):
        parts[0].stand.export_records()
    with pytest.raises(StandError):
        parts[0].stand.skip_update()
    whole.close()
    for sh in parts:
        sh.stand.close()


@pytest.mark.parametrize("B", [1, 3])
def test_host_buffer_step_equals_the_device_buffer_step(B):
    """stand_step_host (logits in pinned host memory, results copied back, stream synchronised) against
    stand_step on device buffers: same emitted tokens, trees and tables, step by step."""
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand, StandError
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=B, steps=20, dtype=inputs.DTYPE_BF16)
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    streams = inputs.token_streams(w, 9, 300)
    mk = lambda staging: Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 9, 1 << 14, parent, host_staging=staging)
    dev, host = mk(False), mk(True)
    tail = torch.from_numpy(streams[:, 5:8].copy())
    lens = np.full(w.B, 8, np.int64)
    dev.reset_sequences(tail, torch.from_numpy(lens))
    host.reset_sequences(tail, torch.from_numpy(lens))
    h_em = torch.empty((w.B, dev.D + 1), dtype=torch.int32).pin_memory()
    h_ne = torch.empty(w.B, dtype=torch.int32).pin_memory()
    h_tr = torch.empty((w.B, w.N), dtype=torch.int32).pin_memory()
    for s in range(20):
        logits = inputs.logits_numpy(w, streams, lens, depth, s, 9, "p80")
        h_logits = torch.from_numpy(logits.view(np.int16)).view(torch.bfloat16).pin_memory()
        em, ne, tr = (t.cpu().numpy() for t in dev.step(harness.to_device_logits(logits)))
        host.step_host(h_logits, h_em, h_ne, h_tr)
        assert np.array_equal(em, h_em.numpy()) and np.array_equal(ne, h_ne.numpy()) and np.array_equal(tr, h_tr.numpy()), s
        lens = dev.state_dump()["len"]
    assert dev.table_dict() == host.table_dict()
    # a context made without the staging buffer refuses the host entry point
    with pytest.raises(StandError):
        dev.step_host(h_logits, h_em, h_ne, h_tr)
    dev.close(); host.close()


def test_table_persists_across_trajectories_and_resume_from_a_checkpoint():
    """Sec. 5.1: the N-gram module is kept across trajectories (stand_reset_sequences restarts the sequences only).
    And a run resumed in a fresh context from dumped table + state continues exactly like the original."""
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand
    w = inputs.scaled(inputs.WORKLOADS["cfg1"], B=3, V=4000, steps=40)
    loop = harness.ClosedLoop(w, seed=9, peak_mode="p80", table_slots=1 << 14)
    try:
        for _ in range(20):
            loop.step()
        n_ctx = len(loop.orc.table())
        # a new trajectory: same prompts, sequences restart, the table stays
        tail = np.full((w.B, w.order_max), -1, np.int32)
        tail[:, :] = loop.streams[:, 8 - w.order_max:8]
        lens = np.full(w.B, 8, np.int64)
        loop.gpu.reset_sequences(torch.from_numpy(tail), torch.from_numpy(lens))
        loop.orc.reset_sequences(tail, lens)
        loop.lens = lens
        assert len(loop.gpu.table_dict()) == n_ctx
        for _ in range(10):
            loop.step()
        assert loop.hard == [] and loop.check_state_and_table() == []
        assert len(loop.orc.table()) >= n_ctx and sum(loop.gpu.stats()["lookup_hits"]) > 0
        # checkpoint, resume elsewhere, and run both on the same logits
        other = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 9, 1 << 15, loop.parent)
        other.table_load(*loop.gpu.table_dump())
        other.state_load(loop.gpu.state_dump())
        for s in range(5):
            logits = inputs.logits_numpy(w, loop.streams, loop.lens, loop.depth, 100 + s, 9, "p80")
            dl = harness.to_device_logits(logits)
            a = [t.cpu().numpy().copy() for t in loop.gpu.step(dl)]
            b = [t.cpu().numpy().copy() for t in other.step(dl)]
            assert all(np.array_equal(x, y) for x, y in zip(a, b)), s
            loop.lens = loop.gpu.state_dump()["len"]
        assert other.table_dict() == loop.gpu.table_dict()
        other.close()
    finally:
        loop.close()


def test_bulk_update_and_table_roundtrip():
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand
    w = inputs.scaled(inputs.WORKLOADS["cfg5"], V=2000)
    ctx, ids, probs = inputs.pregrow_records(w, 1, 6000)
    parent = inputs.topology(w.N, w.D, w.kb)
    g = Stand(1, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, 1 << 16, parent)
    o = so.Oracle(1, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, parent)
    g.ngram_update_bulk(torch.from_numpy(ctx), torch.from_numpy(ids), torch.from_numpy(probs))
    o.update_bulk(ctx, ids, probs)
    ot = o.table()
    assert harness.compare_tables(g.table_dict(), ot, 1e-5) == []
    assert g.stats()["inserts"] == len(ot) and g.stats()["drops"] == 0
    # dump -> load into a fresh context -> same contents
    g2 = Stand(1, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, 1 << 15, parent)
    g2.table_load(*g.table_dump())
    assert g2.table_dict() == g.table_dict()
    g.close(); g2.close(); o.close()


def test_full_table_drops_updates_and_never_hangs():
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand
    w = inputs.scaled(inputs.WORKLOADS["cfg5"], V=2000)
    ctx, ids, probs = inputs.pregrow_records(w, 2, 3000)
    parent = inputs.topology(w.N, w.D, w.kb)
    g = Stand(1, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, 64, parent, max_probe=4)
    g.ngram_update_bulk(torch.from_numpy(ctx), torch.from_numpy(ids), torch.from_numpy(probs))
    st = g.stats()
    assert st["drops"] > 0 and st["inserts"] <= 64
    assert len(g.table_dict()) == st["inserts"]
    g.close()


# ------------------------------------------------- steps in flight, failure path
@pytest.mark.parametrize("shape", ["cfg1", "B4", "B20"])
def test_back_to_back_steps_equal_synchronised_steps(shape):
    """200 stand_step calls queued with nothing between them and no host synchronisation, against the same
    steps run one at a time.  Small grids leave most of the GPU free, so a kernel of the next step that started
    before the previous step's state was complete would read stale trees, candidate lists or tails here."""
    torch = _torch()
    from paper_2506_04708_b200.binding import Stand
    base = inputs.WORKLOADS["cfg1"]
    w = {"cfg1": inputs.scaled(base, steps=200), "B4": inputs.scaled(base, B=4, V=4096, steps=200),
         "B20": inputs.scaled(base, B=20, V=4096, steps=200)}[shape]
    parent = inputs.topology(w.N, w.D, w.kb)
    depth = inputs.node_depths(parent)
    streams = inputs.token_streams(w, 7, 8 + (w.steps + 2) * (w.D + 2))
    tail = torch.from_numpy(streams[:, 5:8].copy())
    lens0 = torch.full((w.B,), 8, dtype=torch.int64)
    mk = lambda: Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 7, 1 << 14, parent)
    # pass 1, one step at a time: the closed loop makes each step's logits from the lengths so far
    a = mk()
    a.reset_sequences(tail, lens0)
    gen = inputs.DeviceLogits(w, streams, depth, 7, pool=2, device=a.dev, peak_mode="p80")
    logits, want = [], []
    lens = torch.empty(w.B, dtype=torch.int64, device=a.dev)
    for s in range(w.steps):
        a.lens_device(lens)
        buf = torch.empty((w.B, w.N, w.V), dtype=torch.float32, device=a.dev)
        gen.make(buf, lens, s)
        out = a.step(buf)
        torch.cuda.synchronize()
        logits.append(buf)
        want.append([t.clone() for t in out])
    # pass 2, a fresh context: the same logits, every step writing its own result buffers, nothing else queued
    b = mk()
    b.reset_sequences(tail, lens0)
    i32 = dict(dtype=torch.int32, device=b.dev)
    got = [(torch.empty((w.B, b.D + 1), **i32), torch.empty(w.B, **i32), torch.empty((w.B, w.N), **i32)) for _ in range(w.steps)]
    torch.cuda.synchronize()
    for s in range(w.steps):
        b.step(logits[s], out=got[s])
    torch.cuda.synchronize()
    for s in range(w.steps):
        for x, y in zip(got[s], want[s]):
            assert torch.equal(x, y), s
    assert sum(int(t[1].sum()) for t in want) > 1.2 * w.B * w.steps  # drafts were accepted: the state mattered
    sa, sb = a.state_dump(), b.state_dump()
    assert all(np.array_equal(sa[k], sb[k]) for k in sa)
    assert a.table_dict() == b.table_dict()
    assert b.stats()["wait_timeouts"] == 0
    a.close(); b.close()


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_clean():
    """The streaming kernel's loader is told to give up its first wait at once (nothing has been copied yet, so
    nothing is in flight): the kernel returns, the failure is reported in-band, and the next call works."""
    from paper_2506_04708_b200 import binding
    torch = _torch()
    g = torch.Generator(device="cuda:0").manual_seed(3)
    dl = torch.randn((1501, 40000), generator=g, device="cuda:0") * 2.5  # large enough for the streaming kernel
    x = dl[:1].cpu().numpy()
    good = [t.cpu().numpy() for t in binding.row_stats(dl, 0.8, 8)]
    binding.set_wait_limit(0)
    try:
        lse, ids, vals, probs = (t.cpu().numpy() for t in binding.row_stats(dl, 0.8, 8))
    finally:
        binding.set_wait_limit(-1)
    assert np.isnan(lse).all() and (ids == -1).all() and (probs == 0).all()
    again = [t.cpu().numpy() for t in binding.row_stats(dl, 0.8, 8)]
    assert all(np.array_equal(p, q) for p, q in zip(good, again))
    olse, oids, _, oprobs, _ = so.row_stats(x[0], float(np.float32(0.8)), 8)
    assert np.array_equal(again[1][0], oids) and abs(again[0][0] - olse) < 1e-5 * max(1, abs(olse))


def test_smoke_entry():
    import __graft_entry__
    __graft_entry__.smoke()

"""Closed-loop comparison of the CUDA library with the CPU oracle on seeded synthetic workloads.

The margin rule.  The library may differ from the oracle only on a decision that the oracle logged with a margin
below MARGIN_TOL, and a difference is excused only by the logged decision that can explain it:

  * a sequence whose emitted tokens differ first at position j: an accept test or the final sample AT THE NODE
    THAT DECIDED position j (the oracle's path node j; node j - 1 when one side's walk ended there);
  * a sequence whose emitted tokens agree but whose drafted tree differs first at node v: the Gumbel selection
    at v's parent, or a table difference at one of the contexts v's parent looked up in this step, where that
    table difference is itself excused;
  * a table difference: an "other ids kept" difference at a context whose truncation was decided by less than
    the margin in this step, or any difference at a context that an excused sequence fed in this step with
    the rows of its differing path.

Everything else is a hard mismatch.  After any difference the library is reset to the oracle's state and table,
so that the two run on in step, and the event is counted.
"""
import numpy as np

from oracle import stand_oracle as so
from paper_2506_04708_b200 import inputs

MARGIN_TOL = 1e-6  # a decision may differ from the oracle's only if the oracle logged a margin below this


def value_tol(dtype):
    """Relative tolerance of probabilities and stored values: 1e-5 for fp32 inputs, 4e-3 for bf16 inputs."""
    return 1e-5 if dtype == inputs.DTYPE_F32 else 4e-3


def to_device_logits(a, device="cuda:0"):
    import torch
    t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
    t = t.to(device)
    return t.view(torch.bfloat16) if a.dtype == np.uint16 else t


def compare_tables(gpu_table, orc_table, tol, low_margin_keys=()):
    """Returns a list of differences between two {key: (count, {id: prob})} maps."""
    diffs = []
    if set(gpu_table) != set(orc_table):
        diffs.append(("keys", sorted(set(gpu_table) ^ set(orc_table))[:5]))
        return diffs
    for key, (cnt, items) in orc_table.items():
        gcnt, gitems = gpu_table[key]
        if gcnt != cnt:
            diffs.append(("count", key, gcnt, cnt))
            continue
        if set(gitems) != set(items):
            if key not in low_margin_keys:
                diffs.append(("ids", key, sorted(gitems), sorted(items)))
            continue
        for t, pv in items.items():
            if abs(gitems[t] - pv) > tol * abs(pv) + 1e-30:
                diffs.append(("prob", key, t, gitems[t], pv))
                break
    return diffs


_KEY_DTYPE = np.dtype([("a", np.int32), ("b", np.int32), ("c", np.int32), ("d", np.int32)])


def _sorted_items(ids, probs):
    """Rows of (id, prob) pairs ordered by id, unused entries (id < 0) last."""
    key = np.where(ids < 0, np.iinfo(np.int32).max, ids)
    order = np.argsort(key, axis=1, kind="stable")
    return np.take_along_axis(ids, order, 1), np.take_along_axis(probs, order, 1)


def table_differences(gpu_arrays, orc_arrays, tol):
    """Every difference between two tables given as (keys [M,4], counts, n_items, ids [M,K], probs [M,K]) arrays:
    {context tuple: kind}, kind in "missing_gpu", "missing_oracle", "count", "ids", "prob"."""
    gk, gc, gn, gi, gp = gpu_arrays
    ok, oc, on, oi, op = orc_arrays
    gv = np.ascontiguousarray(gk, np.int32).view(_KEY_DTYPE).ravel()
    ov = np.ascontiguousarray(ok, np.int32).view(_KEY_DTYPE).ravel()
    as_key = lambda row: tuple(int(t) for t in row if t >= 0)
    out = {}
    _, ig, io = np.intersect1d(gv, ov, assume_unique=True, return_indices=True)
    if len(ig) != len(gv):
        for row in np.asarray(gk)[np.setdiff1d(np.arange(len(gv)), ig)]:
            out[as_key(row)] = "missing_oracle"
    if len(io) != len(ov):
        for row in np.asarray(ok)[np.setdiff1d(np.arange(len(ov)), io)]:
            out[as_key(row)] = "missing_gpu"
    if len(ig) == 0:
        return out
    keys = np.asarray(gk)[ig]
    bad_count = np.asarray(gc)[ig].astype(np.int64) != np.asarray(oc)[io].astype(np.int64)
    gids, gpr = _sorted_items(np.asarray(gi)[ig], np.asarray(gp, np.float64)[ig])
    oids, opr = _sorted_items(np.asarray(oi)[io], np.asarray(op, np.float64)[io])
    bad_ids = (gids != oids).any(axis=1) | (np.asarray(gn)[ig] != np.asarray(on)[io])
    live = oids >= 0
    bad_prob = ((np.abs(gpr - opr) > tol * np.abs(opr) + 1e-30) & live & (gids == oids)).any(axis=1)
    for i in np.nonzero(bad_count | bad_ids | bad_prob)[0]:
        out[as_key(keys[i])] = "count" if bad_count[i] else ("ids" if bad_ids[i] else "prob")
    return out


def compare_states(gs, os_, tol):
    diffs = []
    for k in ("tail", "len", "tree", "cand_n", "step"):
        if not np.array_equal(np.asarray(gs[k]), np.asarray(os_[k])):
            diffs.append(k)
    if "cand_n" not in diffs:
        B, N = os_["cand_n"].shape
        for b in range(B):
            for u in range(N):
                n = os_["cand_n"][b, u]
                g = dict(zip(gs["cand_id"][b, u, :n].tolist(), gs["cand_phi"][b, u, :n].tolist()))
                o = dict(zip(os_["cand_id"][b, u, :n].tolist(), os_["cand_phi"][b, u, :n].tolist()))
                if set(g) != set(o) or any(abs(g[t] - o[t]) > tol * abs(o[t]) for t in o):
                    diffs.append(("cand", b, u, g, o))
    return diffs


def resync_gpu_from_oracle(gpu, orc):
    keys, counts, n_items, ids, probs = orc.table_arrays()
    gpu.table_load(keys, counts, n_items, ids, probs.astype(np.float32), clear=True)
    gpu.state_load(orc.state())


def first_difference(em_g, ne_g, em_o, ne_o, tr_g, tr_o):
    """("emitted", j), ("tree", v) or None for one sequence."""
    if ne_g != ne_o or not np.array_equal(em_g, em_o):
        return "emitted", int(np.nonzero(em_g != em_o)[0][0])
    if not np.array_equal(tr_g, tr_o):
        return "tree", int(np.nonzero(tr_g != tr_o)[0][0])
    return None


def fed_contexts(old_tail, emitted, n_max):
    """The contexts a sequence feeds in one step: for every emitted position, the 1..n_max tokens before it."""
    seq = [int(t) for t in old_tail if t >= 0]
    keys = set()
    for tok in emitted:
        for n in range(1, n_max + 1):
            if len(seq) >= n:
                keys.add(tuple(seq[-n:]))
        seq.append(int(tok))
    return keys


def lookup_contexts(new_tail, tree, parent, u, n_max):
    """The contexts node u looks up when its children are drafted: the sequence followed by the path root..u."""
    chain = []
    w = u
    while w != 0:
        chain.append(int(tree[w]))
        w = int(parent[w])
    seq = [int(t) for t in new_tail if t >= 0] + chain[::-1]
    return {tuple(seq[-n:]) for n in range(1, n_max + 1) if len(seq) >= n}


class StepJudge:
    """Applies the margin rule to one step of all sequences."""

    def __init__(self, parent, n_max, tol):
        self.parent, self.n_max, self.tol = np.asarray(parent), n_max, tol

    def judge(self, gpu_out, orc_out, margin_ints, margins, path_o, old_tail, new_tail, tables):
        """gpu_out / orc_out: (emitted, n_emitted, tree) arrays; path_o: the oracle's accepted paths; old_tail /
        new_tail: the oracle's sequence tails before and after the step; tables: callable returning
        (gpu arrays, oracle arrays), called only when the tables have to be looked at.
        Returns (hard, excused, looked): lists of findings, and whether the tables were compared."""
        em_g, ne_g, tr_g = gpu_out
        em_o, ne_o, tr_o = orc_out
        low = margin_ints[margins < MARGIN_TOL]
        merge_keys = {tuple(int(t) for t in rec[4:8] if t >= 0) for rec in low[low[:, 0] == so.MARGIN_MERGE]}
        diffs = {}
        for b in range(len(ne_o)):
            d = first_difference(em_g[b], ne_g[b], em_o[b], ne_o[b], tr_g[b], tr_o[b])
            if d is not None:
                diffs[b] = d
        hard, excused = [], []
        if not diffs and not merge_keys:
            return hard, excused, False
        allowed = set()  # contexts at which the two tables may differ in any way after this step
        for b, (what, j) in sorted(diffs.items()):
            if what != "emitted":
                continue
            m = int(min(ne_g[b], ne_o[b]))
            nodes = set()
            if j < ne_o[b]:
                nodes.add(int(path_o[b, j]))
            if j >= 1 and m == j:  # one walk ended at position j - 1 with the token the other accepted there
                nodes.add(int(path_o[b, j - 1]))
            recs = low[(low[:, 1] == b) & ((low[:, 0] == so.MARGIN_ACCEPT) | (low[:, 0] == so.MARGIN_FINAL))]
            if any(int(r[2]) in nodes for r in recs):
                excused.append(("decision", b, j))
                allowed |= fed_contexts(old_tail[b], em_g[b, :ne_g[b]], self.n_max)
                allowed |= fed_contexts(old_tail[b], em_o[b, :ne_o[b]], self.n_max)
            else:
                hard.append(("emitted", b, j, em_g[b].tolist(), em_o[b].tolist()))
        tdiff = table_differences(*tables(), self.tol)
        excused_keys = set()
        for key, kind in tdiff.items():
            if key in allowed or (kind == "ids" and key in merge_keys):
                excused_keys.add(key)
            else:
                hard.append(("table", key, kind))
        if excused_keys and not any(w == "emitted" for w, _ in diffs.values()):
            excused.append(("merge", sorted(excused_keys)[:3]))
        for b, (what, v) in sorted(diffs.items()):
            if what != "tree":
                continue
            u = int(self.parent[v])
            recs = low[(low[:, 1] == b) & (low[:, 0] == so.MARGIN_GUMBEL) & (low[:, 2] == u)]
            if len(recs):
                excused.append(("gumbel", b, v))
            elif lookup_contexts(new_tail[b], tr_o[b], self.parent, u, self.n_max) & excused_keys:
                excused.append(("lookup", b, v))
            else:
                hard.append(("tree", b, v, tr_g[b].tolist(), tr_o[b].tolist()))
        return hard, excused, True


class ClosedLoop:
    """Runs the same seeded workload through both sides, step by step."""

    def __init__(self, w, seed=0, peak_mode="add8", table_slots=None, prompt=8, device="cuda:0", device_logits=False,
                 parent=None, deterministic=False, seq_base=0, tail=None, **stand_kw):
        from paper_2506_04708_b200.binding import Stand
        self.w, self.seed, self.peak_mode = w, seed, peak_mode
        self.parent = inputs.topology(w.N, w.D, w.kb) if parent is None else np.ascontiguousarray(parent, np.int32)
        self.depth = inputs.node_depths(self.parent)
        self.streams = inputs.token_streams(w, seed, prompt + (w.steps + 2) * (w.D + 2))
        slots = table_slots or w.table_slots
        self.gpu = Stand(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, seed, slots, self.parent, device=device,
                         deterministic=deterministic, seq_base=seq_base, **stand_kw)
        self.orc = so.Oracle(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, seed, self.parent,
                             deterministic=deterministic, seq_base=seq_base)
        import torch
        if tail is None:
            tail = np.full((w.B, w.order_max), -1, np.int32)
            take = min(prompt, w.order_max)
            tail[:, w.order_max - take:] = self.streams[:, prompt - take:prompt]
        self.lens = np.full(w.B, prompt, np.int64)
        self.gpu.reset_sequences(torch.from_numpy(tail), torch.from_numpy(self.lens))
        self.orc.reset_sequences(tail, self.lens)
        self.gen = None
        if device_logits:
            # full-size workloads: the logits are made on the device (as the benchmark does) and copied to the host
            # for the oracle; both sides still see the same bytes
            self.gen = inputs.DeviceLogits(w, self.streams, self.depth, seed, pool=1, device=self.gpu.dev,
                                           peak_mode=peak_mode)
            tdtype = torch.bfloat16 if w.dtype == inputs.DTYPE_BF16 else torch.float32
            self.dev_buf = torch.empty((w.B, w.N, w.V), dtype=tdtype, device=self.gpu.dev)
        self.judge = StepJudge(self.parent, w.order_max, value_tol(w.dtype))
        self.step_no = 0
        self.tolerated = 0
        self.tolerated_by = {"decision": 0, "gumbel": 0, "lookup": 0, "merge": 0}
        self.emitted_total = 0
        self.hard = []

    def step(self, logits=None):
        """One step of both sides on the workload's logits (or on `logits`, a host array for both)."""
        w = self.w
        if logits is not None:
            dl = to_device_logits(logits, self.gpu.dev)
        elif self.gen is not None:
            import torch
            dl = self.gen.make(self.dev_buf, torch.from_numpy(np.asarray(self.lens, np.int64)).to(self.gpu.dev), self.step_no)
            host = dl.cpu()
            logits = host.view(torch.int16).numpy().view(np.uint16) if w.dtype == inputs.DTYPE_BF16 else host.numpy()
        else:
            logits = inputs.logits_numpy(w, self.streams, self.lens, self.depth, self.step_no, self.seed, self.peak_mode)
            dl = to_device_logits(logits, self.gpu.dev)
        old_tail = self.orc.state()["tail"]
        gpu_out = tuple(t.cpu().numpy() for t in self.gpu.step(dl))
        orc_out = self.orc.step(logits)
        ints, margins = self.orc.take_margins()
        state = self.orc.state()
        hard, excused, looked = self.judge.judge(
            gpu_out, orc_out, ints, margins, self.orc.path(), old_tail, state["tail"],
            lambda: (self.gpu.table_dump(), self.orc.table_arrays()))
        for h in hard:
            self.hard.append((self.step_no,) + h)
        for e in excused:
            self.tolerated += 1
            self.tolerated_by[e[0]] += 1
        if hard or excused:
            resync_gpu_from_oracle(self.gpu, self.orc)
        self.lens = state["len"]
        self.emitted_total += int(orc_out[1].sum())
        self.step_no += 1
        return orc_out

    def check_state_and_table(self):
        tol = value_tol(self.w.dtype)
        d = compare_states(self.gpu.state_dump(), self.orc.state(), tol)
        d += sorted(table_differences(self.gpu.table_dump(), self.orc.table_arrays(), tol).items())
        return d

    def close(self):
        self.gpu.close()
        self.orc.close()

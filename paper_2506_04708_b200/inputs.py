"""Seeded synthetic inputs: static tree topologies, token streams, logits.

This module serves the CUDA path and the CPU oracle alike and contains none of
the method's arithmetic (no softmax, no sampling, no table logic): it only
makes the arrays that both sides are fed.  The five workloads mirror the shapes,
sizes and value distributions of the benchmark configurations: peaked-Gaussian
logit rows, token streams that mix copied spans with Zipf-distributed fresh
tokens, and static draft trees that are wide near the root with a long
single-node tail (the shape the paper's optimised tree has, Sec. 5.4).
"""
from dataclasses import dataclass, replace
import itertools
import math

import numpy as np

DTYPE_F32, DTYPE_BF16 = 0, 1


@dataclass(frozen=True)
class Workload:
    name: str
    B: int            # sequences
    N: int            # tree nodes per sequence, root included
    D: int            # maximum depth (edges)
    kb: int           # maximum children per node
    V: int            # vocabulary
    dtype: int        # DTYPE_F32 / DTYPE_BF16
    T: float          # sampling temperature
    order_max: int    # N-gram orders 1..order_max
    topk: int         # entries kept per context
    steps: int
    table_slots: int  # power of two
    sigma: float      # std of the Gaussian part of a logit row
    copy_prob: float  # share of stream segments that copy an earlier span
    span_max: int     # span lengths are uniform in [8, span_max]
    zipf_s: float
    extra_peaks: int = 0      # up to this many further planted peaks per row
    stream_kind: str = "own"  # "own" | "pool" (shared span pool) | "fork" (beams forked from roots)
    pregrow_contexts: int = 0


WORKLOADS = {
    "cfg1": Workload("cfg1", 1, 8, 4, 2, 32000, DTYPE_F32, 1.0, 3, 8, 1000, 1 << 20, 2.5, 0.5, 64, 1.1),
    "cfg2": Workload("cfg2", 1, 64, 8, 4, 151936, DTYPE_BF16, 0.6, 4, 10, 4096, 1 << 22, 2.5, 0.6, 128, 1.05),
    "cfg3": Workload("cfg3", 16, 32, 6, 4, 151936, DTYPE_BF16, 0.8, 4, 10, 8192, 1 << 22, 2.5, 0.6, 128, 1.05,
                     stream_kind="pool"),
    "cfg4": Workload("cfg4", 64, 16, 4, 3, 128256, DTYPE_F32, 1.0, 3, 8, 2048, 1 << 23, 3.0, 0.5, 64, 1.1,
                     extra_peaks=2),
    "cfg5": Workload("cfg5", 256, 24, 6, 3, 151936, DTYPE_BF16, 0.7, 4, 10, 1024, 1 << 24, 2.5, 0.6, 128, 1.05,
                     stream_kind="fork", pregrow_contexts=10_000_000),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller copy of a workload (same recipe) for parity tests."""
    return replace(w, **kw)


# ---------------------------------------------------------------------------
# Static tree topology.
# ---------------------------------------------------------------------------
def topology(N: int, D: int, kb: int) -> np.ndarray:
    """Parent array of a static draft tree with N nodes (root = node 0).

    A node is the sequence of sibling ranks on its path, each < kb, at most D
    long; its cost is sum(rank + 1).  The leftmost chain down to depth D is
    always taken; the other nodes are added by increasing (cost, depth, path)
    until N - 1 non-root nodes exist.  Nodes are numbered breadth-first
    (depth, then path), so the children of a node are consecutive and ordered by rank.
    """
    chosen = {tuple([0] * d) for d in range(1, D + 1)}
    cand = []
    for d in range(1, D + 1):
        for p in itertools.product(range(kb), repeat=d):
            cand.append((sum(o + 1 for o in p), d, p))
    cand.sort()
    for _, _, p in cand:
        if len(chosen) >= N - 1:
            break
        chosen.add(p)
    nodes = sorted(chosen, key=lambda p: (len(p), p))[: N - 1]
    index = {(): 0}
    for i, p in enumerate(nodes):
        index[p] = i + 1
    parent = np.full(len(nodes) + 1, -1, np.int32)
    for p in nodes:
        parent[index[p]] = index[p[:-1]]
    return parent


def node_depths(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), np.int32)
    for u in range(1, len(parent)):
        d[u] = d[parent[u]] + 1
    return d


# ---------------------------------------------------------------------------
# Token streams.
# ---------------------------------------------------------------------------
def _zipf_sampler(V: int, s: float):
    ranks = np.arange(1, V + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-s))
    cdf /= cdf[-1]
    # fixed affine permutation rank -> id
    a = 2654435761 % V
    while math.gcd(a, V) != 1:
        a += 1
    off = 40503 % V

    def draw(rng, n):
        r = np.searchsorted(cdf, rng.random(n), side="right").astype(np.int64)
        r = np.minimum(r, V - 1)
        return ((a * r + off) % V).astype(np.int32)

    return draw


def _one_stream(rng, length, w: Workload, draw, pool=None, prefix=None):
    out = np.empty(length + w.span_max, np.int32)
    n = 0
    if prefix is not None:
        n = min(len(prefix), length)
        out[:n] = prefix[:n]
    while n < length:
        L = int(rng.integers(8, w.span_max + 1))
        copy = rng.random() < w.copy_prob
        if copy and pool is not None:
            span = pool[int(rng.integers(0, len(pool)))]
            span = span[:L]
            L = len(span)
            out[n:n + L] = span
        elif copy and n >= 8:
            L = min(L, n)
            start = int(rng.integers(0, n - L + 1))
            out[n:n + L] = out[start:start + L]
        else:
            out[n:n + L] = draw(rng, L)
        n += L
    return out[:length]


def token_streams(w: Workload, seed: int, length: int) -> np.ndarray:
    """[B, length] int32 token streams, seeded per (seed, sequence)."""
    draw = _zipf_sampler(w.V, w.zipf_s)
    streams = np.empty((w.B, length), np.int32)
    if w.stream_kind == "pool":
        prng = np.random.default_rng([seed, 0xC0FFEE])
        pool = [draw(prng, int(prng.integers(8, w.span_max + 1))) for _ in range(4096)]
        for b in range(w.B):
            streams[b] = _one_stream(np.random.default_rng([seed, b]), length, w, draw, pool=pool)
    elif w.stream_kind == "fork":
        n_roots = min(32, w.B)
        roots = [_one_stream(np.random.default_rng([seed, 1_000_000 + r]), length, w, draw) for r in range(n_roots)]
        for b in range(w.B):
            if b < n_roots:
                streams[b] = roots[b]
            else:
                streams[b] = _one_stream(np.random.default_rng([seed, b]), length, w, draw,
                                         prefix=roots[b % n_roots][:256])
    else:
        for b in range(w.B):
            streams[b] = _one_stream(np.random.default_rng([seed, b]), length, w, draw)
    return streams


# ---------------------------------------------------------------------------
# Logits.
# ---------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def peak_indices(w: Workload, streams: np.ndarray, lens: np.ndarray, depth: np.ndarray) -> np.ndarray:
    """[B, N] index of the planted peak of every row: the stream token at the
    position the row predicts (sequence length + node depth)."""
    pos = lens.astype(np.int64)[:, None] + depth.astype(np.int64)[None, :]
    pos = np.minimum(pos, streams.shape[1] - 1)
    return np.take_along_axis(streams, pos, axis=1).astype(np.int64)


def logits_numpy(w: Workload, streams, lens, depth, step: int, seed: int, peak_mode: str = "add8") -> np.ndarray:
    """One step's logits [B, N, V] on the host: float32, or uint16 bf16 bit patterns.

    Row (b, u) = sigma * N(0,1) noise with a planted peak at the stream token of
    the predicted position.  peak_mode "add8": +8 is added to that entry (the
    contract reading).  "p80": the entry is set so that it holds 70-90% (80% on
    average, varied per row) of the row's mass before rounding; this exercises deep
    accept paths and table hits.
    """
    rng = np.random.default_rng([seed, 7_000_000 + step])
    x = rng.standard_normal((w.B, w.N, w.V), dtype=np.float32) * np.float32(w.sigma)
    idx = peak_indices(w, streams, np.asarray(lens), depth)
    bb, uu = np.meshgrid(np.arange(w.B), np.arange(w.N), indexing="ij")
    if peak_mode == "add8":
        x[bb, uu, idx] += np.float32(8.0)
    elif peak_mode == "p80":
        z = x.astype(np.float64) / w.T
        z[bb, uu, idx] = -np.inf
        m = z.max(axis=2, keepdims=True)
        lse = (m + np.log(np.exp(z - m).sum(axis=2, keepdims=True)))[:, :, 0]
        mass = 0.7 + 0.2 * (((idx * 40503 + step * 9176 + uu * 131) % 1009) / 1009.0)  # 0.7 .. 0.9 per row
        x[bb, uu, idx] = (w.T * (np.log(mass / (1.0 - mass)) + lse)).astype(np.float32)
    else:
        raise ValueError(peak_mode)
    for e in range(w.extra_peaks):
        h = (idx * 2654435761 + 97 * (e + 1) + step) % w.V
        on = ((idx + e + step) % 3) > e  # 0..extra_peaks further peaks per row
        x[bb[on], uu[on], h[on]] += np.float32(8.0)
    if w.dtype == DTYPE_BF16:
        return f32_to_bf16_bits(x)
    return x


class DeviceLogits:
    """The same recipe on the GPU with torch (plumbing: device memory and RNG only).

    A pool of noise tensors is made once; a step's logits are a pool entry with the
    peaks planted by position.  Used for the full-size workloads, where host generation
    would take minutes per step.
    """

    def __init__(self, w: Workload, streams: np.ndarray, depth: np.ndarray, seed: int, pool: int, device,
                 peak_mode: str = "add8"):
        import torch
        self.torch = torch
        self.w, self.peak_mode = w, peak_mode
        self.dev = device
        self.streams = torch.from_numpy(streams.astype(np.int64)).to(device)
        self.depth = torch.from_numpy(depth.astype(np.int64)).to(device)
        self.tdtype = torch.bfloat16 if w.dtype == DTYPE_BF16 else torch.float32
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        self.pool = []
        for _ in range(pool):
            t = torch.empty((w.B, w.N, w.V), dtype=torch.float32, device=device)
            t.normal_(0.0, w.sigma, generator=g)
            self.pool.append(t.to(self.tdtype))
            del t

    def make(self, out, lens_dev, step: int):
        """Writes step `step`'s logits into `out` ([B,N,V], device). lens_dev: int64 [B] on the device."""
        torch, w = self.torch, self.w
        out.copy_(self.pool[step % len(self.pool)])
        pos = lens_dev[:, None] + self.depth[None, :]
        pos = pos.clamp_(max=self.streams.shape[1] - 1)
        idx = torch.gather(self.streams, 1, pos)  # [B, N]
        rows = out.view(w.B * w.N, w.V)
        ar = torch.arange(w.B * w.N, device=self.dev)
        flat = idx.reshape(-1)
        if self.peak_mode == "add8":
            rows[ar, flat] = (rows[ar, flat].float() + 8.0).to(self.tdtype)
        else:
            z = rows.float() / w.T
            z[ar, flat] = float("-inf")
            lse = torch.logsumexp(z, dim=1)
            uu = ar % w.N
            mass = 0.7 + 0.2 * (((flat * 40503 + step * 9176 + uu * 131) % 1009).double() / 1009.0)
            rows[ar, flat] = (w.T * (torch.log(mass / (1.0 - mass)) + lse.double())).to(self.tdtype)
        for e in range(w.extra_peaks):
            h = (flat * 2654435761 + 97 * (e + 1) + step) % w.V
            on = ((flat + e + step) % 3) > e
            rows[ar[on], h[on]] = (rows[ar[on], h[on]].float() + 8.0).to(self.tdtype)
        return out


# ---------------------------------------------------------------------------
# Records for growing a table before a run (cfg5: ~10M contexts).
# ---------------------------------------------------------------------------
def pregrow_records(w: Workload, seed: int, n_tokens: int):
    """Synthetic compressed rows for a corpus of n_tokens stream tokens.

    Returns (ctx [M, order_max] int32 windows, -1 padded at the front; ids [M, topk]
    int32; probs [M, topk] float32).  Row i predicts corpus token i+1: id 0 is that
    token, the other ids are hashed, the probabilities are a normalised exp of
    hashed normals sorted in decreasing order.
    """
    one = replace(w, B=1, stream_kind="own")
    corpus = token_streams(one, seed + 12345, n_tokens + 1)[0].astype(np.int64)
    return records_from_corpus(w, corpus, seed)


def records_from_corpus(w: Workload, corpus: np.ndarray, seed: int):
    """The same rows for a given token sequence (len(corpus) - 1 rows): a table fed with them has "read" that text
    before, as the N-gram module of a run that has met the text in earlier trajectories has."""
    corpus = np.asarray(corpus, np.int64)
    n_tokens = len(corpus) - 1
    M = n_tokens
    ctx = np.full((M, w.order_max), -1, np.int32)
    for t in range(w.order_max):
        # window column t holds corpus[i - (order_max-1-t)]
        shift = w.order_max - 1 - t
        ctx[shift:, t] = corpus[: M - shift]
    ids = np.empty((M, w.topk), np.int64)
    ids[:, 0] = corpus[1: M + 1]
    for t in range(1, w.topk):
        ids[:, t] = (corpus[1: M + 1] * 40503 + 7919 * t + corpus[:M] * 31) % w.V
    # make the ids of a row distinct: bump duplicates deterministically
    for t in range(1, w.topk):
        for _ in range(64):
            dup = (ids[:, t:t + 1] == ids[:, :t]).any(axis=1)
            if not dup.any():
                break
            ids[dup, t] = (ids[dup, t] + 1 + t) % w.V
        assert not (ids[:, t:t + 1] == ids[:, :t]).any()
    rng = np.random.default_rng([seed, 555])
    e = np.exp(rng.standard_normal((M, w.topk)) * 1.5)
    e = -np.sort(-e, axis=1)
    probs = (e / e.sum(axis=1, keepdims=True) * 0.9).astype(np.float32)
    return ctx, ids.astype(np.int32), probs

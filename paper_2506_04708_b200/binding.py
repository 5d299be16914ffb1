"""Thin ctypes binding over the C-ABI library (include/stand.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
libstand.so.  torch is used for device memory and streams.  There is no CPU
fallback: if the library has not been built, loading raises.
"""
import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libstand.so")

STAND_MAX_TOPK, STAND_MAX_ORDER, STAND_MAX_NODES = 12, 4, 640
DTYPE_F32, DTYPE_BF16 = 0, 1

EXPORTS = [
    "stand_workspace_bytes", "stand_init", "stand_destroy", "stand_reset_sequences", "stand_verify_tree",
    "stand_ngram_update", "stand_ngram_update_bulk", "stand_export_records", "stand_export_records_packed",
    "stand_ngram_update_packed", "stand_skip_update", "stand_draft_tree", "stand_step", "stand_step_host",
    "stand_row_stats_scratch_bytes", "stand_row_stats", "stand_row_stats_static", "stand_get_stats",
    "stand_last_path", "stand_tree_depth", "stand_table_dump", "stand_table_load", "stand_state_dump",
    "stand_state_load", "stand_profile_row_pass", "stand_profile_stages", "stand_node_accepts", "stand_prune_tree",
    "stand_initial_tree", "stand_launch_count", "stand_set_wait_limit", "stand_strerror",
]


class StandConfig(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("N", C.c_int32), ("V", C.c_int32), ("topk", C.c_int32), ("order_max", C.c_int32),
        ("dtype", C.c_int32), ("temperature", C.c_float), ("max_probe", C.c_int32), ("seed", C.c_uint64),
        ("table_slots", C.c_uint64), ("parent", C.c_void_p), ("deterministic", C.c_int32),
        ("host_staging", C.c_int32), ("seq_base", C.c_int32), ("reserved", C.c_int32),
    ]


class StandStats(C.Structure):
    _fields_ = [
        ("steps", C.c_uint64), ("emitted_tokens", C.c_uint64), ("records", C.c_uint64), ("inserts", C.c_uint64),
        ("drops", C.c_uint64), ("bad_tokens", C.c_uint64), ("lookups", C.c_uint64),
        ("lookup_hits", C.c_uint64 * STAND_MAX_ORDER), ("max_probe_seen", C.c_uint64), ("wait_timeouts", C.c_uint64),
    ]


class StandError(RuntimeError):
    pass


_lib = None


def lib():
    """Loads libstand.so (built by paper_2506_04708_b200/build.py); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise StandError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_04708_b200.build` "
                         "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, u64, u32, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_uint32, C.c_float
    L.stand_workspace_bytes.restype = C.c_size_t
    L.stand_workspace_bytes.argtypes = [C.POINTER(StandConfig)]
    L.stand_init.argtypes = [C.POINTER(StandConfig), vp, C.c_size_t, C.POINTER(vp)]
    L.stand_destroy.argtypes = [vp]
    L.stand_reset_sequences.argtypes = [vp, vp, vp, vp]
    L.stand_verify_tree.argtypes = [vp, vp, vp, vp, vp]
    L.stand_ngram_update.argtypes = [vp, vp]
    L.stand_ngram_update_bulk.argtypes = [vp, vp, vp, vp, i64, vp]
    L.stand_export_records.argtypes = [vp, vp, vp, vp, vp]
    L.stand_export_records.restype = C.c_int
    L.stand_export_records_packed.argtypes = [vp, vp, vp]
    L.stand_export_records_packed.restype = C.c_int
    L.stand_ngram_update_packed.argtypes = [vp, vp, i64, vp]
    L.stand_ngram_update_packed.restype = C.c_int
    L.stand_skip_update.argtypes = [vp]
    L.stand_skip_update.restype = C.c_int
    L.stand_draft_tree.argtypes = [vp, vp, vp]
    L.stand_step.argtypes = [vp, vp, vp, vp, vp, vp]
    L.stand_step_host.argtypes = [vp, vp, vp, vp, vp, vp]
    L.stand_row_stats_scratch_bytes.restype = C.c_size_t
    L.stand_row_stats_scratch_bytes.argtypes = [i64, i32, i32, i32]
    L.stand_row_stats.argtypes = [vp, i64, i32, i32, f32, i32, vp, C.c_size_t, vp, vp, vp, vp, vp]
    L.stand_row_stats_static.argtypes = [vp, i64, i32, i32, f32, i32, vp, vp, vp, vp, vp]
    L.stand_row_stats_static.restype = C.c_int
    L.stand_get_stats.argtypes = [vp, C.POINTER(StandStats)]
    L.stand_last_path.argtypes = [vp, vp, vp, vp, vp]
    L.stand_tree_depth.argtypes = [vp]
    L.stand_tree_depth.restype = i32
    L.stand_table_dump.argtypes = [vp, vp, vp, vp, vp, vp, u64, vp, vp]
    L.stand_table_load.argtypes = [vp, vp, vp, vp, vp, vp, u64, i32, vp]
    L.stand_state_dump.argtypes = [vp, vp, vp, vp, vp, vp, vp, C.POINTER(u32), vp]
    L.stand_state_load.argtypes = [vp, vp, vp, vp, vp, vp, vp, u32, vp]
    L.stand_profile_row_pass.argtypes = [vp, vp, vp]
    L.stand_profile_row_pass.restype = C.c_int
    L.stand_profile_stages.argtypes = [vp, C.POINTER(vp)]
    L.stand_profile_stages.restype = C.c_int
    L.stand_node_accepts.argtypes = [vp, vp, i32]
    L.stand_node_accepts.restype = C.c_int
    L.stand_prune_tree.argtypes = [vp, i32, vp, i32, vp, vp]
    L.stand_prune_tree.restype = C.c_int
    L.stand_initial_tree.argtypes = [i32, vp, vp, vp, i32, C.POINTER(i32)]
    L.stand_initial_tree.restype = C.c_int
    L.stand_launch_count.argtypes = [vp]
    L.stand_launch_count.restype = u64
    L.stand_set_wait_limit.argtypes = [i64]
    L.stand_set_wait_limit.restype = C.c_int
    L.stand_strerror.argtypes = [C.c_int]
    L.stand_strerror.restype = C.c_char_p
    for name in ["stand_init", "stand_destroy", "stand_reset_sequences", "stand_verify_tree", "stand_ngram_update",
                 "stand_ngram_update_bulk", "stand_draft_tree", "stand_step", "stand_step_host", "stand_row_stats",
                 "stand_get_stats", "stand_last_path", "stand_table_dump", "stand_table_load", "stand_state_dump",
                 "stand_state_load"]:
        getattr(L, name).restype = C.c_int
    _lib = L
    return L


def _check(rc, what):
    if rc != 0:
        raise StandError(f"{what}: {lib().stand_strerror(rc).decode()} ({rc})")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_config(B, N, V, topk, order_max, dtype, temperature, seed, table_slots, parent, max_probe=0,
                host_staging=False, deterministic=False, seq_base=0):
    par = np.ascontiguousarray(parent, np.int32)
    cfg = StandConfig(B, N, V, topk, order_max, dtype, float(temperature), max_probe, seed, table_slots,
                      par.ctypes.data, int(bool(deterministic)), int(bool(host_staging)), int(seq_base), 0)
    cfg._keepalive = par
    return cfg


def workspace_bytes(cfg):
    return lib().stand_workspace_bytes(C.byref(cfg))


class Stand:
    """One decoder context.  Tensors are torch CUDA tensors; results are written in place."""

    def __init__(self, B, N, V, topk, order_max, dtype, temperature, seed, table_slots, parent, max_probe=0,
                 host_staging=False, device="cuda:0", deterministic=False, seq_base=0):
        import torch
        self.torch = torch
        self.dev = torch.device(device)
        self.B, self.N, self.V, self.K, self.n_max, self.dtype = B, N, V, topk, order_max, dtype
        self.cfg = make_config(B, N, V, topk, order_max, dtype, temperature, seed, table_slots, parent, max_probe,
                               host_staging, deterministic, seq_base)
        self.seq_base = seq_base
        self._bulk_keep = None
        need = workspace_bytes(self.cfg)
        if need == 0:
            raise StandError("invalid configuration")
        with torch.cuda.device(self.dev):
            self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=self.dev)
            base = self.workspace.data_ptr()
            self._ws_off = (-base) % 256
            h = C.c_void_p()
            _check(lib().stand_init(C.byref(self.cfg), C.c_void_p(base + self._ws_off), need, C.byref(h)), "stand_init")
        self.h = h
        self.D = lib().stand_tree_depth(self.h)
        i32 = dict(dtype=torch.int32, device=self.dev)
        self.emitted = torch.full((B, self.D + 1), -1, **i32)
        self.n_emitted = torch.zeros(B, **i32)
        self.tree = torch.full((B, N), -1, **i32)

    def close(self):
        if getattr(self, "h", None):
            lib().stand_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    # ---- the hot path ------------------------------------------------------------
    def reset_sequences(self, tail, length, stream=None):
        t = tail.to(device=self.dev, dtype=self.torch.int32).contiguous()
        l = length.to(device=self.dev, dtype=self.torch.int64).contiguous()
        assert t.numel() == self.B * self.n_max and l.numel() == self.B
        _check(lib().stand_reset_sequences(self.h, _ptr(t), _ptr(l), _stream(stream)), "stand_reset_sequences")
        self.torch.cuda.current_stream().synchronize() if stream is None else stream.synchronize()

    def _logits_ok(self, logits):
        t = self.torch
        want = t.bfloat16 if self.dtype == DTYPE_BF16 else t.float32
        assert logits.is_cuda and logits.dtype == want and logits.is_contiguous()
        assert logits.numel() == self.B * self.N * self.V

    def verify_tree(self, logits, stream=None):
        self._logits_ok(logits)
        _check(lib().stand_verify_tree(self.h, _ptr(logits), _ptr(self.emitted), _ptr(self.n_emitted), _stream(stream)),
               "stand_verify_tree")
        return self.emitted, self.n_emitted

    def ngram_update(self, stream=None):
        _check(lib().stand_ngram_update(self.h, _stream(stream)), "stand_ngram_update")

    def ngram_update_bulk(self, ctx, ids, probs, stream=None, sync=True):
        """Rows [M, order_max] / [M, topk] / [M, topk].  sync=False returns without waiting for the kernels
        and keeps the three tensors alive until the next bulk update."""
        t = self.torch
        ctx = ctx.to(device=self.dev, dtype=t.int32).contiguous()
        ids = ids.to(device=self.dev, dtype=t.int32).contiguous()
        probs = probs.to(device=self.dev, dtype=t.float32).contiguous()
        M = ctx.numel() // self.n_max
        assert ids.numel() == M * self.K and probs.numel() == M * self.K
        _check(lib().stand_ngram_update_bulk(self.h, _ptr(ctx), _ptr(ids), _ptr(probs), M, _stream(stream)),
               "stand_ngram_update_bulk")
        if sync:
            (t.cuda.current_stream() if stream is None else stream).synchronize()  # inputs must outlive the kernels
            self._bulk_keep = None
        else:
            self._bulk_keep = (ctx, ids, probs)

    def export_records(self, stream=None):
        """The accepted rows of the last verification as bulk-update rows: (ctx [B*(D+1), order_max] int32,
        ids [B*(D+1), topk] int32, probs [B*(D+1), topk] float32), device tensors; rows past a path are blank."""
        t = self.torch
        rows = self.B * (self.D + 1)
        ctx = t.empty((rows, self.n_max), dtype=t.int32, device=self.dev)
        ids = t.empty((rows, self.K), dtype=t.int32, device=self.dev)
        probs = t.empty((rows, self.K), dtype=t.float32, device=self.dev)
        _check(lib().stand_export_records(self.h, _ptr(ctx), _ptr(ids), _ptr(probs), _stream(stream)),
               "stand_export_records")
        return ctx, ids, probs

    def export_records_packed(self, out=None, stream=None):
        """The same rows in one int32 tensor [B*(D+1), order_max + 2*topk]: context, ids, probabilities (as bits)."""
        t = self.torch
        if out is None:
            out = t.empty((self.B * (self.D + 1), self.n_max + 2 * self.K), dtype=t.int32, device=self.dev)
        _check(lib().stand_export_records_packed(self.h, _ptr(out), _stream(stream)), "stand_export_records_packed")
        return out

    def ngram_update_packed(self, rows, stream=None):
        """Applies packed rows (as export_records_packed writes them, of any number of contexts) in row order.
        Does not wait for the kernels: `rows` is kept alive until the next such call."""
        assert rows.is_cuda and rows.dtype == self.torch.int32 and rows.is_contiguous()
        assert rows.shape[-1] == self.n_max + 2 * self.K
        _check(lib().stand_ngram_update_packed(self.h, _ptr(rows), rows.numel() // rows.shape[-1], _stream(stream)),
               "stand_ngram_update_packed")
        self._bulk_keep = rows

    def skip_update(self):
        _check(lib().stand_skip_update(self.h), "stand_skip_update")

    def draft_tree(self, stream=None):
        _check(lib().stand_draft_tree(self.h, _ptr(self.tree), _stream(stream)), "stand_draft_tree")
        return self.tree

    def step(self, logits, stream=None, out=None):
        """out: (emitted [B, D+1], n_emitted [B], tree [B, N]) int32 device tensors to write instead of the
        context's own result tensors."""
        self._logits_ok(logits)
        em, ne, tr = out if out is not None else (self.emitted, self.n_emitted, self.tree)
        _check(lib().stand_step(self.h, _ptr(logits), _ptr(em), _ptr(ne), _ptr(tr), _stream(stream)), "stand_step")
        return em, ne, tr

    def step_host(self, host_logits, host_emitted, host_n_emitted, host_tree, stream=None):
        """Host tensors in, host tensors out (pinned memory recommended); synchronises."""
        assert not host_logits.is_cuda and host_logits.is_contiguous()
        _check(lib().stand_step_host(self.h, _ptr(host_logits), _ptr(host_emitted), _ptr(host_n_emitted),
                                     _ptr(host_tree), _stream(stream)), "stand_step_host")

    # ---- inspection ----------------------------------------------------------------
    def stats(self):
        s = StandStats()
        _check(lib().stand_get_stats(self.h, C.byref(s)), "stand_get_stats")
        d = {k: getattr(s, k) for k, _ in StandStats._fields_ if k != "lookup_hits"}
        d["lookup_hits"] = list(s.lookup_hits)
        return d

    def last_path(self):
        t = self.torch
        W = self.D + 1
        path = t.empty((self.B, W), dtype=t.int32, device=self.dev)
        ids = t.empty((self.B, W, self.K), dtype=t.int32, device=self.dev)
        probs = t.empty((self.B, W, self.K), dtype=t.float32, device=self.dev)
        _check(lib().stand_last_path(self.h, _ptr(path), _ptr(ids), _ptr(probs), _stream(None)), "stand_last_path")
        t.cuda.current_stream().synchronize()
        return path, ids, probs

    def profile_row_pass(self, ev_before=None, ev_after=None):
        """torch.cuda.Event pair (already created, enable_timing=True) recorded around the row-pass kernel."""
        a = None if ev_before is None else C.c_void_p(ev_before.cuda_event)
        b = None if ev_after is None else C.c_void_p(ev_after.cuda_event)
        _check(lib().stand_profile_row_pass(self.h, a, b), "stand_profile_row_pass")

    def profile_stages(self, events=None):
        """Five torch.cuda.Event (already recorded once, enable_timing=True) recorded at the stage boundaries of
        every later step: before/after the row pass, after verification, after the update, after drafting."""
        if events is None:
            _check(lib().stand_profile_stages(self.h, None), "stand_profile_stages")
            return
        arr = (C.c_void_p * 5)(*[C.c_void_p(e.cuda_event) for e in events])
        _check(lib().stand_profile_stages(self.h, arr), "stand_profile_stages")

    def node_accepts(self, reset=False):
        """How often each tree node lay on the accepted path (numpy uint64 [N])."""
        out = np.zeros(self.N, np.uint64)
        _check(lib().stand_node_accepts(self.h, out.ctypes.data, int(reset)), "stand_node_accepts")
        return out

    def lens_device(self, out):
        """Copies the sequence lengths into `out` (int64 [B], device) on the current stream."""
        _check(lib().stand_state_dump(self.h, None, _ptr(out), None, None, None, None, None, _stream(None)),
               "stand_state_dump")
        return out

    def launch_count(self):
        return lib().stand_launch_count(self.h)

    def table_dump(self, cap=None):
        """(keys [M,4], counts [M], n_items [M], ids [M,K], probs [M,K]) as numpy arrays."""
        t = self.torch
        total = t.zeros(1, dtype=t.int64, device=self.dev)
        if cap is None:
            _check(lib().stand_table_dump(self.h, None, None, None, None, None, 0, _ptr(total), _stream(None)),
                   "stand_table_dump")
            cap = int(total.item())
        keys = t.empty((max(cap, 1), 4), dtype=t.int32, device=self.dev)
        counts = t.empty(max(cap, 1), dtype=t.int32, device=self.dev)
        n_items = t.empty(max(cap, 1), dtype=t.int32, device=self.dev)
        ids = t.empty((max(cap, 1), self.K), dtype=t.int32, device=self.dev)
        probs = t.empty((max(cap, 1), self.K), dtype=t.float32, device=self.dev)
        _check(lib().stand_table_dump(self.h, _ptr(keys), _ptr(counts), _ptr(n_items), _ptr(ids), _ptr(probs), cap,
                                      _ptr(total), _stream(None)), "stand_table_dump")
        M = min(int(total.item()), cap)
        return (keys[:M].cpu().numpy(), counts[:M].cpu().numpy().view(np.uint32), n_items[:M].cpu().numpy(),
                ids[:M].cpu().numpy(), probs[:M].cpu().numpy())

    def table_snapshot(self):
        """The table's contents as device tensors (keys, counts, n_items, ids, probs), for table_restore."""
        t = self.torch
        total = t.zeros(1, dtype=t.int64, device=self.dev)
        _check(lib().stand_table_dump(self.h, None, None, None, None, None, 0, _ptr(total), _stream(None)), "stand_table_dump")
        cap = max(int(total.item()), 1)
        snap = (t.empty((cap, 4), dtype=t.int32, device=self.dev), t.empty(cap, dtype=t.int32, device=self.dev),
                t.empty(cap, dtype=t.int32, device=self.dev), t.empty((cap, self.K), dtype=t.int32, device=self.dev),
                t.empty((cap, self.K), dtype=t.float32, device=self.dev))
        _check(lib().stand_table_dump(self.h, *(_ptr(x) for x in snap), cap, _ptr(total), _stream(None)), "stand_table_dump")
        t.cuda.current_stream().synchronize()
        return snap + (min(int(total.item()), cap),)

    def table_restore(self, snap):
        """Empties the table and loads a snapshot made by table_snapshot (device to device)."""
        _check(lib().stand_table_load(self.h, *(_ptr(x) for x in snap[:5]), snap[5], 1, _stream(None)), "stand_table_load")
        self.torch.cuda.current_stream().synchronize()

    def table_dict(self):
        keys, counts, n_items, ids, probs = self.table_dump()
        out = {}
        for i in range(len(keys)):
            key = tuple(int(x) for x in keys[i] if x >= 0)
            out[key] = (int(counts[i]), {int(ids[i, j]): float(probs[i, j]) for j in range(n_items[i])})
        return out

    def table_load(self, keys, counts, n_items, ids, probs, clear=True):
        t = self.torch
        M = len(keys)
        dk = t.from_numpy(np.ascontiguousarray(keys, np.int32)).to(self.dev)
        dc = t.from_numpy(np.ascontiguousarray(counts, np.uint32).view(np.int32)).to(self.dev)
        dn = t.from_numpy(np.ascontiguousarray(n_items, np.int32)).to(self.dev)
        di = t.from_numpy(np.ascontiguousarray(ids, np.int32)).to(self.dev)
        dp = t.from_numpy(np.ascontiguousarray(probs, np.float32)).to(self.dev)
        _check(lib().stand_table_load(self.h, _ptr(dk), _ptr(dc), _ptr(dn), _ptr(di), _ptr(dp), M, int(clear),
                                      _stream(None)), "stand_table_load")
        t.cuda.current_stream().synchronize()

    def state_dump(self):
        t = self.torch
        i32 = dict(dtype=t.int32, device=self.dev)
        tail = t.empty((self.B, self.n_max), **i32)
        length = t.empty(self.B, dtype=t.int64, device=self.dev)
        tree = t.empty((self.B, self.N), **i32)
        cn = t.empty((self.B, self.N), **i32)
        ci = t.empty((self.B, self.N, self.K), **i32)
        cp = t.empty((self.B, self.N, self.K), dtype=t.float32, device=self.dev)
        step = C.c_uint32()
        _check(lib().stand_state_dump(self.h, _ptr(tail), _ptr(length), _ptr(tree), _ptr(cn), _ptr(ci), _ptr(cp),
                                      C.byref(step), _stream(None)), "stand_state_dump")
        t.cuda.current_stream().synchronize()
        return dict(tail=tail.cpu().numpy(), len=length.cpu().numpy(), tree=tree.cpu().numpy(),
                    cand_n=cn.cpu().numpy(), cand_id=ci.cpu().numpy(), cand_phi=cp.cpu().numpy(), step=step.value)

    def state_load(self, st):
        t = self.torch
        f = lambda a, dt: t.from_numpy(np.ascontiguousarray(a, dt)).to(self.dev)
        tail, length, tree = f(st["tail"], np.int32), f(st["len"], np.int64), f(st["tree"], np.int32)
        cn, ci, cp = f(st["cand_n"], np.int32), f(st["cand_id"], np.int32), f(st["cand_phi"], np.float32)
        _check(lib().stand_state_load(self.h, _ptr(tail), _ptr(length), _ptr(tree), _ptr(cn), _ptr(ci), _ptr(cp),
                                      int(st["step"]), _stream(None)), "stand_state_load")
        t.cuda.current_stream().synchronize()


def row_stats(logits, temperature, topk, stream=None):
    """Context-free row pass: (lse [rows], ids [rows,k], values [rows,k], probs [rows,k]) torch tensors."""
    import torch
    assert logits.is_cuda and logits.is_contiguous() and logits.dim() == 2
    rows, V = logits.shape
    dtype = DTYPE_BF16 if logits.dtype == torch.bfloat16 else DTYPE_F32
    assert logits.dtype in (torch.bfloat16, torch.float32)
    need = lib().stand_row_stats_scratch_bytes(rows, V, dtype, topk)
    if need == 0:
        raise StandError("stand_row_stats: invalid shape")
    dev = logits.device
    scratch = torch.empty(need + 256, dtype=torch.uint8, device=dev)
    off = (-scratch.data_ptr()) % 256
    lse = torch.empty(rows, dtype=torch.float32, device=dev)
    ids = torch.empty((rows, topk), dtype=torch.int32, device=dev)
    vals = torch.empty((rows, topk), dtype=torch.float32, device=dev)
    probs = torch.empty((rows, topk), dtype=torch.float32, device=dev)
    _check(lib().stand_row_stats(_ptr(logits), rows, V, dtype, float(temperature), topk,
                                 C.c_void_p(scratch.data_ptr() + off), need, _ptr(lse), _ptr(ids), _ptr(vals),
                                 _ptr(probs), _stream(stream)), "stand_row_stats")
    (torch.cuda.current_stream() if stream is None else stream).synchronize()
    return lse, ids, vals, probs


STATIC_SCRATCH_BYTES = 8 << 20


def row_stats_static(logits, temperature, topk, out=None, stream=None):
    """stand_row_stats_static: the row pass with the library's built-in scratch buffer, for callers that
    cannot allocate device memory.  `out` = (lse, ids, values, probs) tensors the caller already owns;
    when it is None they are made here (a convenience for tests -- the C call itself allocates nothing).
    Raises StandError when the shape needs more scratch than the built-in buffer holds."""
    import torch
    assert logits.is_cuda and logits.is_contiguous() and logits.dim() == 2
    assert logits.dtype in (torch.bfloat16, torch.float32)
    rows, V = logits.shape
    dtype = DTYPE_BF16 if logits.dtype == torch.bfloat16 else DTYPE_F32
    dev = logits.device
    if out is None:
        out = (torch.empty(rows, dtype=torch.float32, device=dev),
               torch.empty((rows, topk), dtype=torch.int32, device=dev),
               torch.empty((rows, topk), dtype=torch.float32, device=dev),
               torch.empty((rows, topk), dtype=torch.float32, device=dev))
    lse, ids, vals, probs = out
    with torch.cuda.device(dev):
        _check(lib().stand_row_stats_static(_ptr(logits), rows, V, dtype, float(temperature), topk, _ptr(lse), _ptr(ids),
                                            _ptr(vals), _ptr(probs), _stream(stream)), "stand_row_stats_static")
    (torch.cuda.current_stream() if stream is None else stream).synchronize()
    return out


def set_wait_limit(polls):
    """Polls the streaming kernel's loader spends on one wait (0: give up at once; negative: the default)."""
    _check(lib().stand_set_wait_limit(int(polls)), "stand_set_wait_limit")


def initial_tree(levels=20, capacity=None):
    """App. A.1 Algorithm 1: (parent, depth, order, total_nodes); at most `capacity` nodes are returned."""
    total = C.c_int32()
    _check(lib().stand_initial_tree(levels, None, None, None, 0, C.byref(total)), "stand_initial_tree")
    n = total.value if capacity is None else min(capacity, total.value)
    parent, depth, order = (np.zeros(n, np.int32) for _ in range(3))
    _check(lib().stand_initial_tree(levels, parent.ctypes.data, depth.ctypes.data, order.ctypes.data, n, C.byref(total)),
           "stand_initial_tree")
    return parent, depth, order, total.value


def prune_tree(parent, counts, keep):
    """Keeps the `keep` most often accepted nodes: (new parent array, old index of every kept node)."""
    par = np.ascontiguousarray(parent, np.int32)
    cnt = np.ascontiguousarray(counts, np.uint64)
    out, old = np.zeros(keep, np.int32), np.zeros(keep, np.int32)
    _check(lib().stand_prune_tree(par.ctypes.data, len(par), cnt.ctypes.data, keep, out.ctypes.data, old.ctypes.data),
           "stand_prune_tree")
    return out, old

"""ctypes access to the CPU oracle (``stand_oracle.cpp``).

TEST INFRASTRUCTURE: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg only.  Nothing here touches the CUDA library.
All arithmetic lives in the C++ file; this module only marshals numpy arrays.
"""
import ctypes as C
import numpy as np

from .build_oracle import build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.so_uniform.restype = C.c_double
        _lib.so_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, C.c_int]
        _lib.so_create.restype = C.c_void_p
        _lib.so_create.argtypes = [C.c_int] * 6 + [C.c_double, C.c_uint64, C.c_void_p]
        _lib.so_table_size.restype = C.c_int64
        _lib.so_margin_count.restype = C.c_int64
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def as_raw(logits):
    """numpy view of a logits array: float32 stays, bf16 comes as uint16 bit patterns."""
    a = np.ascontiguousarray(logits)
    assert a.dtype in (np.float32, np.uint16), a.dtype
    return a, (0 if a.dtype == np.float32 else 1)


def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().so_philox(_p(c), _p(k), _p(out))
    return out


def uniform(seed, b, step, node, slot, open_interval=False):
    return lib().so_uniform(seed, b, step, node, slot, int(open_interval))


SLOT_FINAL = 0x40000000
SLOT_GUMBEL = 0x80000000


def row_stats(row, T, k, want_p=False):
    a, dt = as_raw(row)
    V = a.shape[-1]
    lse = C.c_double()
    ids = np.zeros(k, np.int32)
    vals = np.zeros(k, np.float64)
    probs = np.zeros(k, np.float64)
    p = np.zeros(V, np.float64) if want_p else None
    lib().so_row_stats(_p(a), dt, V, C.c_double(T), k, C.byref(lse), _p(ids), _p(vals), _p(probs),
                       _p(p) if want_p else None)
    return lse.value, ids, vals, probs, p


def inverse_cdf(w, U):
    w = np.ascontiguousarray(w, dtype=np.float64)
    m = C.c_double()
    lib().so_inverse_cdf.restype = C.c_int
    y = lib().so_inverse_cdf(_p(w), len(w), C.c_double(U), C.byref(m))
    return y, m.value


def verify_children(p, cand_id, cand_phi, child, u_acc, u_final):
    p = np.ascontiguousarray(p, np.float64)
    ci = np.ascontiguousarray(cand_id, np.int32)
    cp = np.ascontiguousarray(cand_phi, np.float64)
    ch = np.ascontiguousarray(child, np.int32)
    ua = np.ascontiguousarray(u_acc, np.float64)
    res = C.c_int32(-1)
    acc = lib().so_verify_children(_p(p), len(p), _p(ci), _p(cp), len(ci), _p(ch), len(ch), _p(ua),
                                   C.c_double(u_final), C.byref(res))
    return acc, res.value


def verify_children_deterministic(p, child, u_acc, u_final):
    p = np.ascontiguousarray(p, np.float64)
    ch = np.ascontiguousarray(child, np.int32)
    ua = np.ascontiguousarray(u_acc, np.float64)
    res = C.c_int32(-1)
    acc = lib().so_verify_children_deterministic(_p(p), len(p), _p(ch), len(ch), _p(ua), C.c_double(u_final),
                                                 C.byref(res))
    return acc, res.value


def most_probable(ids, phi, m):
    ids = np.ascontiguousarray(ids, np.int32)
    phi = np.ascontiguousarray(phi, np.float64)
    out = np.full(max(m, 1), -1, np.int32)
    n = lib().so_most_probable(_p(ids), _p(phi), len(ids), m, _p(out))
    return out[:n]


def gumbel_top(ids, phi, U, m):
    ids = np.ascontiguousarray(ids, np.int32)
    phi = np.ascontiguousarray(phi, np.float64)
    U = np.ascontiguousarray(U, np.float64)
    out = np.full(max(m, 1), -1, np.int32)
    n = lib().so_gumbel_top(_p(ids), _p(phi), _p(U), len(ids), m, _p(out))
    return out[:n]


MARGIN_ACCEPT, MARGIN_FINAL, MARGIN_GUMBEL, MARGIN_MERGE = 0, 1, 2, 3


class Oracle:
    def __init__(self, B, N, V, topk, order_max, dtype, temperature, seed, parent, deterministic=False, seq_base=0):
        self.B, self.N, self.V, self.K, self.n_max, self.dtype = B, N, V, topk, order_max, dtype
        self.parent = np.ascontiguousarray(parent, np.int32)
        assert len(self.parent) == N
        # the temperature is a float32 in the library's configuration: use the same value
        self.T = float(np.float32(temperature))
        self.h = C.c_void_p(lib().so_create(B, N, V, topk, order_max, dtype, C.c_double(self.T), seed,
                                            _p(self.parent)))
        self.D = lib().so_depth(self.h)
        if deterministic:
            lib().so_set_deterministic(self.h, 1)
        if seq_base:
            lib().so_set_seq_base(self.h, int(seq_base))

    def close(self):
        if self.h:
            lib().so_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def reset_sequences(self, tail, length):
        t = np.ascontiguousarray(tail, np.int32).reshape(self.B, self.n_max)
        l = np.ascontiguousarray(length, np.int64).reshape(self.B)
        lib().so_reset_sequences(self.h, _p(t), _p(l))

    def _check(self, logits):
        a, dt = as_raw(logits)
        assert dt == self.dtype and a.size == self.B * self.N * self.V
        return a

    def verify(self, logits):
        a = self._check(logits)
        em = np.full((self.B, self.D + 1), -1, np.int32)
        ne = np.zeros(self.B, np.int32)
        lib().so_verify(self.h, _p(a), _p(em), _p(ne))
        return em, ne

    def update(self):
        lib().so_update(self.h)

    def draft(self):
        tr = np.full((self.B, self.N), -1, np.int32)
        lib().so_draft(self.h, _p(tr))
        return tr

    def step(self, logits):
        a = self._check(logits)
        em = np.full((self.B, self.D + 1), -1, np.int32)
        ne = np.zeros(self.B, np.int32)
        tr = np.full((self.B, self.N), -1, np.int32)
        lib().so_step(self.h, _p(a), _p(em), _p(ne), _p(tr))
        return em, ne, tr

    def path(self):
        p = np.full((self.B, self.D + 1), -1, np.int32)
        lib().so_get_path(self.h, _p(p))
        return p

    def fresh(self):
        ids = np.full((self.B, self.D + 1, self.K), -1, np.int32)
        pr = np.zeros((self.B, self.D + 1, self.K), np.float64)
        lib().so_get_fresh(self.h, _p(ids), _p(pr))
        return ids, pr

    def update_bulk(self, ctx, ids, probs):
        ctx = np.ascontiguousarray(ctx, np.int32).reshape(-1, self.n_max)
        ids = np.ascontiguousarray(ids, np.int32).reshape(-1, self.K)
        probs = np.ascontiguousarray(probs, np.float32).reshape(-1, self.K)
        assert len(ctx) == len(ids) == len(probs)
        lib().so_update_bulk(self.h, _p(ctx), _p(ids), _p(probs), C.c_int64(len(ctx)))

    def table_size(self):
        return lib().so_table_size(self.h)

    def table(self):
        """dict: key tuple (order_n tokens) -> (count, {id: prob})."""
        M = self.table_size()
        keys = np.zeros((M, 4), np.int32)
        counts = np.zeros(M, np.uint32)
        n_items = np.zeros(M, np.int32)
        ids = np.zeros((M, self.K), np.int32)
        probs = np.zeros((M, self.K), np.float64)
        lib().so_table_dump(self.h, _p(keys), _p(counts), _p(n_items), _p(ids), _p(probs))
        out = {}
        for i in range(M):
            key = tuple(int(t) for t in keys[i] if t >= 0)
            out[key] = (int(counts[i]), {int(ids[i, t]): float(probs[i, t]) for t in range(n_items[i])})
        return out

    def table_arrays(self):
        M = self.table_size()
        keys = np.zeros((M, 4), np.int32)
        counts = np.zeros(M, np.uint32)
        n_items = np.zeros(M, np.int32)
        ids = np.zeros((M, self.K), np.int32)
        probs = np.zeros((M, self.K), np.float64)
        lib().so_table_dump(self.h, _p(keys), _p(counts), _p(n_items), _p(ids), _p(probs))
        return keys, counts, n_items, ids, probs

    def table_get(self, key):
        k = np.ascontiguousarray(key, np.int32)
        cnt = C.c_uint32()
        ids = np.zeros(self.K + 1, np.int32)
        pr = np.zeros(self.K + 1, np.float64)
        n = lib().so_table_get(self.h, _p(k), len(k), C.byref(cnt), _p(ids), _p(pr))
        if n < 0:
            return None
        return cnt.value, ids[:n].copy(), pr[:n].copy()

    def state(self):
        tail = np.zeros((self.B, self.n_max), np.int32)
        length = np.zeros(self.B, np.int64)
        tree = np.zeros((self.B, self.N), np.int32)
        cn = np.zeros((self.B, self.N), np.int32)
        ci = np.zeros((self.B, self.N, self.K), np.int32)
        cp = np.zeros((self.B, self.N, self.K), np.float64)
        step = C.c_uint32()
        lib().so_get_state(self.h, _p(tail), _p(length), _p(tree), _p(cn), _p(ci), _p(cp), C.byref(step))
        return dict(tail=tail, len=length, tree=tree, cand_n=cn, cand_id=ci, cand_phi=cp, step=step.value)

    def take_margins(self):
        n = lib().so_margin_count(self.h)
        ints = np.zeros((n, 8), np.int32)
        m = np.zeros(n, np.float64)
        if n:
            lib().so_margin_take(self.h, _p(ints), _p(m))
        return ints, m

"""The C-ABI library without a GPU: it loads, exports every symbol that include/stand.h declares,
and its host-side argument checks answer without touching a device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2506_04708_b200 import binding, build as lib_build, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "stand.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stand_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 20
    raw = C.CDLL(binding.LIB_PATH)
    for name in names:
        assert hasattr(raw, name), name
    assert sorted(binding.EXPORTS) == names


def test_config_struct_matches_the_header(tmp_path):
    """The ctypes structures against the C compiler's view of include/stand.h."""
    import subprocess
    fields_c = [n for n, _ in binding.StandConfig._fields_]
    fields_s = [n for n, _ in binding.StandStats._fields_]
    prog = ['#include <stdio.h>', '#include <stddef.h>', '#include "stand.h"', 'int main(void) {',
            'printf("%zu %zu\\n", sizeof(stand_config), sizeof(stand_stats));']
    prog += [f'printf("%zu\\n", offsetof(stand_config, {n}));' for n in fields_c]
    prog += [f'printf("%zu\\n", offsetof(stand_stats, {n}));' for n in fields_s]
    prog += ['printf("%d %d %d\\n", STAND_MAX_TOPK, STAND_MAX_ORDER, STAND_MAX_NODES);', 'return 0; }']
    src = tmp_path / "layout.c"
    src.write_text("\n".join(prog))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    nums = [int(t) for t in out]
    assert nums[0] == C.sizeof(binding.StandConfig) and nums[1] == C.sizeof(binding.StandStats)
    at = 2
    for n in fields_c:
        assert getattr(binding.StandConfig, n).offset == nums[at], n
        at += 1
    for n in fields_s:
        assert getattr(binding.StandStats, n).offset == nums[at], n
        at += 1
    assert nums[at:] == [binding.STAND_MAX_TOPK, binding.STAND_MAX_ORDER, binding.STAND_MAX_NODES]


def test_workspace_bytes_and_rejections(lib):
    w = inputs.WORKLOADS["cfg1"]
    parent = inputs.topology(w.N, w.D, w.kb)
    good = binding.make_config(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, 1 << 10, parent)
    need = binding.workspace_bytes(good)
    assert need >= (1 << 10) * 128
    bigger = binding.make_config(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, 1 << 11, parent)
    assert binding.workspace_bytes(bigger) - need == (1 << 10) * 128  # one slot = 128 bytes
    staged = binding.make_config(w.B, w.N, w.V, w.topk, w.order_max, w.dtype, w.T, 0, 1 << 10, parent,
                                 host_staging=True)
    assert binding.workspace_bytes(staged) - need >= w.B * w.N * w.V * 4

    def bad(**kw):
        args = dict(B=w.B, N=w.N, V=w.V, topk=w.topk, order_max=w.order_max, dtype=w.dtype, temperature=w.T, seed=0,
                    table_slots=1 << 10, parent=parent)
        args.update(kw)
        return binding.workspace_bytes(binding.make_config(**args))

    assert bad(B=0) == 0
    assert bad(V=1) == 0
    assert bad(topk=13) == 0
    assert bad(order_max=5) == 0
    assert bad(dtype=7) == 0
    assert bad(temperature=0.0) == 0
    assert bad(table_slots=1000) == 0                      # not a power of two
    assert bad(parent=np.array([0] * w.N, np.int32)) == 0  # the root's parent must be -1
    wrong = parent.copy()
    wrong[1], wrong[2] = 2, 0
    assert bad(parent=wrong) == 0                          # a parent must come before its child
    # stand_init refuses before it touches the device
    h = C.c_void_p()
    assert lib.stand_init(C.byref(good), None, need, C.byref(h)) == -2
    assert lib.stand_init(C.byref(good), C.c_void_p(0x1000), need - 1, C.byref(h)) == -2
    assert lib.stand_init(C.byref(good), C.c_void_p(0x1001), need, C.byref(h)) == -2
    assert lib.stand_init(None, C.c_void_p(0x1000), need, C.byref(h)) == -1
    assert lib.stand_destroy(None) == -1
    assert lib.stand_step(None, None, None, None, None, None) == -1
    # sequence sharding: a negative first-sequence index, or one that overflows with B, is not a configuration
    assert bad(seq_base=-1) == 0
    assert bad(seq_base=2**31 - 1) == 0
    assert bad(seq_base=12345) == need
    assert lib.stand_export_records(None, None, None, None, None) == -1
    assert lib.stand_skip_update(None) == -1
    assert lib.stand_ngram_update_bulk(None, None, None, None, 0, None) == -1


def test_strerror_and_scratch_size(lib):
    assert lib.stand_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4):
        assert lib.stand_strerror(code) not in (b"ok", b"unknown error code")
    assert lib.stand_strerror(-99) == b"unknown error code"
    assert lib.stand_row_stats_scratch_bytes(0, 1000, 0, 8) == 0
    assert lib.stand_row_stats_scratch_bytes(4, 1000, 0, 13) == 0
    a = lib.stand_row_stats_scratch_bytes(4, 151936, 1, 10)
    b = lib.stand_row_stats_scratch_bytes(8, 151936, 1, 10)
    assert 0 < a < b
    assert lib.stand_launch_count(None) == 0 and lib.stand_tree_depth(None) == -1

"""CPU-side checks of the C boundary: the library loads, exports every symbol the header declares,
and rejects bad arguments on the host before touching a device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_03566_b200 import build as b
    b.build()
    from paper_2506_03566_b200.binding import load_library
    return load_library()


def declared_symbols():
    names = []
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            text = open(os.path.join(ROOT, "include", f)).read()
            names += re.findall(r"POSS_API\s+[\w\s\*]+?\b(poss_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2506_03566_b200.binding import EXPORTS
    names = declared_symbols()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), n
        assert n in EXPORTS, f"{n} has no Python prototype"
    assert set(EXPORTS) == set(names)


def test_host_side_argument_checks(lib):
    from paper_2506_03566_b200.binding import poss_config, poss_weights
    import poss_synth as ps
    from paper_2506_03566_b200.binding import make_config
    assert lib.poss_workspace_bytes(None) == 0
    good = make_config(ps.CONFIGS["c2"], 2048)
    assert lib.poss_workspace_bytes(C.byref(good)) > 0
    assert lib.poss_workspace_bytes(C.byref(good)) % 256 == 0
    for field, value in [("head_dim", 48), ("max_topk", 17), ("max_depth", 0), ("dtype", 7), ("hidden", 4100),
                         ("n_kv_heads", 5), ("max_total", 300)]:
        bad = make_config(ps.CONFIGS["c2"], 2048)
        setattr(bad, field, value)
        assert lib.poss_workspace_bytes(C.byref(bad)) == 0, field
    ctx = C.c_void_p()
    w = poss_weights()
    assert lib.poss_init(C.byref(ctx), C.byref(good), None, None, 0, None) == 1          # INVALID
    assert lib.poss_init(C.byref(ctx), C.byref(good), C.byref(w), None, 0, None) == 1    # NULL weights
    bad = make_config(ps.CONFIGS["c2"], 2048)
    bad.head_dim = 48
    assert lib.poss_init(C.byref(ctx), C.byref(bad), C.byref(w), None, 0, None) == 2     # SHAPE
    bad = make_config(ps.CONFIGS["c2"], 2048)
    bad.max_topk = 99
    assert lib.poss_init(C.byref(ctx), C.byref(bad), C.byref(w), None, 0, None) == 3     # CAPACITY
    assert lib.poss_destroy(None) == 1
    assert lib.poss_draft_round(None, None, 0, None, None, 1, 1, 1, 1, None, None, None, None, None, None, None) == 1
    assert lib.poss_launch_count(None) == 0


def test_workspace_grows_with_the_model(lib):
    import poss_synth as ps
    from paper_2506_03566_b200.binding import make_config
    small = lib.poss_workspace_bytes(C.byref(make_config(ps.CONFIGS["t_bf16"], 512)))
    big = lib.poss_workspace_bytes(C.byref(make_config(ps.CONFIGS["c2"], 2048)))
    assert 0 < small < big < (2 << 30)


def test_attention_key_cut_depends_on_the_key_count_alone_and_sits_at_absolute_positions(lib):
    """The tcgen05 attention cuts its keys into 128-key groups at absolute positions, two per 256-key unit, one partial
    per unit: every key count from 1 to 10240 is covered exactly once, the keys before any position fall into the
    same groups and units whatever comes after them (what makes a tree's root row equal to its single-row decode bit
    for bit), and counts past 10240 are reported as not covered."""
    k, n = C.c_int(), C.c_int()
    assert lib.poss_attention_plan(0, C.byref(k), C.byref(n)) == 1
    assert lib.poss_attention_plan(5, None, C.byref(n)) == 1
    for total in list(range(1, 2600)) + [4096, 4097, 8192, 8193, 8273, 10239, 10240]:
        assert lib.poss_attention_plan(total, C.byref(k), C.byref(n)) == 0
        assert k.value == (128 if total <= 128 else 256) and 1 <= n.value <= 40
        assert (n.value - 1) * 256 < total <= n.value * 256              # no empty unit, nothing left out
    k.value, n.value = -1, -1
    assert lib.poss_attention_plan(10241, C.byref(k), C.byref(n)) == 2    # POSS_E_SHAPE
    assert (k.value, n.value) == (-1, -1)

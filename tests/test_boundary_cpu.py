"""C-ABI boundary and host partitioner, without a GPU: the library loads, exports every symbol the
header declares, validates arguments before touching CUDA, and the partitioner covers every tile once."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2607_09207_b200 import build as pd_build
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    pd_build.build()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names.update(re.findall(r"\b(pdattn_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    L = pdattn.lib()
    syms = declared_symbols()
    assert len(syms) >= 12
    for name in syms:
        assert hasattr(L, name), name
    assert set(pdattn.EXPORTS) <= set(syms)


def test_header_and_library_from_plain_c(tmp_path):
    """The public header parses as C99 (no C++ in it), the symbols link, and the entry points that need no GPU
    behave as documented when called from C."""
    import shutil
    import subprocess
    cc = shutil.which("gcc") or shutil.which("cc")
    if cc is None:
        pytest.skip("no C compiler")
    exe = str(tmp_path / "abi_check")
    lib_dir = os.path.dirname(pd_build.LIB)
    subprocess.check_call([cc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"),
                           os.path.join(ROOT, "tests", "c", "abi_check.c"), "-o", exe, "-L", lib_dir, "-lpdattn",
                           "-Wl,-rpath," + lib_dir])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=60)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "abi_check: ok" in out.stdout


def test_status_strings():
    L = pdattn.lib()
    assert L.pdattn_status_string(0) == b"ok"
    seen = {L.pdattn_status_string(-i) for i in range(0, 9)}
    assert len(seen) == 9


def test_tuning_setters_check_their_ranges():
    L = pdattn.lib()
    for mode in (-1, 0, 1, 2):
        assert L.pdattn_set_merge_mode(mode) == pdattn.OK
    for mode in (-2, 3, 100):
        assert L.pdattn_set_merge_mode(mode) == pdattn.INVALID_ARG
    L.pdattn_set_merge_mode(-1)
    assert L.pdattn_set_dynamic_spans(-2) == pdattn.INVALID_ARG
    assert L.pdattn_set_dynamic_spans(9) == pdattn.INVALID_ARG
    assert L.pdattn_set_dynamic_spans(0) == pdattn.OK
    assert L.pdattn_set_dynamic_spans(-1) == pdattn.OK
    for mode in (-1, 0, 1):
        assert L.pdattn_set_host_zero_copy(mode) == pdattn.OK
    assert L.pdattn_set_host_zero_copy(2) == pdattn.INVALID_ARG
    assert L.pdattn_set_host_zero_copy(-1) == pdattn.OK
    for mode in (-1, 0, 1):
        assert L.pdattn_set_short_piece_path(mode) == pdattn.OK
    for mode in (-2, 2):
        assert L.pdattn_set_short_piece_path(mode) == pdattn.INVALID_ARG
    assert L.pdattn_set_short_piece_path(-1) == pdattn.OK


def test_workspace_size_and_shape_checks():
    n = pdattn.workspace_size(256, 28, 4, 128)
    assert 0 < n < 64 << 20 and n % 256 == 0
    assert pdattn.workspace_size(256, 64, 4, 128) > n          # G = 16 needs wider partial slots
    for bad, code in [((4, 28, 4, 96, 16), pdattn.UNSUPPORTED), ((4, 28, 4, 128, 8), pdattn.UNSUPPORTED), ((4, 28, 4, 128, 48), pdattn.UNSUPPORTED), ((4, 28, 4, 128, 128), pdattn.UNSUPPORTED),
                      ((4, 30, 4, 128, 16), pdattn.INVALID_ARG), ((4, 68, 4, 128, 16), pdattn.UNSUPPORTED),
                      ((-1, 28, 4, 128, 16), pdattn.INVALID_ARG)]:
        with pytest.raises(pdattn.PdattnError) as e:
            pdattn.workspace_size(*bad)
        assert e.value.status == code


def test_decode_rejects_bad_arguments_before_any_cuda_call():
    L = pdattn.lib()
    assert L.pdattn_decode_ex(None, None) == pdattn.INVALID_ARG
    a = pdattn.Args()
    a.num_seqs, a.num_q_heads, a.num_kv_heads, a.head_dim, a.block_size = 0, 4, 1, 64, 16
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.OK          # empty batch: no-op
    a.num_seqs = 2
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.INVALID_ARG  # null pointers
    for f in ("q", "k_cache", "v_cache", "out", "block_table", "context_lens"):
        setattr(a, f, 0x1000)
    a.workspace = 0x1000
    a.max_blocks_per_seq, a.num_blocks = 4, 8
    a.kv_block_stride, a.kv_head_stride, a.kv_token_stride = 1024, 1024, 64
    a.workspace_bytes = 16
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.WORKSPACE_TOO_SMALL
    a.workspace_bytes = 1 << 30
    a.q = 0x1004
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.MISALIGNED
    a.q = 0x1000
    a.kv_token_stride = 68
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.UNSUPPORTED
    a.head_dim = 80
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.UNSUPPORTED
    # a context longer than its block_table row can describe (4 pages of 16 tokens): refused from the host copy of
    # the lengths, in every entry point that takes one, before anything is launched
    a.head_dim, a.kv_token_stride = 64, 64
    lens = (ctypes.c_int32 * 2)(64, 65)
    a.context_lens_host = ctypes.cast(lens, ctypes.c_void_p).value
    assert L.pdattn_decode_ex(ctypes.byref(a), None) == pdattn.INVALID_ARG
    assert L.pdattn_decode_multi(ctypes.byref(a), 2, None) == pdattn.INVALID_ARG
    assert L.pdattn_decode_static_scratch(ctypes.byref(a), None, None) == pdattn.INVALID_ARG


def test_short_form_needs_a_binding():
    import threading
    res = []
    t = threading.Thread(target=lambda: res.append(
        pdattn.lib().pdattn_decode(None, None, None, None, None, 1, 4, 1, 64, 16, 1.0, None, None)))
    t.start()
    t.join()
    assert res == [pdattn.NOT_BOUND]


PIECE_COST = 2     # cost of starting a unit, in tiles (the partitioner's constant)


def walk_spans(lens, Hkv, n_ctas, dyn=8):
    """Re-walk the plan the way a CTA does and return the list of (unit, tile) each span covers."""
    spans, plan = pdattn.plan_host(lens, Hkv, n_ctas, dynamic_per_cta=dyn)
    nt = [(int(L) + 63) // 64 if L > 0 else 0 for L in lens]
    cover = []
    for c in range(len(spans) - 1):
        unit, tb = int(spans[c, 0]), int(spans[c, 1])
        rem = int(spans[c + 1, 2] - spans[c, 2])
        assert rem >= 0
        mine = []
        while rem > 0 and unit < len(lens) * Hkv:
            n = nt[unit // Hkv]
            if tb >= n:
                unit, tb = unit + 1, 0
                continue
            te = min(n, tb + rem)
            mine += [(unit, t) for t in range(tb, te)]
            rem -= te - tb
            unit, tb = unit + 1, 0
        assert rem == 0
        cover.append(mine)
    return cover, plan


def span_cost(mine):
    """tiles plus the start-up cost of every unit the span touches"""
    return len(mine) + PIECE_COST * len({u for u, _ in mine})


@pytest.mark.parametrize("case", ["cfg1", "cfg2", "cfg5", "zeros", "short", "one"])
@pytest.mark.parametrize("n_ctas", [1, 7, 148])
@pytest.mark.parametrize("dyn", [0, 8])
def test_partitioner_covers_every_tile_exactly_once(case, n_ctas, dyn):
    lens, Hkv = {
        "cfg1": (W.config_lengths(1), 1), "cfg2": (W.config_lengths(2), 4), "cfg5": (W.config_lengths(5), 4),
        "zeros": (np.array([0, 5, 0, 0, 300, 0]), 2), "short": (np.arange(1, 40), 3), "one": (np.array([1]), 8),
    }[case]
    cover, plan = walk_spans(lens, Hkv, n_ctas, dyn)
    want = [(s * Hkv + g, t) for s, L in enumerate(lens) for g in range(Hkv) for t in range((int(L) + 63) // 64)]
    flat = [x for mine in cover for x in mine]
    assert plan.total_tiles == len(want)
    assert flat == want                      # contiguous, ordered, nothing twice, nothing missing
    assert plan.n_static == n_ctas and len(cover) == plan.n_static + plan.n_dynamic
    assert dyn > 0 or plan.n_dynamic == 0
    assert plan.n_dynamic <= 8 * n_ctas


@pytest.mark.parametrize("case", ["cfg1", "cfg2", "cfg5", "zeros", "short", "one", "long"])
@pytest.mark.parametrize("n_ctas", [7, 148])
@pytest.mark.parametrize("dyn", [0, 8])
def test_merge_words_describe_every_cut_unit(case, n_ctas, dyn):
    """The fourth word of a span says how the units that span boundaries cut are put together again.  Rebuilt here
    from the coverage alone: for a unit that starts in span c and has tiles in later spans, word c holds the number
    of spans up to the last one that begins inside the unit and one bit per such span that holds tiles; every span
    that begins inside a unit says how far back the unit's first span lies.  Chains longer than 15 spans say so."""
    lens, Hkv = {
        "cfg1": (W.config_lengths(1), 1), "cfg2": (W.config_lengths(2), 4), "cfg5": (W.config_lengths(5), 4),
        "zeros": (np.array([0, 5, 0, 0, 300, 0]), 2), "short": (np.arange(1, 40), 3), "one": (np.array([1]), 8),
        "long": (np.array([40000, 3, 70000]), 1),
    }[case]
    spans, plan = pdattn.plan_host(lens, Hkv, n_ctas, dynamic_per_cta=dyn)
    cover, _ = walk_spans(lens, Hkv, n_ctas, dyn)
    n = len(cover)
    word = [int(spans[k, 3]) for k in range(n)]
    first_span, holders = {}, {}
    for k, mine in enumerate(cover):
        for u in sorted({u for u, _ in mine}):
            first_span.setdefault(u, k)
            holders.setdefault(u, []).append(k)
    seen_owner = set()
    for u, ks in holders.items():
        if len(ks) == 1:
            continue                                         # not cut
        c = first_span[u]
        seen_owner.add(c)
        inside = [k for k in range(c + 1, n) if int(spans[k, 0]) == u and int(spans[k, 1]) > 0]
        assert inside and inside == list(range(c + 1, c + 1 + len(inside)))       # a run right behind span c
        assert set(ks[1:]) <= set(inside)
        run = (word[c] >> 16) & 31
        if len(inside) > 15:
            assert run == 31
        else:
            assert run == len(inside)
            assert (word[c] & 0x7fff) == sum(1 << (k - c - 1) for k in ks[1:])
        for k in inside:
            back = (word[k] >> 24) & 31
            assert back == (k - c if k - c <= 15 else 31)
    for k in range(n):
        if k not in seen_owner:
            assert (word[k] >> 16) & 31 == 0                 # no unit runs past this span's end
        if int(spans[k, 1]) == 0:
            assert (word[k] >> 24) & 31 == 0                 # begins at a unit's first tile


def test_partitioner_balances_cost_not_tiles():
    """Config 2: CTAs inside long sequences get more tiles than CTAs that walk many short ones, and the
    cost (tiles + 2 per unit touched) is even to within one unit's start-up plus the cut unit."""
    lens = W.config_lengths(2)
    cover, plan = walk_spans(lens, 4, 148, dyn=0)
    costs = np.array([span_cost(m) for m in cover])
    tiles = np.array([len(m) for m in cover])
    assert costs.max() - costs.min() <= 2 * PIECE_COST + 1
    assert tiles.max() - tiles.min() > 4
    units = np.array([len({u for u, _ in m}) for m in cover])
    assert np.corrcoef(units, tiles)[0, 1] < -0.8       # more units to start -> fewer tiles


def test_runtime_spans_are_a_quarter_of_the_cost_and_shrink_along_the_stream():
    """Config 2 with up to 4 run-time spans per CTA: the static spans share 3/4 of the cost evenly, the run-time spans
    the rest, falling linearly from 1.75 to 0.25 of their mean cost (to within the cut unit's start-up); there are
    as many of them as keeps the smallest at 8 cost units (the partitioner's minimum), and none is empty."""
    lens = W.config_lengths(2)
    cover, plan = walk_spans(lens, 4, 148, dyn=4)
    assert plan.n_static == 148 and 148 < plan.n_dynamic <= 4 * 148
    costs = np.array([span_cost(m) for m in cover], dtype=np.float64)
    stat, dyn = costs[:148], costs[148:]
    assert all(len(m) > 0 for m in cover)
    assert stat.max() - stat.min() <= 2 * PIECE_COST + 1
    total = stat.sum() + dyn.sum()
    assert abs(dyn.sum() / total - 0.25) < 0.01
    mean = dyn.mean()
    n = len(dyn)
    want = mean * (1.75 - 1.5 * (np.arange(n) + 0.5) / n)
    assert np.abs(dyn - want).max() <= 2 * PIECE_COST + 2
    assert dyn[:8].mean() > 5 * dyn[-8:].mean()
    assert 8 - 1 <= 0.25 * mean <= 8 + 1                 # the smallest span's nominal cost


def test_partitioner_spreads_the_straggler_phase_over_all_sms():
    """8 sequences x 4 KV heads = 32 units must still occupy all 148 CTAs."""
    lens = W.config_lengths(5)
    cover, plan = walk_spans(lens, 4, 148)
    assert all(len(m) > 0 for m in cover[:148]) and plan.n_dynamic > 0
    splits = {}
    for c, mine in enumerate(cover):
        for u, _ in mine:
            splits.setdefault(u, set()).add(c)
    assert min(len(v) for v in splits.values()) >= 3


def test_partitioner_small_batches_use_static_spans_only():
    cover, plan = walk_spans(W.config_lengths(1), 1, 148)
    assert plan.n_dynamic == 0 and plan.total_tiles == 8
    assert sum(len(m) for m in cover) == 8 and max(len(m) for m in cover) <= 2


def test_partitioner_depends_on_lengths_only():
    lens = W.config_lengths(2, num_seqs=32)
    a = pdattn.plan_host(lens, 4, 148, 8)
    b = pdattn.plan_host(lens.copy(), 4, 148, 8)
    assert np.array_equal(a[0], b[0])
    assert [getattr(a[1], f) for f, _ in a[1]._fields_] == [getattr(b[1], f) for f, _ in b[1]._fields_]


def test_partitioner_respects_max_spans():
    lens = W.config_lengths(2)
    spans, plan = pdattn.plan_host(lens, 4, 148, 8, max_spans=200)
    assert plan.n_static == 148 and 0 < plan.n_dynamic <= 52

"""Pins of the fp64 oracle against closed forms, invariants and brute force (CPU only).

Each test would fail under a plausible mistake in the oracle: a dropped or doubled token, a
wrong page/slot/head index, a missing scale, a sign error in the exponent, a transposed operand.
"""
import math

import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import workloads as W

BF16 = torch.bfloat16


def f64(t):
    return t.to(torch.float32).to(torch.float64).numpy()


def dense_kv(w, s):
    """Independent gather of sequence s into dense [L, Hkv, d] fp64 arrays (numpy indexing)."""
    L = int(w.context_lens_host[s])
    bs = w.block_size
    k = f64(w.k_cache)
    v = f64(w.v_cache)
    bt = w.block_table.numpy()
    K = np.stack([k[bt[s, t // bs], :, t % bs, :] for t in range(L)]) if L else np.zeros((0, w.num_kv_heads, w.head_dim))
    V = np.stack([v[bt[s, t // bs], :, t % bs, :] for t in range(L)]) if L else np.zeros((0, w.num_kv_heads, w.head_dim))
    return K, V


def brute(w):
    """Textbook softmax(q K^T scale) V per head on the dense gather."""
    S, Hq, d = w.q.shape
    G = Hq // w.num_kv_heads
    q = f64(w.q)
    out = np.zeros((S, Hq, d))
    for s in range(S):
        K, V = dense_kv(w, s)
        if K.shape[0] == 0:
            continue
        for h in range(Hq):
            x = (K[:, h // G, :] @ q[s, h]) * float(np.float32(w.scale))
            p = np.exp(x - x.max())
            p /= p.sum()
            out[s, h] = p @ V[:, h // G, :]
    return out


def test_context_len_one_returns_v_exactly():
    w = W.make_custom([1, 1, 1], Hq=6, Hkv=2, d=64, seed=11)
    out = orc.decode_workload(w)
    v = f64(w.v_cache)
    bt = w.block_table.numpy()
    for s in range(3):
        for h in range(6):
            assert np.array_equal(out[s, h], v[bt[s, 0], h // 3, 0])


@pytest.mark.parametrize("how", ["equal_keys", "zero_scale", "zero_q"])
def test_uniform_weights_return_mean_of_v(how):
    w = W.make_custom([37, 64, 5], Hq=4, Hkv=2, d=64, seed=12, poison=False)
    if how == "equal_keys":
        w.k_cache[:] = w.k_cache[0, 0, 0][None, None, None, :]
    elif how == "zero_scale":
        w.scale = 0.0
    else:
        w.q.zero_()
    out = orc.decode_workload(w)
    for s in range(3):
        _, V = dense_kv(w, s)
        for h in range(4):
            np.testing.assert_allclose(out[s, h], V[:, h // 2].mean(0), rtol=1e-13, atol=1e-15)


def test_page_permutation_leaves_bits_unchanged():
    w = W.make_custom([100, 33, 256], Hq=4, Hkv=1, d=64, seed=13, num_blocks=64)
    ref = orc.decode_workload(w)
    rng = np.random.default_rng(5)
    perm = rng.permutation(64)                      # new id of old page p is perm[p]
    w2 = w.clone()
    inv = np.argsort(perm)
    w2.k_cache = w.k_cache[torch.from_numpy(inv)]
    w2.v_cache = w.v_cache[torch.from_numpy(inv)]
    bt = w.block_table.numpy().copy()
    valid = bt >= 0
    bt[valid] = perm[bt[valid]]
    w2.block_table = torch.from_numpy(bt.astype(np.int32))
    out = orc.decode_workload(w2)
    assert np.array_equal(ref, out)


def test_brute_force_dense_on_tiny_inputs():
    for seed, (Hq, Hkv, d) in enumerate([(4, 1, 64), (6, 2, 32), (7, 7, 16), (8, 2, 128)]):
        w = W.make_custom([1, 2, 15, 16, 17, 50, 0], Hq=Hq, Hkv=Hkv, d=d, seed=20 + seed, num_blocks=32)
        np.testing.assert_allclose(orc.decode_workload(w), brute(w), rtol=1e-12, atol=1e-14)


def test_tiny_config_matches_brute_force():
    w = W.make_config(1)
    np.testing.assert_allclose(orc.decode_workload(w), brute(w), rtol=1e-12, atol=1e-14)


def test_context_len_two_is_a_sigmoid_blend():
    w = W.make_custom([2], Hq=2, Hkv=1, d=32, seed=14)
    out = orc.decode_workload(w)
    K, V = dense_kv(w, 0)
    q = f64(w.q)
    for h in range(2):
        x = (K[:, 0] @ q[0, h]) * float(np.float32(w.scale))
        sg = 1.0 / (1.0 + math.exp(-(x[0] - x[1])))
        np.testing.assert_allclose(out[0, h], sg * V[0, 0] + (1 - sg) * V[1, 0], rtol=1e-13, atol=1e-15)


def test_dominant_key_selects_its_value():
    w = W.make_custom([70], Hq=1, Hkv=1, d=64, seed=15, poison=False)
    w.k_cache.zero_()
    w.q[:] = 1.0
    w.scale = 1.0
    bt = w.block_table.numpy()
    t = 37
    w.k_cache[bt[0, t // 16], 0, t % 16, :] = 1.0      # score 64, all others 0
    out = orc.decode_workload(w)
    _, V = dense_kv(w, 0)
    # the 69 other weights are e^-64 = 1.6e-28 each
    assert np.abs(out[0, 0] - V[t, 0]).max() < 1e-20


def test_score_shift_invariance():
    """Adding the same constant to every score of a head (an extra dimension with q = 1 and a
    constant key) must not change the output."""
    w = W.make_custom([45, 16], Hq=2, Hkv=1, d=32, seed=16, poison=False)
    base = orc.decode_workload(w)
    S, Hq, d = w.q.shape
    q2 = torch.zeros(S, Hq, d + 32, dtype=BF16)
    q2[..., :d] = w.q
    q2[..., d] = 1.0
    k2 = torch.zeros(w.num_blocks, 1, 16, d + 32, dtype=BF16)
    k2[..., :d] = w.k_cache
    k2[..., d] = 3.0
    v2 = torch.zeros_like(k2)
    v2[..., :d] = w.v_cache
    out = orc.decode(q2, k2, v2, w.block_table, w.context_lens, w.scale)
    np.testing.assert_allclose(out[..., :d], base, rtol=1e-12, atol=1e-14)
    assert np.all(out[..., d:] == 0)


def test_convex_hull_and_linearity_in_v():
    w = W.make_custom([90, 3], Hq=4, Hkv=2, d=64, seed=17, poison=False)
    out = orc.decode_workload(w)
    for s in range(2):
        _, V = dense_kv(w, s)
        for h in range(4):
            lo, hi = V[:, h // 2].min(0), V[:, h // 2].max(0)
            assert np.all(out[s, h] >= lo - 1e-12) and np.all(out[s, h] <= hi + 1e-12)
    w2 = w.clone()
    w2.v_cache = (w.v_cache.to(torch.float32) * 2.0).to(BF16)     # exact in bf16
    np.testing.assert_allclose(orc.decode_workload(w2), 2.0 * out, rtol=1e-14, atol=0)


def test_split_merge_identity():
    """Attention over [0,L) equals the (m, l, acc) merge of partials over [0,c) and [c,L): pins
    the combine formula independently of any GPU code."""
    w = W.make_custom([200], Hq=4, Hkv=2, d=64, seed=18)
    full = orc.decode_workload(w)
    args = (w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale)
    for h in range(4):
        for cuts in ([64], [1], [199], [64, 128], [16, 17, 150]):
            edges = [0] + cuts + [200]
            parts = [orc.partial(*args, 0, h, a, b) for a, b in zip(edges[:-1], edges[1:])]
            ms, ls, accs = zip(*parts)
            got = orc.merge(ms, ls, np.stack(accs))
            np.testing.assert_allclose(got, full[0, h], rtol=1e-12, atol=1e-15)


def test_library_softmax_matmul_on_identity_table():
    """With an identity block table the pool is a dense [L, d] array: compare with torch's fp64
    softmax and matmul."""
    L, d, Hq, Hkv = 80, 64, 4, 2
    w = W.make_custom([L], Hq=Hq, Hkv=Hkv, d=d, seed=19, num_blocks=8, poison=False)
    w.block_table = torch.arange(5, dtype=torch.int32)[None, :]
    out = orc.decode_workload(w)
    K = w.k_cache.to(torch.float64).permute(1, 0, 2, 3).reshape(Hkv, -1, d)[:, :L]
    V = w.v_cache.to(torch.float64).permute(1, 0, 2, 3).reshape(Hkv, -1, d)[:, :L]
    q = w.q.to(torch.float64)[0]
    for h in range(Hq):
        p = torch.softmax((K[h // 2] @ q[h]) * float(np.float32(w.scale)), dim=0)
        np.testing.assert_allclose(out[0, h], (p @ V[h // 2]).numpy(), rtol=1e-12, atol=1e-15)


def test_gqa_head_map_is_contiguous_groups():
    """q head h reads KV head h // G: make KV head 1 the only one that differs."""
    w = W.make_custom([20], Hq=6, Hkv=3, d=32, seed=21, poison=False)
    w.v_cache.zero_()
    w.v_cache[:, 1] = 1.0
    out = orc.decode_workload(w)
    for h in range(6):
        expect = 1.0 if h // 2 == 1 else 0.0
        np.testing.assert_allclose(out[0, h], expect, rtol=1e-14)


def test_poisoned_tail_and_unowned_pages_do_not_matter():
    w = W.make_custom([1, 17, 100], Hq=4, Hkv=1, d=64, seed=22, num_blocks=32, poison=False)
    clean = orc.decode_workload(w)
    W.poison_unused(w)
    assert torch.isnan(w.k_cache.float()).any()
    out = orc.decode_workload(w)
    assert np.array_equal(clean, out)


def test_zero_length_and_empty_batch():
    w = W.make_custom([0, 5], Hq=2, Hkv=1, d=32, seed=23)
    out = orc.decode_workload(w)
    assert np.all(out[0] == 0) and np.isfinite(out).all()
    e = W.make_custom([], Hq=2, Hkv=1, d=32, seed=23)
    assert orc.decode_workload(e).shape == (0, 2, 32)


def test_out_of_range_pages_are_skipped_and_counted():
    w = W.make_custom([48], Hq=2, Hkv=1, d=32, seed=24, num_blocks=16, poison=False)
    ref_w = w.clone()
    bt = w.block_table.clone()
    bt[0, 1] = 99                                     # tokens 16..31 unreachable
    w.block_table = bt
    out, bad = orc.decode_workload(w, return_bad=True)
    assert bad == 16 * 2
    # equals attention over tokens 0..15 and 32..47 of the intact cache
    args = (ref_w.q, ref_w.k_cache, ref_w.v_cache, ref_w.block_table, ref_w.context_lens, ref_w.scale)
    for h in range(2):
        a = orc.partial(*args, 0, h, 0, 16)
        b = orc.partial(*args, 0, h, 32, 48)
        got = orc.merge([a[0], b[0]], [a[1], b[1]], np.stack([a[2], b[2]]))
        np.testing.assert_allclose(out[0, h], got, rtol=1e-12, atol=1e-15)


def test_strided_token_major_pool_gives_same_result():
    """The same logical cache stored [page, slot, head, dim] (token-major) through strides."""
    w = W.make_custom([40, 9], Hq=4, Hkv=2, d=32, seed=25)
    ref = orc.decode_workload(w)
    k_nhd = w.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v_nhd = w.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert k_nhd.stride() != w.k_cache.stride()
    out = orc.decode(w.q, k_nhd, v_nhd, w.block_table, w.context_lens, w.scale)
    assert np.array_equal(ref, out)


def test_bf16_rounding_helper():
    xs = np.array([0.0, 1.0, 1.00390625, 1.005859375, -2.5, 3.3895313892515355e38, 1e-40, 0.1])
    got = orc.bf16_rne(xs)
    want = torch.tensor(xs, dtype=torch.float64).to(torch.float32).to(BF16).to(torch.float64).numpy()
    # 1.00390625 = 1 + 2^-8 is a tie: rounds to even (1.0); 1.005859375 = 1 + 1.5*2^-8 rounds up
    assert got[2] == 1.0 and got[3] == 1.0078125
    np.testing.assert_array_equal(got, want)


def test_append_then_attend_equals_the_longer_cache():
    """Oracle append pin: take a cache of L + 1 tokens, cut the last token out (poison its slot), append
    it back: the bits of the caches and the attention output are those of the original."""
    lens = [16, 33, 1]                               # the appended token lands at slot 0, 1 and 1 of a page
    full = W.make_custom([L + 1 for L in lens], Hq=4, Hkv=2, d=32, seed=26, num_blocks=16)
    ref_out = orc.decode_workload(full)
    cut = full.clone()
    bt = full.block_table.numpy()
    k_new = torch.zeros(3, 2, 32, dtype=BF16)
    v_new = torch.zeros(3, 2, 32, dtype=BF16)
    for s, L in enumerate(lens):
        page, slot = bt[s, L // 16], L % 16
        k_new[s] = full.k_cache[page, :, slot]
        v_new[s] = full.v_cache[page, :, slot]
        cut.k_cache[page, :, slot] = float("nan")
        cut.v_cache[page, :, slot] = float("nan")
    cut.context_lens = torch.tensor(lens, dtype=torch.int32)
    assert orc.append_kv(cut.k_cache, cut.v_cache, cut.block_table, cut.context_lens, k_new, v_new) == 0
    assert cut.context_lens.tolist() == [L + 1 for L in lens]
    assert torch.equal(cut.k_cache.view(torch.int16), full.k_cache.view(torch.int16))
    assert torch.equal(cut.v_cache.view(torch.int16), full.v_cache.view(torch.int16))
    assert np.array_equal(orc.decode_workload(cut), ref_out)


def test_multi_token_queries_match_a_dense_causal_softmax():
    """Several new tokens per sequence: textbook masked softmax on the dense gather, the mask written as a
    matrix (query token j of T sees key t iff t <= L - T + j), against the oracle's T truncated decode steps."""
    rng = np.random.default_rng(5)
    for seed, (Hq, Hkv, d, T) in enumerate([(4, 2, 32, 2), (6, 2, 64, 3), (4, 1, 128, 4), (8, 8, 16, 1)]):
        lens = [T, T + 1, 16, 17, 63, 64, 65, 130, 2]
        w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, seed=40 + seed, num_blocks=64)
        S = len(lens)
        G = Hq // Hkv
        q = W.normal_bf16(S * T * Hq * d, 900 + seed, 1).view(S, T, Hq, d)
        got = orc.decode_multi(q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale)
        qf = f64(q)
        for s in range(S):
            K, V = dense_kv(w, s)
            L = K.shape[0]
            mask = np.array([[t <= L - T + j for t in range(L)] for j in range(T)])
            for h in range(Hq):
                x = (qf[s, :, h, :] @ K[:, h // G, :].T) * float(np.float32(w.scale))      # [T, L]
                x = np.where(mask, x, -np.inf)
                for j in range(T):
                    if not mask[j].any():
                        assert not got[s, j, h].any()            # a query token that sees no key: zeros
                        continue
                    p = np.exp(x[j] - x[j].max())
                    p /= p.sum()
                    np.testing.assert_allclose(got[s, j, h], p @ V[:, h // G, :], rtol=1e-12, atol=1e-14)
        # the last query token is the plain decode step
        last = orc.decode(q[:, T - 1].contiguous(), w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale)
        assert np.array_equal(got[:, T - 1], last)


def test_e4m3_table_matches_the_library_cast():
    vals = orc.e4m3_to_double(np.arange(256))
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(vals), np.isnan(ref)) and np.isnan(vals).sum() == 2
    assert np.array_equal(vals[~np.isnan(vals)], ref[~np.isnan(ref)])
    assert vals[0x38] == 1.0 and vals[0x7E] == 448.0 and vals[0x01] == 2.0 ** -9 and vals[0xB8] == -1.0


def test_fp8_cache_oracle_against_the_bf16_oracle_on_the_same_values():
    """e4m3 values are exact in bf16: with unit scales the fp8 oracle must reproduce the bf16 oracle bit for
    bit on pools that hold the decoded values (V transposed back); scales enter as a factor on the scores
    (K) and on the output (V)."""
    lens = [1, 2, 15, 16, 17, 50, 0, 129]
    for seed, (Hq, Hkv, d, bs) in enumerate([(4, 1, 64, 16), (6, 2, 128, 16), (8, 8, 32, 32)]):
        w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=60 + seed, num_blocks=64)
        one = torch.ones(Hkv)
        k8, v8 = W.fp8_caches(w, one, one)
        kd, vd = W.fp8_dequantized(k8, v8)
        ref = orc.decode(w.q, kd, vd, w.block_table, w.context_lens, w.scale)
        got = orc.decode_fp8(w.q, k8, v8, one, one, w.block_table, w.context_lens, w.scale)
        assert np.array_equal(got, ref)
        # power-of-two scales stay exact: K scale acts like the softmax scale, V scale like a factor on the output
        got2 = orc.decode_fp8(w.q, k8, v8, 0.5 * one, 4.0 * one, w.block_table, w.context_lens, w.scale)
        ref2 = 4.0 * orc.decode(w.q, kd, vd, w.block_table, w.context_lens, float(np.float32(w.scale)) * 0.5)
        np.testing.assert_allclose(got2, ref2, rtol=1e-12, atol=1e-14)
    # per-head scales address the right KV head
    w = W.make_custom([40, 70], Hq=4, Hkv=2, d=32, seed=70, num_blocks=16)
    k8, v8 = W.fp8_caches(w, torch.ones(2), torch.ones(2))
    base = orc.decode_fp8(w.q, k8, v8, torch.ones(2), torch.ones(2), w.block_table, w.context_lens, w.scale)
    scaled = orc.decode_fp8(w.q, k8, v8, torch.ones(2), torch.tensor([1.0, 3.0]), w.block_table, w.context_lens, w.scale)
    assert np.array_equal(scaled[:, :2], base[:, :2]) and np.allclose(scaled[:, 2:], 3.0 * base[:, 2:], rtol=1e-15)


def test_e4m3_encoder_matches_the_library_cast_and_round_trips():
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.normal(size=20000) * 3, rng.uniform(-448, 448, size=20000), rng.normal(size=5000) * 1e-2,
                        orc.e4m3_to_double(np.arange(0x7f)), [0.0, -0.0, 447.9, 448.0, 464.0, 1e9, -1e9]]).astype(np.float32)
    got = orc.e4m3_encode(x)
    inr = np.abs(x) <= 448
    ref = torch.from_numpy(x[inr]).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got[inr], ref)
    assert np.all(got[~inr] & 0x7f == 0x7e)                                   # saturation to the largest finite code
    codes = np.delete(np.arange(256, dtype=np.uint8), [0x7f, 0xff])
    vals = orc.e4m3_to_double(codes).astype(np.float32)
    back = orc.e4m3_encode(vals)
    assert np.array_equal(back[codes != 0x80], codes[codes != 0x80]) and back[codes == 0x80][0] in (0x00, 0x80)
    # a tie goes to the even code: 17 lies halfway between 16 (code 0x58) and 18 (0x59)
    assert orc.e4m3_encode(np.array([17.0, 19.0], dtype=np.float32)).tolist() == [0x58, 0x5a]


def test_pair_list_equals_the_rows_of_the_full_output():
    """decode(pairs=P) must return, row by row, exactly what the full output holds at (seq, head) = P[i]: an
    off-by-one in the pair indexing, a swapped (head, seq) order, an output row written at the pair's own
    index instead of its position in the list, or a stale row for a repeated pair would all show."""
    w = W.make_custom([1, 17, 100, 0, 256, 33, 64], Hq=6, Hkv=2, d=32, seed=81, num_blocks=64)
    full = orc.decode_workload(w)
    pairs = np.array([[4, 5], [0, 0], [6, 3], [1, 2], [4, 5], [3, 1], [2, 4], [6, 0], [1, 2], [5, 5]], dtype=np.int32)
    for nt in (1, 3):
        got = orc.decode_workload(w, pairs=pairs, num_threads=nt)
        assert got.shape == (len(pairs), 32)
        for i, (s, h) in enumerate(pairs):
            assert np.array_equal(got[i], full[s, h]), (i, s, h)
    # pairs of a sequence with a bad page count their own skipped tokens only
    bt = w.block_table.clone()
    bt[2, 3] = -7                                       # tokens 48..63 of sequence 2
    w.block_table = bt
    _, bad = orc.decode_workload(w, pairs=np.array([[2, 0], [2, 5], [4, 1]]), return_bad=True)
    assert bad == 2 * 16


def test_fp8_append_then_attend_equals_the_longer_cache():
    """fp8 append pin: take an fp8 cache of L + 1 tokens, lift the last token's decoded values times the scale
    out, poison its slot in K (a row) and in the transposed V page (a column), append it back.  The code bytes
    of both pools must be those of the original: a V column written as a row, a slot/dim swap, the wrong page,
    a scale applied the wrong way round or a length not advanced would all show.  Then the skip rules."""
    lens = [16, 33, 1, 47]                            # the appended token lands at slot 0, 1, 1 and 15
    bs, Hkv, d = 16, 2, 32
    full = W.make_custom([L + 1 for L in lens], Hq=4, Hkv=Hkv, d=d, bs=bs, seed=82, num_blocks=16)
    ks, vs = torch.tensor([0.5, 2.0]), torch.tensor([4.0, 0.25])          # powers of two: value = scale * code exactly
    k8, v8 = W.fp8_caches(full, ks, vs)
    ref_out = orc.decode_fp8(full.q, k8, v8, ks, vs, full.block_table, full.context_lens, full.scale)
    k8c, v8c = k8.clone(), v8.clone()
    bt = full.block_table.numpy()
    k_new = torch.zeros(len(lens), Hkv, d, dtype=BF16)
    v_new = torch.zeros(len(lens), Hkv, d, dtype=BF16)
    kval = orc.e4m3_to_double(k8.numpy()).reshape(k8.shape)               # [page, head, slot, dim]
    vval = orc.e4m3_to_double(v8.numpy()).reshape(v8.shape)               # [page, head, dim, slot]
    for s, L in enumerate(lens):
        page, slot = int(bt[s, L // bs]), L % bs
        k_new[s] = torch.from_numpy(kval[page, :, slot, :] * ks.numpy()[:, None]).to(BF16)
        v_new[s] = torch.from_numpy(vval[page, :, :, slot] * vs.numpy()[:, None]).to(BF16)
        k8c[page, :, slot, :] = 0x7f
        v8c[page, :, :, slot] = 0x7f
    assert not torch.equal(k8c, k8) and not torch.equal(v8c, v8)
    cl = torch.tensor(lens, dtype=torch.int32)
    assert orc.append_kv_fp8(k8c, v8c, ks, vs, full.block_table, cl, k_new, v_new) == 0
    assert cl.tolist() == [L + 1 for L in lens]
    assert torch.equal(k8c, k8) and torch.equal(v8c, v8)
    assert np.array_equal(orc.decode_fp8(full.q, k8c, v8c, ks, vs, full.block_table, cl, full.scale), ref_out)
    # skip rules: a bad page id and a full table row leave pools and length untouched and are counted
    bt2 = full.block_table.clone()
    cl2 = torch.tensor([5, 5, 5, 5], dtype=torch.int32)
    bt2[1, 0] = 99
    bt2[2, 0] = -1
    before_k, before_v = k8c.clone(), v8c.clone()
    MB = bt2.shape[1]
    cl2[3] = MB * bs                                   # row full
    skipped = orc.append_kv_fp8(k8c, v8c, ks, vs, bt2, cl2, k_new, v_new)
    assert skipped == 3 and cl2.tolist() == [6, 5, 5, MB * bs]
    page0 = int(bt2[0, 0])
    changed_k = (k8c != before_k).any(dim=(1, 2, 3)).nonzero().flatten().tolist()
    changed_v = (v8c != before_v).any(dim=(1, 2, 3)).nonzero().flatten().tolist()
    assert set(changed_k) <= {page0} and set(changed_v) <= {page0}
    assert torch.equal(k8c[page0, :, 5, :], torch.from_numpy(orc.e4m3_encode(
        k_new[0].float().numpy() / ks.numpy()[:, None])))
    assert torch.equal(v8c[page0, :, :, 5], torch.from_numpy(orc.e4m3_encode(
        v_new[0].float().numpy() / vs.numpy()[:, None])))


def test_fp8_multi_token_queries_match_a_dense_causal_softmax():
    """decode_fp8_multi against a textbook masked softmax on the decoded values (scale * code), the mask written
    as a matrix: a wrong truncation per query token, a transposed V page or a scale on the wrong operand shows."""
    for seed, (Hq, Hkv, d, bs, T) in enumerate([(4, 2, 32, 16, 2), (6, 2, 64, 32, 3), (4, 1, 128, 16, 4)]):
        lens = [T, T + 1, 16, 17, 63, 64, 65, 130, 2]
        w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=90 + seed, num_blocks=64)
        S, G = len(lens), Hq // Hkv
        ks = torch.linspace(0.5, 1.5, Hkv)
        vs = torch.linspace(2.0, 0.75, Hkv)
        k8, v8 = W.fp8_caches(w, ks, vs)
        q = W.normal_bf16(S * T * Hq * d, 950 + seed, 1).view(S, T, Hq, d)
        got = orc.decode_fp8_multi(q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale)
        kval = orc.e4m3_to_double(k8.numpy()).reshape(k8.shape) * ks.double().numpy()[None, :, None, None]
        vval = orc.e4m3_to_double(v8.numpy()).reshape(v8.shape) * vs.double().numpy()[None, :, None, None]
        bt = w.block_table.numpy()
        qf = f64(q)
        for s in range(S):
            L = lens[s]
            K = np.stack([kval[bt[s, t // bs], :, t % bs, :] for t in range(L)])      # [L, Hkv, d]
            V = np.stack([vval[bt[s, t // bs], :, :, t % bs] for t in range(L)])      # [L, Hkv, d]
            mask = np.array([[t <= L - T + j for t in range(L)] for j in range(T)])
            for h in range(Hq):
                x = (qf[s, :, h, :] @ K[:, h // G, :].T) * float(np.float32(w.scale))
                x = np.where(mask, x, -np.inf)
                for j in range(T):
                    if not mask[j].any():
                        assert not got[s, j, h].any()
                        continue
                    p = np.exp(x[j] - x[j].max())
                    p /= p.sum()
                    np.testing.assert_allclose(got[s, j, h], p @ V[:, h // G, :], rtol=1e-12, atol=1e-14)


def test_a_nan_in_a_live_slot_propagates_while_a_bad_page_is_masked():
    """The bad-page rule is a mask, not a marker value: a NaN key in a slot the sequence owns must reach that KV
    head's outputs (and only those), in the bf16 path, the pair path and the fp8 path."""
    w = W.make_custom([40, 20], Hq=4, Hkv=2, d=32, seed=83, num_blocks=16, poison=False)
    bt = w.block_table.numpy()
    w.k_cache[int(bt[0, 1]), 1, 3, 5] = float("nan")            # token 19 of sequence 0, KV head 1
    out = orc.decode_workload(w)
    assert np.isnan(out[0, 2:]).all() and np.isfinite(out[0, :2]).all() and np.isfinite(out[1]).all()
    got = orc.decode_workload(w, pairs=np.array([[0, 3], [0, 0]]))
    assert np.isnan(got[0]).all() and np.isfinite(got[1]).all()
    one = torch.ones(2)
    k8, v8 = W.fp8_caches(w, one, one)
    assert k8[int(bt[0, 1]), 1, 3, 5] == 0x7f
    out8 = orc.decode_fp8(w.q, k8, v8, one, one, w.block_table, w.context_lens, w.scale)
    assert np.isnan(out8[0, 2:]).all() and np.isfinite(out8[0, :2]).all() and np.isfinite(out8[1]).all()

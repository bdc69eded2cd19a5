"""GPU parity of pdattn_decode_fp8 (e4m3 KV cache with per-head scales) against the fp64 oracle of the same
cache.  Tolerance as everywhere: |gpu - ref| <= max(2e-3, 1e-2 * |ref|), nothing NaN/Inf.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def scales(Hkv, seed):
    rng = np.random.default_rng(seed)
    ks = torch.tensor(rng.uniform(0.5, 2.0, size=Hkv), dtype=torch.float32, device=DEV)
    vs = torch.tensor(rng.uniform(0.5, 2.0, size=Hkv), dtype=torch.float32, device=DEV)
    return ks, vs


def run_fp8(w, k8, v8, ks, vs, host_lens=True, ws=None):
    if ws is None:
        ws = pdattn.alloc_workspace(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size)
    out = torch.full_like(w.q, float("nan"))
    pdattn.decode_fp8(w.q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, out, ws,
                      context_lens_host=w.context_lens_host if host_lens else None)
    return out, pdattn.check(ws)


def assert_parity(out, ref, what):
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    bad = err > np.maximum(2e-3, 1e-2 * np.abs(ref))
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; "
                           f"max abs err {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}")


def reference(w, k8, v8, ks, vs, **kw):
    return orc.decode_fp8(w.q.cpu(), k8.cpu(), v8.cpu(), ks.cpu(), vs.cpu(), w.block_table.cpu(), w.context_lens.cpu(),
                          w.scale, **kw)


@pytest.mark.parametrize("host_lens", [True, False])
@pytest.mark.parametrize("Hq,Hkv", [(28, 4), (8, 2), (64, 4), (5, 5), (12, 1)])
def test_ragged_lengths_and_head_groupings(Hq, Hkv, host_lens):
    """8- and 16-row tiles, contexts around page and tile edges, NaN codes in every unused slot."""
    lens = [1, 2, 3, 4, 5, 15, 16, 17, 31, 33, 47, 49, 63, 64, 65, 127, 129, 191, 193, 255, 257, 1000, 0, 4097, 577]
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=128, seed=400 + Hq, device=DEV)       # unused slots poisoned
    ks, vs = scales(Hkv, Hq)
    k8, v8 = W.fp8_caches(w, ks, vs)
    out, st = run_fp8(w, k8, v8, ks, vs, host_lens)
    assert st == pdattn.OK
    assert_parity(out, reference(w, k8, v8, ks, vs), f"fp8 Hq={Hq} Hkv={Hkv}")


@pytest.mark.parametrize("bs", [32, 64])
@pytest.mark.parametrize("Hq,Hkv", [(28, 4), (32, 2)])
def test_larger_pages(Hq, Hkv, bs):
    lens = [1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 127, 129, 1000, 0, 4097]
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=128, bs=bs, seed=420 + bs, device=DEV)
    ks, vs = scales(Hkv, bs)
    k8, v8 = W.fp8_caches(w, ks, vs)
    for host in (True, False):
        out, st = run_fp8(w, k8, v8, ks, vs, host)
        assert st == pdattn.OK
        assert_parity(out, reference(w, k8, v8, ks, vs), f"fp8 page size {bs} Hq={Hq} Hkv={Hkv}")


def test_scaled_rollout_config_and_run_to_run_bits():
    w = W.make_config(2, device=DEV, num_seqs=24, len_div=2)
    ks, vs = scales(4, 1)
    k8, v8 = W.fp8_caches(w, ks, vs)
    out, st = run_fp8(w, k8, v8, ks, vs)
    assert st == pdattn.OK
    assert_parity(out, reference(w, k8, v8, ks, vs), "fp8 config 2 scaled")
    again, _ = run_fp8(w, k8, v8, ks, vs)
    assert torch.equal(out, again)


def test_single_long_sequence_and_peaked_scores():
    w = W.make_custom([30000], Hq=7, Hkv=1, d=128, seed=41, device=DEV)
    ks, vs = scales(1, 2)
    k8, v8 = W.fp8_caches(w, ks, vs)
    out, st = run_fp8(w, k8, v8, ks, vs)
    assert st == pdattn.OK
    assert_parity(out, reference(w, k8, v8, ks, vs), "fp8 one long sequence")
    wp = dataclasses.replace(W.make_custom([700, 130, 64], Hq=8, Hkv=2, d=128, seed=42, device=DEV), scale=0.7)
    ks, vs = scales(2, 3)
    k8, v8 = W.fp8_caches(wp, ks, vs)
    out, st = run_fp8(wp, k8, v8, ks, vs)
    assert st == pdattn.OK
    assert_parity(out, reference(wp, k8, v8, ks, vs), "fp8 peaked softmax")


def test_context_len_one_returns_the_scaled_code_value():
    w = W.make_custom([1, 1, 1], Hq=4, Hkv=2, d=128, seed=43, device=DEV)
    ks = torch.ones(2, device=DEV)
    vs = torch.tensor([1.0, 0.25], device=DEV)                 # exact factors
    k8, v8 = W.fp8_caches(w, ks, vs)
    out, st = run_fp8(w, k8, v8, ks, vs)
    assert st == pdattn.OK
    ref = reference(w, k8, v8, ks, vs)
    assert np.array_equal(out.float().cpu().numpy().astype(np.float64), ref)        # e4m3 values are exact in bf16


def test_out_of_range_page_ids_are_masked_and_reported():
    w = W.make_custom([200, 48], Hq=8, Hkv=2, d=128, seed=44, device=DEV, num_blocks=64, poison=False)
    ks, vs = scales(2, 4)
    k8, v8 = W.fp8_caches(w, ks, vs)
    bt = w.block_table.clone()
    bt[0, 3] = 64
    bt[1, 1] = -5
    wb = dataclasses.replace(w, block_table=bt)
    out, st = run_fp8(wb, k8, v8, ks, vs)
    assert st == pdattn.BAD_PAGE_INDEX
    ref, bad = reference(wb, k8, v8, ks, vs, return_bad=True)
    assert bad == 2 * 16 * 8
    assert_parity(out, ref, "fp8 bad pages masked")


def test_rejects_what_it_cannot_do():
    assert pdattn.lib().pdattn_decode_fp8(None, None, None, None) == pdattn.INVALID_ARG
    # a grouped call over the fp8 cache scores the shared tiles with warp-level MMAs: at most 48 query rows a group
    w = W.make_custom([200] * 8, Hq=28, Hkv=4, d=128, seed=45, device=DEV)
    ks, vs = scales(4, 5)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ws = pdattn.alloc_grouped_workspace(8, 28, 4, 128)
    pt = torch.tensor([1], dtype=torch.int32, device=DEV)
    st = pdattn.decode_grouped_fp8(w.q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, torch.empty_like(w.q),
                                   ws, w.context_lens_host, 8, pt, [1], check=False)
    assert st == pdattn.UNSUPPORTED                  # 8 * 7 = 56 rows


@pytest.mark.parametrize("host_lens", [True, False])
@pytest.mark.parametrize("Hq,Hkv,bs", [(4, 1, 16), (16, 2, 16), (32, 2, 32), (12, 4, 64)])
def test_head_dim_64(Hq, Hkv, bs, host_lens):
    """K rows of 64 bytes land under the copy engine's 64-byte swizzle; 8- and 16-row tiles; every page size."""
    lens = [1, 2, 3, 15, 16, 17, 31, 33, 47, 49, 63, 64, 65, 127, 129, 191, 193, 255, 257, 1000, 0, 4097, 577]
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=64, bs=bs, seed=460 + Hq, device=DEV)
    ks, vs = scales(Hkv, Hq + 1)
    k8, v8 = W.fp8_caches(w, ks, vs)
    out, st = run_fp8(w, k8, v8, ks, vs, host_lens)
    assert st == pdattn.OK
    assert_parity(out, reference(w, k8, v8, ks, vs), f"fp8 d=64 Hq={Hq} Hkv={Hkv} bs={bs}")
    again, _ = run_fp8(w, k8, v8, ks, vs, host_lens)
    assert torch.equal(out, again)


def test_head_dim_64_append_then_decode():
    lens = [0, 1, 15, 16, 17, 63, 64, 300]
    w = W.make_custom(lens, Hq=8, Hkv=2, d=64, seed=47, device=DEV, headroom_tokens=40)
    ks, vs = scales(2, 6)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ck8, cv8 = k8.cpu().clone(), v8.cpu().clone()
    ws = pdattn.alloc_workspace(len(lens), 8, 2, 64)
    dlens, clens = w.context_lens.clone(), w.context_lens.cpu().clone()
    for step in range(20):
        k_new = W.normal_bf16(len(lens) * 2 * 64, 600 + step, 3, device=DEV).view(len(lens), 2, 64)
        v_new = W.normal_bf16(len(lens) * 2 * 64, 600 + step, 4, device=DEV).view(len(lens), 2, 64)
        pdattn.append_kv_fp8(k_new, v_new, k8, v8, ks, vs, w.block_table, dlens, ws)
        assert orc.append_kv_fp8(ck8, cv8, ks.cpu(), vs.cpu(), w.block_table.cpu(), clens, k_new.cpu(), v_new.cpu()) == 0
    assert pdattn.check(ws) == pdattn.OK
    assert torch.equal(dlens.cpu(), clens) and torch.equal(k8.cpu(), ck8) and torch.equal(v8.cpu(), cv8)
    wl = dataclasses.replace(w, context_lens=dlens, context_lens_host=clens.numpy().astype(np.int32))
    out, st = run_fp8(wl, k8, v8, ks, vs, ws=ws)
    assert st == pdattn.OK
    assert_parity(out, orc.decode_fp8(w.q.cpu(), ck8, cv8, ks.cpu(), vs.cpu(), w.block_table.cpu(), clens, w.scale),
                  "fp8 d=64 decode after appends")


@pytest.mark.parametrize("Hq,Hkv,group,d,bs", [(40, 8, 8, 128, 16), (28, 4, 4, 128, 16), (8, 2, 8, 64, 16), (16, 4, 6, 128, 32)])
def test_grouped_over_the_fp8_cache(Hq, Hkv, group, d, bs):
    """GRPO groups on an fp8 cache: groups that share 0, 1, 5 and 16 tiles; the shared tiles are read once per
    group (warp-MMA prefix kernel on the widened codes) and merged with every member's own tiles."""
    rng = np.random.default_rng(Hq * 10 + group)
    shared_tokens = [0, 70, 330, 1024]
    lens, tiles = [], []
    for stok in shared_tokens:
        tiles.append(stok // 64)
        for j in range(group):
            lens.append(stok + (1 if j == 0 else int(rng.integers(1, 700))))
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=70 + group, device=DEV, poison=False)
    bt = w.block_table.clone()
    for gi, stok in enumerate(shared_tokens):
        pages = stok // bs
        for j in range(1, group):
            bt[gi * group + j, :pages] = bt[gi * group, :pages]
    w = dataclasses.replace(w, block_table=bt)
    W.poison_unused(w)
    ks, vs = scales(Hkv, group)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ws = pdattn.alloc_grouped_workspace(w.num_seqs, Hq, Hkv, d, bs)
    pt = torch.tensor(tiles, dtype=torch.int32, device=DEV)
    out = torch.full_like(w.q, float("nan"))
    pdattn.decode_grouped_fp8(w.q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, out, ws,
                              w.context_lens_host, group, pt, tiles)
    assert pdattn.check(ws) == pdattn.OK
    assert_parity(out, reference(w, k8, v8, ks, vs), f"fp8 grouped Hq={Hq} Hkv={Hkv} group={group} d={d} bs={bs}")
    again = torch.full_like(w.q, float("nan"))
    pdattn.decode_grouped_fp8(w.q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, again, ws,
                              w.context_lens_host, group, pt, tiles)
    assert pdattn.check(ws) == pdattn.OK and torch.equal(out, again)


def test_host_buffer_form_over_the_fp8_cache():
    """pdattn_decode_host_fp8: the step's q / block_table / context_lens in pinned host memory, out read back."""
    w = W.make_config(2, device=DEV, num_seqs=12, len_div=4)
    ks, vs = scales(4, 9)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ref, st = run_fp8(w, k8, v8, ks, vs)
    assert st == pdattn.OK
    ws = pdattn.alloc_workspace(w.num_seqs, 28, 4, 128)
    qh, bth, lh = w.q.cpu().pin_memory(), w.block_table.cpu().pin_memory(), w.context_lens.cpu().pin_memory()
    oh = torch.full_like(qh, float("nan")).pin_memory()
    staging = torch.empty(pdattn.host_staging_size(w.num_seqs, 28, 128, w.max_blocks_per_seq), dtype=torch.uint8, device=DEV)
    pdattn.decode_host_fp8(qh, bth, lh, oh, k8, v8, ks, vs, w.scale, staging, ws)
    torch.cuda.synchronize()
    assert pdattn.check(ws) == pdattn.OK and torch.equal(ref.cpu(), oh)
    assert_parity(oh, reference(w, k8, v8, ks, vs), "fp8 host-buffer form")


@pytest.mark.parametrize("bs", [16, 32])
def test_append_writes_the_same_codes_as_the_oracle_and_decode_follows(bs):
    """A growing loop on the fp8 cache: quantising append (codes bit-exact against the CPU), then a decode step."""
    lens = [0, 1, 15, 16, 17, 63, 64, 300]
    steps = 35
    w = W.make_custom(lens, Hq=8, Hkv=2, d=128, bs=bs, seed=47, device=DEV, headroom_tokens=steps + 5, poison=False)
    ks, vs = scales(2, 6)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ck8, cv8 = k8.cpu().clone(), v8.cpu().clone()
    clens = w.context_lens.cpu().clone()
    dlens = w.context_lens.clone()
    ws = pdattn.alloc_workspace(len(lens), 8, 2, 128, bs)
    for step in range(steps):
        k_new = W.normal_bf16(len(lens) * 2 * 128, 500 + step, 3, device=DEV).view(len(lens), 2, 128)
        v_new = W.normal_bf16(len(lens) * 2 * 128, 500 + step, 4, device=DEV).view(len(lens), 2, 128)
        pdattn.append_kv_fp8(k_new, v_new, k8, v8, ks, vs, w.block_table, dlens, ws)
        assert orc.append_kv_fp8(ck8, cv8, ks.cpu(), vs.cpu(), w.block_table.cpu(), clens, k_new.cpu(), v_new.cpu()) == 0
    assert pdattn.check(ws) == pdattn.OK
    assert torch.equal(dlens.cpu(), clens)
    assert torch.equal(k8.cpu(), ck8) and torch.equal(v8.cpu(), cv8)
    wl = dataclasses.replace(w, context_lens=dlens, context_lens_host=clens.numpy().astype(np.int32))
    out, st = run_fp8(wl, k8, v8, ks, vs, host_lens=False, ws=ws)
    assert st == pdattn.OK
    assert_parity(out, orc.decode_fp8(w.q.cpu(), ck8, cv8, ks.cpu(), vs.cpu(), w.block_table.cpu(), clens, w.scale),
                  "fp8 decode after appends")
    # a full table row and a bad page id leave the sequence untouched and are reported
    bt = w.block_table.clone()
    bt[0, int(clens[0]) // bs] = -1
    pdattn.append_kv_fp8(k_new, v_new, k8, v8, ks, vs, bt, dlens, ws)
    assert pdattn.check(ws) == pdattn.BAD_PAGE_INDEX
    assert int(dlens[0]) == int(clens[0]) and int(dlens[1]) == int(clens[1]) + 1


def test_page_permutation_and_plan_source_leave_the_bits_unchanged():
    w = W.make_custom([100, 33, 256, 5000, 777], Hq=28, Hkv=4, d=128, seed=48, device=DEV, num_blocks=512)
    ks, vs = scales(4, 7)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ref, st = run_fp8(w, k8, v8, ks, vs)
    assert st == pdattn.OK
    perm = torch.from_numpy(np.random.default_rng(3).permutation(512)).to(DEV)
    inv = torch.argsort(perm)
    bt = w.block_table.clone().long()
    valid = bt >= 0
    bt[valid] = perm[bt[valid]]
    w2 = dataclasses.replace(w, block_table=bt.to(torch.int32))
    out, st = run_fp8(w2, k8[inv].contiguous(), v8[inv].contiguous(), ks, vs)
    assert st == pdattn.OK and torch.equal(ref, out)
    dev_plan, st = run_fp8(w, k8, v8, ks, vs, host_lens=False)          # spans computed on the device
    assert st == pdattn.OK and torch.equal(ref, dev_plan)


@pytest.mark.parametrize("Hq,Hkv,T,bs", [(28, 4, 2, 16), (8, 2, 4, 16), (8, 2, 2, 32)])
def test_several_query_tokens_over_the_fp8_cache(Hq, Hkv, T, bs):
    lens = [T, T + 1, 15, 16, 17, 63, 64, 65, 66, 67, 127, 128, 129, 130, 131, 255, 257, 1000, 0, 2, 64 * 9 + 2]
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=128, bs=bs, seed=430 + T, device=DEV)
    ks, vs = scales(Hkv, 10 + T)
    k8, v8 = W.fp8_caches(w, ks, vs)
    S = len(lens)
    q = W.normal_bf16(S * T * Hq * 128, 21, 7, device=DEV).view(S, T, Hq, 128)
    ws = pdattn.alloc_multi_workspace(S, Hq, Hkv, 128, bs, T)
    out = torch.full_like(q, float("nan"))
    pdattn.decode_fp8(q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, out, ws,
                      context_lens_host=w.context_lens_host)
    assert pdattn.check(ws) == pdattn.OK
    ref = orc.decode_fp8_multi(q.cpu(), k8.cpu(), v8.cpu(), ks.cpu(), vs.cpu(), w.block_table.cpu(),
                               w.context_lens.cpu(), w.scale)
    assert_parity(out, ref, f"fp8, T={T}, Hq={Hq} Hkv={Hkv} bs={bs}")

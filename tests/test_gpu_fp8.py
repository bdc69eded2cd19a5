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
    w = W.make_custom([100], Hq=4, Hkv=2, d=64, seed=45, device=DEV)
    ks, vs = scales(2, 5)
    k8, v8 = W.fp8_caches(w, ks, vs)
    ws = pdattn.alloc_workspace(1, 4, 2, 64)
    out = torch.empty_like(w.q)
    args = (w.block_table, w.context_lens, w.scale, out, ws)
    assert pdattn.decode_fp8(w.q, k8, v8, ks, vs, *args, check=False) == pdattn.UNSUPPORTED       # head_dim 64
    assert pdattn.lib().pdattn_decode_fp8(None, None, None, None) == pdattn.INVALID_ARG


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

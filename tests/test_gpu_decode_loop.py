"""The growing decode loop on the GPU: KV append (bit-exact byte/index work) followed by decode attention
with the device-side planner, step after step, against the oracle's append + attention; and the loop's
token count against the closed form of the paper's decode-history feature."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"
BF16 = torch.bfloat16


def new_rows(S, Hkv, d, step, seed=77):
    k = W.normal_bf16(S * Hkv * d, seed, 100 + 2 * step, DEV).view(S, Hkv, d)
    v = W.normal_bf16(S * Hkv * d, seed, 101 + 2 * step, DEV).view(S, Hkv, d)
    return k, v


@pytest.mark.parametrize("token_major", [False, True])
def test_append_is_bit_exact_over_page_boundaries(token_major):
    lens = [0, 1, 15, 16, 17, 31, 100, 255]
    w = W.make_custom(lens, Hq=8, Hkv=4, d=128, seed=41, device=DEV, headroom_tokens=40, poison=True)
    if token_major:
        w = dataclasses.replace(w, k_cache=w.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3),
                                v_cache=w.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3))
    ref = w.to("cpu")
    ref = dataclasses.replace(ref, k_cache=ref.k_cache.clone(), v_cache=ref.v_cache.clone(),
                              context_lens=ref.context_lens.clone())
    ws = pdattn.alloc_workspace(len(lens), 8, 4, 128)
    for step in range(35):                                    # crosses two page boundaries per sequence
        k_new, v_new = new_rows(len(lens), 4, 128, step)
        pdattn.append_kv(k_new, v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, workspace=ws)
        assert orc.append_kv(ref.k_cache, ref.v_cache, ref.block_table, ref.context_lens, k_new.cpu(), v_new.cpu()) == 0
    assert pdattn.check(ws) == pdattn.OK
    assert torch.equal(w.context_lens.cpu(), ref.context_lens)
    assert w.context_lens.cpu().tolist() == [L + 35 for L in lens]
    # same bits everywhere, the NaN poison of untouched slots included
    assert torch.equal(w.k_cache.cpu().view(torch.int16), ref.k_cache.view(torch.int16))
    assert torch.equal(w.v_cache.cpu().view(torch.int16), ref.v_cache.view(torch.int16))


def test_append_with_page_size_32_and_head_dim_64():
    lens = [0, 31, 32, 33, 64]
    w = W.make_custom(lens, Hq=4, Hkv=2, d=64, bs=32, seed=43, device=DEV, headroom_tokens=40)
    ref = w.to("cpu")
    ref = dataclasses.replace(ref, k_cache=ref.k_cache.clone(), v_cache=ref.v_cache.clone(),
                              context_lens=ref.context_lens.clone())
    for step in range(34):
        k_new, v_new = new_rows(len(lens), 2, 64, step)
        pdattn.append_kv(k_new, v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens)
        assert orc.append_kv(ref.k_cache, ref.v_cache, ref.block_table, ref.context_lens, k_new.cpu(), v_new.cpu()) == 0
    assert torch.equal(w.context_lens.cpu(), ref.context_lens)
    assert torch.equal(w.k_cache.cpu().view(torch.int16), ref.k_cache.view(torch.int16))
    assert torch.equal(w.v_cache.cpu().view(torch.int16), ref.v_cache.view(torch.int16))


def test_append_skips_and_reports_bad_targets():
    w = W.make_custom([16, 5, 31], Hq=4, Hkv=2, d=64, seed=42, device=DEV, num_blocks=32, headroom_tokens=20)
    bt = w.block_table.clone()
    bt[0, 1] = 32                      # sequence 0's next token would go to a page outside the pool
    w = dataclasses.replace(w, block_table=bt[:, :2].contiguous())      # and sequence 2's row is full at 32
    ref = w.to("cpu")
    ref = dataclasses.replace(ref, k_cache=ref.k_cache.clone(), v_cache=ref.v_cache.clone(),
                              context_lens=ref.context_lens.clone())
    ws = pdattn.alloc_workspace(3, 4, 2, 64)
    skipped = 0
    for step in range(3):
        k_new, v_new = new_rows(3, 2, 64, step)
        pdattn.append_kv(k_new, v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, workspace=ws)
        skipped += orc.append_kv(ref.k_cache, ref.v_cache, ref.block_table, ref.context_lens, k_new.cpu(), v_new.cpu())
    assert skipped == 3 + 2            # sequence 0 every step, sequence 2 once its row is full
    assert pdattn.check(ws) == pdattn.BAD_PAGE_INDEX
    assert w.context_lens.cpu().tolist() == ref.context_lens.tolist() == [16, 8, 32]
    assert torch.equal(w.k_cache.cpu().view(torch.int16), ref.k_cache.view(torch.int16))


def test_growing_decode_loop_matches_the_oracle_every_step():
    """append + attention with no host copy of the lengths, so the loop needs no host work that depends on them"""
    w = W.make_config(2, device=DEV, num_seqs=12, len_div=8, headroom_tokens=24)
    ref = w.to("cpu")
    ref = dataclasses.replace(ref, k_cache=ref.k_cache.clone(), v_cache=ref.v_cache.clone(),
                              context_lens=ref.context_lens.clone())
    S = w.num_seqs
    L0 = w.context_lens_host.astype(np.int64)
    ws = pdattn.alloc_workspace(S, 28, 4, 128)
    out = torch.empty_like(w.q)
    tokens = 0
    steps = 20
    for step in range(steps):
        k_new, v_new = new_rows(S, 4, 128, step)
        pdattn.append_kv(k_new, v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, workspace=ws)
        pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws,
                         context_lens_host=None)
        tokens += int(w.context_lens.sum().item())
        orc.append_kv(ref.k_cache, ref.v_cache, ref.block_table, ref.context_lens, k_new.cpu(), v_new.cpu())
        if step % 4 == 3 or step == 0:
            want = orc.decode(ref.q, ref.k_cache, ref.v_cache, ref.block_table, ref.context_lens, ref.scale)
            got = out.float().cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            assert np.all(np.abs(got - want) <= np.maximum(2e-3, 1e-2 * np.abs(want))), step
    assert pdattn.check(ws) == pdattn.OK
    # history tokens read over the loop: sum_i (r * p_i + r (r - 1) / 2) in the paper's convention (the step
    # sees p + t - 1 tokens) plus r per request in this library's (the current token is already cached)
    r = steps
    assert tokens == sum(W.h_dec(int(p), r) + r for p in L0)


def test_a_decode_step_replays_as_a_cuda_graph():
    """append + device-side plan + decode + combine captured once and replayed: no host work per step.
    (The first, uncaptured calls do the one-time set-up: function attributes, driver entry points.)"""
    w = W.make_config(2, device=DEV, num_seqs=16, len_div=4, headroom_tokens=40)
    S = w.num_seqs
    ws = pdattn.alloc_workspace(S, 28, 4, 128)
    out = torch.empty_like(w.q)
    k_new, v_new = new_rows(S, 4, 128, 0)
    lens0 = w.context_lens.clone()
    k0, v0 = w.k_cache.clone(), w.v_cache.clone()

    def step(stream=None):
        pdattn.append_kv(k_new, v_new, w.k_cache, w.v_cache, w.block_table, w.context_lens, workspace=ws,
                         stream=stream)
        pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws,
                         context_lens_host=None, stream=stream)

    for _ in range(12):
        step()
    torch.cuda.synchronize()
    eager = out.clone()

    def reset():
        w.context_lens.copy_(lens0)
        w.k_cache.copy_(k0)
        w.v_cache.copy_(v0)

    reset()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        step(stream=side)
    torch.cuda.synchronize()
    reset()
    for _ in range(12):
        graph.replay()
    torch.cuda.synchronize()
    assert pdattn.check(ws) == pdattn.OK
    assert w.context_lens.cpu().tolist() == [int(L) + 12 for L in lens0.cpu().tolist()]
    assert torch.equal(out, eager)

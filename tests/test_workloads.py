"""Input generators: determinism, config shapes, byte/token accounting (CPU only)."""
import os

import numpy as np
import torch

from paper_2607_09207_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden", "kv_accounting.txt")


def _gold(kind):
    rows = []
    for line in open(GOLD):
        parts = line.split()
        if parts and parts[0] == kind:
            rows.append([int(x) for x in parts[1:]])
    return rows


def test_per_token_kv_footprint_matches_printed_formula():
    for L, Hkv, d, b, tp, want in _gold("bkv"):
        assert 2 * L * Hkv * d * b // tp == want
        if L == 1 and tp == 1 and b == 2:
            w = W.make_custom([3], Hq=Hkv, Hkv=Hkv, d=d, num_blocks=4)
            assert w.kv_bytes_per_token() == want


def test_history_tokens_over_a_rollout_match_h_dec():
    """Summing this repo's context_len (which includes the current token) over the decode steps of
    one request gives H_dec + r: the paper counts the history before the step, p + t - 1."""
    for p, r, want in _gold("hdec"):
        assert W.h_dec(p, r) == want
        paper_convention = sum(p + t - 1 for t in range(1, r + 1))
        ours = sum(p + t for t in range(1, r + 1))
        assert paper_convention == want and ours == want + r


def test_values_are_pure_functions_of_seed_tensor_index():
    a = W.normal_bf16(5000, 7, W.T_K)
    b = W.normal_bf16(5000, 7, W.T_K, chunk=777)
    assert torch.equal(a, b)
    assert not torch.equal(a, W.normal_bf16(5000, 8, W.T_K))
    assert not torch.equal(a, W.normal_bf16(5000, 7, W.T_V))
    x = W.normal_bf16(1 << 18, 3, W.T_Q).float()
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01
    assert x.abs().max().item() < 4.5


def test_tiny_config_shape():
    w = W.make_config(1)
    assert w.q.shape == (4, 4, 64) and w.k_cache.shape == (64, 1, 16, 64)
    assert w.context_lens_host.tolist() == [1, 17, 100, 256]
    assert w.unique_pages() == 26 and w.logical_tokens() == 374
    bt = w.block_table.numpy()
    used = np.concatenate([bt[s, : -(-int(w.context_lens_host[s]) // 16)] for s in range(4)])
    assert len(set(used.tolist())) == 26 and used.min() >= 0 and used.max() < 64
    # unowned pages and tail slots are poisoned, owned slots are finite
    k = w.k_cache.float()
    assert torch.isnan(k).any()
    for s in range(4):
        L = int(w.context_lens_host[s])
        for t in range(L):
            assert torch.isfinite(k[bt[s, t // 16], 0, t % 16]).all()
    assert torch.isnan(k[bt[1, 1], 0, 1:]).all()        # L = 17: slots 1..15 of its 2nd page


def test_length_distributions_of_the_configs():
    l2 = W.config_lengths(2)
    assert l2.shape == (256,) and l2.min() >= 513 and l2.max() <= 512 + 8192
    assert 2000 < np.median(l2) < 3200
    l3 = W.config_lengths(3)
    assert l3.shape == (512,) and l3.min() >= 1025 and l3.max() <= 1024 + 16384
    l4 = W.config_lengths(4)
    assert l4.shape == (128,) and l4.min() >= 1 and l4.max() <= 32768
    l5 = W.config_lengths(5)
    assert l5.shape == (8,) and l5.min() >= 32768 and l5.max() <= 65536
    assert np.array_equal(l2, W.config_lengths(2))


def test_grpo_groups_share_prompt_pages():
    w = W.make_config(3, num_seqs=16, len_div=8, poison=False)     # prompt 128 tokens = 8 pages
    bt = w.block_table.numpy()
    for g in range(2):
        rows = bt[8 * g: 8 * g + 8]
        assert (rows[:, :8] == rows[0, :8]).all()
        priv = [set(r[8: -(-int(L) // 16)].tolist()) for r, L in zip(rows, w.context_lens_host[8 * g: 8 * g + 8])]
        allp = [p for s in priv for p in s]
        assert len(allp) == len(set(allp))                        # private pages are disjoint
    assert w.unique_kv_bytes() < w.logical_kv_bytes()
    assert bt[0, 0] != bt[8, 0]


def test_unique_bytes_count_only_occupied_slots():
    w = W.make_custom([17, 1], Hq=2, Hkv=1, d=64, num_blocks=8)
    assert w.unique_kv_bytes() == 18 * w.kv_bytes_per_token()


def test_head_scales_config4():
    w = W.make_config(4, num_seqs=4, len_div=64, poison=False)
    k = w.k_cache.float()
    stds = k.permute(1, 0, 2, 3).reshape(8, -1).std(dim=1)
    assert stds.min() > 0.45 and stds.max() < 2.1 and (stds.max() - stds.min()) > 0.2


def test_balanced_shards_cover_everything_once():
    lens = W.config_lengths(2)
    for ws in (1, 2, 3, 8):
        shards = W.balanced_shards(lens, ws)
        allidx = np.concatenate(shards)
        assert sorted(allidx.tolist()) == list(range(len(lens)))
        loads = np.array([lens[s].sum() for s in shards])
        assert loads.max() - loads.min() <= lens.max()

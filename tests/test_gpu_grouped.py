"""Shared-prefix (GRPO group) decode: the prompt tiles of a group are read once and scored against the
query rows of all its samples.  The result must be the plain definition the oracle computes."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_grouped(w, group, prefix_tiles_host):
    ws = pdattn.alloc_grouped_workspace(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim)
    pt = torch.tensor(prefix_tiles_host, dtype=torch.int32, device=DEV)
    out = torch.empty_like(w.q)
    pdattn.decode_grouped(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws,
                          w.context_lens_host, group, pt, np.asarray(prefix_tiles_host, dtype=np.int32))
    st = pdattn.check(ws)
    return out, st


def assert_parity(out, ref, what):
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), what
    err = np.abs(got - ref)
    bad = err > np.maximum(2e-3, 1e-2 * np.abs(ref))
    assert not bad.any(), f"{what}: {int(bad.sum())} bad, max err {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"


def test_scaled_grpo_config_all_outputs():
    w = W.make_config(3, device=DEV, num_seqs=32, len_div=4)          # prompt 256 tokens = 4 tiles, 4 groups of 8
    out, st = run_grouped(w, 8, [4, 4, 4, 4])
    assert st == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), "config 3 scaled, grouped")
    again, _ = run_grouped(w, 8, [4, 4, 4, 4])
    assert torch.equal(out, again)                                    # run to run
    plain = pdattn.decode_workload(w)
    assert_parity(plain, orc.decode_workload(w.to("cpu")), "config 3 scaled, plain")


@pytest.mark.parametrize("Hq,Hkv,group", [(40, 8, 8), (28, 4, 4), (8, 2, 8), (6, 6, 3), (32, 4, 6)])
def test_groups_with_uneven_prefixes_and_head_counts(Hq, Hkv, group):
    """Groups that share 0, 1, 5 and 16 tiles; members only a token longer than the prefix; prefix
    lengths that are not whole tiles in the table (only whole tiles are declared shared)."""
    rng = np.random.default_rng(Hq * 100 + group)
    shared_tokens = [0, 70, 330, 1024]                  # -> 0, 1, 5, 16 whole tiles
    lens, tiles = [], []
    for st in shared_tokens:
        tiles.append(st // 64)
        for j in range(group):
            extra = 1 if j == 0 else int(rng.integers(1, 700))
            lens.append(st + extra)
    # build with whole shared pages = floor(shared tokens / 16)
    w = None
    parts = []
    # one workload with per-group shared pages: build rows by hand
    S = len(lens)
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=128, seed=50 + group, device=DEV, poison=False)
    bt = w.block_table.clone()
    for gi, st in enumerate(shared_tokens):
        pages = st // 16
        lead = gi * group
        for j in range(1, group):
            bt[lead + j, :pages] = bt[lead, :pages]
    w = dataclasses.replace(w, block_table=bt)
    W.poison_unused(w)
    out, status = run_grouped(w, group, tiles)
    assert status == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), f"Hq={Hq} Hkv={Hkv} group={group}")


@pytest.mark.parametrize("factor", [-1.0, 0.0, -4.0])
def test_grouped_with_negative_and_zero_scale(factor):
    """A negative scale turns the row max into a min of the raw scores (the tcgen05 kernel keeps raw scores and
    moves the sign into the staged query rows); a zero scale gives uniform weights."""
    lens = [640 + 3, 640 + 200, 640 + 64, 640 + 1, 128 + 5, 128 + 77, 128 + 300, 128 + 31]
    w = W.make_custom(lens, Hq=28, Hkv=4, d=128, seed=77, device=DEV, poison=False)
    bt = w.block_table.clone()
    for lead, pages in ((0, 40), (4, 8)):
        for j in range(1, 4):
            bt[lead + j, :pages] = bt[lead, :pages]
    w = dataclasses.replace(w, block_table=bt, scale=w.scale * factor)
    W.poison_unused(w)
    out, status = run_grouped(w, 4, [10, 2])
    assert status == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), f"scale factor {factor}")


def test_a_group_of_sixteen_passed_as_smaller_groups(prefix_engine):
    """Sixteen samples of one prompt are more query rows than a unit holds (16 * 7 = 112 > 64): the caller passes
    them as groups of eight (of four for the warp-MMA kernel, which takes 48 rows) with the same number of
    shared tiles."""
    rng = np.random.default_rng(5)
    lens = [768 + int(x) for x in rng.integers(1, 500, size=32)]
    w = W.make_custom(lens, Hq=28, Hkv=4, d=128, seed=81, device=DEV, poison=False)
    bt = w.block_table.clone()
    for lead in (0, 16):
        for j in range(1, 16):
            bt[lead + j, :48] = bt[lead, :48]
    w = dataclasses.replace(w, block_table=bt)
    W.poison_unused(w)
    part = 4 if prefix_engine == "warp_mma" else 8
    out, status = run_grouped(w, part, [12] * (32 // part))
    assert status == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), "two prompts x sixteen samples")


@pytest.mark.parametrize("bs", [32, 64])
def test_grouped_with_larger_pages(bs):
    lens = [200, 70, 65, 1000, 129, 500, 66, 300]
    w = W.make_custom(lens, Hq=16, Hkv=4, d=128, bs=bs, seed=61, device=DEV, poison=False)
    bt = w.block_table.clone()
    n = 64 // bs
    for j in range(1, 4):
        bt[j, :n] = bt[0, :n]                       # group 0 shares one 64-token tile (two 32-token pages or one page)
    for j in range(5, 8):
        bt[j, :n] = bt[4, :n]
    w = dataclasses.replace(w, block_table=bt)
    W.poison_unused(w)
    out, status = run_grouped(w, 4, [1, 1])
    assert status == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), f"grouped, page size {bs}")


def test_full_size_grpo_config_every_output(full_reference):
    """Configuration 3 at full size through the grouped entry point (the 16 shared prompt tiles of each of the 64
    groups read once): every output element against the oracle, and run to run bitwise."""
    w = W.make_config(3, device=DEV)
    tiles = [16] * 64
    out, st = run_grouped(w, 8, tiles)
    assert st == pdattn.OK
    ref = full_reference(3, w)
    assert ref.shape == tuple(out.shape)
    assert_parity(out, ref, f"config 3 full, grouped, all {ref.size} outputs")
    again, _ = run_grouped(w, 8, tiles)
    assert torch.equal(out, again)
    del w
    torch.cuda.empty_cache()


@pytest.mark.parametrize("d", [128, 64])
def test_grouped_with_peaked_scores_moves_the_softmax_reference(d):
    """Score spread of about 25 in the log2 domain: the running max of a row jumps by more than 2^8 between
    tiles again and again, so the accumulator of the shared tiles is rescaled (in tensor memory for the
    tcgen05 kernel, which only follows the max when it grew by that much), and a few tokens carry the weight."""
    lens = [1024 + 1 + 37 * j for j in range(16)]
    w = W.make_custom(lens, Hq=10, Hkv=2, d=d, seed=77, device=DEV, poison=False)
    bt = w.block_table.clone()
    for j in range(16):
        bt[j, :64] = bt[j - j % 8, :64]                  # two groups of 8 share 64 pages = 16 tiles
    w = dataclasses.replace(w, block_table=bt, scale=w.scale * 16.0)
    W.poison_unused(w)
    out, status = run_grouped(w, 8, [16, 16])
    assert status == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), f"grouped, peaked scores, d={d}")
    again, _ = run_grouped(w, 8, [16, 16])
    assert torch.equal(out, again)


def test_grouped_bad_page_ids_in_the_shared_tiles_are_masked_and_reported():
    lens = [300 + 11 * j for j in range(8)]
    w = W.make_custom(lens, Hq=8, Hkv=2, d=128, seed=78, device=DEV, num_blocks=256, poison=False)
    bt = w.block_table.clone()
    for j in range(1, 8):
        bt[j, :16] = bt[0, :16]                          # one group shares 16 pages = 4 tiles
    bt[:, 5] = 256                                       # one past the pool, in the second shared tile
    bt[:, 9] = -3
    wb = dataclasses.replace(w, block_table=bt)
    out, status = run_grouped(wb, 8, [4])
    assert status == pdattn.BAD_PAGE_INDEX
    ref, bad = orc.decode_workload(wb.to("cpu"), return_bad=True)
    assert bad == 8 * 2 * 16 * 8                         # 8 rows, two pages of 16 tokens, 8 heads
    assert_parity(out, ref, "grouped, bad pages in the shared tiles masked")


@pytest.mark.parametrize("Hq,Hkv,group,d", [(28, 4, 8, 128), (32, 4, 8, 128), (16, 2, 8, 64)])
def test_groups_of_56_and_64_query_rows(Hq, Hkv, group, d, prefix_engine):
    """The 7B shape (28 q / 4 KV heads) in groups of 8 is 56 rows per unit, 32 / 4 is 64: every lane pair of
    the tensor-memory kernel is in use.  The warp-MMA kernel takes at most 48 rows and says so."""
    rng = np.random.default_rng(group + Hq)
    lens = [512 + int(rng.integers(1, 300)) for _ in range(2 * group)]
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, seed=90 + Hq, device=DEV, poison=False)
    bt = w.block_table.clone()
    for j in range(2 * group):
        bt[j, :32] = bt[j - j % group, :32]              # each group shares 32 pages = 8 tiles
    w = dataclasses.replace(w, block_table=bt)
    W.poison_unused(w)
    if prefix_engine == "warp_mma":
        ws = pdattn.alloc_grouped_workspace(w.num_seqs, Hq, Hkv, d)
        pt = torch.tensor([8, 8], dtype=torch.int32, device=DEV)
        st = pdattn.decode_grouped(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale,
                                   torch.empty_like(w.q), ws, w.context_lens_host, group, pt, [8, 8], check=False)
        assert st == pdattn.UNSUPPORTED
        return
    out, status = run_grouped(w, group, [8, 8])
    assert status == pdattn.OK
    assert_parity(out, orc.decode_workload(w.to("cpu")), f"Hq={Hq} Hkv={Hkv} group={group} d={d}")


def test_grouped_rejects_what_it_cannot_do():
    w = W.make_config(3, device=DEV, num_seqs=16, len_div=4)
    ws = pdattn.alloc_grouped_workspace(16, 40, 8, 128)
    pt = torch.tensor([4, 4], dtype=torch.int32, device=DEV)
    out = torch.empty_like(w.q)
    args = (w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws, w.context_lens_host)
    assert pdattn.decode_grouped(*args, 8, pt, [4, 4], check=False) == pdattn.OK
    assert pdattn.decode_grouped(*args, 5, pt, [4, 4], check=False) == pdattn.INVALID_ARG        # 16 % 5
    assert pdattn.decode_grouped(*args, 16, pt, [4], check=False) == pdattn.UNSUPPORTED          # 16 * 5 rows > 64
    too_long = [int(w.context_lens_host[:8].min()) // 64 + 1, 4]
    assert pdattn.decode_grouped(*args, 8, pt, too_long, check=False) == pdattn.INVALID_ARG      # prefix >= a member
    small = pdattn.alloc_workspace(16, 40, 8, 128)
    a2 = args[:7] + (small,) + args[8:]
    assert pdattn.decode_grouped(*a2, 8, pt, [4, 4], check=False) == pdattn.WORKSPACE_TOO_SMALL

"""GPU parity: libpdattn (through its C ABI) against the fp64 CPU oracle, element by element, plus
the structured suites that pin indexing exactly (probe positions, needles, poison, bitwise invariances).

Tolerance (bf16 output, fp32 accumulation): an element passes when
    |gpu - ref| <= max(2e-3, 1e-2 * |ref|)
and nothing is NaN/Inf.
"""
import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16
DEV = "cuda"


def run(w, use_host_lens=True, ws=None, out=None):
    if ws is None:
        ws = pdattn.alloc_workspace(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size)
    out = pdattn.decode_workload(w, out=out, workspace=ws, use_host_lens=use_host_lens)
    st = pdattn.check(ws)
    return out, st


def assert_parity(out, ref, what=""):
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    tol = np.maximum(2e-3, 1e-2 * np.abs(ref))
    bad = err > tol
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; "
                           f"max abs err {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}")
    return err.max()


def check_against_oracle(w_gpu, what, use_host_lens=True, pairs=None):
    out, st = run(w_gpu, use_host_lens)
    assert st == pdattn.OK
    wc = w_gpu.to("cpu")
    if pairs is None:
        ref = orc.decode_workload(wc)
        assert_parity(out, ref, what)
    else:
        ref = orc.decode_workload(wc, pairs=pairs)
        got = out[torch.as_tensor(pairs[:, 0], device=DEV), torch.as_tensor(pairs[:, 1], device=DEV)]
        assert_parity(got, ref, what)
    return out


# ---------------------------------------------------------------------------- oracle parity

def test_tiny_config():
    check_against_oracle(W.make_config(1, device=DEV), "config 1")


def test_tiny_config_device_side_plan():
    check_against_oracle(W.make_config(1, device=DEV), "config 1 / device plan", use_host_lens=False)


@pytest.mark.parametrize("cfg,num_seqs,len_div", [(2, 24, 2), (3, 16, 4), (4, 12, 4), (5, 2, 8)])
def test_scaled_configs_all_outputs(cfg, num_seqs, len_div):
    """Every output element of a shrunk configuration: several tiles per unit, ragged tails,
    units cut by span boundaries, G = 7 / 5 / 8 / 7."""
    check_against_oracle(W.make_config(cfg, device=DEV, num_seqs=num_seqs, len_div=len_div), f"config {cfg} scaled")


@pytest.mark.parametrize("host_lens", [True, False])
def test_ragged_lengths_around_tile_and_page_edges(host_lens):
    lens = [1, 2, 15, 16, 17, 31, 32, 33, 47, 48, 49, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 257,
            511, 513, 1000, 0, 3, 64 * 9 + 1]
    for (Hq, Hkv, d) in [(28, 4, 128), (4, 1, 64), (16, 2, 64), (32, 2, 128), (3, 3, 128)]:
        w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, seed=100 + Hq, device=DEV)
        check_against_oracle(w, f"ragged Hq={Hq} Hkv={Hkv} d={d}", use_host_lens=host_lens)


def test_many_short_sequences():
    rng = np.random.default_rng(7)
    lens = rng.integers(0, 150, size=700)
    check_against_oracle(W.make_custom(lens, Hq=8, Hkv=2, d=128, seed=5, device=DEV), "many short")


@pytest.mark.parametrize("Hq,Hkv,d,bs", [(28, 4, 128, 16), (64, 4, 128, 16), (16, 2, 64, 16), (32, 2, 64, 32)])
def test_batches_of_two_to_eleven_tile_pieces(Hq, Hkv, d, bs):
    """Hundreds of pieces per CTA, each spread over two to six consumer warps: every hand-off slot of
    the chained merge is reused many times, with 8- and 16-row tiles (one slot only at d = 128)."""
    rng = np.random.default_rng(17)
    lens = rng.integers(65, 700, size=1200)
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=19, device=DEV)
    out = check_against_oracle(w, f"mid-length pieces Hq={Hq} Hkv={Hkv} d={d} bs={bs}",
                               pairs=sample_pairs(w, 600, seed=23))
    again, st = run(w)
    assert st == pdattn.OK and torch.equal(out, again)      # the order of every sum is fixed


@pytest.mark.parametrize("Hq,Hkv,d,bs", [(28, 4, 128, 16), (8, 2, 64, 32), (5, 5, 128, 64), (16, 2, 64, 16)])
@pytest.mark.parametrize("kind", ["one_tile", "ragged", "few_tiles"])
def test_short_piece_kernel_same_bits_as_the_default_kernel(Hq, Hkv, d, bs, kind):
    """The short-piece instantiation (every warp walks 32 units at a time, a warp of its own stages the query
    rows) against the oracle, and bit for bit against the all-purpose instantiation: same tile dealing, same
    order of every sum.  A batch in which no sequence is cut needs no combine launch."""
    rng = np.random.default_rng(31)
    S = 1500
    lens = {"one_tile": rng.integers(1, 65, size=S), "ragged": rng.integers(0, 260, size=S),
            "few_tiles": rng.integers(40, 700, size=S)}[kind]
    if kind == "ragged":
        lens[rng.integers(S, size=40)] = 0                    # empty sequences inside the 32-unit windows
        lens[rng.integers(S, size=3)] = rng.integers(3000, 9000, size=3)   # and a few long ones cut over many spans
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=37, device=DEV)
    try:
        pdattn.set_merge_mode(2)
        pdattn.set_short_piece_path(0)
        base, st = run(w)
        assert st == pdattn.OK
        pdattn.set_short_piece_path(1)
        out = check_against_oracle(w, f"short-piece kernel, {kind}", pairs=sample_pairs(w, 800, seed=41))
        assert torch.equal(out, base)
        for _ in range(3):
            again, st = run(w)
            assert st == pdattn.OK and torch.equal(out, again)
        # by itself the library takes this kernel for batches of mostly one-tile sequences
        pdattn.set_merge_mode(-1)
        pdattn.set_short_piece_path(-1)
        auto, st = run(w)
        assert st == pdattn.OK and torch.equal(out, auto)
        if kind == "one_tile":
            assert pdattn.last_launch_count() == 1            # nothing is cut: no combine launch
    finally:
        pdattn.set_merge_mode(-1)
        pdattn.set_short_piece_path(-1)


def test_single_long_sequence_is_split_over_all_sms():
    w = W.make_custom([40000], Hq=7, Hkv=1, d=128, seed=6, device=DEV)
    check_against_oracle(w, "one long sequence")


def test_peaked_softmax_with_head_scales():
    w = W.make_config(4, device=DEV, num_seqs=6, len_div=8)
    w.scale = w.scale * 4.0                       # score std up to ~8: near one-hot weights
    check_against_oracle(w, "peaked")


def test_negative_and_zero_scale():
    w = W.make_custom([300, 77], Hq=8, Hkv=2, d=128, seed=8, device=DEV)
    for sc in (-0.1, 0.0):
        w.scale = sc
        check_against_oracle(w, f"scale {sc}")


# ---------------------------------------------------------------------------- full-size configs

def sample_pairs(w, n, seed):
    rng = np.random.default_rng(seed)
    L = w.context_lens_host
    seqs = set(rng.integers(0, len(L), size=n).tolist())
    seqs.update([int(np.argmax(L)), int(np.argmin(L)), 0, len(L) - 1])
    pairs = [(s, int(h)) for s in sorted(seqs) for h in rng.choice(w.num_q_heads, size=3, replace=False)]
    return np.array(pairs, dtype=np.int32)


@pytest.mark.parametrize("cfg", [2, 3, 4, 5])
def test_full_size_configs_every_output(cfg, full_reference):
    """The benchmark's configurations at full size in the benchmark's launch configuration: every output
    element against the oracle (all (sequence, head) rows, computed once per session), and the bitwise
    properties that hold at any size."""
    w = W.make_config(cfg, device=DEV)
    out, st = run(w)
    assert st == pdattn.OK
    ref = full_reference(cfg, w)
    assert ref.shape == tuple(out.shape)
    assert_parity(out, ref, f"config {cfg} full, all {ref.size} outputs")
    out2, st = run(w)
    assert st == pdattn.OK and torch.equal(out, out2)                      # run to run
    out3, _ = run(w, use_host_lens=False)
    assert torch.equal(out, out3)                                          # host plan == device plan
    del w
    torch.cuda.empty_cache()


# ---------------------------------------------------------------------------- exact pins

def test_context_len_one_returns_v_bits():
    w = W.make_custom([1] * 9, Hq=28, Hkv=4, d=128, seed=9, device=DEV)
    out, st = run(w)
    assert st == pdattn.OK
    bt = w.block_table.cpu().numpy()
    for s in range(9):
        for h in range(28):
            assert torch.equal(out[s, h], w.v_cache[bt[s, 0], h // 7, 0])


def boundary_positions(L):
    c = {0, L - 1}
    for e in range(16, L, 16):
        c.update([e - 1, e])
    return sorted(p for p in c if 0 <= p < L)


@pytest.mark.parametrize("L", [1, 2, 16, 64, 128, 1024, 4096, 32768])
def test_probe_positions_power_of_two(L):
    """K = 0 gives uniform weights 1/L; V[t, j] = 1 iff t == pos_j.  out[j] must be exactly 2^-k:
    a dropped token would give 0 and a double-counted one 2^-(k-1)."""
    d = 128
    w = W.make_custom([L], Hq=7, Hkv=1, d=d, seed=10, device=DEV, poison=False)
    w.k_cache.zero_()
    w.v_cache.zero_()
    pos = boundary_positions(L)
    if len(pos) > d:
        rng = np.random.default_rng(L)
        keep = {0, L - 1, L - 2, 63, 64, 65} & set(pos)
        rest = [p for p in pos if p not in keep]
        pos = sorted(keep | set(rng.choice(rest, size=d - len(keep), replace=False).tolist()))
    bt = w.block_table.cpu().numpy()
    for j, t in enumerate(pos):
        w.v_cache[bt[0, t // 16], 0, t % 16, j] = 1.0
    W.poison_unused(w)
    out, st = run(w)
    assert st == pdattn.OK
    got = out.float().cpu().numpy()
    want = np.zeros(d, dtype=np.float32)
    want[: len(pos)] = 1.0 / L
    for h in range(7):
        assert np.array_equal(got[0, h], want), (L, h, got[0, h][: len(pos)], 1.0 / L)


@pytest.mark.parametrize("L", [3, 17, 100, 1000, 8191, 8193, 50001])
def test_probe_positions_any_length(L):
    d = 128
    w = W.make_custom([L], Hq=4, Hkv=1, d=d, seed=11, device=DEV, poison=False)
    w.k_cache.zero_()
    w.v_cache.zero_()
    pos = boundary_positions(L)
    if len(pos) > d:
        rng = np.random.default_rng(L)
        keep = {0, L - 1, L - 2} & set(pos)
        rest = [p for p in pos if p not in keep]
        pos = sorted(keep | set(rng.choice(rest, size=d - len(keep), replace=False).tolist()))
    bt = w.block_table.cpu().numpy()
    for j, t in enumerate(pos):
        w.v_cache[bt[0, t // 16], 0, t % 16, j] = 1.0
    W.poison_unused(w)
    out, _ = run(w)
    got = out.float().cpu().numpy().astype(np.float64)
    want = np.zeros(d)
    want[: len(pos)] = 1.0 / L
    # 1/L rounded to bf16, allowing one bf16 ulp for the fp32 reciprocal and partial-sum merges
    assert np.all(np.abs(got[0] - want[None, :]) <= want[None, :] * 2.0 ** -7 + 0)
    assert np.all(got[0, :, len(pos):] == 0)
    assert np.all(got[0, :, : len(pos)] > 0.9 / L)          # nothing dropped


@pytest.mark.parametrize("L", [70, 1000, 20000])
def test_needle_returns_its_value_bits(L):
    """One key aligned with q outweighs all others by e^60 or more: out must equal that token's V bit for bit,
    wherever the needle sits relative to page, tile and span boundaries."""
    d = 128
    w = W.make_custom([L], Hq=7, Hkv=1, d=d, seed=12, device=DEV, poison=False)
    w.k_cache.zero_()
    w.q[:] = 1.0
    w.scale = 1.0
    bt = w.block_table.cpu().numpy()
    pos = boundary_positions(L)
    if len(pos) > 24:
        rng = np.random.default_rng(L)
        pos = sorted({0, L - 1} | set(rng.choice(pos, size=22, replace=False).tolist()))
    ws = pdattn.alloc_workspace(1, 7, 1, d)
    for t in pos:
        page, slot = bt[0, t // 16], t % 16
        w.k_cache[page, 0, slot, :] = 1.0                   # score 128, all others 0
        out, st = run(w, ws=ws)
        assert st == pdattn.OK
        for h in range(7):
            assert torch.equal(out[0, h], w.v_cache[page, 0, slot]), (L, t, h)
        w.k_cache[page, 0, slot, :] = 0.0


def test_poisoned_tail_slots_and_unowned_pages_do_not_matter():
    lens = [1, 17, 100, 256, 1000, 63, 65, 4097]
    clean = W.make_custom(lens, Hq=28, Hkv=4, d=128, seed=13, device=DEV, poison=False)
    ref, _ = run(clean)
    W.poison_unused(clean)
    assert torch.isnan(clean.v_cache.float()).any()
    out, st = run(clean)
    assert st == pdattn.OK
    assert torch.equal(ref, out)


def test_shared_versus_copied_prefix_pages_bitwise():
    """GRPO group: 8 samples point at the same prompt pages (run A) or at private copies of them (run B)."""
    w = W.make_config(3, device=DEV, num_seqs=16, len_div=4, poison=False)   # prompt 256 tokens = 16 pages
    out_a, st = run(w)
    assert st == pdattn.OK
    NB = w.num_blocks
    bt = w.block_table.clone()
    extra = 2 * 7 * 16
    k2 = torch.cat([w.k_cache, torch.zeros(extra, *w.k_cache.shape[1:], dtype=BF16, device=DEV)])
    v2 = torch.cat([w.v_cache, torch.zeros(extra, *w.v_cache.shape[1:], dtype=BF16, device=DEV)])
    nxt = NB
    for s in range(16):
        if s % 8 == 0:
            continue
        for j in range(16):
            src = int(bt[s, j])
            k2[nxt] = w.k_cache[src]
            v2[nxt] = w.v_cache[src]
            bt[s, j] = nxt
            nxt += 1
    import dataclasses
    wb = dataclasses.replace(w, k_cache=k2, v_cache=v2, block_table=bt)
    out_b, st = run(wb)
    assert st == pdattn.OK
    assert torch.equal(out_a, out_b)
    assert_parity(out_a, orc.decode_workload(w.to("cpu")), "shared prefix")


def test_page_permutation_bitwise():
    w = W.make_custom([100, 33, 256, 5000, 777], Hq=28, Hkv=4, d=128, seed=14, device=DEV, num_blocks=512)
    ref, _ = run(w)
    perm = torch.from_numpy(np.random.default_rng(3).permutation(512)).to(DEV)
    inv = torch.argsort(perm)
    import dataclasses
    bt = w.block_table.clone().long()
    valid = bt >= 0
    bt[valid] = perm[bt[valid]]
    w2 = dataclasses.replace(w, k_cache=w.k_cache[inv].contiguous(), v_cache=w.v_cache[inv].contiguous(),
                             block_table=bt.to(torch.int32))
    out, st = run(w2)
    assert st == pdattn.OK
    assert torch.equal(ref, out)


@pytest.mark.parametrize("L", [64, 4096, 65536])
def test_integer_values_are_exact(L):
    """K = 0, V small integers, L a power of two: out = bf16(sum / L) exactly in any summation order."""
    w = W.make_custom([L], Hq=8, Hkv=2, d=64, seed=15, device=DEV, poison=False)
    w.k_cache.zero_()
    NBs = w.v_cache.shape
    ints = torch.randint(-3, 4, NBs, device=DEV, generator=torch.Generator(DEV).manual_seed(L))
    w.v_cache.copy_(ints.to(BF16))
    out, _ = run(w)
    bt = w.block_table[0, : L // 16].long()
    vs = ints[bt].permute(1, 0, 2, 3).reshape(2, L, 64).sum(1).double() / L         # [Hkv, d]
    want = vs.to(torch.float32).to(BF16)
    for h in range(8):
        assert torch.equal(out[0, h], want[h // 4])


def test_padded_query_rows_are_never_written():
    for Hq, Hkv in [(28, 4), (40, 8), (4, 1), (5, 5), (18, 2)]:
        w = W.make_custom([100, 0, 3000, 64], Hq=Hq, Hkv=Hkv, d=128, seed=16, device=DEV)
        S, n = 4, 4 * Hq * 128
        buf = torch.full((n + 2048,), 7.0, dtype=BF16, device=DEV)
        out = buf[1024: 1024 + n].view(S, Hq, 128)
        assert out.data_ptr() % 16 == 0
        run(w, out=out)
        assert torch.all(buf[:1024] == 7.0) and torch.all(buf[1024 + n:] == 7.0)
        assert_parity(out, orc.decode_workload(w.to("cpu")), f"guarded out Hq={Hq}")


def test_zero_length_sequences_give_zeros_and_empty_batch_is_a_noop():
    w = W.make_custom([0, 50, 0, 0], Hq=8, Hkv=2, d=128, seed=17, device=DEV)
    out = torch.full_like(w.q, 5.0)
    run(w, out=out)
    assert torch.all(out[0] == 0) and torch.all(out[2:] == 0)
    assert_parity(out, orc.decode_workload(w.to("cpu")), "zero lengths")
    allz = W.make_custom([0, 0], Hq=8, Hkv=2, d=128, seed=17, device=DEV)
    out = torch.full_like(allz.q, 5.0)
    for host in (True, False):
        run(allz, out=out, use_host_lens=host)
        assert torch.all(out == 0)
    e = W.make_custom([], Hq=8, Hkv=2, d=128, seed=17, device=DEV)
    ws = pdattn.alloc_workspace(1, 8, 2, 128)
    pdattn.decode_workload(e, workspace=ws)


def test_out_of_range_page_ids_are_masked_and_reported():
    w = W.make_custom([200, 48], Hq=8, Hkv=2, d=128, seed=18, device=DEV, num_blocks=64, poison=False)
    ws = pdattn.alloc_workspace(2, 8, 2, 128)
    bt = w.block_table.clone()
    bt[0, 3] = 64            # one past the pool
    bt[1, 1] = -5
    import dataclasses
    wb = dataclasses.replace(w, block_table=bt)
    out, st = run(wb, ws=ws)
    assert st == pdattn.BAD_PAGE_INDEX
    ref, bad = orc.decode_workload(wb.to("cpu"), return_bad=True)
    assert bad == 2 * 16 * 8
    assert_parity(out, ref, "bad pages masked")
    out, st = run(w, ws=ws)                      # the word was cleared by the check
    assert st == pdattn.OK
    # garbage past the used range of a row is never read
    bt2 = w.block_table.clone()
    bt2[1, 3:] = 1 << 30
    out2, st = run(dataclasses.replace(w, block_table=bt2), ws=ws)
    assert st == pdattn.OK and torch.equal(out, out2)


def test_a_context_longer_than_its_table_row_is_masked_and_reported_without_reading_past_the_row():
    """Device-side plan (no host copy of the lengths to refuse the call with): the last sequence claims 200 tokens
    while its block_table row describes 128.  The entries past the row's end would lie past the end of the table's
    allocation; they are not read, those tokens count as a bad page, and the result is the attention over the 128
    tokens the row does describe.  With the host copy the call is refused instead."""
    import dataclasses
    w = W.make_custom([100, 128], Hq=8, Hkv=2, d=128, seed=21, device=DEV, num_blocks=64, poison=False)
    assert w.max_blocks_per_seq == 8
    lens = torch.tensor([100, 200], dtype=torch.int32, device=DEV)
    wl = dataclasses.replace(w, context_lens=lens, context_lens_host=np.array([100, 200], dtype=np.int32))
    ws = pdattn.alloc_workspace(2, 8, 2, 128)
    out, st = run(wl, use_host_lens=False, ws=ws)
    assert st == pdattn.BAD_PAGE_INDEX
    assert_parity(out, orc.decode_workload(w.to("cpu")), "tokens past the row masked")
    out2 = torch.empty_like(w.q)
    st = pdattn.decode_ex(wl.q, wl.k_cache, wl.v_cache, wl.block_table, wl.context_lens, wl.scale, out2, ws,
                          context_lens_host=wl.context_lens_host, check=False)
    assert st == pdattn.INVALID_ARG


def test_device_planner_refuses_a_batch_whose_tile_count_overflows():
    """Without a host copy of the lengths the planning kernel sums tile counts itself; a batch beyond 2^30 tiles gets
    an empty plan (nothing is read or computed) and pdattn_check says so.  With the host copy the call is refused."""
    S = 64
    w = W.make_custom([16] * S, Hq=8, Hkv=8, d=128, seed=22, device=DEV, num_blocks=64, poison=False)
    huge = torch.full((S,), 1 << 30, dtype=torch.int32, device=DEV)
    ws = pdattn.alloc_workspace(S, 8, 8, 128)
    out = torch.full_like(w.q, 7.0)
    st = pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, huge, w.scale, out, ws, context_lens_host=None,
                          check=False)
    assert st == pdattn.OK
    assert pdattn.check(ws) == pdattn.UNSUPPORTED
    assert torch.all(out == 7.0)                       # nothing was written
    st = pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, huge, w.scale, out, ws,
                          context_lens_host=np.full(S, 1 << 30, dtype=np.int32), check=False)
    assert st == pdattn.INVALID_ARG
    out2, st = run(w, use_host_lens=False, ws=ws)      # the workspace is usable afterwards
    assert st == pdattn.OK
    assert_parity(out2, orc.decode_workload(w.to("cpu")), "after a refused batch")


def test_token_major_cache_layout_through_strides():
    """[page, slot, head, dim] pools passed through the stride arguments give the same bits."""
    w = W.make_custom([333, 64, 1500], Hq=28, Hkv=4, d=128, seed=19, device=DEV)
    ref, _ = run(w)
    import dataclasses
    k = w.k_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v = w.v_cache.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert k.stride(1) == 128 and k.stride(2) == 4 * 128
    out, st = run(dataclasses.replace(w, k_cache=k, v_cache=v))
    assert st == pdattn.OK and torch.equal(ref, out)


def test_short_form_with_binding_and_host_buffer_form(merge_mode):
    w = W.make_config(2, device=DEV, num_seqs=12, len_div=4)
    ref, _ = run(w)
    ws = pdattn.alloc_workspace(w.num_seqs, 28, 4, 128)
    lens_host = w.context_lens_host.copy()
    pdattn.bind(w.max_blocks_per_seq, w.num_blocks, ws, lens_host)
    out = torch.empty_like(w.q)
    pdattn.decode(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.num_seqs, 28, 4, 128, 16,
                  w.scale, out)
    assert pdattn.check(ws) == pdattn.OK and torch.equal(ref, out)
    # one launch when the cut units are merged inside the decode kernel, else the combine kernel follows
    assert pdattn.last_launch_count() == (1 if merge_mode == "chain" else 2)
    pdattn.bind(w.max_blocks_per_seq, w.num_blocks, ws, None)
    out.zero_()
    pdattn.decode(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.num_seqs, 28, 4, 128, 16,
                  w.scale, out)
    assert pdattn.check(ws) == pdattn.OK and torch.equal(ref, out)
    assert pdattn.last_launch_count() == 3
    # host-buffer form
    qh = w.q.cpu().pin_memory()
    bth = w.block_table.cpu().pin_memory()
    lh = w.context_lens.cpu().pin_memory()
    oh = torch.empty_like(qh).pin_memory()
    staging = torch.empty(pdattn.host_staging_size(w.num_seqs, 28, 128, w.max_blocks_per_seq), dtype=torch.uint8,
                          device=DEV)
    try:
        for mode in (0, 1):     # through the staging copies; pinned q and out used in place by the kernels
            pdattn.set_host_zero_copy(mode)
            oh.fill_(float("nan"))
            pdattn.decode_host(qh, bth, lh, oh, w.k_cache, w.v_cache, w.scale, staging, ws)
            torch.cuda.synchronize()
            assert pdattn.check(ws) == pdattn.OK and torch.equal(ref.cpu(), oh)
        # the same call with its arguments marshalled once, over buffers the caller rewrites in place: the lengths
        # shrink (the gather kernel fetches fewer table entries), the garbage past the used part is never read
        step = pdattn.HostStep(qh, bth, lh, oh, w.k_cache, w.v_cache, w.scale, staging, ws)
        oh.fill_(float("nan"))
        step()
        torch.cuda.synchronize()
        assert torch.equal(ref.cpu(), oh)
        shorter = torch.clamp(lh - 37, min=0)
        import dataclasses
        ws2 = dataclasses.replace(w, context_lens=shorter.to(DEV), context_lens_host=shorter.numpy().copy())
        ref2, _ = run(ws2)
        lh.copy_(shorter)
        for s_, L_ in enumerate(shorter.tolist()):
            bth[s_, (L_ + 15) // 16:] = 1 << 30
        step()
        torch.cuda.synchronize()
        assert pdattn.check(ws) == pdattn.OK and torch.equal(ref2.cpu(), oh)
        lh.copy_(w.context_lens.cpu())
        bth.copy_(w.block_table.cpu())
        # pageable q and out: the in-place form does not apply and the copies are taken
        qp, op = w.q.cpu(), torch.full_like(w.q.cpu(), float("nan"))
        pdattn.decode_host(qp, bth, lh, op, w.k_cache, w.v_cache, w.scale, staging, ws)
        torch.cuda.synchronize()
        assert pdattn.check(ws) == pdattn.OK and torch.equal(ref.cpu(), op)
    finally:
        pdattn.set_host_zero_copy(-1)


def test_workspace_too_small_and_misaligned_are_rejected_on_gpu():
    w = W.make_custom([10], Hq=4, Hkv=1, d=64, seed=20, device=DEV)
    out = torch.empty_like(w.q)
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    st = pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, small, check=False)
    assert st == pdattn.WORKSPACE_TOO_SMALL
    ws = pdattn.alloc_workspace(1, 4, 1, 64)
    st = pdattn.decode_ex(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws[16:],
                          check=False)
    assert st == pdattn.MISALIGNED


@pytest.fixture
def runtime_spans():
    pdattn.set_dynamic_spans(8)
    yield
    pdattn.set_dynamic_spans(-1)


@pytest.mark.parametrize("cfg,num_seqs,len_div", [(2, 48, 1), (5, 2, 2), (3, 24, 2)])
def test_runtime_span_scheduling_is_correct_and_deterministic(runtime_spans, cfg, num_seqs, len_div):
    """With run-time spans the CTA that processes a span varies from run to run; the output bits must not."""
    w = W.make_config(cfg, device=DEV, num_seqs=num_seqs, len_div=len_div)
    _, plan = pdattn.plan_host(w.context_lens_host, w.num_kv_heads, 148, dynamic_per_cta=8)
    assert plan.n_dynamic > 0
    out = check_against_oracle(w, f"config {cfg} with run-time spans")
    for _ in range(4):
        again, st = run(w)
        assert st == pdattn.OK and torch.equal(out, again)
    dev_plan, st = run(w, use_host_lens=False)
    assert st == pdattn.OK and torch.equal(out, dev_plan)


def test_page_sizes_32_and_64_and_wide_gqa_groups():
    """block_size 32 and 64 (two pages, one page per tile) and G in 9..16 (two MMA column tiles per warp)."""
    lens = [1, 31, 32, 33, 63, 64, 65, 100, 1000, 4097, 0, 129]
    for (Hq, Hkv, d, bs) in [(28, 4, 128, 32), (4, 1, 64, 32), (24, 2, 128, 32), (32, 2, 128, 16), (10, 1, 64, 16),
                             (28, 4, 128, 64), (6, 2, 64, 64), (24, 2, 128, 64)]:
        w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=200 + Hq + bs, device=DEV)
        for host in (True, False):
            check_against_oracle(w, f"bs={bs} Hq={Hq} Hkv={Hkv} d={d}", use_host_lens=host)
    w = W.make_config(2, device=DEV, num_seqs=32)
    for bs in (32, 64):
        wb = W.make_custom(w.context_lens_host, Hq=28, Hkv=4, d=128, bs=bs, seed=77, device=DEV)
        check_against_oracle(wb, f"7B-shaped lengths, page size {bs}")


def test_an_expired_wait_is_reported_and_leaves_the_context_usable():
    """Failure path without a fault: a wait that nothing satisfies runs into its limit (2 ms here), the
    kernel sets the timeout bit and returns; the check reports it once; the next decode step is fine."""
    w = W.make_config(1, device=DEV)
    ws = pdattn.alloc_workspace(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim)
    ref, st = run(w, ws=ws)
    assert st == pdattn.OK
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    assert pdattn.wait_limit_probe(ws, 2000) == pdattn.OK
    t1.record()
    assert pdattn.check(ws) == pdattn.DEVICE_TIMEOUT
    assert 1.5 < t0.elapsed_time(t1) < 200.0                       # it waited about its limit, not forever
    assert pdattn.check(ws) == pdattn.OK                           # the word is sticky until read, then clear
    out, st = run(w, ws=ws)
    assert st == pdattn.OK and torch.equal(out, ref)
    assert pdattn.wait_limit_probe(ws, 0) == pdattn.INVALID_ARG


@pytest.mark.parametrize("per_cta", [0, 2])
def test_full_config2_with_a_fixed_number_of_runtime_spans(per_cta):
    """The default picks the number of run-time spans from the batch shape (4 per CTA here); static spans only
    and another count must give the same attention within tolerance (the cuts differ, so not the same bits)."""
    w = W.make_config(2, device=DEV)
    pdattn.set_dynamic_spans(per_cta)
    try:
        check_against_oracle(w, f"config 2, {per_cta} run-time spans per CTA", pairs=sample_pairs(w, 24, seed=31))
    finally:
        pdattn.set_dynamic_spans(-1)

"""GPU parity of pdattn_decode_multi (several new tokens per sequence, causal among them) against the oracle.

Tolerance as everywhere: |gpu - ref| <= max(2e-3, 1e-2 * |ref|), nothing NaN/Inf.
"""
import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def queries(w, T, seed):
    S, Hq, d = w.q.shape
    return W.normal_bf16(S * T * Hq * d, seed, 7, device=DEV).view(S, T, Hq, d)


def run_multi(w, q, host_lens=True, ws=None):
    S, T, Hq, d = q.shape
    if ws is None:
        ws = pdattn.alloc_multi_workspace(S, Hq, w.num_kv_heads, d, w.block_size, T)
    out = torch.full_like(q, float("nan"))
    pdattn.decode_multi(q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws,
                        context_lens_host=w.context_lens_host if host_lens else None)
    return out, pdattn.check(ws)


def assert_parity(out, ref, what):
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    bad = err > np.maximum(2e-3, 1e-2 * np.abs(ref))
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; "
                           f"max abs err {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}")


def reference(w, q):
    wc = w.to("cpu")
    return orc.decode_multi(q.cpu(), wc.k_cache, wc.v_cache, wc.block_table, wc.context_lens, wc.scale)


@pytest.mark.parametrize("host_lens", [True, False])
@pytest.mark.parametrize("Hq,Hkv,d,bs,T", [(28, 4, 128, 16, 2), (8, 2, 128, 16, 4), (8, 2, 64, 16, 2),
                                          (16, 4, 128, 32, 3), (3, 3, 128, 16, 16), (10, 2, 64, 32, 3), (28, 4, 128, 64, 2)])
def test_ragged_lengths_around_tile_and_page_edges(Hq, Hkv, d, bs, T, host_lens):
    """8-row and 16-row tiles, the new tokens straddling page and tile edges, sequences shorter than T
    (their first query tokens see nothing and give zeros), empty sequences."""
    lens = [T, T + 1, 15, 16, 17, 63, 64, 65, 66, 67, 127, 128, 129, 130, 131, 191, 193, 255, 257, 1000, 0, 2, 1,
            64 * 9 + 1, 64 * 9 + 2]
    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=300 + Hq + T, device=DEV)
    q = queries(w, T, 11)
    out, st = run_multi(w, q, host_lens)
    assert st == pdattn.OK
    assert_parity(out, reference(w, q), f"Hq={Hq} Hkv={Hkv} d={d} bs={bs} T={T}")


def test_scaled_rollout_config_with_two_query_tokens():
    """Units cut by span boundaries: the merge across spans carries all T * G rows."""
    w = W.make_config(2, device=DEV, num_seqs=24, len_div=2)
    q = queries(w, 2, 12)
    out, st = run_multi(w, q)
    assert st == pdattn.OK
    assert_parity(out, reference(w, q), "config 2 scaled, T = 2")
    again, _ = run_multi(w, q)
    assert torch.equal(out, again)


def test_single_long_sequence_split_over_all_sms():
    w = W.make_custom([40000], Hq=8, Hkv=2, d=128, seed=13, device=DEV)
    q = queries(w, 4, 14)
    out, st = run_multi(w, q)
    assert st == pdattn.OK
    assert_parity(out, reference(w, q), "one long sequence, T = 4")


def test_one_query_token_is_the_plain_decode_step_bitwise():
    w = W.make_config(2, device=DEV, num_seqs=16, len_div=4)
    out, st = run_multi(w, w.q.unsqueeze(1).contiguous())
    assert st == pdattn.OK
    assert torch.equal(out[:, 0], pdattn.decode_workload(w))


def test_last_query_token_agrees_with_the_plain_step_and_padded_rows_stay_untouched():
    w = W.make_custom([70, 300, 129], Hq=6, Hkv=2, d=128, seed=15, device=DEV)
    q = queries(w, 3, 16)
    out, st = run_multi(w, q)
    assert st == pdattn.OK
    wq = W.make_custom([70, 300, 129], Hq=6, Hkv=2, d=128, seed=15, device=DEV)
    import dataclasses
    plain = pdattn.decode_workload(dataclasses.replace(wq, q=q[:, 2].contiguous()))
    assert_parity(out[:, 2], plain.float().cpu().numpy().astype(np.float64), "last query token vs plain step")
    assert not torch.isnan(out).any()                    # every row of out was written, none twice with garbage


def test_rejects_what_it_cannot_do():
    w = W.make_custom([100, 200], Hq=28, Hkv=4, d=128, seed=17, device=DEV)
    ws = pdattn.alloc_workspace(2, 28, 4, 128)
    q3 = queries(w, 3, 18)                               # 3 * 7 = 21 rows > 16
    out = torch.empty_like(q3)
    args = (w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale)
    assert pdattn.decode_multi(q3, *args, out, ws, check=False) == pdattn.UNSUPPORTED
    q2 = queries(w, 2, 19)                               # 14 rows: needs the larger workspace
    assert pdattn.decode_multi(q2, *args, torch.empty_like(q2), ws, check=False) == pdattn.WORKSPACE_TOO_SMALL
    with pytest.raises(pdattn.PdattnError):
        pdattn.multi_workspace_size(2, 28, 4, 128, 16, 3)
    assert pdattn.lib().pdattn_decode_multi(None, 2, None) == pdattn.INVALID_ARG

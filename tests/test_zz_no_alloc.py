"""pdattn_decode_static_scratch: the decode step for callers that may not allocate device memory and
have no workspace to hand over (an engine whose KV-cache pool already owns the whole GPU, or a plug-in
whose host forbids allocation inside the step).  Its scratch is an array built into the library, shared
by every call on the device and never cleared between calls, so the check is made on two calls in a row
with different batches: stale partials of the first must not leak into the second.

Collected last on purpose (file name), so a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import pdattn_oracle as orc
from paper_2607_09207_b200 import pdattn
from paper_2607_09207_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def reference(w):
    ws = pdattn.alloc_workspace(w.num_seqs, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size)
    out = pdattn.decode_workload(w, workspace=ws)
    assert pdattn.check(ws) == pdattn.OK
    return out


def assert_close(got, ref, what):
    """got: bf16 output of the library; ref: the fp64 oracle's output for the same inputs."""
    g = got.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all(), what
    assert np.all(np.abs(g - ref) <= np.maximum(2e-3, 1e-2 * np.abs(ref))), what


def test_static_scratch_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    # batch A: long sequences cut by span boundaries (partials in use); batch B: another shape and
    # head configuration, fewer spans in use, so slots written by A stay behind untouched
    wa = W.make_config(2, device=DEV, num_seqs=40, len_div=1)
    wb = W.make_custom([5000, 17, 0, 900, 64, 3333], Hq=40, Hkv=8, d=128, seed=31, device=DEV)
    ref_a, ref_b = reference(wa), reference(wb)              # the entry point that takes a workspace
    orc_a, orc_b = orc.decode_workload(wa.to("cpu")), orc.decode_workload(wb.to("cpu"))
    status = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    out_a = torch.empty_like(wa.q)
    out_b = torch.empty_like(wb.q)
    pdattn.decode_static_scratch(wa.q, wa.k_cache, wa.v_cache, wa.block_table, wa.context_lens, wa.scale, out_a,
                                 context_lens_host=wa.context_lens_host, status_out=status)
    pdattn.decode_static_scratch(wb.q, wb.k_cache, wb.v_cache, wb.block_table, wb.context_lens, wb.scale, out_b,
                                 context_lens_host=None, status_out=status)      # device-side plan this time
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the expected value is the oracle's; within the tolerance every parity test uses
    assert_close(out_a, orc_a, "first call")
    assert_close(out_b, orc_b, "second call")
    # same plan, same kernels as the entry point that takes a workspace: the bits agree as well
    assert torch.equal(out_a, ref_a) and torch.equal(out_b, ref_b)
    # and again in the other order, through the same array
    out_a2 = torch.empty_like(wa.q)
    pdattn.decode_static_scratch(wa.q, wa.k_cache, wa.v_cache, wa.block_table, wa.context_lens, wa.scale, out_a2,
                                 context_lens_host=wa.context_lens_host)
    torch.cuda.synchronize()
    assert_close(out_a2, orc_a, "third call")
    assert torch.equal(out_a2, ref_a)


def test_static_scratch_reports_bad_pages_and_rejects_oversized_batches():
    import dataclasses
    w = W.make_custom([200, 48], Hq=8, Hkv=2, d=128, seed=32, device=DEV, num_blocks=64, poison=False)
    bt = w.block_table.clone()
    bt[0, 2] = 64
    wb = dataclasses.replace(w, block_table=bt)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = torch.empty_like(w.q)
    pdattn.decode_static_scratch(wb.q, wb.k_cache, wb.v_cache, wb.block_table, wb.context_lens, wb.scale, out,
                                 context_lens_host=wb.context_lens_host, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1
    pdattn.decode_static_scratch(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out,
                                 context_lens_host=w.context_lens_host, status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0           # the error word does not survive into the next call
    # more sequences than the built-in array is sized for: refused with a message, nothing launched
    S = 65537
    q = torch.zeros(S, 4, 64, dtype=torch.bfloat16, device=DEV)
    k = torch.zeros(8, 1, 16, 64, dtype=torch.bfloat16, device=DEV)
    table = torch.zeros(S, 1, dtype=torch.int32, device=DEV)
    lens = torch.ones(S, dtype=torch.int32, device=DEV)
    st = pdattn.decode_static_scratch(q, k, k, table, lens, 1.0, torch.empty_like(q), check=False)
    assert st == pdattn.WORKSPACE_TOO_SMALL
    assert b"65537 sequences" in pdattn.lib().pdattn_last_cuda_error()

"""Randomised mix of shapes, lengths, page sizes, merge modes, span settings and entry points (plain, several
query tokens, fp8 cache, fp8 with several query tokens, grouped with either prefix kernel) against the oracle.
Fixed seeds: the cases are the same on every run.
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


def parity(out, ref):
    got = out.float().cpu().numpy().astype(np.float64)
    if not np.isfinite(got).all():
        return "non-finite output"
    err = np.abs(got - ref)
    bad = err > np.maximum(2e-3, 1e-2 * np.abs(ref))
    return None if not bad.any() else f"{int(bad.sum())} elements out of tolerance, max abs err {err.max():.3e}"


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_mix_of_everything(seed):
    rng = np.random.default_rng(seed)
    failures = []
    shapes = [(28,4),(8,2),(40,8),(32,2),(5,5),(12,1),(64,4),(16,16),(7,1)]
    n = attempts = 0
    try:
        while n < 60 and attempts < 200:
            attempts += 1
            Hq, Hkv = shapes[rng.integers(len(shapes))]
            d = int(rng.choice([64, 128])); bs = int(rng.choice([16, 32, 64]))
            S = int(rng.integers(1, 40))
            kind = rng.choice(["short", "mid", "long", "mixed"])
            hi = {"short": 130, "mid": 1200, "long": 9000, "mixed": 3000}[kind]
            lens = rng.integers(0, hi, size=S)
            if kind == "mixed": lens[rng.integers(S)] = int(rng.integers(20000, 60000))
            mode = int(rng.choice([-1, 0, 1, 2])); dyn = int(rng.choice([-1, 0, 3, 8])); host = bool(rng.integers(2))
            short = int(rng.choice([-1, 0, 1]))
            pdattn.set_merge_mode(mode); pdattn.set_dynamic_spans(dyn); pdattn.set_short_piece_path(short)
            variant = rng.choice(["plain", "multi", "fp8", "grouped", "fp8multi"])
            G = Hq // Hkv
            desc = f"{variant} Hq={Hq} Hkv={Hkv} d={d} bs={bs} S={S} {kind} mode={mode} dyn={dyn} short={short} host={host}"
            try:
                w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=int(rng.integers(1 << 30)), device=DEV)
                wc = w.to("cpu")
                if variant == "plain":
                    ws = pdattn.alloc_workspace(S, Hq, Hkv, d, bs)
                    out = pdattn.decode_workload(w, workspace=ws, use_host_lens=host)
                    st = pdattn.check(ws); msg = parity(out, orc.decode_workload(wc))
                elif variant in ("multi", "fp8multi"):
                    T = int(rng.integers(1, max(2, 16 // G + 1)))
                    q = W.normal_bf16(S * T * Hq * d, 5, 7, device=DEV).view(S, T, Hq, d)
                    ws = pdattn.alloc_multi_workspace(S, Hq, Hkv, d, bs, T)
                    out = torch.full_like(q, float("nan"))
                    if variant == "multi":
                        pdattn.decode_multi(q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws, context_lens_host=w.context_lens_host if host else None)
                        ref = orc.decode_multi(q.cpu(), wc.k_cache, wc.v_cache, wc.block_table, wc.context_lens, wc.scale)
                    else:
                        ks = torch.tensor(rng.uniform(0.5, 2, Hkv), dtype=torch.float32, device=DEV); vs = torch.tensor(rng.uniform(0.5, 2, Hkv), dtype=torch.float32, device=DEV)
                        k8, v8 = W.fp8_caches(w, ks, vs)
                        pdattn.decode_fp8(q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, out, ws, context_lens_host=w.context_lens_host if host else None)
                        ref = orc.decode_fp8_multi(q.cpu(), k8.cpu(), v8.cpu(), ks.cpu(), vs.cpu(), wc.block_table, wc.context_lens, wc.scale)
                    st = pdattn.check(ws); msg = parity(out, ref); desc += f" T={T}"
                elif variant == "fp8":
                    ks = torch.tensor(rng.uniform(0.5, 2, Hkv), dtype=torch.float32, device=DEV); vs = torch.tensor(rng.uniform(0.5, 2, Hkv), dtype=torch.float32, device=DEV)
                    k8, v8 = W.fp8_caches(w, ks, vs)
                    ws = pdattn.alloc_workspace(S, Hq, Hkv, d, bs); out = torch.full_like(w.q, float("nan"))
                    pdattn.decode_fp8(w.q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, out, ws, context_lens_host=w.context_lens_host if host else None)
                    st = pdattn.check(ws); msg = parity(out, orc.decode_fp8(w.q.cpu(), k8.cpu(), v8.cpu(), ks.cpu(), vs.cpu(), wc.block_table, wc.context_lens, wc.scale))
                else:
                    if G > 8: continue
                    gs = int(rng.choice([g for g in (1, 2, 3, 4, 8) if g * G <= 64]))
                    ng = int(rng.integers(1, 6)); S = gs * ng
                    pt = rng.integers(0, 20, size=ng)
                    lens = np.concatenate([pt[i] * 64 + rng.integers(1, 400, size=gs) for i in range(ng)])
                    w = W.make_custom(lens, Hq=Hq, Hkv=Hkv, d=d, bs=bs, seed=int(rng.integers(1 << 30)), device=DEV, poison=False)
                    bt = w.block_table.clone()
                    for i in range(ng):
                        pg = int(pt[i]) * 64 // bs
                        for j in range(1, gs): bt[i * gs + j, :pg] = bt[i * gs, :pg]
                    w = dataclasses.replace(w, block_table=bt); W.poison_unused(w)
                    eng = int(rng.choice([0, 1])) if gs * G <= 48 else 1
                    f8 = bool(rng.integers(2)) and gs * G <= 48     # the same groups over an e4m3 copy of the pools
                    pdattn.set_prefix_engine(eng)
                    ws = pdattn.alloc_grouped_workspace(S, Hq, Hkv, d, bs); out = torch.full_like(w.q, float("nan"))
                    ptd = torch.tensor(pt, dtype=torch.int32, device=DEV)
                    if f8:
                        ks = torch.tensor(rng.uniform(0.5, 2, Hkv), dtype=torch.float32, device=DEV); vs = torch.tensor(rng.uniform(0.5, 2, Hkv), dtype=torch.float32, device=DEV)
                        k8, v8 = W.fp8_caches(w, ks, vs)
                        pdattn.decode_grouped_fp8(w.q, k8, v8, ks, vs, w.block_table, w.context_lens, w.scale, out, ws, w.context_lens_host, gs, ptd, pt.astype(np.int32))
                        ref = orc.decode_fp8(w.q.cpu(), k8.cpu(), v8.cpu(), ks.cpu(), vs.cpu(), w.block_table.cpu(), w.context_lens.cpu(), w.scale)
                    else:
                        pdattn.decode_grouped(w.q, w.k_cache, w.v_cache, w.block_table, w.context_lens, w.scale, out, ws, w.context_lens_host, gs, ptd, pt.astype(np.int32))
                        ref = orc.decode_workload(w.to("cpu"))
                    st = pdattn.check(ws); msg = parity(out, ref); desc += f" gs={gs} pt={pt.tolist()} eng={eng} fp8={f8}"
                    pdattn.set_prefix_engine(-1)
                n += 1
                if st != pdattn.OK or msg:
                    failures.append(f"{desc}: status {st}, {msg}")
            except Exception as e:
                failures.append(f"{desc}: {e!r}")
    finally:
        pdattn.set_merge_mode(-1)
        pdattn.set_dynamic_spans(-1)
        pdattn.set_short_piece_path(-1)
        pdattn.set_prefix_engine(-1)
    assert not failures, "\n".join(failures)
    assert n == 60
